"""Paged caches (block tables): the CUDA path on scattered blocks against the oracle on contiguous sequences.
Paging changes addresses only, so scores, indices and outputs must agree exactly as in the contiguous case --
and byte for byte with the CUDA path's own contiguous run."""
import pytest

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import __graft_entry__ as entry

entry._load_build_module().build()

import oracle
import paper_2606_06467_b200 as clsa
from _harness import GpuProblem, check_attention, check_scores, check_topk_band, check_topk_exact_on_gpu_scores
from workloads import MID, RAGGED, TINY, Workload

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg,bs", [
    (MID.replace(num_seqs=3, ctx=5000 + 7, top_k=384, num_layers=3), 16),
    (RAGGED.replace(num_seqs=5, ctx=9000, ragged_min=100, num_short=2, top_k=700, num_layers=2), 64),
    (TINY.replace(num_seqs=2, ctx=3000, top_k=128, num_layers=2), 32),
    (MID.replace(num_seqs=2, ctx=2500, top_k=256, num_layers=2, num_q_heads=20, num_kv_heads=4), 256),
], ids=["mid-bs16", "ragged-bs64", "tiny-bs32", "paper-heads-bs256"])
def test_paged_decode_matches_oracle_and_contiguous_run(cfg, bs):
    w = Workload(cfg)
    kc, vc = w.host_kv_full()
    prob = oracle.problem_from_workload(w, k_cache=kc, v_cache=vc, idx_k_cache=w.host_kidx_cache())
    ref_scores = prob.index_scores(w.q_idx_bits())
    ref_idx, ref_cnt = prob.topk(ref_scores)
    flat = GpuProblem(w)
    flat_outs = flat.decode_step()
    torch.cuda.synchronize()
    g = GpuProblem(w, block_size=bs)
    gs = g.index_scores()
    check_scores(gs, ref_scores, w)
    assert torch.equal(gs.nan_to_num(7.0), flat.index_scores().nan_to_num(7.0))
    outs = g.decode_step()
    torch.cuda.synchronize()
    assert g.status() == 0
    check_topk_exact_on_gpu_scores(prob, gs, g.idx, g.count, w)
    check_topk_band(ref_scores, ref_idx, ref_cnt, g.idx, g.count, w)
    assert torch.equal(g.idx, flat.idx) and torch.equal(g.count, flat.count)
    idx_np, cnt_np = g.idx.cpu().numpy(), g.count.cpu().numpy()
    for l in range(g.L):
        check_attention(prob, w, l, outs[l], None, idx_np, cnt_np)
        assert torch.equal(outs[l].view(torch.int16), flat_outs[l].view(torch.int16))
    # separate calls on the paged layout too, with LSE
    out0, lse0 = g.sparse_attn(0)
    check_attention(prob, w, 0, out0, lse0, idx_np, cnt_np)


def test_layers_call_on_paged_caches_never_follows_a_bad_entry():
    """clsa_sparse_attn_layers on paged caches with a caller-built index that has corrupt entries, a shorter count and
    a sequence whose length lies outside its bounds must come out as in the contiguous case: bad entries skipped and
    flagged (no block-table lookup, no row fetched), every other row equal to the contiguous run byte for byte, the
    caller's index untouched."""
    import numpy as np
    w = Workload(MID.replace(num_seqs=4, ctx=5000, top_k=256, num_layers=3, seed=123))
    kc, vc = w.host_kv_full()
    prob = oracle.problem_from_workload(w, k_cache=kc, v_cache=vc, idx_k_cache=w.host_kidx_cache())
    flat, g = GpuProblem(w), GpuProblem(w, block_size=16)
    gi, gc = flat.topk(flat.index_scores())
    idx_np, cnt_np = gi.cpu().numpy().copy(), gc.cpu().numpy().copy()
    bad = idx_np.copy()
    bad[0, 0, 3] = 2 ** 31 - 1
    bad[0, 0, 100] = -5
    bad[2, 0, 255] = int(w.seq_len[2]) + 4000          # past the sequence and past its row of the block table
    cnt = cnt_np.copy()
    cnt[3, 0] = 200                                    # a shorter selection: entries 200.. must be ignored
    bad[3, 0, 200:] = 10 ** 9
    results = []
    for prob_gpu in (flat, g):
        idx_t, cnt_t = torch.from_numpy(bad).to(prob_gpu.dev), torch.from_numpy(cnt).to(prob_gpu.dev)
        keep = idx_t.clone()
        outs = [prob_gpu.new_out() for _ in range(3)]
        clsa.clsa_sparse_attn_layers(prob_gpu.params, [prob_gpu.t["q_layers"][l] for l in range(3)], idx_t, cnt_t, outs, prob_gpu.ws)
        torch.cuda.synchronize()
        assert prob_gpu.status() == clsa.CLSA_DEV_BAD_INDEX
        clsa.clsa_clear_status(prob_gpu.ws)
        assert torch.equal(idx_t, keep)
        results.append(outs)
    ref_idx = -np.ones_like(idx_np); ref_cnt = cnt.copy()
    for b, drop in ((0, [3, 100]), (1, []), (2, [255]), (3, [])):
        row = np.delete(idx_np[b, 0, :cnt[b, 0]], drop)
        ref_idx[b, 0, :row.size] = row
        ref_cnt[b, 0] = row.size
    for l in range(3):
        check_attention(prob, w, l, results[1][l], None, ref_idx, ref_cnt)
        assert torch.equal(results[1][l].view(torch.int16), results[0][l].view(torch.int16))
    # a sequence whose length is out of bounds: zeros for it, flagged, the others unchanged
    g.t["seq_len"][1] = 10 ** 6
    idx_t, cnt_t = torch.from_numpy(idx_np).to(g.dev), torch.from_numpy(cnt_np).to(g.dev)
    outs = [g.new_out() for _ in range(3)]
    clsa.clsa_sparse_attn_layers(g.params, [g.t["q_layers"][l] for l in range(3)], idx_t, cnt_t, outs, g.ws)
    torch.cuda.synchronize()
    assert g.status() & clsa.CLSA_DEV_BAD_SEQLEN
    clsa.clsa_clear_status(g.ws)
    clean = [flat.new_out() for _ in range(3)]
    clsa.clsa_sparse_attn_layers(flat.params, [flat.t["q_layers"][l] for l in range(3)], gi, gc, clean, flat.ws)
    torch.cuda.synchronize()
    for l in range(3):
        assert (outs[l][1].float() == 0).all()
        for b in (0, 2, 3):
            assert torch.equal(outs[l][b].view(torch.int16), clean[l][b].view(torch.int16))


def test_paged_arguments_are_validated():
    w = Workload(MID.replace(num_seqs=2, ctx=1000, top_k=64, num_layers=1))
    g = GpuProblem(w, block_size=16)
    s = g.new_scores()
    for bad_bs in (8, 24, 8192):
        g.params.block_size = bad_bs
        with pytest.raises(clsa.ClsaError) as e:
            clsa.clsa_index_scores(g.params, g.t["q_idx"], s, g.score_stride, g.ws)
        assert e.value.status == clsa.CLSA_ERR_INVALID_ARG
    g.params.block_size = 16
    g.params.max_blocks_per_seq = 10          # 160 < 1000 positions
    with pytest.raises(clsa.ClsaError) as e:
        clsa.clsa_topk(g.params, s, g.score_stride, g.idx, g.count, g.ws)
    assert e.value.status == clsa.CLSA_ERR_INVALID_ARG
    g.params.max_blocks_per_seq = g.t["block_table"].shape[1]
    g.params.q_per_seq = 4                    # chunked scores need the extent of the (paged) row space
    g.params.num_cache_rows = 0
    with pytest.raises(clsa.ClsaError) as e:
        clsa.clsa_index_scores(g.params, g.t["q_idx"], s, g.score_stride, g.ws)
    assert e.value.status == clsa.CLSA_ERR_INVALID_ARG
