"""Prefill chunk (T > 1 queries per sequence, causal): the tcgen05 score GEMM, per-row causal top-k and sparse
attention with one index row per query, against the oracle."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import __graft_entry__ as entry

entry._load_build_module().build()

import oracle
import paper_2606_06467_b200 as clsa
from _harness import GpuProblem, check_attention, check_scores, check_topk_band, check_topk_exact_on_gpu_scores
from workloads import MID, TINY, Workload

pytestmark = pytest.mark.gpu


def _fused_equals_pair(g, gi, gc):
    """clsa_index_topk against clsa_index_scores + clsa_topk on the same problem: the same index, bit for bit."""
    idx = torch.full_like(gi, -7)
    cnt = torch.full_like(gc, -7)
    clsa.clsa_index_topk(g.params, g.t["q_idx"], idx, cnt, g.ws)
    torch.cuda.synchronize()
    assert g.status() == 0
    assert torch.equal(cnt, gc)
    assert torch.equal(idx, gi)


def _full_oracle(w):
    kc, vc = w.host_kv_full()
    return oracle.problem_from_workload(w, k_cache=kc, v_cache=vc, idx_k_cache=w.host_kidx_cache())


@pytest.mark.parametrize("B,T,n,d_idx,causal,ragged", [
    (1, 128, 1024, 128, 1, 0), (2, 200, 3000, 128, 1, 0), (1, 300, 2500, 64, 1, 0), (2, 77, 1111, 128, 0, 0),
    (3, 150, 2000, 128, 1, 500), (1, 513, 700, 64, 1, 0),
    (2, 401, 2500, 128, 1, 0), (1, 650, 1500, 64, 0, 0)])   # the last two: several query rows per attention block, with a tail
def test_chunk_scores_topk_attention(B, T, n, d_idx, causal, ragged):
    base = MID if d_idx == 128 else TINY
    cfg = base.replace(num_seqs=B, ctx=n, q_per_seq=T, causal=causal, top_k=96, num_layers=2, seed=900 + T + n,
                       ragged_min=ragged, num_short=0)
    w = Workload(cfg)
    g = GpuProblem(w)
    prob = _full_oracle(w)
    ref_scores = prob.index_scores(w.q_idx_bits())
    gs = g.index_scores()
    torch.cuda.synchronize()
    assert g.status() == 0
    check_scores(gs, ref_scores, w)
    gi, gc = g.topk(gs)
    check_topk_exact_on_gpu_scores(prob, gs, gi, gc, w)
    ref_idx, ref_cnt = prob.topk(ref_scores)
    check_topk_band(ref_scores, ref_idx, ref_cnt, gi, gc, w)
    _fused_equals_pair(g, gi, gc)
    idx_np, cnt_np = gi.cpu().numpy().copy(), gc.cpu().numpy().copy()
    for l in range(2):
        out, lse = g.sparse_attn(l, reverse=l)
        check_attention(prob, w, l, out, lse, idx_np, cnt_np)
    # the layers of a chunk as one call (no layer waits for its predecessor; two layers per launch where the group of
    # query heads leaves a head tile free): the separate calls of those shapes, bit for bit
    outs = [g.new_out() for _ in range(2)]
    clsa.clsa_sparse_attn_layers(g.params, [g.t["q_layers"][l] for l in range(2)], g.idx, g.count, outs, g.ws)
    for l in range(2):
        check_attention(prob, w, l, outs[l], None, idx_np, cnt_np)
        singles = [g.sparse_attn(l, shared_gpu=sg, keep_rows=1 if l == 0 else 0, lse=False)[0] for sg in (1, 2, 3, 4)]
        assert any(torch.equal(outs[l].view(torch.int16), x.view(torch.int16)) for x in singles), l
    assert g.status() == 0


@pytest.mark.parametrize("B,T,n,d_idx,causal,ragged,bs", [
    (2, 200, 3000, 128, 1, 0, 16), (1, 300, 2500, 64, 1, 0, 64), (3, 150, 2000, 128, 1, 500, 128),
    (2, 77, 1111, 128, 0, 0, 256), (1, 260, 5000, 128, 1, 0, 1024), (2, 130, 300, 64, 1, 0, 32),
    (2, 333, 2100, 128, 1, 0, 16)])
def test_chunk_on_paged_caches(B, T, n, d_idx, causal, ragged, bs):
    """Paging changes addresses only: the chunk's scores are bit-identical to the contiguous run, and the rest of
    the chunk path (top-k, attention through the block table) agrees with the oracle."""
    base = MID if d_idx == 128 else TINY
    cfg = base.replace(num_seqs=B, ctx=n, q_per_seq=T, causal=causal, top_k=96, num_layers=1, seed=700 + T + n + bs,
                       ragged_min=ragged, num_short=0)
    w = Workload(cfg)
    flat, g = GpuProblem(w), GpuProblem(w, block_size=bs)
    prob = _full_oracle(w)
    ref_scores = prob.index_scores(w.q_idx_bits())
    gs = g.index_scores()
    torch.cuda.synchronize()
    assert g.status() == 0
    check_scores(gs, ref_scores, w)
    assert torch.equal(gs.nan_to_num(7.0), flat.index_scores().nan_to_num(7.0))
    gi, gc = g.topk(gs)
    check_topk_exact_on_gpu_scores(prob, gs, gi, gc, w)
    _fused_equals_pair(g, gi, gc)
    out, lse = g.sparse_attn(0)
    check_attention(prob, w, 0, out, lse, gi.cpu().numpy().copy(), gc.cpu().numpy().copy())
    assert g.status() == 0


@pytest.mark.parametrize("B,T,n,d_idx,k,causal,ragged,bs", [
    (1, 300, 20000, 128, 512, 1, 0, 0), (2, 130, 9000, 64, 96, 1, 7000, 0), (1, 257, 40000, 128, 2048, 1, 0, 0),
    (2, 140, 12000, 128, 300, 0, 0, 0), (1, 200, 20000, 128, 512, 1, 0, 16), (2, 129, 9000, 64, 200, 1, 6500, 64),
    (1, 64, 70000, 128, 1024, 1, 0, 256)])
def test_fused_chunk_routing_on_long_rows(B, T, n, d_idx, k, causal, ragged, bs):
    """Rows longer than the candidate list: the pivot comes from a sample of the keys, the filter runs in the GEMM's
    epilogue, the select works on the candidates alone. The index must equal the materialising pair's bit for bit
    (same tensor-core scores, exact selection) and agree with the oracle under the usual rules; contiguous and paged."""
    base = MID if d_idx == 128 else TINY
    cfg = base.replace(num_seqs=B, ctx=n, q_per_seq=T, causal=causal, top_k=k, num_layers=1, seed=4000 + T + n + bs,
                       ragged_min=ragged, num_short=0)
    w = Workload(cfg)
    g = GpuProblem(w, block_size=bs)
    prob = oracle.problem_from_workload(w, idx_k_cache=w.host_kidx_cache())
    ref_scores = prob.index_scores(w.q_idx_bits())
    gs = g.index_scores()
    gi, gc = g.topk(gs)
    check_topk_exact_on_gpu_scores(prob, gs, gi, gc, w)
    ref_idx, ref_cnt = prob.topk(ref_scores)
    check_topk_band(ref_scores, ref_idx, ref_cnt, gi, gc, w)
    _fused_equals_pair(g, gi, gc)


def test_fused_chunk_routing_hands_back_rows_it_cannot_finish():
    """Long runs of equal scores at the threshold defeat the candidate list (it would have to hold all of them). Such
    rows are recomputed through the scratch matrix and still come out bit-identical to the materialising pair; when
    more rows need that than the scratch holds (64), the surplus rows get count 0 and CLSA_DEV_ROUTING_OVERFLOW is
    raised, and every other row is still right."""
    n, T, k = 16000, 100, 256
    w = Workload(MID.replace(num_seqs=1, ctx=n, q_per_seq=T, causal=1, top_k=k, num_layers=1, seed=77))
    g = GpuProblem(w)
    keys = g.t["idx_k_cache"]
    # queries 0..39: their own key rows are far away; make 9000 cached keys copies of query-aligned directions so that
    # for the first 40 queries thousands of scores tie exactly at the top
    q = g.t["q_idx"][0]                                   # [T, d]
    keys[1000:10000] = 0                                  # 9000 all-zero keys: score exactly 0 for every query
    big = torch.zeros_like(keys[0]); big[0] = 1.0
    # rows 0..39 get a negative component on dim 0 for all other keys -> zero-score keys rank at the top for them
    g.t["q_idx"][0, :40, :] = 0
    g.t["q_idx"][0, :40, 0] = -1.0
    keys[:1000, 0] = keys[:1000, 0].abs() + 0.5           # positive dim 0 -> negative scores for queries 0..39
    keys[10000:, 0] = keys[10000:, 0].abs() + 0.5
    gs = g.index_scores()
    gi, gc = g.topk(gs)
    torch.cuda.synchronize()
    assert (gs[0, :40, 1000:10000] == 0).all()
    _fused_equals_pair(g, gi, gc)                         # 40 rows handed back: all fit the scratch
    # now all 100 queries tie the same way: 100 rows need the scratch, 64 get it
    g.t["q_idx"][0, :, :] = 0
    g.t["q_idx"][0, :, 0] = -1.0
    gs = g.index_scores()
    gi, gc = g.topk(gs)
    idx = torch.full_like(gi, -7)
    cnt = torch.full_like(gc, -7)
    clsa.clsa_index_topk(g.params, g.t["q_idx"], idx, cnt, g.ws)
    torch.cuda.synchronize()
    assert g.status() == clsa.CLSA_DEV_ROUTING_OVERFLOW
    clsa.clsa_clear_status(g.ws)
    done = cnt[0] > 0
    assert int(done.sum()) == 64 and int((cnt[0] == 0).sum()) == T - 64
    assert torch.equal(idx[0][done], gi[0][done]) and torch.equal(cnt[0][done], gc[0][done])
    assert (idx[0][~done] == -1).all()


def test_gemm_row_equals_decode_gemv():
    """Row t of the chunk GEMM is the decode kernel's result for the same query against the same keys."""
    w = Workload(MID.replace(num_seqs=1, ctx=4096, q_per_seq=256, causal=0, top_k=64, num_layers=1, seed=31))
    g = GpuProblem(w)
    gs = g.index_scores()
    for t in (0, 100, 255):
        wd = Workload(MID.replace(num_seqs=1, ctx=4096, top_k=64, num_layers=1, seed=31))
        gd = GpuProblem(wd, layers=1)
        gd.params.idx_k_cache = g.t["idx_k_cache"].data_ptr()
        q = g.t["q_idx"][:, t:t + 1].contiguous()
        s = gd.new_scores()
        clsa.clsa_index_scores(gd.params, q, s, gd.score_stride, gd.ws)
        a, b = s[0, 0, :4096].cpu().numpy(), gs[0, t, :4096].cpu().numpy()
        assert np.abs(a - b).max() <= 1e-4 * max(1.0, np.abs(a).max())


def test_misaligned_score_rows_use_the_scalar_store_path():
    w = Workload(MID.replace(num_seqs=1, ctx=1500, q_per_seq=130, causal=1, top_k=32, num_layers=1, seed=5))
    g = GpuProblem(w)
    prob = oracle.problem_from_workload(w, idx_k_cache=w.host_kidx_cache())
    ref = prob.index_scores(w.q_idx_bits())
    stride = 1501                                    # odd stride: rows are not 32-byte aligned
    s = torch.full((1, 130, stride), float("nan"), dtype=torch.float32, device=g.dev)
    clsa.clsa_index_scores(g.params, g.t["q_idx"], s, stride, g.ws)
    got = s.cpu().numpy().astype(np.float64)
    for t in range(130):
        v = w.visible(0, t)
        assert np.abs(got[0, t, :v] - ref[0, t, :v]).max() <= 1e-4 * max(1.0, np.abs(ref[0, t, :v]).max())
        assert np.isnan(got[0, t, v:]).all()
