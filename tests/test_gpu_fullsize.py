"""Full-size parity: the mid, headline (128K x 16) and ragged workloads through `clsa_decode_step`, i.e. in the
launch configuration bench.py times. Scores and the top-k are checked completely; the attention output of the
first two and the last layer is checked completely against the oracle fed the GPU's index (the oracle works on a
calloc-backed full-size host cache in which only the selected rows are filled)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import __graft_entry__ as entry

entry._load_build_module().build()

import oracle
import paper_2606_06467_b200 as clsa
from _harness import (GpuProblem, check_attention, check_scores, check_topk_band, check_topk_exact_on_gpu_scores,
                      oracle_scores_and_topk)
from workloads import HEADLINE, MID, RAGGED, Workload

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg", [MID, HEADLINE, RAGGED], ids=lambda c: c.name)
def test_full_size_decode_step(cfg):
    w = Workload(cfg)
    g = GpuProblem(w)
    prob, ref_scores, ref_idx, ref_cnt = oracle_scores_and_topk(w)
    # the step as the bench runs it
    outs = g.decode_step()
    torch.cuda.synchronize()
    assert g.status() == 0
    idx_np, cnt_np = g.idx.cpu().numpy().copy(), g.count.cpu().numpy().copy()
    # scores and selection, completely
    gs = g.index_scores()
    check_scores(gs, ref_scores, w)
    check_topk_exact_on_gpu_scores(prob, gs, g.idx, g.count, w)
    band_rows = check_topk_band(ref_scores, ref_idx, ref_cnt, g.idx, g.count, w)
    print(f"{cfg.name}: rows whose set differs from the fp64 oracle only inside the 1e-3 band: {band_rows}")
    if cfg.planted:
        for b in range(cfg.num_seqs):
            planted = w.planted_positions(b)
            s = ref_scores[b, 0, : w.seq_len[b]]
            tau = np.sort(s)[-cfg.top_k]
            sure = planted[s[planted] > tau * (1 + 1e-3)]
            assert np.isin(sure, idx_np[b, 0]).all()
            assert sure.size >= 0.8 * planted.size
    if cfg.dup_frac:
        # exact-duplicate keys give bit-identical scores, so ties are broken by position on both sides
        src = w.row_source()
        for b in (0, cfg.num_seqs - 1):
            s0, n = int(w.seq_start[b]), int(w.seq_len[b])
            local = src[s0: s0 + n] - s0
            dup = np.nonzero(local != np.arange(n))[0]
            dup = dup[local[local[dup]] == local[dup]]
            sc = gs[b, 0].cpu().numpy()
            np.testing.assert_array_equal(sc[dup].view(np.uint32), sc[local[dup]].view(np.uint32))
    # attention: oracle on the GPU's index
    kc, vc = w.host_kv_sparse(idx_np, cnt_np)
    full = oracle.problem_from_workload(w, k_cache=kc, v_cache=vc)
    for l in sorted({0, 1, cfg.num_layers - 1}):
        mx, mean = check_attention(full, w, l, outs[l], None, idx_np, cnt_np)
        print(f"{cfg.name} layer {l}: max abs err {mx:.2e}, mean abs err {mean:.2e}")
    # the index buffers are the same bytes after the L launches as after the top-k alone
    g2_idx, g2_cnt = g.topk(gs)
    np.testing.assert_array_equal(g2_idx.cpu().numpy(), idx_np)
    np.testing.assert_array_equal(g2_cnt.cpu().numpy(), cnt_np)


def test_full_size_prefill_chunk():
    """Config 5: 131072 cached tokens + a 4096-query causal chunk. The GPU runs the whole chunk; the oracle checks
    64 sampled query rows completely (a query row of a causal chunk is exactly a decode problem whose sequence
    ends at that query) and cheap invariants cover every row."""
    from workloads import PREFILL

    cfg = PREFILL
    w = Workload(cfg)
    g = GpuProblem(w, layers=2)            # queries of layers 0 and 1 stand for "first" and "any other" layer
    T, n, k = cfg.q_per_seq, cfg.ctx, cfg.top_k
    gs = g.index_scores()
    gi, gc = g.topk(gs)
    # the fused routing (scores never materialised) gives the same index, bit for bit
    fi, fc = torch.full_like(gi, -7), torch.full_like(gc, -7)
    clsa.clsa_index_topk(g.params, g.t["q_idx"], fi, fc, g.ws)
    torch.cuda.synchronize()
    assert g.status() == 0 and torch.equal(fc, gc) and torch.equal(fi, gi)
    outs = [g.sparse_attn(l, reverse=l, lse=False)[0] for l in range(2)]
    torch.cuda.synchronize()
    assert g.status() == 0
    # every row: count, range, order, finiteness
    vis = torch.arange(T, device=g.dev) + (n - T + 1)
    assert torch.equal(gc[0].long(), torch.clamp(vis, max=k))
    assert (gi[0, :, 1:] > gi[0, :, :-1]).all() and (gi[0, :, 0] >= 0).all()
    assert (gi[0, :, -1].long() < vis).all()
    for o in outs:
        assert torch.isfinite(o.float()).all()
    # sampled rows against the oracle
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([[0, 1, T - 1, T - 2, 127, 128], rng.integers(0, T, 58)]))
    kidx = w.host_kidx_cache()
    qi = w.q_idx_bits()[0, rows]                                            # [R, d_idx]
    R = rows.size
    seq_len = np.array([w.visible(0, int(t)) for t in rows], dtype=np.int32)
    sub_prob = oracle.Problem(num_seqs=R, num_q_heads=cfg.num_q_heads, num_kv_heads=cfg.num_kv_heads,
                              head_dim=cfg.head_dim, idx_dim=cfg.idx_dim, top_k=k, sm_scale=cfg.sm_scale,
                              seq_start=np.zeros(R, dtype=np.int64), seq_len=seq_len, idx_k_cache=kidx)
    ref_scores = sub_prob.index_scores(qi.reshape(R, 1, -1))
    got_scores = gs[0, torch.from_numpy(rows).to(g.dev)].cpu().numpy().astype(np.float64)
    for i in range(R):
        v = seq_len[i]
        r = ref_scores[i, 0, :v]
        assert (np.abs(got_scores[i, :v] - r) <= 1e-4 * np.maximum(1.0, np.abs(r))).all()
        assert np.isnan(got_scores[i, v:n]).all()
    ref_idx, ref_cnt = sub_prob.topk(ref_scores)
    gpu_idx = gi[0, torch.from_numpy(rows).to(g.dev)].cpu().numpy()
    exact_idx, _ = sub_prob.topk(np.where(np.isnan(got_scores), -np.inf, got_scores)[:, None, : ref_scores.shape[2]])
    band = 0
    for i in range(R):
        np.testing.assert_array_equal(gpu_idx[i], np.sort(exact_idx[i, 0]))      # exact on the GPU's own scores
        a, b = set(gpu_idx[i].tolist()), set(ref_idx[i, 0].tolist())
        if a != b:
            s = ref_scores[i, 0, : seq_len[i]]
            tau = np.sort(s)[-k]
            diff = np.array(sorted(a ^ b))
            assert (np.abs(s[diff] - tau) <= 1e-3 * abs(tau)).all()
            band += 1
    print(f"prefill: sampled rows differing from the fp64 oracle inside the band only: {band} of {R}")
    # attention of the sampled rows, oracle fed the GPU's index
    idx_s = gpu_idx.reshape(R, 1, k)
    cnt_s = np.minimum(seq_len, k).reshape(R, 1).astype(np.int32)
    kc = np.zeros((w.total_rows, cfg.num_kv_heads, cfg.head_dim), dtype=np.uint16)
    vc = np.zeros_like(kc)
    touched = np.unique(idx_s)
    kc[touched] = w.kv_rows_bits("k", touched).reshape(-1, cfg.num_kv_heads, cfg.head_dim)
    vc[touched] = w.kv_rows_bits("v", touched).reshape(-1, cfg.num_kv_heads, cfg.head_dim)
    att_prob = oracle.Problem(num_seqs=R, num_q_heads=cfg.num_q_heads, num_kv_heads=cfg.num_kv_heads,
                              head_dim=cfg.head_dim, idx_dim=cfg.idx_dim, top_k=k, sm_scale=cfg.sm_scale,
                              seq_start=np.zeros(R, dtype=np.int64), seq_len=seq_len, k_cache=kc, v_cache=vc)
    for l in range(2):
        q = w.q_layer_bits(l)[0, rows].reshape(R, 1, cfg.num_q_heads, cfg.head_dim)
        o_ref, _ = att_prob.sparse_attn(q, idx_s, cnt_s)
        got = outs[l][0, torch.from_numpy(rows).to(g.dev)].float().cpu().numpy().astype(np.float64)
        err = np.abs(got - o_ref[:, 0])
        assert err.max() <= 2e-2 and err.mean() <= 2e-3
        print(f"prefill layer {l}: max abs err {err.max():.2e}, mean abs err {err.mean():.2e}")
