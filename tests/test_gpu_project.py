"""clsa_project_append (Eq. 2 and the cache append) against the oracle.

Tolerance: the oracle's sum is exact in fp64; the GPU accumulates d_model bf16 x bf16 products in fp32 on the
tensor cores (at most about d_model/16 * 2^-23 relative to the running sum, a few 1e-5 here) and rounds once to
bf16 (half an ulp = 2^-8 relative at most). So |gpu - exact| <= 2^-8 |exact| + 1e-4, and against the oracle's own
bf16 rounding the two may disagree only by one step of the bf16 grid, next to a rounding tie of the exact value
(checked where the grid step, 2^-8 |exact| or more, is far above the fp32 error: |exact| >= 1/16)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import __graft_entry__ as entry

entry._load_build_module().build()

import oracle
import paper_2606_06467_b200 as clsa
from _harness import GpuProblem, check_scores, check_topk_exact_on_gpu_scores
from workloads import MID, RAGGED, TINY, Workload
from workloads import generator as g

pytestmark = pytest.mark.gpu

ABS_TOL, REL_TOL = 1e-4, 2.0 ** -8


def bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def run_gpu(gp, proj, with_kv=True):
    c = gp.cfg
    q = torch.full((c.num_seqs, c.q_per_seq, c.idx_dim), float("nan"), dtype=torch.bfloat16, device=gp.dev)
    clsa.clsa_project_append(gp.params, c.d_model, proj["h"], proj["w_q_idx"], proj["w_k_idx"],
                             proj["w_k"] if with_kv else None, proj["w_v"] if with_kv else None, q,
                             gp.t["idx_k_cache"], gp.t["k_cache"] if with_kv else None,
                             gp.t["v_cache"] if with_kv else None, gp.ws)
    torch.cuda.synchronize()
    return q


def target_rows(w, block_size=0):
    c = w.cfg
    rows = np.empty((c.num_seqs, c.q_per_seq), dtype=np.int64)
    table = w.block_table(block_size)[0] if block_size else None
    for b in range(c.num_seqs):
        for t in range(c.q_per_seq):
            s = int(w.seq_len[b]) - c.q_per_seq + t
            rows[b, t] = (int(table[b, s // block_size]) * block_size + s % block_size) if block_size else int(w.seq_start[b]) + s
    return rows


def compare(got_bits, exact):
    """got_bits uint16 [..], exact float64 [..] (the unrounded product)."""
    got = g.bf16_bits_to_f64(got_bits)
    assert np.isfinite(got).all()
    err = np.abs(got - exact)
    assert (err <= REL_TOL * np.abs(exact) + ABS_TOL).all(), float(err.max())
    want_bits = oracle.round_bf16(exact)
    diff = got_bits != want_bits
    assert diff.mean() < 0.02, float(diff.mean())
    big = diff & (np.abs(exact) >= 1.0 / 16)
    if big.any():  # a disagreement is one step on the bf16 grid, next to a tie of the exact value
        assert (np.abs(got_bits[big].astype(np.int32) - want_bits[big].astype(np.int32)) == 1).all()
    return float(diff.mean())


CASES = [
    (TINY.replace(ctx=700, top_k=64, num_layers=1), 0),                                        # 1 row: a ragged row tile
    (MID.replace(num_seqs=8, ctx=900, top_k=64, num_layers=1), 0),
    (MID.replace(num_seqs=16, ctx=515, top_k=64, num_layers=1), 0),                            # the headline's batch
    (MID.replace(num_seqs=20, ctx=300, top_k=64, num_layers=1, num_q_heads=20, num_kv_heads=4), 0),  # two row tiles, 4 KV heads
    (RAGGED.replace(num_seqs=37, ctx=1200, ragged_min=64, num_short=2, top_k=96, num_layers=1), 0),  # packed ragged rows
    (RAGGED.replace(num_seqs=70, ctx=400, ragged_min=64, num_short=2, top_k=96, num_layers=1), 16),  # two row blocks, paged
    (MID.replace(num_seqs=2, ctx=600, q_per_seq=50, causal=1, top_k=64, num_layers=1, d_model=1056), 32),  # T > 1, paged
]


@pytest.mark.parametrize("cfg,bs", CASES, ids=["tiny", "b8", "b16", "b20-heads20/4", "ragged37", "ragged70-paged", "chunk-paged"])
def test_project_append_matches_oracle(cfg, bs):
    w = Workload(cfg)
    c = w.cfg
    gp = GpuProblem(w, block_size=bs)
    proj = w.projection_to_device(gp.dev)
    before = {n: gp.t[n].clone() for n in ("idx_k_cache", "k_cache", "v_cache")}
    q = run_gpu(gp, proj)
    assert gp.status() == 0
    h = g.bf16_bits_to_f64(w.hidden_bits()).reshape(c.num_seqs * c.q_per_seq, c.d_model)
    hb = w.hidden_bits().reshape(-1, c.d_model)
    rows = target_rows(w, bs).reshape(-1)
    rows_t = torch.from_numpy(rows).to(gp.dev)
    compare(bits(q).reshape(len(rows), -1), oracle.linear(hb, w.weight_bits("q_idx")))
    compare(bits(gp.t["idx_k_cache"][rows_t]), oracle.linear(hb, w.weight_bits("k_idx")))
    compare(bits(gp.t["k_cache"][rows_t]).reshape(len(rows), -1), oracle.linear(hb, w.weight_bits("k")))
    compare(bits(gp.t["v_cache"][rows_t]).reshape(len(rows), -1), oracle.linear(hb, w.weight_bits("v")))
    # nothing but the target rows changed
    keep = torch.ones(gp.t["idx_k_cache"].shape[0], dtype=torch.bool, device=gp.dev)
    keep[rows_t] = False
    for n in before:
        assert torch.equal(gp.t[n][keep].view(torch.int16), before[n][keep].view(torch.int16)), n
    assert len(set(rows.tolist())) == len(rows)
    del h


def test_selector_weights_reproduce_components_of_h_exactly():
    """With 0/1 weights every sum has one term: the result must be the chosen element of h, bit for bit, at the
    right feature of the right matrix (operand order, KV-head layout, the k-permutation inside the MMAs)."""
    cfg = MID.replace(num_seqs=5, ctx=260, top_k=32, num_layers=1, d_model=2560)
    w = Workload(cfg)
    c = w.cfg
    gp = GpuProblem(w)
    proj = w.projection_to_device(gp.dev)
    rng = np.random.default_rng(7)
    cols = {}
    for name, n_out in (("w_q_idx", c.idx_dim), ("w_k_idx", c.idx_dim), ("w_k", c.num_kv_heads * c.head_dim),
                        ("w_v", c.num_kv_heads * c.head_dim)):
        pick = rng.permutation(c.d_model)[:n_out]
        cols[name] = pick
        sel = torch.zeros((n_out, c.d_model), dtype=torch.bfloat16, device=gp.dev)
        sel[torch.arange(n_out, device=gp.dev), torch.from_numpy(pick).to(gp.dev)] = 1.0
        proj[name] = sel
    q = run_gpu(gp, proj)
    hb = w.hidden_bits().reshape(c.num_seqs, c.d_model)
    rows = torch.from_numpy(target_rows(w).reshape(-1)).to(gp.dev)
    np.testing.assert_array_equal(bits(q).reshape(c.num_seqs, -1), hb[:, cols["w_q_idx"]])
    np.testing.assert_array_equal(bits(gp.t["idx_k_cache"][rows]), hb[:, cols["w_k_idx"]])
    np.testing.assert_array_equal(bits(gp.t["k_cache"][rows]).reshape(c.num_seqs, -1), hb[:, cols["w_k"]])
    np.testing.assert_array_equal(bits(gp.t["v_cache"][rows]).reshape(c.num_seqs, -1), hb[:, cols["w_v"]])


def test_indexer_branch_only_leaves_k_and_v_alone_and_is_deterministic():
    w = Workload(MID.replace(num_seqs=16, ctx=300, top_k=32, num_layers=1))
    gp = GpuProblem(w)
    proj = w.projection_to_device(gp.dev)
    k0, v0 = gp.t["k_cache"].clone(), gp.t["v_cache"].clone()
    q1 = run_gpu(gp, proj, with_kv=False)
    assert torch.equal(gp.t["k_cache"].view(torch.int16), k0.view(torch.int16))
    assert torch.equal(gp.t["v_cache"].view(torch.int16), v0.view(torch.int16))
    kidx1 = gp.t["idx_k_cache"].clone()
    q2 = run_gpu(gp, proj, with_kv=True)
    assert torch.equal(q1.view(torch.int16), q2.view(torch.int16))
    assert torch.equal(kidx1.view(torch.int16), gp.t["idx_k_cache"].view(torch.int16))


def test_appended_rows_feed_the_rest_of_the_path():
    """project -> index scores -> top-k on the GPU; the oracle scores the GPU's own projected query against the
    GPU's own cache, so the check isolates 'the later kernels see the appended row'."""
    w = Workload(MID.replace(num_seqs=4, ctx=3000, top_k=128, num_layers=2))
    c = w.cfg
    gp = GpuProblem(w)
    proj = w.projection_to_device(gp.dev)
    q = run_gpu(gp, proj)
    gp.t["q_idx"] = q
    scores = gp.index_scores()
    idx, cnt = gp.topk(scores)
    torch.cuda.synchronize()
    prob = oracle.problem_from_workload(w, idx_k_cache=bits(gp.t["idx_k_cache"]))
    ref = prob.index_scores(bits(q))
    check_scores(scores, ref, w)
    check_topk_exact_on_gpu_scores(prob, scores, idx, cnt, w)
    # the newest token's score is q . k of the two freshly projected rows
    hb = w.hidden_bits().reshape(c.num_seqs, c.d_model)
    for b in range(c.num_seqs):
        qe = g.bf16_bits_to_f64(oracle.round_bf16(oracle.linear(hb[b: b + 1], w.weight_bits("q_idx"))))[0]
        ke = g.bf16_bits_to_f64(oracle.round_bf16(oracle.linear(hb[b: b + 1], w.weight_bits("k_idx"))))[0]
        got = float(scores[b, 0, int(w.seq_len[b]) - 1])
        assert abs(got - float(qe @ ke)) <= 0.05 * max(1.0, abs(float(qe @ ke)))  # one-ulp input differences allowed
    outs = gp.decode_step()
    torch.cuda.synchronize()
    assert gp.status() == 0 and all(torch.isfinite(o.float()).all() for o in outs)


def test_bad_sequence_length_is_flagged_not_written():
    w = Workload(MID.replace(num_seqs=3, ctx=200, top_k=32, num_layers=1))
    gp = GpuProblem(w)
    proj = w.projection_to_device(gp.dev)
    gp.t["seq_len"][1] = 0
    before = gp.t["idx_k_cache"].clone()
    run_gpu(gp, proj)
    assert gp.status() & clsa.CLSA_DEV_BAD_SEQLEN
    rows = target_rows(w).reshape(-1)
    changed = (gp.t["idx_k_cache"].view(torch.int16) != before.view(torch.int16)).any(dim=1).nonzero().flatten().cpu().numpy()
    assert set(changed.tolist()) == {int(rows[0]), int(rows[2])}
    clsa.clsa_clear_status(gp.ws)
