"""Top-k on many long rows (the prefill-chunk route: one-sweep kernel + general kernel for the rows it hands back).

The selection is integer work: the GPU's index must equal, bit for bit, the oracle's TopK of the same fp32 scores,
whichever of the two kernels finished the row. The score matrices below are built so that both kernels get work:
i.i.d. rows (the one-sweep kernel finishes them), and rows that defeat its sampled pivot or overflow its candidate
list (runs of equal scores, two-valued rows, clustered maxima, quantised tails with ties at the threshold)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import __graft_entry__ as entry

entry._load_build_module().build()

import oracle
import paper_2606_06467_b200 as clsa
from _harness import GpuProblem, check_scores, check_topk_band, check_topk_exact_on_gpu_scores
from workloads import MID, RAGGED, Workload

pytestmark = pytest.mark.gpu

ROWS = 640  # more than 4 x 148 rows: the many-rows route


def crafted_rows(rng, rows, n, k):
    """float32 [rows, n]: eleven kinds of row, cycling."""
    x = rng.standard_normal((rows, n)).astype(np.float32) * 11.3
    pos = np.arange(n)
    for r in range(rows):
        kind = r % 11
        if kind == 1:
            x[r] = 3.25                                            # all equal
        elif kind == 2:
            x[r] = np.round(x[r] / 4) * 4                          # coarse grid: ties everywhere
        elif kind == 3:
            x[r] = pos.astype(np.float32)                          # increasing
        elif kind == 4:
            x[r] = -pos.astype(np.float32)                         # decreasing
        elif kind == 5:
            x[r] = 0.0
            x[r, ::100] = 1.0                                      # two values, threshold inside the zeros
        elif kind == 6:
            hi = x[r] > 17.0
            x[r, hi] = np.round(x[r, hi] * 2) / 2                  # quantised tail: ties at the threshold
        elif kind == 7:
            x[r] = np.abs(x[r]) * 1e-3
            start = int(rng.integers(0, n - k))
            x[r, start:start + k // 2] += 50.0                     # half of the answer in one contiguous run
        elif kind == 8:
            x[r] = -np.abs(x[r]) - 1.0                             # all negative
            x[r, rng.integers(0, n, 5)] = -0.0
        elif kind == 9:
            x[r] = np.exp(x[r] / 4)                                # heavy right tail
        elif kind == 10:
            x[r] = x[r] * 1e-30                                    # tiny magnitudes (low exponents)
    return x


@pytest.mark.parametrize("n,k", [(20000, 2048), (7001, 512), (50000, 2048), (9000, 4096)])
def test_many_rows_on_crafted_scores(n, k):
    w = Workload(MID.replace(num_seqs=1, ctx=n, q_per_seq=ROWS, causal=0, top_k=k, num_layers=1))
    g = GpuProblem(w, layers=1)
    rng = np.random.default_rng(n + k)
    sc = torch.full((1, ROWS, g.score_stride), float("nan"), dtype=torch.float32, device=g.dev)
    sc[0, :, :n] = torch.from_numpy(crafted_rows(rng, ROWS, n, k)).to(g.dev)
    gi, gc = g.topk(sc)
    torch.cuda.synchronize()
    assert g.status() == 0
    prob = oracle.problem_from_workload(w)
    check_topk_exact_on_gpu_scores(prob, sc, gi, gc, w)
    first = gi.clone()
    gi2, _ = g.topk(sc)
    assert torch.equal(first, gi2)


def test_many_rows_causal_chunk_against_oracle():
    """Scores from the chunk GEMM, causal rows of different visible lengths."""
    cfg = MID.replace(num_seqs=1, ctx=9000 + ROWS, q_per_seq=ROWS, causal=1, top_k=512, num_layers=1, seed=4242)
    w = Workload(cfg)
    g = GpuProblem(w, layers=1)
    prob = oracle.problem_from_workload(w, idx_k_cache=w.host_kidx_cache())
    ref = prob.index_scores(w.q_idx_bits())
    gs = g.index_scores()
    check_scores(gs, ref, w)
    gi, gc = g.topk(gs)
    torch.cuda.synchronize()
    assert g.status() == 0
    check_topk_exact_on_gpu_scores(prob, gs, gi, gc, w)
    ri, rc = prob.topk(ref)
    check_topk_band(ref, ri, rc, gi, gc, w)


def test_many_rows_ragged_sequences_short_and_long():
    """Several sequences per chunk: rows shorter than k (everything selected), rows that fit the candidate list
    whole, and long rows, in one launch."""
    cfg = RAGGED.replace(num_seqs=4, ctx=14000, ragged_min=300, num_short=1, q_per_seq=160, causal=1, top_k=1024,
                         num_layers=1, dup_frac=0.05, seed=77)
    w = Workload(cfg)
    lens = sorted(int(x) for x in w.seq_len)
    assert lens[0] < 1024 + 160 and lens[-1] > 6144 + 160, lens
    g = GpuProblem(w, layers=1)
    prob = oracle.problem_from_workload(w, idx_k_cache=w.host_kidx_cache())
    gs = g.index_scores()
    gi, gc = g.topk(gs)
    torch.cuda.synchronize()
    assert g.status() == 0
    check_topk_exact_on_gpu_scores(prob, gs, gi, gc, w)


def test_many_rows_misaligned_rows_and_non_finite_scores_keep_the_contract():
    n, k = 12000, 700
    w = Workload(MID.replace(num_seqs=1, ctx=n, q_per_seq=ROWS, causal=0, top_k=k, num_layers=1))
    g = GpuProblem(w, layers=1)
    rng = np.random.default_rng(5)
    stride = n + 1                                   # odd stride: most rows are not 16-byte aligned
    sc = torch.from_numpy(rng.standard_normal((1, ROWS, stride)).astype(np.float32)).to(g.dev)
    clsa.clsa_topk(g.params, sc, stride, g.idx, g.count, g.ws)
    prob = oracle.problem_from_workload(w)
    check_topk_exact_on_gpu_scores(prob, sc, g.idx, g.count, w)
    g2 = GpuProblem(w, layers=1)
    sc2 = torch.from_numpy(rng.standard_normal((1, ROWS, g2.score_stride)).astype(np.float32)).to(g.dev)
    sc2[0, ::3, ::7] = float("nan")
    sc2[0, 1::3, ::5] = float("inf")
    sc2[0, 1::3, 1::5] = float("-inf")
    gi, gc = g2.topk(sc2)
    torch.cuda.synchronize()
    assert g2.status() == 0
    gi, gc = gi.cpu().numpy(), gc.cpu().numpy()
    assert (gc == k).all()
    assert (np.diff(gi[0], axis=1) > 0).all() and (gi[0, :, 0] >= 0).all() and (gi[0, :, -1] < n).all()
    assert np.isin(gi[0, 1::3], np.arange(0, n, 5)).all()   # +inf outranks every finite score
    finite_rows = torch.arange(2, ROWS, 3, device=g.dev)      # rows without NaN/inf: exact against the oracle
    sub = Workload(MID.replace(num_seqs=1, ctx=n, q_per_seq=len(finite_rows), causal=0, top_k=k, num_layers=1))
    check_topk_exact_on_gpu_scores(oracle.problem_from_workload(sub), sc2[:, finite_rows], g2.idx[:, finite_rows],
                                   g2.count[:, finite_rows], sub)


@pytest.mark.parametrize("B,k,n_max", [(ROWS, 800, 16000), (40, 2048, 131072), (64, 2048, 100000), (150, 512, 40000),
                                       (34, 4096, 131072), (48, 3000, 131072)],
                         ids=["640x16000", "40x131072", "64x100000", "150x40000", "34x131072-k4096", "48x131072-k3000"])
def test_many_sequences_one_query_each(B, k, n_max):
    """The same route when the rows are sequences of different lengths (a decode batch), not the queries of one
    chunk: 640 rows, and batches just large enough that their clusters would not all be resident at once (the
    one-sweep kernel takes those too, unless k is so large that its candidate list would overflow: k = 4096 of
    131072 stays with the cluster kernel). Selection only, on random scores, against the oracle's sort."""
    rng = np.random.default_rng(99 + B)
    lens = rng.integers(500, n_max + 1, B).astype(np.int32)
    lens[:3] = (n_max, k - 1, 6145)                    # longest, shorter than k, just above the candidate list's capacity
    dev = torch.device("cuda:0")
    stride = (n_max + 63) // 64 * 64
    sc_host = (rng.standard_normal((B, 1, stride)) * 11.3).astype(np.float32)
    sc = torch.from_numpy(sc_host).to(dev)
    seq_len = torch.from_numpy(lens).to(dev)
    seq_start = torch.zeros(B, dtype=torch.int64, device=dev)
    kv = torch.zeros((8, 8, 128), dtype=torch.bfloat16, device=dev)
    ik = torch.zeros((8, 128), dtype=torch.bfloat16, device=dev)
    p = clsa.make_params(num_seqs=B, q_per_seq=1, num_q_heads=32, num_kv_heads=8, head_dim=128, idx_dim=128, top_k=k,
                         num_layers=1, max_seq_len=n_max, sm_scale=0.1, seq_start=seq_start, seq_len=seq_len, k_cache=kv,
                         v_cache=kv, idx_k_cache=ik)
    ws = torch.zeros(clsa.clsa_workspace_bytes(p), dtype=torch.uint8, device=dev)
    idx = torch.full((B, 1, k), -7, dtype=torch.int32, device=dev)
    cnt = torch.full((B, 1), -7, dtype=torch.int32, device=dev)
    clsa.clsa_topk(p, sc, stride, idx, cnt, ws)
    torch.cuda.synchronize()
    assert clsa.clsa_device_status(ws) == 0
    prob = oracle.Problem(num_seqs=B, q_per_seq=1, num_q_heads=32, num_kv_heads=8, head_dim=128, idx_dim=128, top_k=k,
                          sm_scale=0.1, seq_start=np.zeros(B, np.int64), seq_len=lens)
    ref_idx, ref_cnt = prob.topk(sc_host.astype(np.float64))
    gi, gc = idx.cpu().numpy(), cnt.cpu().numpy()
    np.testing.assert_array_equal(gc, ref_cnt)
    for b in range(B):
        c = gc[b, 0]
        np.testing.assert_array_equal(gi[b, 0, :c], np.sort(ref_idx[b, 0, :c]))
        assert (gi[b, 0, c:] == -1).all()
