"""Seeded random shapes through every entry point against the oracle: head layouts, indexer widths, decode and chunk
launches, ragged lengths, duplicates, contiguous and paged caches, budgets from 1 to beyond the context. Each case
checks the scores, the exact selection on the GPU's own scores, the band rule against the oracle's scores, every layer in
the three launch shapes, the chained call against the separate calls, and (chunks) the fused routing against the
materialising pair bit for bit."""
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

HEADS = [(8, 1), (32, 8), (20, 4), (16, 2), (32, 2), (5, 5), (32, 16), (16, 16), (48, 3)]


def _draw(seed):
    rng = np.random.default_rng(seed)
    hq, hkv = HEADS[rng.integers(len(HEADS))]
    d_idx = int(rng.choice([64, 128]))
    T = int(rng.choice([1, 1, 1, 200, 640]))
    B = int(rng.integers(1, 9 if T == 1 else 2))
    n = int(rng.integers(max(T, 1), 30000 if T == 1 else int(rng.choice([9000, 30000, 70000])))) + T
    k = int(rng.choice([1, 16, 17, 100, 256, 777, 2048, 5000]))
    ragged = bool(rng.integers(2)) and B > 1
    bs = int(rng.choice([0, 0, 16, 64, 256]))
    L = int(rng.integers(1, 4))
    kw = dict(num_seqs=B, ctx=n, q_per_seq=T, causal=int(T > 1 and rng.integers(2)), top_k=k, num_layers=L, num_q_heads=hq,
              num_kv_heads=hkv, seed=int(rng.integers(1 << 30)), idx_dim=d_idx, dup_frac=float(rng.choice([0.0, 0.0, 0.2])))
    if ragged:
        kw.update(ragged_min=max(T, min(n, int(rng.integers(1, 300)))), num_short=0)
    return (MID if d_idx == 128 else TINY).replace(**kw), bs


@pytest.mark.parametrize("seed", list(range(100, 116)))
def test_random_shape(seed):
    cfg, bs = _draw(seed)
    T, L = cfg.q_per_seq, cfg.num_layers
    w = Workload(cfg)
    g = GpuProblem(w, block_size=bs)
    kc, vc = w.host_kv_full()
    prob = oracle.problem_from_workload(w, k_cache=kc, v_cache=vc, idx_k_cache=w.host_kidx_cache())
    ref = prob.index_scores(w.q_idx_bits())
    gs = g.index_scores()
    check_scores(gs, ref, w)
    gi, gc = g.topk(gs)
    check_topk_exact_on_gpu_scores(prob, gs, gi, gc, w)
    ri, rc = prob.topk(ref)
    check_topk_band(ref, ri, rc, gi, gc, w)
    if T > 1:
        fi, fc = torch.full_like(gi, -7), torch.full_like(gc, -7)
        clsa.clsa_index_topk(g.params, g.t["q_idx"], fi, fc, g.ws)
        torch.cuda.synchronize()
        assert g.status() == 0
        assert torch.equal(fc, gc) and torch.equal(fi, gi)
    idx_np, cnt_np = gi.cpu().numpy().copy(), gc.cpu().numpy().copy()
    singles = []
    for l in range(L):
        out, lse = g.sparse_attn(l, reverse=l & 1, keep_rows=1, only_q_pending=int(l > 0))
        check_attention(prob, w, l, out, lse, idx_np, cnt_np)
        pair = []
        for shape in (1, 2, 3, 4):
            o, s = g.sparse_attn(l, shared_gpu=shape)
            check_attention(prob, w, l, o, s, idx_np, cnt_np)
            pair.append(o)
        singles.append(pair)
    if T == 1:
        outs = g.decode_step()
        torch.cuda.synchronize()
        for l in range(L):
            rows = outs[l].shape[0] * outs[l].shape[1]
            a, b1, b2, b3, b4 = (x.reshape(rows, -1).view(torch.int16) for x in [outs[l]] + singles[l])
            same = (a == b1).all(dim=1) | (a == b2).all(dim=1) | (a == b3).all(dim=1) | (a == b4).all(dim=1)
            assert bool(same.all()), "chain differs from the separate calls"
    assert g.status() == 0
