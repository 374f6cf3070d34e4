"""Pins for the CPU oracle: every function is checked against something other than itself.

What pins what (a plausible slip in the oracle -- a dropped term, a wrong sign or index, a
transposed operand, a wrong head mapping -- fails at least one of these):
  scores  : numpy float64 matmul (library routine), unit-vector / self / zero closed forms,
            causal visibility counts, the hand example (Eq. 3).
  TopK    : two independently written selectors, Python's sorted() as brute force on tiny inputs,
            closed-form special cases, order-theoretic invariants on random inputs (Eq. 3).
  attention: scipy softmax + numpy einsum (library), the independent dense routine for k >= n
            (Eq. 1 vs Eq. 4), closed forms (uniform logits, constant V, single token, dominant
            logit), invariances (permutation, logit shift, GQA grouping), the hand example.
  chain   : one index reused by all layers; decode_step == the separate calls.
  projections + append (Eq. 2): the rounding against every bf16 value, constructed ties, a double-rounding
            trap and torch's float32 -> bf16 conversion (library); the product against numpy float64 matmul
            with asymmetric shapes; selector weights (a projected row must reproduce chosen components
            of h exactly, which fixes operand order and the [Hkv][D] layout); untouched rows stay
            byte-identical; contiguous and paged placement; the newest token's score in closed form.
"""
import json
import math
import os

import numpy as np
import pytest
from scipy.special import logsumexp, softmax

import oracle
from workloads import generator as g

GOLD = os.path.join(os.path.dirname(__file__), "golden", "hand_example.json")


def bf16(x):
    return g.f64_to_bf16_bits(np.asarray(x, dtype=np.float64))


def f64(bits):
    return g.bf16_bits_to_f64(bits)


def rand_bits(rng, shape, scale=1.0):
    return bf16(rng.standard_normal(shape) * scale)


def make_problem(rng, B=2, T=1, Hq=4, Hkv=2, D=8, d_idx=6, k=5, lens=(9, 13), causal=0, sm_scale=None, pad=3):
    lens = np.asarray(lens, dtype=np.int32)
    starts = np.zeros(B, dtype=np.int64)
    acc = 2
    for b in range(B):
        starts[b] = acc
        acc += int(lens[b]) + pad
    rows = acc + 1
    kc, vc = rand_bits(rng, (rows, Hkv, D)), rand_bits(rng, (rows, Hkv, D))
    ik = rand_bits(rng, (rows, d_idx))
    p = oracle.Problem(num_seqs=B, q_per_seq=T, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, idx_dim=d_idx,
                       top_k=k, causal=causal, sm_scale=(1 / math.sqrt(D) if sm_scale is None else sm_scale),
                       seq_start=starts, seq_len=lens, k_cache=kc, v_cache=vc, idx_k_cache=ik)
    return p


# ======================================================================================= scores
def test_scores_match_numpy_matmul():
    rng = np.random.default_rng(1)
    for causal, T in ((0, 1), (1, 4), (0, 3)):
        p = make_problem(rng, B=3, T=T, lens=(17, 5, 31), d_idx=7, causal=causal)
        q = rand_bits(rng, (p.B, p.T, p.d_idx))
        got = p.index_scores(q)
        for b in range(p.B):
            keys = f64(p.idx_k_cache[p.seq_start[b]: p.seq_start[b] + p.seq_len[b]])
            ref = f64(q[b]) @ keys.T  # [T, n]
            for t in range(T):
                v = p.seq_len[b] - T + t + 1 if causal else p.seq_len[b]
                np.testing.assert_allclose(got[b, t, :v], ref[t, :v], rtol=1e-14, atol=1e-14)
                assert np.isnan(got[b, t, v:]).all(), "positions past the visible prefix must not be scored"


def test_scores_closed_forms():
    rng = np.random.default_rng(2)
    d = 8
    q = rand_bits(rng, (1, 1, d))
    rows = np.zeros((d + 2, d), dtype=np.uint16)
    for j in range(d):
        rows[j, j] = bf16(1.0)          # unit vector e_j -> score q[j]
    rows[d] = q[0, 0]                   # the query itself -> |q|^2
    rows[d + 1] = bf16(np.zeros(d))     # zero row -> 0
    p = oracle.Problem(num_seqs=1, num_q_heads=1, num_kv_heads=1, head_dim=2, idx_dim=d, top_k=1, sm_scale=1.0,
                       seq_start=[0], seq_len=[d + 2], idx_k_cache=rows)
    s = p.index_scores(q)[0, 0]
    np.testing.assert_array_equal(s[:d], f64(q[0, 0]))
    assert s[d] == float((f64(q[0, 0]) ** 2).sum())
    assert s[d + 1] == 0.0
    zero = p.index_scores(bf16(np.zeros((1, 1, d))))[0, 0]
    assert (zero == 0.0).all()


def test_scores_linearity_and_no_scaling():
    # scores(2 q) = 2 scores(q) exactly (power-of-two scaling is exact in bf16): there is no hidden
    # normalisation, activation or 1/sqrt(d) whose effect would depend on |q|.
    rng = np.random.default_rng(3)
    p = make_problem(rng, B=1, lens=(40,), d_idx=16)
    q = rand_bits(rng, (1, 1, 16))
    q2 = bf16(2.0 * f64(q))
    np.testing.assert_array_equal(p.index_scores(q2), 2.0 * p.index_scores(q))
    qn = bf16(-f64(q))
    np.testing.assert_array_equal(p.index_scores(qn), -p.index_scores(q))


def test_hand_example_scores_and_topk():
    gold = json.load(open(GOLD))["index"]
    p = oracle.Problem(num_seqs=1, num_q_heads=1, num_kv_heads=1, head_dim=2, idx_dim=2, top_k=2, sm_scale=1.0,
                       seq_start=[0], seq_len=[5], idx_k_cache=bf16(gold["k_idx"]))
    s = p.index_scores(bf16(gold["q_idx"]).reshape(1, 1, 2))
    np.testing.assert_array_equal(s[0, 0], np.array(gold["scores"], dtype=np.float64))
    for k, want in gold["topk"].items():
        pk = oracle.Problem(num_seqs=1, num_q_heads=1, num_kv_heads=1, head_dim=2, idx_dim=2, top_k=int(k),
                            sm_scale=1.0, seq_start=[0], seq_len=[5], idx_k_cache=bf16(gold["k_idx"]))
        for sel in ("sort", "select"):
            idx, cnt = pk.topk(s, selector=sel)
            assert cnt[0, 0] == len(want)
            got = idx[0, 0, : cnt[0, 0]]
            if sel == "sort":
                assert got.tolist() == want          # rank order: score descending, index ascending
            assert sorted(got.tolist()) == sorted(want)
            assert (idx[0, 0, cnt[0, 0]:] == -1).all()


# ======================================================================================= TopK
def _topk_problem(n, k, T=1, causal=0, B=1):
    return oracle.Problem(num_seqs=B, q_per_seq=T, num_q_heads=1, num_kv_heads=1, head_dim=2, idx_dim=2, top_k=k,
                          causal=causal, sm_scale=1.0, seq_start=np.arange(B) * n, seq_len=[n] * B)


def _sets(idx, cnt):
    return [sorted(idx[b, t, : cnt[b, t]].tolist()) for b in range(idx.shape[0]) for t in range(idx.shape[1])]


def test_topk_brute_force_tiny():
    rng = np.random.default_rng(4)
    for n in range(1, 9):
        for k in range(1, 10):
            for trial in range(6):
                sc = rng.integers(-2, 3, size=(1, 1, n)).astype(np.float64)  # many ties
                p = _topk_problem(n, k)
                want = sorted(sorted(range(n), key=lambda s: (-sc[0, 0, s], s))[:k])
                for sel in ("sort", "select"):
                    idx, cnt = p.topk(sc, selector=sel)
                    assert cnt[0, 0] == min(n, k)
                    assert _sets(idx, cnt)[0] == want, (n, k, sel, sc)


def test_topk_special_cases():
    n, k = 50, 7
    p = _topk_problem(n, k)
    for sel in ("sort", "select"):
        idx, cnt = p.topk(np.full((1, 1, n), 3.25), selector=sel)
        assert _sets(idx, cnt)[0] == list(range(k))                       # all equal -> lowest indices
        idx, cnt = p.topk(np.arange(n, dtype=np.float64).reshape(1, 1, n), selector=sel)
        assert _sets(idx, cnt)[0] == list(range(n - k, n))                # increasing -> the last k
        sc = np.where(np.arange(n) % 10 == 9, 1.0, 0.0).reshape(1, 1, n)  # 5 ones, the rest zeros
        idx, cnt = p.topk(sc, selector=sel)
        assert _sets(idx, cnt)[0] == sorted([9, 19, 29, 39, 49] + [0, 1])  # then the lowest-index zeros
        sc = np.zeros((1, 1, n)); sc[0, 0, 0] = -0.0; sc[0, 0, 1:] = -1.0; sc[0, 0, 30] = 0.0
        p1 = _topk_problem(n, 1)
        idx, cnt = p1.topk(sc, selector=sel)
        assert idx[0, 0, 0] == 0                                          # -0.0 ties with +0.0, lower index wins
        sc = np.zeros((1, 1, n)); sc[0, 0, 17] = 5.0; sc[0, 0, 33] = 5.0
        idx, cnt = p1.topk(sc, selector=sel)
        assert idx[0, 0, 0] == 17                                         # k = 1 -> first arg-max
        pbig = _topk_problem(n, n + 13)
        idx, cnt = pbig.topk(np.random.default_rng(0).standard_normal((1, 1, n)), selector=sel)
        assert cnt[0, 0] == n and _sets(idx, cnt)[0] == list(range(n))    # k >= n -> everything
        assert (idx[0, 0, n:] == -1).all()


def test_topk_two_selectors_agree_and_invariants():
    rng = np.random.default_rng(5)
    for n, k, quant in ((1000, 64, None), (777, 100, 0.25), (4096, 256, None), (300, 299, 1.0), (64, 64, 0.5)):
        B, T = 3, 2
        sc = rng.standard_normal((B, T, n))
        if quant:
            sc = np.round(sc / quant) * quant
        p = _topk_problem(n, k, T=T, causal=1, B=B)
        i0, c0 = p.topk(sc, selector="sort")
        i1, c1 = p.topk(sc, selector="select")
        np.testing.assert_array_equal(c0, c1)
        assert _sets(i0, c0) == _sets(i1, c1)
        for b in range(B):
            for t in range(T):
                v = n - T + t + 1
                c = c0[b, t]
                assert c == min(k, v)
                sel = i0[b, t, :c]
                assert len(set(sel.tolist())) == c and sel.min() >= 0 and sel.max() < v
                mask = np.zeros(v, bool); mask[sel] = True
                s = sc[b, t, :v]
                if c < v:
                    thr = s[mask].min()
                    assert thr >= s[~mask].max()
                    # among scores equal to the threshold the selected ones have the smallest indices
                    eq = np.nonzero(s == thr)[0]
                    chosen = mask[eq]
                    assert not (np.diff(chosen.astype(int)) > 0).any()
                # rank order of selector 1: non-increasing score, ties by increasing index
                ss = s[sel]
                assert (np.diff(ss) <= 0).all()
                tie = np.diff(ss) == 0
                assert (np.diff(sel)[tie] > 0).all()


# ======================================================================================= attention
def _np_attention(p, q, sets):
    """Library-built reference: scipy softmax + numpy einsum, explicit contiguous GQA groups."""
    G = p.Hq // p.Hkv
    out = np.zeros((p.B, p.T, p.Hq, p.D)); lse = np.zeros((p.B, p.T, p.Hq))
    scale = p._s.sm_scale
    for b in range(p.B):
        for t in range(p.T):
            rows = p.seq_start[b] + np.asarray(sets[b][t], dtype=np.int64)
            K = f64(p.k_cache[rows]); V = f64(p.v_cache[rows])          # [c, Hkv, D]
            Kq = np.repeat(K, G, axis=1); Vq = np.repeat(V, G, axis=1)   # head h uses KV head h // G
            z = scale * np.einsum("hd,chd->hc", f64(q[b, t]), Kq)
            w = softmax(z, axis=1)
            out[b, t] = np.einsum("hc,chd->hd", w, Vq)
            lse[b, t] = logsumexp(z, axis=1)
    return out, lse


def test_dense_matches_library_softmax():
    rng = np.random.default_rng(6)
    for causal, T in ((0, 1), (1, 3)):
        p = make_problem(rng, B=2, T=T, Hq=6, Hkv=2, D=8, lens=(11, 23), causal=causal)
        q = rand_bits(rng, (p.B, p.T, p.Hq, p.D))
        sets = [[list(range(p.visible(b, t))) for t in range(T)] for b in range(p.B)]
        ref_o, ref_l = _np_attention(p, q, sets)
        o, l = p.dense_attn(q)
        np.testing.assert_allclose(o, ref_o, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(l, ref_l, rtol=1e-12, atol=1e-13)


def test_sparse_matches_library_softmax_on_random_subsets():
    rng = np.random.default_rng(7)
    p = make_problem(rng, B=2, T=2, Hq=4, Hkv=2, D=16, k=6, lens=(20, 33), causal=1)
    q = rand_bits(rng, (p.B, p.T, p.Hq, p.D))
    idx = -np.ones((p.B, p.T, p.k), dtype=np.int32); cnt = np.zeros((p.B, p.T), dtype=np.int32)
    sets = [[None] * p.T for _ in range(p.B)]
    for b in range(p.B):
        for t in range(p.T):
            c = int(rng.integers(1, p.k + 1))
            s = rng.choice(p.visible(b, t), size=c, replace=False)
            idx[b, t, :c] = s; cnt[b, t] = c; sets[b][t] = s.tolist()
    ref_o, ref_l = _np_attention(p, q, sets)
    o, l = p.sparse_attn(q, idx, cnt)
    np.testing.assert_allclose(o, ref_o, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(l, ref_l, rtol=1e-12, atol=1e-13)


def test_sparse_with_k_ge_n_equals_dense_routine():
    rng = np.random.default_rng(8)
    for causal, T in ((0, 1), (1, 4)):
        p = make_problem(rng, B=2, T=T, Hq=4, Hkv=1, D=8, d_idx=4, k=64, lens=(21, 40), causal=causal)
        q_idx = rand_bits(rng, (p.B, p.T, p.d_idx))
        q = rand_bits(rng, (p.B, p.T, p.Hq, p.D))
        idx, cnt = p.topk(p.index_scores(q_idx))
        for b in range(p.B):
            for t in range(T):
                assert cnt[b, t] == p.visible(b, t)
        o_s, l_s = p.sparse_attn(q, idx, cnt)
        o_d, l_d = p.dense_attn(q)
        np.testing.assert_allclose(o_s, o_d, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(l_s, l_d, rtol=1e-12, atol=1e-13)


def test_attention_closed_forms():
    rng = np.random.default_rng(9)
    p = make_problem(rng, B=1, Hq=2, Hkv=1, D=4, k=6, lens=(12,), sm_scale=0.5)
    s0 = int(p.seq_start[0])
    sel = np.array([[[2, 5, 7, 11, -1, -1]]], dtype=np.int32); cnt = np.array([[4]], dtype=np.int32)
    q = rand_bits(rng, (1, 1, 2, 4))
    # (a) identical selected K rows -> uniform weights: O = mean of V rows, lse = z + ln c
    p.k_cache[s0 + sel[0, 0, :4]] = p.k_cache[s0 + 2]
    o, l = p.sparse_attn(q, sel, cnt)
    v = f64(p.v_cache[s0 + sel[0, 0, :4], 0])
    z = 0.5 * (f64(q[0, 0]) @ f64(p.k_cache[s0 + 2, 0]))
    np.testing.assert_allclose(o[0, 0], np.broadcast_to(v.mean(0), (2, 4)), rtol=1e-14)
    np.testing.assert_allclose(l[0, 0], z + math.log(4), rtol=1e-14)
    # (b) all V rows equal -> O is that row whatever the weights
    p2 = make_problem(rng, B=1, Hq=2, Hkv=1, D=4, k=6, lens=(12,))
    p2.v_cache[:] = p2.v_cache[0]
    o, _ = p2.sparse_attn(q, sel, cnt)
    np.testing.assert_allclose(o[0, 0], np.broadcast_to(f64(p2.v_cache[0, 0]), (2, 4)), rtol=1e-14)
    # (c) one selected token -> O = its V row, lse = its logit
    one = np.array([[[9, -1, -1, -1, -1, -1]]], dtype=np.int32)
    o, l = p2.sparse_attn(q, one, np.array([[1]], dtype=np.int32))
    z9 = p2._s.sm_scale * (f64(q[0, 0]) @ f64(p2.k_cache[int(p2.seq_start[0]) + 9, 0]))
    np.testing.assert_allclose(l[0, 0], z9, rtol=1e-14)
    # (d) one logit far above the rest -> O tends to that token's V row
    p3 = make_problem(rng, B=1, Hq=1, Hkv=1, D=4, k=6, lens=(12,), sm_scale=1.0)
    s3 = int(p3.seq_start[0])
    qd = bf16(np.array([[[[8.0, 0, 0, 0]]]]))
    p3.k_cache[s3: s3 + 12] = bf16(np.zeros((12, 1, 4)))
    p3.k_cache[s3 + 7, 0] = bf16([16.0, 0, 0, 0])        # logit 128 against zeros
    o, l = p3.sparse_attn(qd, sel, cnt)
    np.testing.assert_allclose(o[0, 0, 0], f64(p3.v_cache[s3 + 7, 0]), atol=1e-40, rtol=1e-14)
    np.testing.assert_allclose(l[0, 0, 0], 128.0, rtol=1e-14)
    # (e) empty selection -> zeros and -inf
    o, l = p3.sparse_attn(qd, -np.ones((1, 1, 6), np.int32), np.zeros((1, 1), np.int32))
    assert (o == 0).all() and np.isneginf(l).all()


def test_attention_invariances():
    rng = np.random.default_rng(10)
    p = make_problem(rng, B=1, Hq=4, Hkv=2, D=8, k=8, lens=(30,))
    s0 = int(p.seq_start[0])
    q = rand_bits(rng, (1, 1, 4, 8))
    sel = rng.choice(30, size=8, replace=False).astype(np.int32).reshape(1, 1, 8)
    cnt = np.array([[8]], dtype=np.int32)
    o, l = p.sparse_attn(q, sel, cnt)
    # permutation of the index row
    perm = sel[:, :, ::-1].copy()
    o2, l2 = p.sparse_attn(q, perm, cnt)
    np.testing.assert_allclose(o2, o, rtol=1e-13); np.testing.assert_allclose(l2, l, rtol=1e-13)
    # heads of one group with equal queries give equal outputs; heads of different groups do not
    qq = q.copy(); qq[0, 0, 1] = qq[0, 0, 0]; qq[0, 0, 2] = qq[0, 0, 0]
    o3, _ = p.sparse_attn(qq, sel, cnt)
    np.testing.assert_array_equal(o3[0, 0, 0], o3[0, 0, 1])          # heads 0,1 -> KV head 0
    assert np.abs(o3[0, 0, 0] - o3[0, 0, 2]).max() > 1e-3           # head 2 -> KV head 1
    # convex hull and weights summing to one (constant-one V column comes back as one)
    v = f64(p.v_cache[s0 + sel[0, 0]])
    for h in range(4):
        gk = h // 2
        assert (o[0, 0, h] <= v[:, gk].max(0) + 1e-12).all() and (o[0, 0, h] >= v[:, gk].min(0) - 1e-12).all()
    # adding one shared direction e to every selected key shifts each logit by the same amount:
    # O unchanged, lse shifted by sm_scale * q.e   (values chosen exactly representable)
    p4 = make_problem(rng, B=1, Hq=1, Hkv=1, D=4, k=4, lens=(10,), sm_scale=1.0)
    s4 = int(p4.seq_start[0])
    p4.k_cache[:, :, 3] = bf16(0.0)
    q4 = rand_bits(rng, (1, 1, 1, 4)); q4[0, 0, 0, 3] = bf16(2.0)
    sel4 = np.array([[[1, 4, 6, 9]]], dtype=np.int32); c4 = np.array([[4]], dtype=np.int32)
    o_a, l_a = p4.sparse_attn(q4, sel4, c4)
    p4.k_cache[:, :, 3] = bf16(1.5)
    o_b, l_b = p4.sparse_attn(q4, sel4, c4)
    np.testing.assert_allclose(o_b, o_a, rtol=1e-12)
    np.testing.assert_allclose(l_b - l_a, 3.0, rtol=1e-12)


def test_hand_example_attention():
    gold = json.load(open(GOLD))["attention"]
    V = bf16(np.array(gold["v"], dtype=np.float64)).reshape(5, 1, 2)

    def run(q, K, sel, scale):
        k = len(sel)
        p = oracle.Problem(num_seqs=1, num_q_heads=1, num_kv_heads=1, head_dim=2, idx_dim=2, top_k=k,
                           sm_scale=scale, seq_start=[0], seq_len=[5],
                           k_cache=bf16(np.array(K, dtype=np.float64)).reshape(5, 1, 2), v_cache=V)
        return p.sparse_attn(bf16(np.array(q, dtype=np.float64)).reshape(1, 1, 1, 2),
                             np.array(sel, dtype=np.int32).reshape(1, 1, k), np.array([[k]], dtype=np.int32))

    u = gold["uniform"]
    for case in u["cases"]:
        o, l = run(u["q"], u["k"], case["sel"], 1.0)
        want = np.array(case["out"], float) if "out" in case else np.array(case["out_times_3"], float) / 3
        np.testing.assert_allclose(o[0, 0, 0], want, rtol=1e-15)
        np.testing.assert_allclose(l[0, 0, 0], math.log(case["lse_ln_of"]), rtol=1e-15, atol=1e-16)
    t = gold["two_to_one"]
    o, l = run(t["q"], t["k"], t["sel"], math.log(2.0))
    np.testing.assert_allclose(o[0, 0, 0], np.array(t["out_times_3"], float) / 3, rtol=1e-14)
    np.testing.assert_allclose(l[0, 0, 0], math.log(t["lse_ln_of"]), rtol=1e-14)


# ======================================================================================= chain
def test_decode_step_reuses_one_index_for_every_layer():
    rng = np.random.default_rng(11)
    p = make_problem(rng, B=2, T=1, Hq=4, Hkv=2, D=8, d_idx=6, k=5, lens=(19, 4))
    L = 3
    q_idx = rand_bits(rng, (p.B, p.T, p.d_idx))
    ql = rand_bits(rng, (L, p.B, p.T, p.Hq, p.D))
    step = p.decode_step(q_idx, ql)
    sc = p.index_scores(q_idx)
    idx, cnt = p.topk(sc)
    np.testing.assert_array_equal(step["idx"], idx)
    np.testing.assert_array_equal(step["count"], cnt)
    assert cnt.tolist() == [[5], [4]]                      # the 4-token sequence selects all of its tokens
    for l in range(L):
        o, lse = p.sparse_attn(ql[l], idx, cnt)
        np.testing.assert_array_equal(step["out"][l], o)
        np.testing.assert_array_equal(step["lse"][l], lse)
    # layers differ only through their queries: feeding the same query to two layers gives the same output
    ql2 = ql.copy(); ql2[2] = ql2[0]
    step2 = p.decode_step(q_idx, ql2)
    np.testing.assert_array_equal(step2["out"][2], step2["out"][0])


def test_oracle_on_tiny_workload_shape():
    """The 'tiny' benchmark shape end to end through the oracle, cross-checked with the library reference."""
    from workloads import TINY, Workload

    w = Workload(TINY.replace(ctx=512, top_k=32, num_layers=2))
    kc, vc = w.host_kv_full()
    p = oracle.problem_from_workload(w, k_cache=kc, v_cache=vc, idx_k_cache=w.host_kidx_cache())
    ql = np.stack([w.q_layer_bits(l) for l in range(2)])
    step = p.decode_step(w.q_idx_bits(), ql)
    sc = f64(w.q_idx_bits()[0, 0]) @ f64(w.kidx_bits(0)).T
    np.testing.assert_allclose(step["scores"][0, 0], sc, rtol=1e-13, atol=1e-13)
    want = sorted(sorted(range(512), key=lambda s: (-sc[s], s))[:32])
    assert sorted(step["idx"][0, 0].tolist()) == want
    ref_o, ref_l = _np_attention(p, ql[1], [[step["idx"][0, 0].tolist()]])
    np.testing.assert_allclose(step["out"][1], ref_o, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(step["lse"][1], ref_l, rtol=1e-12)


def test_paged_layout_gives_the_same_results_as_contiguous_sequences():
    """Paging is addressing only: the oracle on a block-table layout (blocks scattered by a permutation) must
    return exactly what it returns on contiguous sequences."""
    from workloads import RAGGED, Workload

    w = Workload(RAGGED.replace(num_seqs=4, ctx=700, ragged_min=40, num_short=1, top_k=64, num_layers=2,
                                num_q_heads=8, num_kv_heads=2))
    kc, vc = w.host_kv_full()
    kidx = w.host_kidx_cache()
    ql = np.stack([w.q_layer_bits(l) for l in range(2)])
    flat = oracle.problem_from_workload(w, k_cache=kc, v_cache=vc, idx_k_cache=kidx).decode_step(w.q_idx_bits(), ql)
    for bs in (16, 64):
        table, nblocks = w.block_table(bs)
        assert sorted(table[table >= 0].tolist()).count(0) >= 1 and nblocks == sum((int(n) + bs - 1) // bs for n in w.seq_len)
        paged = oracle.problem_from_workload(w, k_cache=w.paginate_host(kc, bs), v_cache=w.paginate_host(vc, bs),
                                             idx_k_cache=w.paginate_host(kidx, bs), block_table=table, block_size=bs)
        got = paged.decode_step(w.q_idx_bits(), ql)
        for key in ("idx", "count", "out", "lse"):
            np.testing.assert_array_equal(got[key], flat[key])
        for b in range(4):
            n = int(w.seq_len[b])
            np.testing.assert_array_equal(got["scores"][b, 0, :n], flat["scores"][b, 0, :n])


# ======================================================================================= Eq. 2 + append
def test_bf16_rounding_every_value_ties_and_library():
    import torch

    bits = np.arange(65536, dtype=np.uint16)
    finite = (bits & 0x7F80) != 0x7F80
    vals = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).double().numpy()  # torch decodes the bits
    got = oracle.round_bf16(vals[finite])
    np.testing.assert_array_equal(got, bits[finite])  # every finite bf16 number (subnormals, both zeros) is a fixed point
    one = 1.0
    cases = [(one + 2.0 ** -8, 0x3F80),               # tie between 1 and 1 + 2^-7: the even significand wins
             (one + 3 * 2.0 ** -8, 0x3F82),           # tie between odd 1 + 2^-7 and even 1 + 2^-6
             (one + 2.0 ** -8 + 2.0 ** -40, 0x3F81),  # just above a tie: float32 would lose the 2^-40 and round to even
             (one + 2.0 ** -8 - 2.0 ** -40, 0x3F80),
             (-(one + 2.0 ** -8 + 2.0 ** -40), 0xBF81),
             (2.0 ** -134, 0x0000), (2.0 ** -134 * 1.0001, 0x0001), (3 * 2.0 ** -134, 0x0002),  # subnormal grid 2^-133
             (2.0 ** 128, 0x7F80), ((2 - 2.0 ** -8) * 2.0 ** 127, 0x7F80), ((2 - 2.0 ** -7) * 2.0 ** 127, 0x7F7F)]
    for x, want in cases:
        assert int(oracle.round_bf16(np.array([x]))[0]) == want, (x, hex(want))
    rng = np.random.default_rng(50)
    f32 = (rng.standard_normal(200000) * np.exp(rng.uniform(-30, 30, 200000))).astype(np.float32)
    lib_bits = torch.from_numpy(f32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(oracle.round_bf16(f32.astype(np.float64)), lib_bits)  # one rounding on both sides
    x = np.sort(rng.standard_normal(5000))
    r = f64(oracle.round_bf16(x))
    assert (np.diff(r) >= 0).all() and (np.abs(r - x) <= np.abs(x) * 2.0 ** -8).all()  # monotone, half an ulp at most


def test_linear_matches_numpy_matmul():
    rng = np.random.default_rng(51)
    h, w = rand_bits(rng, (5, 11)), rand_bits(rng, (3, 11), 0.3)
    y = oracle.linear(h, w)
    assert y.shape == (5, 3)
    np.testing.assert_allclose(y, f64(h) @ f64(w).T, rtol=0, atol=1e-12)
    e = np.zeros((1, 11)); e[0, 4] = 1.0
    np.testing.assert_array_equal(oracle.linear(bf16(e), w)[0], f64(w)[:, 4])  # a unit state reads column 4 of every row
    np.testing.assert_array_equal(oracle.linear(h, bf16(e))[:, 0], f64(h)[:, 4])


def _selector(n_out, d_model, cols):
    w = np.zeros((n_out, d_model))
    w[np.arange(n_out), cols] = 1.0
    return bf16(w)


@pytest.mark.parametrize("paged", [False, True])
def test_project_append_places_exact_rows_and_touches_nothing_else(paged):
    rng = np.random.default_rng(52)
    B, T, Hkv, D, d_idx, dm = 3, 2, 2, 8, 6, 40
    lens = (9, 13, 4)
    p = make_problem(rng, B=B, T=T, Hq=4, Hkv=Hkv, D=D, d_idx=d_idx, lens=lens, causal=1)
    if paged:
        bs = 4
        nblk = [(n + bs - 1) // bs for n in lens]
        perm = rng.permutation(sum(nblk) + 2)
        table = np.zeros((B, max(nblk)), dtype=np.int32)
        at = 0
        for b in range(B):
            table[b, : nblk[b]] = perm[at: at + nblk[b]]
            at += nblk[b]
        rows = (sum(nblk) + 2) * bs
        p = oracle.Problem(num_seqs=B, q_per_seq=T, num_q_heads=4, num_kv_heads=Hkv, head_dim=D, idx_dim=d_idx, top_k=5,
                           causal=1, sm_scale=1.0, seq_start=np.zeros(B, np.int64), seq_len=np.asarray(lens, np.int32),
                           k_cache=rand_bits(rng, (rows, Hkv, D)), v_cache=rand_bits(rng, (rows, Hkv, D)),
                           idx_k_cache=rand_bits(rng, (rows, d_idx)), block_table=table, block_size=bs)
        row_of = lambda b, s: int(table[b, s // bs]) * bs + s % bs
    else:
        row_of = lambda b, s: int(p.seq_start[b]) + s
    before = (p.idx_k_cache.copy(), p.k_cache.copy(), p.v_cache.copy())
    h = rand_bits(rng, (B, T, dm))
    cq, ck = rng.permutation(dm)[:d_idx], rng.permutation(dm)[:d_idx]
    ckk, cv = rng.permutation(dm)[: Hkv * D], rng.permutation(dm)[: Hkv * D]
    q = p.project_append(h, _selector(d_idx, dm, cq), _selector(d_idx, dm, ck), _selector(Hkv * D, dm, ckk),
                         _selector(Hkv * D, dm, cv))
    touched = set()
    for b in range(B):
        for t in range(T):
            r = row_of(b, lens[b] - T + t)
            touched.add(r)
            np.testing.assert_array_equal(q[b, t], h[b, t, cq])              # bf16 in, selector weights: exact
            np.testing.assert_array_equal(p.idx_k_cache[r], h[b, t, ck])
            np.testing.assert_array_equal(p.k_cache[r].reshape(-1), h[b, t, ckk])  # feature g*D + d lands at [g][d]
            np.testing.assert_array_equal(p.v_cache[r].reshape(-1), h[b, t, cv])
    keep = np.array(sorted(set(range(p.idx_k_cache.shape[0])) - touched))
    assert len(touched) == B * T
    for now, was in zip((p.idx_k_cache, p.k_cache, p.v_cache), before):
        np.testing.assert_array_equal(now[keep], was[keep])


def test_project_append_general_weights_and_indexer_only():
    rng = np.random.default_rng(53)
    B, T, Hkv, D, d_idx, dm = 2, 1, 2, 8, 6, 33
    p = make_problem(rng, B=B, T=T, Hkv=Hkv, D=D, d_idx=d_idx, lens=(9, 13))
    h = rand_bits(rng, (B, T, dm))
    wq, wk = rand_bits(rng, (d_idx, dm), 0.2), rand_bits(rng, (d_idx, dm), 0.2)
    wkk, wv = rand_bits(rng, (Hkv * D, dm), 0.2), rand_bits(rng, (Hkv * D, dm), 0.2)
    k_before = p.k_cache.copy()
    q = p.project_append(h, wq, wk)                    # indexer branch only: K and V stay as they were
    np.testing.assert_array_equal(p.k_cache, k_before)
    hf = f64(h).reshape(B, dm)
    np.testing.assert_array_equal(q.reshape(B, d_idx), oracle.round_bf16(hf @ f64(wq).T))
    q2 = p.project_append(h, wq, wk, wkk, wv)
    np.testing.assert_array_equal(q2, q)
    for b in range(B):
        r = int(p.seq_start[b]) + int(p.seq_len[b]) - 1
        np.testing.assert_array_equal(p.idx_k_cache[r], oracle.round_bf16(hf[b] @ f64(wk).T))
        np.testing.assert_array_equal(p.k_cache[r].reshape(-1), oracle.round_bf16(hf[b] @ f64(wkk).T))
        np.testing.assert_array_equal(p.v_cache[r].reshape(-1), oracle.round_bf16(hf[b] @ f64(wv).T))
    # the appended key is what Eq. 3 then scores: with both indexer weights selecting the same components of h,
    # the newest token's score is the sum of their squares
    cols = np.arange(d_idx) * 3
    sel = _selector(d_idx, dm, cols)
    q3 = p.project_append(h, sel, sel)
    sc = p.index_scores(q3)
    for b in range(B):
        np.testing.assert_allclose(sc[b, 0, int(p.seq_len[b]) - 1], (hf[b, cols] ** 2).sum(), rtol=0, atol=1e-12)
