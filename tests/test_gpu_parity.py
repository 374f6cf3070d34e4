"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs.

Small cases compare every element; they span several tiles of each kernel plus ragged tails and the
degenerate cases (fewer tokens than k, one token, k = 1, duplicate keys, empty selections, corrupt
indices). Full-size cases live in test_gpu_fullsize.py.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import __graft_entry__ as entry

entry._load_build_module().build()

import oracle
import paper_2606_06467_b200 as clsa
from _harness import SCORE_RTOL, GpuProblem, check_attention, check_scores, check_topk_band, check_topk_exact_on_gpu_scores
from workloads import HEADLINE, MID, RAGGED, TINY, Workload

pytestmark = pytest.mark.gpu


def _bf16_bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _full_oracle(w):
    kc, vc = w.host_kv_full()
    return oracle.problem_from_workload(w, k_cache=kc, v_cache=vc, idx_k_cache=w.host_kidx_cache())


def _run_all(w, layers=None, check_lse=True):
    """Scores, top-k, every layer's attention and the chained call, each against the oracle."""
    g = GpuProblem(w, layers=layers)
    prob = _full_oracle(w)
    ref_scores = prob.index_scores(w.q_idx_bits())
    ref_idx, ref_cnt = prob.topk(ref_scores)
    gs = g.index_scores()
    check_scores(gs, ref_scores, w)
    gi, gc = g.topk(gs)
    check_topk_exact_on_gpu_scores(prob, gs, gi, gc, w)
    check_topk_band(ref_scores, ref_idx, ref_cnt, gi, gc, w)
    idx_np, cnt_np = gi.cpu().numpy().copy(), gc.cpu().numpy().copy()
    singles = []
    for l in range(g.L):
        # a launch on its own (the whole GPU on one layer), walking forwards or backwards ...
        out, lse = g.sparse_attn(l, reverse=l & 1)
        check_attention(prob, w, l, out, lse if check_lse else None, idx_np, cnt_np)
        # ... the same when only q is pending (row copies start before the launch waits for its predecessor) ...
        out_e, lse_e = g.sparse_attn(l, reverse=l & 1, only_q_pending=1, keep_rows=1)
        assert torch.equal(out.view(torch.int16), out_e.view(torch.int16)), "hints that do not change the split change nothing"
        # ... and the shapes the chain uses (a few large blocks per layer, one direction): the same result to rounding
        keep = 1 if l + 1 < g.L else 0
        out1, lse1 = g.sparse_attn(l, shared_gpu=1, keep_rows=keep)
        check_attention(prob, w, l, out1, lse1 if check_lse else None, idx_np, cnt_np)
        assert (out.float() - out1.float()).abs().max().item() <= 2e-2
        # ... and its finer variant, which a chain may use for its last layers
        out2, lse2 = g.sparse_attn(l, shared_gpu=2, keep_rows=keep)
        check_attention(prob, w, l, out2, lse2 if check_lse else None, idx_np, cnt_np)
        # ... and the block shape of the launches that compute two layers at once
        out3, lse3 = g.sparse_attn(l, shared_gpu=3, keep_rows=keep)
        check_attention(prob, w, l, out3, lse3 if check_lse else None, idx_np, cnt_np)
        out4, lse4 = g.sparse_attn(l, shared_gpu=4, keep_rows=keep)
        check_attention(prob, w, l, out4, lse4 if check_lse else None, idx_np, cnt_np)
        singles.append((out1, out2, out3, out4))
    # the chain: same index for all layers, byte-identical to the separate calls in the chain's launch shapes
    g.idx.fill_(-7); g.count.fill_(-7)
    outs = g.decode_step()
    torch.cuda.synchronize()
    np.testing.assert_array_equal(g.idx.cpu().numpy(), idx_np)
    np.testing.assert_array_equal(g.count.cpu().numpy(), cnt_np)
    props = torch.cuda.get_device_properties(0)
    fine_layers, paired_layers = clsa.clsa_chain_plan(g.params, props.multi_processor_count, props.clock_rate)
    rows = w.cfg.num_seqs * w.cfg.q_per_seq
    for l in range(g.L):
        # which shape each query row of this layer takes, as clsa_chain_plan reports it
        a, b1, b2, b3, b4 = (x.reshape(rows, -1).view(torch.int16) for x in (outs[l],) + singles[l])
        if l < paired_layers:   # computed together with its neighbour: the single-layer launch of that block shape
            fine = l >= paired_layers - fine_layers
            assert torch.equal(a, b4 if fine else b3), f"layer {l}: chain != separate call (shape {4 if fine else 3})"
            continue
        fine = l >= g.L - fine_layers
        assert torch.equal(a, b2 if fine else b1), f"layer {l}: chain != separate call (shape {2 if fine else 1})"
    g.fine_layers, g.paired_layers = fine_layers, paired_layers
    # the attention half of the chain on its own, fed the index that is already there
    layer_outs = [g.new_out() for _ in range(g.L)]
    clsa.clsa_sparse_attn_layers(g.params, [g.t["q_layers"][l] for l in range(g.L)], g.idx, g.count, layer_outs, g.ws)
    torch.cuda.synchronize()
    for l in range(g.L):
        assert torch.equal(layer_outs[l].view(torch.int16), outs[l].view(torch.int16)), f"layer {l}: layers call"
    np.testing.assert_array_equal(g.idx.cpu().numpy(), idx_np)  # the shared index is read, never written
    assert g.status() == 0
    return g, prob


def test_tiny_config_full():
    _run_all(Workload(TINY))


def test_mid_shape_scaled_down():
    # 32/8 heads, d_idx 128, several spans per row, two sequences
    _run_all(Workload(MID.replace(num_seqs=2, ctx=8192 + 37, top_k=512, num_layers=3)))


def test_ragged_with_duplicates_and_short_sequences():
    w = Workload(RAGGED.replace(num_seqs=6, ctx=9000, ragged_min=100, num_short=2, top_k=700, num_layers=2))
    assert (w.seq_len < 700).sum() >= 2
    g, prob = _run_all(w)
    # duplicates really are exact ties on the GPU: equal keys -> bit-equal fp32 scores
    gs = g.index_scores().cpu().numpy()
    src = w.row_source()
    b = int(np.argmax(w.seq_len))
    s0, n = int(w.seq_start[b]), int(w.seq_len[b])
    local = src[s0: s0 + n] - s0
    dup = np.nonzero(local != np.arange(n))[0]
    dup = dup[local[local[dup]] == local[dup]]   # keep copies whose source position still holds its own base row
    assert dup.size > 10
    np.testing.assert_array_equal(gs[b, 0, dup].view(np.uint32), gs[b, 0, local[dup]].view(np.uint32))


def test_chain_at_the_headline_geometry():
    """The headline's launch geometry at a context the oracle handles in seconds. Groups of 4 query heads: the chain
    computes its 16 layers two per launch, and every layer equals the single-layer launch of that block shape bit for
    bit, and the oracle within tolerance. With an odd number of layers the last one goes alone."""
    w = Workload(MID.replace(num_seqs=16, ctx=4096, top_k=2048, num_layers=16, seed=31))
    g, _ = _run_all(w, check_lse=False)
    assert g.paired_layers == 16 and g.fine_layers == 0
    g, _ = _run_all(Workload(MID.replace(num_seqs=5, ctx=3000, top_k=700, num_layers=3, seed=32)), check_lse=False)
    assert g.paired_layers == 2
    # 20 rows: the step's blocks no longer fit one round of one per SM, and the last pairs take the finer shape
    g, _ = _run_all(Workload(MID.replace(num_seqs=20, ctx=2500, top_k=2048, num_layers=16, seed=34)), check_lse=False)
    if torch.cuda.get_device_properties(0).multi_processor_count == 148:
        assert g.paired_layers == 16 and g.fine_layers in (2, 4, 6), g.fine_layers


def test_chain_of_wide_groups_with_finer_last_layers():
    """16 query heads per KV head: one layer per launch (a warp's two head tiles are taken by the group), 16 layers of
    32 blocks do not fill 148 SMs evenly, so the chain gives its last layers the finer shape; every layer still equals
    the separate call of its shape bit for bit, and the oracle within tolerance."""
    w = Workload(MID.replace(num_seqs=16, ctx=4096, top_k=2048, num_layers=16, num_q_heads=128, num_kv_heads=8, seed=33))
    g, _ = _run_all(w, check_lse=False)
    assert g.paired_layers == 0
    if torch.cuda.get_device_properties(0).multi_processor_count == 148:
        assert 1 <= g.fine_layers <= 3, g.fine_layers


@pytest.mark.parametrize("B,k,heads", [(20, 512, (32, 8)), (5, 1000, (20, 4)), (37, 96, (32, 8)), (3, 4096, (8, 1)), (1, 333, (32, 8)),
                                       (87, 200, (32, 8)), (21, 2048, (32, 8))])
def test_standalone_attention_at_awkward_batch_sizes(B, k, heads):
    """A launch that has the GPU to itself cuts its work at token granularity when whole (row, KV head) units would
    fill the SMs poorly: unit counts that do not divide the SM count (20 and 21 rows: every unit's workers sit in two
    or three blocks, partials merged across blocks), more units than the workers' even shares allow (87 rows: flat
    split, spans across unit boundaries, whole units written by one warp), a group of 5 query heads, a single KV
    head, one sequence; 37 rows fill two rounds exactly and stay with the whole-unit kernel. Every case against the
    oracle, both walking directions, with and without the early row copies."""
    w = Workload(MID.replace(num_seqs=B, ctx=max(2 * k, 3000) + 11, top_k=k, num_layers=2, num_q_heads=heads[0],
                             num_kv_heads=heads[1], seed=500 + B))
    g = GpuProblem(w)
    prob = _full_oracle(w)
    gi, gc = g.topk(g.index_scores())
    idx_np, cnt_np = gi.cpu().numpy().copy(), gc.cpu().numpy().copy()
    for l in range(2):
        out, lse = g.sparse_attn(l, reverse=l, keep_rows=1 - l, only_q_pending=l)
        check_attention(prob, w, l, out, lse, idx_np, cnt_np)
    assert g.status() == 0
    assert g.ws[256: 256 + B * heads[0] * 4].count_nonzero().item() == 0, "the arrival counters are back at zero"


def test_planted_tokens_are_selected():
    w = Workload(HEADLINE.replace(num_seqs=2, ctx=16384, top_k=512, num_layers=1))
    g, prob = _run_all(w)
    sel = g.idx.cpu().numpy()
    for b in range(2):
        planted = w.planted_positions(b)
        assert np.isin(planted, sel[b, 0]).mean() > 0.9


@pytest.mark.parametrize("hq,hkv", [(20, 4), (8, 1), (16, 2), (32, 2), (5, 5), (32, 16)])
def test_head_layouts(hq, hkv):
    # includes the paper's own 20 query / 4 KV heads (group of 5) and the largest supported group (16)
    w = Workload(MID.replace(num_seqs=2, ctx=3000, top_k=300, num_layers=2, num_q_heads=hq, num_kv_heads=hkv, seed=77 + hq))
    _run_all(w)


def test_idx_dim_64_and_stride_padding():
    w = Workload(TINY.replace(num_seqs=3, ctx=5000, top_k=100, num_layers=1, seed=5))
    g = GpuProblem(w)
    prob = _full_oracle(w)
    ref = prob.index_scores(w.q_idx_bits())
    # indexer keys in a padded buffer: token stride 96 elements instead of 64
    padded = torch.zeros((w.total_rows, 96), dtype=torch.bfloat16, device=g.dev)
    padded[:, :64] = g.t["idx_k_cache"]
    g.params.idx_k_cache, g.params.idx_token_stride = padded.data_ptr(), 96
    check_scores(g.index_scores(), ref, w)


@pytest.mark.parametrize("n,k", [(1, 1), (1, 64), (17, 17), (17, 16), (300, 1), (4097, 4096), (2048, 2048), (33, 500)])
def test_degenerate_lengths(n, k):
    w = Workload(MID.replace(num_seqs=2, ctx=n, top_k=k, num_layers=1, seed=1000 + n + k))
    _run_all(w)


def test_topk_on_crafted_scores():
    """Selection alone on score arrays with closed-form answers (ties, signed zeros, monotone ramps)."""
    n, k = 40000, 1000
    w = Workload(MID.replace(num_seqs=5, ctx=n, top_k=k, num_layers=1))
    g = GpuProblem(w, layers=1)
    sc = torch.zeros((5, 1, g.score_stride), dtype=torch.float32, device=g.dev)
    sc[0, 0, :n] = 3.25                                               # all equal -> positions 0..k-1
    sc[1, 0, :n] = torch.arange(n, device=g.dev, dtype=torch.float32)  # increasing -> the last k
    sc[2, 0, :n] = -torch.arange(n, device=g.dev, dtype=torch.float32)  # decreasing -> the first k
    z = torch.zeros(n, device=g.dev); z[::2] = -0.0; z[1::2] = 0.0; z[n // 2:] = -1.0
    sc[3, 0, :n] = z                                                  # +-0 tie -> positions 0..k-1
    two = torch.zeros(n, device=g.dev); two[torch.arange(0, n, 100, device=g.dev)] = 1.0   # 400 ones
    sc[4, 0, :n] = two
    gi, gc = g.topk(sc)
    gi = gi.cpu().numpy()
    assert (gc.cpu().numpy() == k).all()
    np.testing.assert_array_equal(gi[0, 0], np.arange(k))
    np.testing.assert_array_equal(gi[1, 0], np.arange(n - k, n))
    np.testing.assert_array_equal(gi[2, 0], np.arange(k))
    np.testing.assert_array_equal(gi[3, 0], np.arange(k))
    ones = np.arange(0, n, 100)
    rest = np.setdiff1d(np.arange(n), ones)[: k - ones.size]
    np.testing.assert_array_equal(gi[4, 0], np.sort(np.concatenate([ones, rest])))
    # random quantised scores (heavy ties everywhere) against the oracle's sort
    rng = np.random.default_rng(3)
    q = np.round(rng.standard_normal((5, 1, n)) * 4) / 4
    sc[:, :, :n] = torch.from_numpy(q.astype(np.float32)).to(g.dev)
    gi, gc = g.topk(sc)
    prob = oracle.problem_from_workload(w)
    check_topk_exact_on_gpu_scores(prob, sc, gi, gc, w)
    # determinism: a second run gives identical bytes
    first = gi.clone()
    gi2, _ = g.topk(sc)
    assert torch.equal(first, gi2)


def test_attention_accepts_any_order_and_flags_bad_indices():
    w = Workload(MID.replace(num_seqs=2, ctx=6000, top_k=640, num_layers=1, seed=9))
    g = GpuProblem(w)
    prob = _full_oracle(w)
    gi, gc = g.topk(g.index_scores())
    idx_np, cnt_np = gi.cpu().numpy().copy(), gc.cpu().numpy().copy()
    base, base_lse = g.sparse_attn(0)
    check_attention(prob, w, 0, base, base_lse, idx_np, cnt_np)
    # any permutation of the valid entries gives the same result to rounding
    perm = idx_np.copy()
    rng = np.random.default_rng(0)
    for b in range(2):
        perm[b, 0] = rng.permutation(perm[b, 0])
    out_p, lse_p = g.sparse_attn(0, idx=torch.from_numpy(perm).to(g.dev))
    check_attention(prob, w, 0, out_p, lse_p, perm, cnt_np)
    # both sweep directions agree with the oracle
    out_r, lse_r = g.sparse_attn(0, reverse=1)
    check_attention(prob, w, 0, out_r, lse_r, idx_np, cnt_np)
    # empty selection for sequence 1 -> zeros and -inf; sequence 0 untouched
    cnt0 = cnt_np.copy(); cnt0[1, 0] = 0
    out_e, lse_e = g.sparse_attn(0, count=torch.from_numpy(cnt0).to(g.dev))
    assert (out_e[1].float() == 0).all() and torch.isneginf(lse_e[1]).all()
    assert torch.equal(out_e[0].view(torch.int16), base[0].view(torch.int16))
    assert g.status() == 0
    # corrupt entries (out of range, negative) are skipped and flagged, never dereferenced
    bad = idx_np.copy()
    bad[0, 0, 5] = 10 ** 9
    bad[0, 0, 77] = -3
    bad[1, 0, 639] = int(w.seq_len[1])
    out_b, lse_b = g.sparse_attn(0, idx=torch.from_numpy(bad).to(g.dev))
    assert g.status() & clsa.CLSA_DEV_BAD_INDEX
    clsa.clsa_clear_status(g.ws)
    keep = idx_np.copy()
    keep0 = np.delete(keep[0, 0], [5, 77]); keep1 = np.delete(keep[1, 0], [639])
    ref_idx = -np.ones_like(keep); ref_cnt = cnt_np.copy()
    ref_idx[0, 0, : keep0.size] = keep0; ref_cnt[0, 0] = keep0.size
    ref_idx[1, 0, : keep1.size] = keep1; ref_cnt[1, 0] = keep1.size
    check_attention(prob, w, 0, out_b, lse_b, ref_idx, ref_cnt)
    # a count outside [0, k] is clamped and flagged
    cntx = cnt_np.copy(); cntx[0, 0] = 10 ** 6
    out_c, _ = g.sparse_attn(0, count=torch.from_numpy(cntx).to(g.dev))
    assert g.status() & clsa.CLSA_DEV_BAD_COUNT
    assert torch.equal(out_c.view(torch.int16), base.view(torch.int16))
    clsa.clsa_clear_status(g.ws)
    assert g.status() == 0


def test_k_ge_n_equals_dense_attention():
    """With k >= n the sparse path must reproduce dense attention over the whole cache (Eq. 1 vs Eq. 4)."""
    w = Workload(MID.replace(num_seqs=2, ctx=777, top_k=1024, num_layers=1, seed=21))
    g = GpuProblem(w)
    prob = _full_oracle(w)
    g.topk(g.index_scores())
    out, lse = g.sparse_attn(0)
    o_ref, l_ref = prob.dense_attn(w.q_layer_bits(0))
    err = np.abs(out.float().cpu().numpy() - o_ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3
    assert np.abs(lse.cpu().numpy() - l_ref).max() <= 2e-3 * np.abs(l_ref).max()


def test_sequence_longer_than_max_seq_len_is_skipped_and_flagged():
    w = Workload(MID.replace(num_seqs=2, ctx=4000, top_k=128, num_layers=1))
    g = GpuProblem(w)
    g.params.max_seq_len = 3000      # lie about the bound: both sequences exceed it
    s = g.new_scores()
    clsa.clsa_index_scores(g.params, g.t["q_idx"], s, g.score_stride, g.ws)
    clsa.clsa_topk(g.params, s, g.score_stride, g.idx, g.count, g.ws)
    assert g.status() & clsa.CLSA_DEV_BAD_SEQLEN
    assert (g.count.cpu().numpy() == 0).all() and torch.isnan(s).all()


@pytest.mark.parametrize("block_size", [0, 16])
def test_attention_alone_skips_sequences_outside_their_declared_bounds(block_size):
    """clsa_sparse_attn accepts any caller-built index, so it cannot rely on the top-k to have refused a sequence
    whose length lies outside [T, max_seq_len]: such a sequence is treated as count 0 (zeros, lse = -inf) and
    flagged, and its index entries never become addresses -- contiguous and paged caches alike (with paging an
    entry beyond max_blocks_per_seq * block_size would index past the sequence's row of the block table)."""
    w = Workload(MID.replace(num_seqs=3, ctx=4000, top_k=128, num_layers=1, seed=77))
    g = GpuProblem(w, block_size=block_size)
    prob = _full_oracle(w)
    gi, gc = g.topk(g.index_scores())
    idx_np, cnt_np = gi.cpu().numpy().copy(), gc.cpu().numpy().copy()
    base, base_lse = g.sparse_attn(0)
    check_attention(prob, w, 0, base, base_lse, idx_np, cnt_np)
    assert g.status() == 0
    lens = g.t["seq_len"].clone()
    g.t["seq_len"][1] = 10 ** 6            # far beyond max_seq_len (and beyond the block table's row)
    big = idx_np.copy()
    big[1, 0, :] = np.arange(128) * 7000   # positions that would be "valid" for such a length
    out, lse = g.sparse_attn(0, idx=torch.from_numpy(big).to(g.dev))
    torch.cuda.synchronize()
    assert g.status() & clsa.CLSA_DEV_BAD_SEQLEN
    assert (out[1].float() == 0).all() and torch.isneginf(lse[1]).all()
    for b in (0, 2):
        assert torch.equal(out[b].view(torch.int16), base[b].view(torch.int16))
    clsa.clsa_clear_status(g.ws)
    g.t["seq_len"][1] = 0                  # shorter than T
    out, lse = g.sparse_attn(0)
    assert g.status() & clsa.CLSA_DEV_BAD_SEQLEN
    assert (out[1].float() == 0).all() and torch.isneginf(lse[1]).all()
    clsa.clsa_clear_status(g.ws)
    g.t["seq_len"].copy_(lens)
    out, _ = g.sparse_attn(0)
    assert g.status() == 0 and torch.equal(out.view(torch.int16), base.view(torch.int16))


def test_non_finite_scores_never_fault_and_keep_the_index_contract():
    """Scores must be finite by contract; NaN and infinities are ordered by their bit patterns, and whatever the
    order, the result keeps the index contract (count, distinct ascending in-range positions) without faulting."""
    n, k = 50000, 777
    w = Workload(MID.replace(num_seqs=3, ctx=n, top_k=k, num_layers=1))
    g = GpuProblem(w, layers=1)
    rng = np.random.default_rng(12)
    sc = torch.from_numpy(rng.standard_normal((3, 1, g.score_stride)).astype(np.float32)).to(g.dev)
    sc[0, 0, ::7] = float("nan")
    sc[1, 0, ::5] = float("inf")
    sc[1, 0, 1::5] = float("-inf")
    sc[2, 0, :n] = float("nan")
    gi, gc = g.topk(sc)
    torch.cuda.synchronize()
    assert g.status() == 0
    gi, gc = gi.cpu().numpy(), gc.cpu().numpy()
    for b in range(3):
        assert gc[b, 0] == k
        row = gi[b, 0]
        assert (np.diff(row) > 0).all() and row[0] >= 0 and row[-1] < n
    assert np.isin(gi[1, 0], np.arange(0, n, 5)).all()       # +inf outranks every finite score
    # attention on those indices still runs and stays finite (the caches are finite)
    out, _ = g.sparse_attn(0)
    assert torch.isfinite(out.float()).all()


def test_rows_beyond_the_declared_cache_extent_are_refused_not_read():
    """num_cache_rows is the extent of the cache row space; a selected position that maps beyond it is treated like
    an index outside its sequence: skipped and flagged, never dereferenced."""
    w = Workload(MID.replace(num_seqs=2, ctx=1000, top_k=64, num_layers=1))
    g = GpuProblem(w, layers=1)
    g.topk(g.index_scores())
    base, _ = g.sparse_attn(0)
    assert g.status() == 0
    g.params.num_cache_rows = 1500          # the second sequence (rows 1000..1999) now reaches past the extent
    out, _ = g.sparse_attn(0)
    torch.cuda.synchronize()
    assert g.status() & clsa.CLSA_DEV_BAD_INDEX
    assert torch.equal(out[0].view(torch.int16), base[0].view(torch.int16))      # the first sequence is untouched
    assert torch.isfinite(out.float()).all()
    clsa.clsa_clear_status(g.ws)


def test_outputs_may_live_in_pinned_host_memory():
    """The attention outputs are written once with plain stores, so any address the device can reach serves: the
    layers of a decode step store straight into pinned host memory and the host reads the same bits that a device
    buffer would have held (single-block and cluster-merged epilogues both: B = 1 takes the cluster path)."""
    for cfg in (MID.replace(num_seqs=6, ctx=2500, top_k=256, num_layers=3),
                MID.replace(num_seqs=1, ctx=5000, top_k=1024, num_layers=2)):
        w = Workload(cfg)
        g = GpuProblem(w)
        dev_outs = g.decode_step()
        torch.cuda.synchronize()
        host = torch.full((g.L,) + tuple(dev_outs[0].shape), float("nan"), dtype=torch.bfloat16).pin_memory()
        clsa.clsa_sparse_attn_layers(g.params, [g.t["q_layers"][l] for l in range(g.L)], g.idx, g.count,
                                     [host[l] for l in range(g.L)], g.ws)
        torch.cuda.synchronize()
        assert g.status() == 0
        for l in range(g.L):
            assert torch.equal(host[l].view(torch.int16), dev_outs[l].cpu().view(torch.int16)), l


def test_uncleared_workspace_header_is_flagged():
    """The score kernel hands out part of its tiles through two counters in the workspace header, which every launch
    leaves at zero. A header that was never cleared makes it skip tiles; it notices (a ticket beyond the last
    possible one) and sets CLSA_DEV_BAD_WORKSPACE instead of returning wrong scores silently. After
    clsa_clear_status the same workspace works."""
    B, n = 5, 131072                                   # enough tiles for the on-demand part of the schedule
    dev = torch.device("cuda:0")
    gen = torch.Generator(device=dev).manual_seed(3)
    kidx = torch.randn((B * n, 128), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    q = torch.randn((B, 1, 128), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    kv = torch.zeros((8, 8, 128), dtype=torch.bfloat16, device=dev)
    seq_start = torch.arange(B, dtype=torch.int64, device=dev) * n   # the params hold raw pointers: keep these alive
    seq_len = torch.full((B,), n, dtype=torch.int32, device=dev)
    p = clsa.make_params(num_seqs=B, q_per_seq=1, num_q_heads=32, num_kv_heads=8, head_dim=128, idx_dim=128, top_k=64,
                         num_layers=1, max_seq_len=n, sm_scale=0.1, seq_start=seq_start, seq_len=seq_len, k_cache=kv,
                         v_cache=kv, idx_k_cache=kidx)
    good_ws = torch.zeros(clsa.clsa_workspace_bytes(p), dtype=torch.uint8, device=dev)
    want = torch.full((B, 1, n), float("nan"), dtype=torch.float32, device=dev)
    clsa.clsa_index_scores(p, q, want, n, good_ws)
    assert clsa.clsa_device_status(good_ws) == 0
    ref = oracle.Problem(num_seqs=B, num_q_heads=32, num_kv_heads=8, head_dim=128, idx_dim=128, top_k=64, sm_scale=0.1,
                         seq_start=seq_start.cpu().numpy(), seq_len=seq_len.cpu().numpy(),
                         idx_k_cache=_bf16_bits(kidx)).index_scores(_bf16_bits(q), score_stride=n)
    err = np.abs(want.cpu().numpy().astype(np.float64) - ref)
    assert (err <= SCORE_RTOL * np.maximum(1.0, np.abs(ref))).all()
    assert good_ws[:256].count_nonzero().item() == 0                 # the counters are back at zero
    bad_ws = torch.zeros_like(good_ws)
    bad_ws[:256].view(torch.int32)[16] = 1 << 30                     # as if the header had never been cleared
    got = torch.full_like(want, float("nan"))
    clsa.clsa_index_scores(p, q, got, n, bad_ws)
    assert clsa.clsa_device_status(bad_ws) & clsa.CLSA_DEV_BAD_WORKSPACE
    clsa.clsa_clear_status(bad_ws)
    clsa.clsa_index_scores(p, q, got, n, bad_ws)
    assert clsa.clsa_device_status(bad_ws) == 0
    assert torch.equal(got, want)


@pytest.mark.parametrize("d_idx,paged", [(128, 0), (64, 0), (128, 16), (64, 16), (64, 64)])
def test_score_kernel_on_demand_tiles_cover_every_row_once(d_idx, paged):
    """Launches large enough for the on-demand part of the score kernel's schedule (ragged lengths, both indexer
    widths, contiguous and paged caches -- blocks shorter and longer than a warp's run of rows): every visible position gets its score, nothing beyond it is written, a
    second launch on the same workspace gives the same bits (the counters went back to zero), and the values match
    the oracle's fp64 scores within the score tolerance."""
    B, n_max = 24, 131072
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(11 + d_idx)
    lens = rng.integers(1000, n_max + 1, B).astype(np.int32)
    lens[:2] = (n_max, 1)
    gen = torch.Generator(device=dev).manual_seed(5)
    bs = paged if paged else 64
    if paged:
        blocks_per_seq = (n_max + bs - 1) // bs
        nblocks = int(sum((int(x) + bs - 1) // bs for x in lens))
        perm = torch.from_numpy(rng.permutation(nblocks).astype(np.int32))
        table = torch.zeros((B, blocks_per_seq), dtype=torch.int32)
        at = 0
        for b in range(B):
            nb = (int(lens[b]) + bs - 1) // bs
            table[b, :nb] = perm[at: at + nb]
            at += nb
        rows = nblocks * bs
        seq_start = torch.zeros(B, dtype=torch.int64, device=dev)
        table_d = table.to(dev)
    else:
        starts = np.concatenate([[0], np.cumsum((lens.astype(np.int64) + 63) // 64 * 64)[:-1]])
        rows = int(starts[-1] + lens[-1])
        seq_start = torch.from_numpy(starts).to(dev)
        table_d = None
    kidx = torch.randn((rows, d_idx), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    q = torch.randn((B, 1, d_idx), generator=gen, device=dev, dtype=torch.float32).to(torch.bfloat16)
    kv = torch.zeros((8, 8, 128), dtype=torch.bfloat16, device=dev)
    seq_len = torch.from_numpy(lens).to(dev)
    p = clsa.make_params(num_seqs=B, q_per_seq=1, num_q_heads=32, num_kv_heads=8, head_dim=128, idx_dim=d_idx, top_k=64,
                         num_layers=1, max_seq_len=n_max, sm_scale=0.1, seq_start=seq_start, seq_len=seq_len, k_cache=kv,
                         v_cache=kv, idx_k_cache=kidx, block_table=table_d, block_size=bs if paged else 0)
    ws = torch.zeros(clsa.clsa_workspace_bytes(p), dtype=torch.uint8, device=dev)
    outs = []
    for _ in range(2):
        s = torch.full((B, 1, n_max), float("nan"), dtype=torch.float32, device=dev)
        clsa.clsa_index_scores(p, q, s, n_max, ws)
        outs.append(s)
    assert clsa.clsa_device_status(ws) == 0
    assert ws[:256].count_nonzero().item() == 0
    assert torch.equal(outs[0].nan_to_num(nan=-7.0), outs[1].nan_to_num(nan=-7.0))
    got = outs[0][:, 0].cpu().numpy().astype(np.float64)
    ref = oracle.Problem(num_seqs=B, num_q_heads=32, num_kv_heads=8, head_dim=128, idx_dim=d_idx, top_k=64, sm_scale=0.1,
                         seq_start=seq_start.cpu().numpy(), seq_len=lens, idx_k_cache=_bf16_bits(kidx),
                         block_table=table.numpy() if paged else None,
                         block_size=bs if paged else 0).index_scores(_bf16_bits(q), score_stride=n_max)[:, 0]
    for b in range(B):
        n = int(lens[b])
        assert not np.isnan(got[b, :n]).any(), b
        assert np.isnan(got[b, n:]).all(), b
        assert (np.abs(got[b, :n] - ref[b, :n]) <= SCORE_RTOL * np.maximum(1.0, np.abs(ref[b, :n]))).all(), b


def test_gather_probe_runs_the_access_pattern_and_reports_its_duration():
    """The measurement aid: the attention launch's memory accesses without its arithmetic. It writes only into the
    workspace, flags what the attention kernel would flag, and leaves its device-side duration in the header."""
    w = Workload(MID.replace(num_seqs=5, ctx=30000, top_k=1024, num_layers=1, seed=3))
    g = GpuProblem(w)
    gi, gc = g.topk(g.index_scores())
    before = [g.t[k].clone() for k in ("k_cache", "v_cache")]
    clsa.clsa_clear_status(g.ws)
    clsa.clsa_gather_probe(g.params, gi, gc, clsa.make_hints(reverse=1, keep_rows=1), g.ws)
    torch.cuda.synchronize()
    words = g.ws[:32].view(torch.int64).cpu().numpy().view(np.uint64)
    assert int(words[0]) & 0xFFFFFFFF == 0, "no device flag"
    start, end = int(~words[1]) & 0xFFFFFFFFFFFFFFFF, int(words[2])
    assert 0 < end - start < 5_000_000, "duration in nanoseconds of the global timer"
    for k, b in zip(("k_cache", "v_cache"), before):
        assert torch.equal(g.t[k], b)
    bad = gi.clone()
    bad[2, 0, 17] = 10 ** 8
    clsa.clsa_clear_status(g.ws)
    clsa.clsa_gather_probe(g.params, bad, gc, None, g.ws)
    assert g.status() & clsa.CLSA_DEV_BAD_INDEX
    clsa.clsa_clear_status(g.ws)
    # the attention kernel still works on the same workspace afterwards
    out, lse = g.sparse_attn(0)
    check_attention(_full_oracle(w), w, 0, out, lse, gi.cpu().numpy(), gc.cpu().numpy())
