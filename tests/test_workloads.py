"""The synthetic-input generator: determinism, host/torch agreement, and the structure each config promises."""
import numpy as np
import torch

from workloads import HEADLINE, MID, PREFILL, RAGGED, TINY, Workload
from workloads import generator as g


def test_mix64_vector_forms_match_the_scalar_form():
    xs = np.array([0, 1, 2, 0xDEADBEEF, (1 << 63) + 12345, (1 << 64) - 1], dtype=np.uint64)
    want = np.array([g.mix64_int(int(x)) for x in xs], dtype=np.uint64)
    np.testing.assert_array_equal(g.mix64_np(xs), want)
    got = g.mix64_torch(torch.from_numpy(xs.view(np.int64).copy())).numpy().view(np.uint64)
    np.testing.assert_array_equal(got, want)


def test_stream_host_equals_torch_fill_and_is_normal():
    s = g.Stream(0xC15A0001, 3)
    host = s.host_range(0, 200_000)
    t = torch.empty(200_000, dtype=torch.bfloat16)
    s.device_fill(t, chunk=70_001)
    np.testing.assert_array_equal(t.view(torch.int16).numpy().view(np.uint16), host)
    vals = g.bf16_bits_to_f64(host)
    assert abs(vals.mean()) < 0.01 and abs(vals.std() - 1.0) < 0.01
    rows = s.host_rows(np.array([5, 0, 5]), 64)
    np.testing.assert_array_equal(rows[0], host[5 * 64: 6 * 64])
    np.testing.assert_array_equal(rows[1], host[:64])
    np.testing.assert_array_equal(rows[0], rows[2])


def test_bf16_round_trip():
    x = np.array([0.0, 1.0, -2.5, 3.140625, 1e-3, 65280.0])
    b = g.f64_to_bf16_bits(x)
    y = g.bf16_bits_to_f64(b)
    assert (np.abs(y - x) <= np.abs(x) * 2 ** -8).all()
    np.testing.assert_array_equal(g.f64_to_bf16_bits(y), b)
    # ties round to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert g.bf16_bits_to_f64(g.f64_to_bf16_bits(np.array([1 + 2 ** -8])))[0] == 1.0
    assert g.bf16_bits_to_f64(g.f64_to_bf16_bits(np.array([1 + 3 * 2 ** -8])))[0] == 1 + 2 ** -6


def test_config_shapes_and_algorithmic_bytes():
    assert Workload(TINY).algorithmic_bytes() == 1_048_576
    assert Workload(MID).algorithmic_bytes() == 1_140_850_688
    assert Workload(HEADLINE).algorithmic_bytes() == 2_684_354_560
    w = Workload(RAGGED)
    assert w.cfg.num_seqs == 64 and w.seq_len.min() >= 1024 and w.seq_len.max() <= 131072
    assert (w.seq_len < w.cfg.top_k).sum() >= 4
    assert (w.seq_start % 64 == 0).all() and (np.diff(w.seq_start) >= w.seq_len[:-1]).all()
    p = Workload(PREFILL)
    assert p.visible(0, 0) == 131072 + 1 and p.visible(0, 4095) == 131072 + 4096


def test_duplicates_and_planting():
    w = Workload(RAGGED.replace(num_seqs=3, ctx=4096, ragged_min=512, num_short=1, top_k=1024))
    src = w.row_source()
    frac = (src != np.arange(src.size)).mean()
    assert 0.02 < frac < 0.08
    b = 1
    rows = w.kidx_bits(b)
    s0 = int(w.seq_start[b])
    local_src = src[s0: s0 + int(w.seq_len[b])] - s0
    dup = np.nonzero(local_src != np.arange(local_src.size))[0]
    assert dup.size > 0 and (local_src[dup] < dup).all()
    base = g.Stream(w.cfg.seed, 1).host_rows(s0 + local_src[dup], w.cfg.idx_dim)
    np.testing.assert_array_equal(rows[dup], base)          # exact copies of an earlier position's base row
    h = Workload(HEADLINE.replace(num_seqs=2, ctx=8192))
    pos = h.planted_positions(1)
    assert pos.size == 64 and np.unique(pos).size == 64
    keys = g.bf16_bits_to_f64(h.kidx_bits(1))
    q = g.bf16_bits_to_f64(h.q_idx_bits()[1, 0])
    sc = keys @ q
    sigma = np.linalg.norm(q)
    plain = np.delete(sc, pos)
    assert abs(plain.std() / sigma - 1) < 0.05
    assert (sc[pos].mean() - plain.mean()) / sigma > 3.5      # planted tokens sit about +4 sigma up


def test_to_device_matches_host_on_cpu():
    w = Workload(RAGGED.replace(num_seqs=3, ctx=2048, ragged_min=256, num_short=1, top_k=512, num_layers=2))
    d = w.to_device("cpu")
    bits = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits(d["idx_k_cache"])[w.seq_start[2]: w.seq_start[2] + w.seq_len[2]], w.kidx_bits(2))
    k, v = w.host_kv_full()
    np.testing.assert_array_equal(bits(d["k_cache"]), k)
    np.testing.assert_array_equal(bits(d["v_cache"]), v)
    np.testing.assert_array_equal(bits(d["q_layers"][1]), w.q_layer_bits(1))
    np.testing.assert_array_equal(bits(d["q_idx"]), w.q_idx_bits())
    h = Workload(HEADLINE.replace(num_seqs=2, ctx=4096))
    dh = h.to_device("cpu", layers=1)
    np.testing.assert_array_equal(bits(dh["idx_k_cache"])[4096:], h.kidx_bits(1))


def test_projection_inputs_host_equal_device_and_are_scaled_exactly():
    import torch

    w = Workload(TINY.replace(d_model=96))
    d = w.projection_to_device("cpu")
    bits = lambda t: t.view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits(d["h"]), w.hidden_bits())
    for which in ("q_idx", "k_idx", "k", "v"):
        host = w.weight_bits(which)
        assert host.shape == w.weight_shape(which)
        np.testing.assert_array_equal(bits(d["w_" + which]), host)
    assert abs(g.bf16_bits_to_f64(w.weight_bits("k")).std() * 64 - 1.0) < 0.05
