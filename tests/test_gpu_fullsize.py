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
