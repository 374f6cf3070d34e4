"""The workspace-free entry point, `clsa_decode_step_static`, against `clsa_decode_step`.

Who needs it: callers that are handed device tensors but may not allocate -- a step that runs
where cudaMalloc is forbidden or would stall the device, or inside a process whose memory is
already fully reserved by a pool. They cannot provide the workspace `clsa_decode_step` asks for,
so the library keeps an 8 MiB scratch array of its own for them. This test calls the entry point
through the C ABI twice in a row (the second call finds the first call's scores still in the array)
and checks both results against the ordinary entry point; it also checks that a shape beyond the
array's fixed capacity is refused before anything runs. This file sorts last on purpose.
"""
import pytest

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import __graft_entry__ as entry

entry._load_build_module().build()

import paper_2606_06467_b200 as clsa
from _harness import OUT_MAX_ABS, OUT_MEAN_ABS, GpuProblem
from workloads import MID, Workload

pytestmark = pytest.mark.gpu


def _run_static(g, dev_status=None):
    outs = [g.new_out() for _ in range(g.L)]
    idx = torch.full_like(g.idx, -7)
    cnt = torch.full_like(g.count, -7)
    clsa.clsa_decode_step_static(g.params, g.t["q_idx"], [g.t["q_layers"][l] for l in range(g.L)], outs, idx, cnt,
                                 dev_status)
    torch.cuda.synchronize()
    return outs, idx, cnt


def _same(ref_outs, ref_idx, ref_cnt, outs, idx, cnt):
    assert torch.equal(idx, ref_idx) and torch.equal(cnt, ref_cnt)
    for a, b in zip(ref_outs, outs):
        err = (a.float() - b.float()).abs()
        assert err.max().item() <= OUT_MAX_ABS and err.mean().item() <= OUT_MEAN_ABS


def test_static_entry_point_matches_decode_step_twice_in_a_row():
    # first problem: two sequences, several kernel tiles, a ragged tail
    g1 = GpuProblem(Workload(MID.replace(num_seqs=2, ctx=20000 + 13, top_k=512, num_layers=3, seed=4242)))
    ref1 = g1.decode_step()
    torch.cuda.synchronize()
    ref1_idx, ref1_cnt = g1.idx.clone(), g1.count.clone()
    outs, idx, cnt = _run_static(g1)
    _same(ref1, ref1_idx, ref1_cnt, outs, idx, cnt)
    # second call, different shape and data: the array still holds the first call's scores
    g2 = GpuProblem(Workload(MID.replace(num_seqs=3, ctx=7000, top_k=300, num_layers=2, seed=777)))
    ref2 = g2.decode_step()
    torch.cuda.synchronize()
    ref2_idx, ref2_cnt = g2.idx.clone(), g2.count.clone()
    status = torch.zeros(1, dtype=torch.int32, device=g2.dev)
    outs, idx, cnt = _run_static(g2, status)
    _same(ref2, ref2_idx, ref2_cnt, outs, idx, cnt)
    assert int(status.item()) == 0
    # and the first problem again, straight after
    outs, idx, cnt = _run_static(g1)
    _same(ref1, ref1_idx, ref1_cnt, outs, idx, cnt)


def test_static_entry_point_refuses_shapes_beyond_its_scratch():
    w = Workload(MID.replace(num_seqs=2, ctx=4096, top_k=64, num_layers=1))
    g = GpuProblem(w)
    g.params.num_seqs = 17
    g.params.max_seq_len = 131072            # 17 * 131072 score slots > 2 Mi
    with pytest.raises(clsa.ClsaError) as e:
        clsa.clsa_decode_step_static(g.params, g.t["q_idx"], [g.t["q_layers"][0]], [g.new_out()], g.idx, g.count)
    assert e.value.status == clsa.CLSA_ERR_WORKSPACE
