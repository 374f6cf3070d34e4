"""`clsa_decode_step` only enqueues work on the caller's stream (no allocation, no synchronisation), so a step can be
captured into a CUDA graph and replayed; the replay must reproduce the eager result byte for byte."""
import pytest

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import __graft_entry__ as entry

entry._load_build_module().build()

import paper_2606_06467_b200 as clsa
from _harness import GpuProblem
from workloads import MID, Workload

pytestmark = pytest.mark.gpu


def test_decode_step_replays_from_a_cuda_graph():
    w = Workload(MID.replace(num_seqs=4, ctx=12000, top_k=512, num_layers=4, seed=99))
    g = GpuProblem(w)
    eager = g.decode_step()                       # also warms up every per-device cache of the library
    torch.cuda.synchronize()
    eager_idx, eager_cnt = g.idx.clone(), g.count.clone()
    outs = [g.new_out() for _ in range(g.L)]
    qs = [g.t["q_layers"][l] for l in range(g.L)]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        g.idx.fill_(-7)
        g.count.fill_(-7)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            clsa.clsa_decode_step(g.params, g.t["q_idx"], qs, outs, g.idx, g.count, g.ws, stream=side)
    for _ in range(3):
        g.idx.fill_(-7)
        for o in outs:
            o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(g.idx, eager_idx) and torch.equal(g.count, eager_cnt)
        for a, b in zip(outs, eager):
            assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    assert g.status() == 0
