"""Stream ordering behind a chained step.

The layers of `clsa_decode_step` are launched with programmatic dependent launch and, after the first, do not wait
for their predecessors. Everything that follows the call on the stream -- the bench's end event, a copy of the
outputs, the next step's `clsa_topk` rewriting the shared index -- relies on being ordered behind EVERY layer of the
chain, not only the last one. This test pins that: straight after the call, with no synchronisation, it enqueues
plain device copies of all L outputs and a `clsa_topk` on different scores into the same index buffers; the copies
must hold the (oracle-checked) outputs of the original index, repetition after repetition, each behind an L2 flush.
A layer that were still running when the copies or the second top-k started would show up as a stale or torn
output.
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
from _harness import GpuProblem, check_attention
from workloads import MID, Workload

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,ctx,k,L", [(16, 16384, 2048, 16), (3, 6000, 512, 5)])
def test_work_behind_a_chained_step_is_ordered_behind_every_layer(B, ctx, k, L):
    w = Workload(MID.replace(num_seqs=B, ctx=ctx, top_k=k, num_layers=L, seed=123))
    g = GpuProblem(w)
    c = w.cfg
    # reference run, synchronised, checked against the oracle
    ref = g.decode_step()
    torch.cuda.synchronize()
    ref_idx, ref_cnt = g.idx.clone(), g.count.clone()
    kc, vc = w.host_kv_sparse(ref_idx.cpu().numpy(), ref_cnt.cpu().numpy())
    prob = oracle.problem_from_workload(w, k_cache=kc, v_cache=vc, idx_k_cache=w.host_kidx_cache())
    for l in (0, L // 2, L - 1):
        check_attention(prob, w, l, ref[l], None, ref_idx.cpu().numpy(), ref_cnt.cpu().numpy())
    # other scores for the trailing top-k: a different selection lands in the same idx/count buffers
    gen = torch.Generator(device=g.dev).manual_seed(7)
    other = torch.randn((B, 1, g.score_stride), generator=gen, device=g.dev, dtype=torch.float32)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=g.dev)
    qs = [g.t["q_layers"][l] for l in range(L)]
    outs = [g.new_out() for _ in range(L)]
    copies = torch.empty((L,) + tuple(outs[0].shape), dtype=torch.bfloat16, device=g.dev)
    for rep in range(60):
        flush.fill_(rep & 0xff)
        for o in outs:
            o.fill_(float("nan"))
        clsa.clsa_decode_step(g.params, g.t["q_idx"], qs, outs, g.idx, g.count, g.ws)
        for l in range(L):                      # no synchronisation: plain copies queued straight behind the chain
            copies[l].copy_(outs[l], non_blocking=True)
        clsa.clsa_topk(g.params, other, g.score_stride, g.idx, g.count, g.ws)   # rewrites the index the layers read
        torch.cuda.synchronize()
        for l in range(L):
            assert torch.equal(copies[l].view(torch.int16), ref[l].view(torch.int16)), f"repetition {rep}, layer {l}"
        assert not torch.equal(g.idx, ref_idx), "the trailing top-k selected from other scores"
    assert g.status() == 0
