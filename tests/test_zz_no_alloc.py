"""The workspace-free entry point, `clsa_decode_step_static`, against `clsa_decode_step` and the oracle.

Who needs it: callers that are handed device tensors but may not allocate -- a step that runs
where cudaMalloc is forbidden or would stall the device, or inside a process whose memory is
already fully reserved by a pool. They cannot provide the workspace `clsa_decode_step` asks for,
so the library keeps a 16 MiB scratch array of its own for them. This test calls the entry point
through the C ABI twice in a row (the second call finds the first call's contents still in the
array) and checks both results bit for bit against the ordinary entry point and, within the output
tolerance, against the oracle; it plants a bad index entry and reads the flag back through a
caller-owned status word, then checks that the next call is clean again; and it checks that a shape
beyond the array's fixed capacity is refused before anything runs. This file sorts last on purpose.
"""
import pytest

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("no CUDA device", allow_module_level=True)

import __graft_entry__ as entry

entry._load_build_module().build()

import numpy as np

import oracle
import paper_2606_06467_b200 as clsa
from _harness import GpuProblem, check_attention
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
    """The two entry points run the same launches on different scratch: identical bits."""
    assert torch.equal(idx, ref_idx) and torch.equal(cnt, ref_cnt)
    for a, b in zip(ref_outs, outs):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def _against_oracle(g, outs, idx, cnt):
    w = g.w
    kc, vc = w.host_kv_full()
    prob = oracle.problem_from_workload(w, k_cache=kc, v_cache=vc, idx_k_cache=w.host_kidx_cache())
    idx_np, cnt_np = idx.cpu().numpy(), cnt.cpu().numpy()
    ref_idx, ref_cnt = prob.topk(prob.index_scores(w.q_idx_bits()))
    np.testing.assert_array_equal(cnt_np, ref_cnt)
    # the oracle's own index on >= 99 % of the slots (the rest: scores within the tolerance band of the k-th)
    same = sum(len(set(idx_np[b, 0, :cnt_np[b, 0]]) & set(ref_idx[b, 0, :ref_cnt[b, 0]])) for b in range(w.cfg.num_seqs))
    assert same >= 0.99 * int(ref_cnt.sum())
    for l in range(g.L):
        check_attention(prob, w, l, outs[l], None, idx_np, cnt_np)


def test_static_entry_point_matches_decode_step_twice_in_a_row():
    # first problem: two sequences, several kernel tiles, a ragged tail
    g1 = GpuProblem(Workload(MID.replace(num_seqs=2, ctx=20000 + 13, top_k=512, num_layers=3, seed=4242)))
    ref1 = g1.decode_step()
    torch.cuda.synchronize()
    ref1_idx, ref1_cnt = g1.idx.clone(), g1.count.clone()
    outs, idx, cnt = _run_static(g1)
    _same(ref1, ref1_idx, ref1_cnt, outs, idx, cnt)
    _against_oracle(g1, outs, idx, cnt)
    # second call, different shape and data: the array still holds the first call's scores and partials
    g2 = GpuProblem(Workload(MID.replace(num_seqs=3, ctx=7000, top_k=300, num_layers=2, seed=777)))
    ref2 = g2.decode_step()
    torch.cuda.synchronize()
    ref2_idx, ref2_cnt = g2.idx.clone(), g2.count.clone()
    status = torch.zeros(1, dtype=torch.int32, device=g2.dev)
    outs, idx, cnt = _run_static(g2, status)
    _same(ref2, ref2_idx, ref2_cnt, outs, idx, cnt)
    _against_oracle(g2, outs, idx, cnt)
    assert int(status.item()) == 0
    # and the first problem again, straight after
    outs, idx, cnt = _run_static(g1)
    _same(ref1, ref1_idx, ref1_cnt, outs, idx, cnt)


def test_static_entry_point_reports_device_flags_and_recovers():
    """A sequence whose length lies outside its declared bound is skipped and flagged; the flag arrives in the
    caller's own status word, and the call after it -- on the same built-in array -- is clean and correct again
    (every call zeroes the array's counters itself, whoever owns the status word)."""
    g = GpuProblem(Workload(MID.replace(num_seqs=3, ctx=9000, top_k=256, num_layers=2, seed=99)))
    ref = g.decode_step()
    torch.cuda.synchronize()
    ref_idx, ref_cnt = g.idx.clone(), g.count.clone()
    status = torch.zeros(1, dtype=torch.int32, device=g.dev)
    lens = g.t["seq_len"].clone()
    g.t["seq_len"][1] = g.params.max_seq_len + 5
    outs, idx, cnt = _run_static(g, status)
    assert int(status.item()) & clsa.CLSA_DEV_BAD_SEQLEN
    assert int(cnt[1, 0].item()) == 0 and (outs[0][1].float() == 0).all()
    assert torch.equal(outs[0][0].view(torch.int16), ref[0][0].view(torch.int16))   # the other sequences are untouched
    g.t["seq_len"].copy_(lens)
    status.zero_()
    outs, idx, cnt = _run_static(g, status)
    assert int(status.item()) == 0
    _same(ref, ref_idx, ref_cnt, outs, idx, cnt)
    outs, idx, cnt = _run_static(g)          # the built-in status word this time
    _same(ref, ref_idx, ref_cnt, outs, idx, cnt)


def test_static_entry_point_refuses_shapes_beyond_its_scratch():
    w = Workload(MID.replace(num_seqs=2, ctx=4096, top_k=64, num_layers=1))
    g = GpuProblem(w)
    g.params.num_seqs = 17
    g.params.max_seq_len = 4 * 131072        # 17 * 524288 fp32 scores alone exceed the 16 MiB array
    with pytest.raises(clsa.ClsaError) as e:
        clsa.clsa_decode_step_static(g.params, g.t["q_idx"], [g.t["q_layers"][0]], [g.new_out()], g.idx, g.count)
    assert e.value.status == clsa.CLSA_ERR_WORKSPACE
