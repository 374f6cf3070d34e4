"""Shared plumbing of the GPU parity tests: run the CUDA path through the C ABI, run the oracle on the
same seeded inputs, and compare under the stated tolerances.

Tolerances (the acceptance tolerances of this library, with their derivation):
  scores   |gpu - oracle| <= 1e-4 * max(1, |oracle|): bf16 x bf16 products are exact in fp32, so the only
           error is the fp32 accumulation of d_idx <= 128 terms (<= 128 * 2^-24 relative to the sum of
           magnitudes, about 8e-6 * sum|terms|).
  top-k    (a) the GPU index set equals, bit for bit, the oracle's TopK applied to the GPU's own fp32
           scores (the selection itself is integer work and must be exact);
           (b) against the oracle's fp64 scores the sets are identical unless the oracle's k-th and
           (k+1)-th scores differ by less than 1e-3 relative, and then only positions whose oracle
           score lies within 1e-3 * |tau_k| of the k-th score tau_k may differ.
  output   max |gpu - oracle| <= 2e-2 and mean |gpu - oracle| <= 2e-3 (bf16 output rounding is 2^-9
           relative; softmax weights are rounded to bf16 before the PV product).
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2606_06467_b200 as clsa
from workloads import Workload

SCORE_RTOL = 1e-4
BAND = 1e-3
OUT_MAX_ABS = 2e-2
OUT_MEAN_ABS = 2e-3


class GpuProblem:
    """Device tensors, params and workspace of one workload."""

    def __init__(self, w: Workload, device="cuda:0", layers=None, block_size=0):
        self.w, self.cfg = w, w.cfg
        c = w.cfg
        self.dev = torch.device(device)
        self.t = w.to_device(self.dev, layers=layers)
        if block_size:  # same contents, caches rearranged into scattered blocks
            self.t = w.paginate_device(self.t, block_size)
        self.L = c.num_layers if layers is None else layers
        self.params = clsa.make_params(
            num_seqs=c.num_seqs, q_per_seq=c.q_per_seq, num_q_heads=c.num_q_heads, num_kv_heads=c.num_kv_heads,
            head_dim=c.head_dim, idx_dim=c.idx_dim, top_k=c.top_k, num_layers=self.L, causal=c.causal,
            max_seq_len=w.max_seq_len, sm_scale=c.sm_scale, seq_start=self.t["seq_start"], seq_len=self.t["seq_len"],
            k_cache=self.t["k_cache"], v_cache=self.t["v_cache"], idx_k_cache=self.t["idx_k_cache"],
            block_table=self.t.get("block_table"), block_size=block_size)
        self.ws = torch.zeros(clsa.clsa_workspace_bytes(self.params), dtype=torch.uint8, device=self.dev)
        self.score_stride = (w.max_seq_len + 63) // 64 * 64
        B, T = c.num_seqs, c.q_per_seq
        self.idx = torch.full((B, T, c.top_k), -7, dtype=torch.int32, device=self.dev)
        self.count = torch.full((B, T), -7, dtype=torch.int32, device=self.dev)

    def new_scores(self):
        c = self.cfg
        return torch.full((c.num_seqs, c.q_per_seq, self.score_stride), float("nan"), dtype=torch.float32, device=self.dev)

    def new_out(self):
        c = self.cfg
        return torch.full((c.num_seqs, c.q_per_seq, c.num_q_heads, c.head_dim), float("nan"), dtype=torch.bfloat16,
                          device=self.dev)

    def index_scores(self):
        s = self.new_scores()
        clsa.clsa_index_scores(self.params, self.t["q_idx"], s, self.score_stride, self.ws)
        return s

    def topk(self, scores):
        clsa.clsa_topk(self.params, scores, scores.shape[-1], self.idx, self.count, self.ws)
        return self.idx, self.count

    def sparse_attn(self, layer, idx=None, count=None, lse=True, reverse=0, shared_gpu=0, keep_rows=0, only_q_pending=0):
        """One layer through clsa_sparse_attn (all hints zero) or clsa_sparse_attn_hinted."""
        c = self.cfg
        out = self.new_out()
        l = torch.full((c.num_seqs, c.q_per_seq, c.num_q_heads), float("nan"), dtype=torch.float32, device=self.dev) if lse else None
        args = (self.params, self.t["q_layers"][layer], self.idx if idx is None else idx,
                self.count if count is None else count, out, l)
        if reverse or shared_gpu or keep_rows or only_q_pending:
            clsa.clsa_sparse_attn_hinted(*args, clsa.make_hints(reverse, shared_gpu, keep_rows, only_q_pending), self.ws)
        else:
            clsa.clsa_sparse_attn(*args, self.ws)
        return out, l

    def decode_step(self):
        outs = [self.new_out() for _ in range(self.L)]
        clsa.clsa_decode_step(self.params, self.t["q_idx"], [self.t["q_layers"][l] for l in range(self.L)], outs,
                              self.idx, self.count, self.ws)
        return outs

    def status(self) -> int:
        return clsa.clsa_device_status(self.ws)


def oracle_scores_and_topk(w: Workload):
    """Oracle problem (indexer keys only), fp64 scores and TopK for a workload."""
    prob = oracle.problem_from_workload(w, idx_k_cache=w.host_kidx_cache())
    scores = prob.index_scores(w.q_idx_bits())
    idx, cnt = prob.topk(scores)
    return prob, scores, idx, cnt


def check_scores(gpu_scores: torch.Tensor, ref: np.ndarray, w: Workload):
    got = gpu_scores.cpu().numpy().astype(np.float64)
    c = w.cfg
    for b in range(c.num_seqs):
        for t in range(c.q_per_seq):
            v = w.visible(b, t)
            r = ref[b, t, :v]
            err = np.abs(got[b, t, :v] - r)
            assert (err <= SCORE_RTOL * np.maximum(1.0, np.abs(r))).all(), (b, t, err.max())
            assert np.isnan(got[b, t, v:]).all(), "scores past the visible prefix must not be written"


def check_topk_exact_on_gpu_scores(prob, gpu_scores: torch.Tensor, gpu_idx: torch.Tensor, gpu_cnt: torch.Tensor, w: Workload):
    """(a): the selection is exact given the GPU's own fp32 scores; positions ascending; tail -1."""
    sc = gpu_scores.cpu().numpy().astype(np.float64)
    ref_idx, ref_cnt = prob.topk(sc)
    gi, gc = gpu_idx.cpu().numpy(), gpu_cnt.cpu().numpy()
    np.testing.assert_array_equal(gc, ref_cnt)
    c = w.cfg
    for b in range(c.num_seqs):
        for t in range(c.q_per_seq):
            n = gc[b, t]
            assert n == min(c.top_k, w.visible(b, t))
            got = gi[b, t, :n]
            assert (np.diff(got) > 0).all(), "positions must be ascending and distinct"
            np.testing.assert_array_equal(got, np.sort(ref_idx[b, t, :n]))
            assert (gi[b, t, n:] == -1).all()


def check_topk_band(ref_scores: np.ndarray, ref_idx, ref_cnt, gpu_idx: torch.Tensor, gpu_cnt: torch.Tensor, w: Workload):
    """(b): against the oracle's own fp64 scores, only positions inside the 1e-3 band may differ."""
    gi, gc = gpu_idx.cpu().numpy(), gpu_cnt.cpu().numpy()
    np.testing.assert_array_equal(gc, ref_cnt)
    c = w.cfg
    n_band_rows = 0
    for b in range(c.num_seqs):
        for t in range(c.q_per_seq):
            n = gc[b, t]
            got, want = set(gi[b, t, :n].tolist()), set(ref_idx[b, t, :n].tolist())
            if got == want:
                continue
            v = w.visible(b, t)
            s = ref_scores[b, t, :v]
            order = np.sort(s)[::-1]
            tau_k, tau_k1 = order[n - 1], order[n]
            assert tau_k - tau_k1 < BAND * abs(tau_k), "sets differ although the k-th and (k+1)-th scores are well separated"
            diff = np.array(sorted(got ^ want))
            assert (np.abs(s[diff] - tau_k) <= BAND * abs(tau_k)).all(), (b, t, diff[:8])
            n_band_rows += 1
    return n_band_rows


def check_attention(prob, w: Workload, layer: int, gpu_out: torch.Tensor, gpu_lse, idx: np.ndarray, cnt: np.ndarray):
    o_ref, l_ref = prob.sparse_attn(w.q_layer_bits(layer), idx, cnt)
    got = gpu_out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    err = np.abs(got - o_ref)
    assert err.max() <= OUT_MAX_ABS, (layer, err.max())
    assert err.mean() <= OUT_MEAN_ABS, (layer, err.mean())
    if gpu_lse is not None:
        gl = gpu_lse.cpu().numpy().astype(np.float64)
        fin = np.isfinite(l_ref)
        np.testing.assert_array_equal(np.isneginf(gl), ~fin)
        assert np.abs(gl[fin] - l_ref[fin]).max() <= 2e-3 * max(1.0, np.abs(l_ref[fin]).max())
    return err.max(), err.mean()
