"""ctypes front-end of the CPU oracle (`clsa_oracle.c`). TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the bench's CPU-baseline leg may import this package; the
product (the CUDA library and its binding) never does, and this package imports nothing from it.
Arrays are numpy: bf16 tensors travel as uint16 bit patterns, scores/outputs as float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "clsa_oracle.c")
_LIB = os.path.join(_HERE, "libclsa_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2, OpenMP over independent rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Problem(ctypes.Structure):
    _fields_ = [
        ("num_seqs", ctypes.c_int32), ("q_per_seq", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("idx_dim", ctypes.c_int32),
        ("top_k", ctypes.c_int32), ("causal", ctypes.c_int32), ("sm_scale", ctypes.c_double),
        ("seq_start", ctypes.c_void_p), ("seq_len", ctypes.c_void_p),
        ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
        ("kv_token_stride", ctypes.c_int64), ("kv_head_stride", ctypes.c_int64),
        ("idx_k_cache", ctypes.c_void_p), ("idx_token_stride", ctypes.c_int64),
        ("block_table", ctypes.c_void_p), ("block_size", ctypes.c_int32), ("max_blocks_per_seq", ctypes.c_int32),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_visible.restype = ctypes.c_int64
        _lib.oracle_num_threads.restype = ctypes.c_int32
        _lib.oracle_bf16_from_double.restype = ctypes.c_uint16
        _lib.oracle_bf16_from_double.argtypes = [ctypes.c_double]
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _ptr(a):
    return None if a is None else ctypes.c_void_p(a.ctypes.data)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def linear(h, w) -> np.ndarray:
    """Eq. 2 as a plain product: float64 [rows, n_out] = h [rows, d_model] . w[n_out, d_model]^T from bf16 bits."""
    h, w = _c(h, np.uint16), _c(w, np.uint16)
    assert h.ndim == 2 and w.ndim == 2 and h.shape[1] == w.shape[1]
    y = np.empty((h.shape[0], w.shape[0]), dtype=np.float64)
    lib().oracle_linear(_ptr(h), _ptr(w), ctypes.c_int64(h.shape[0]), ctypes.c_int64(w.shape[0]),
                        ctypes.c_int64(h.shape[1]), _ptr(y))
    return y


def round_bf16(x) -> np.ndarray:
    """Nearest-even bf16 bit patterns (uint16) of float64 values, rounded once."""
    x = _c(x, np.float64)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().oracle_round_bf16(_ptr(x), ctypes.c_int64(x.size), _ptr(out))
    return out


class Problem:
    """Shapes plus the caches of one workload, in the layout the paper's problem statement implies.

    k_cache / v_cache: uint16 [rows, Hkv, D] (may be None for score/top-k only use);
    idx_k_cache: uint16 [rows, d_idx]; seq_start int64 [B]; seq_len int32 [B].
    """

    def __init__(self, *, num_seqs, q_per_seq=1, num_q_heads, num_kv_heads, head_dim, idx_dim, top_k,
                 causal=0, sm_scale, seq_start, seq_len, k_cache=None, v_cache=None, idx_k_cache=None,
                 block_table=None, block_size=0):
        self.B, self.T, self.Hq, self.Hkv = int(num_seqs), int(q_per_seq), int(num_q_heads), int(num_kv_heads)
        self.D, self.d_idx, self.k, self.causal = int(head_dim), int(idx_dim), int(top_k), int(causal)
        self.seq_start = _c(seq_start, np.int64)
        self.seq_len = _c(seq_len, np.int32)
        assert self.seq_start.shape == (self.B,) and self.seq_len.shape == (self.B,)
        assert self.Hq % self.Hkv == 0
        self.k_cache = None if k_cache is None else _c(k_cache, np.uint16)
        self.v_cache = None if v_cache is None else _c(v_cache, np.uint16)
        self.idx_k_cache = None if idx_k_cache is None else _c(idx_k_cache, np.uint16)
        s = _Problem()
        s.num_seqs, s.q_per_seq, s.num_q_heads, s.num_kv_heads = self.B, self.T, self.Hq, self.Hkv
        s.head_dim, s.idx_dim, s.top_k, s.causal = self.D, self.d_idx, self.k, self.causal
        s.sm_scale = float(sm_scale)
        s.seq_start, s.seq_len = _ptr(self.seq_start), _ptr(self.seq_len)
        if self.k_cache is not None:
            assert self.k_cache.ndim == 3 and self.k_cache.shape[1:] == (self.Hkv, self.D)
            assert self.v_cache.shape == self.k_cache.shape
            s.k_cache, s.v_cache = _ptr(self.k_cache), _ptr(self.v_cache)
            s.kv_token_stride, s.kv_head_stride = self.Hkv * self.D, self.D
        if self.idx_k_cache is not None:
            assert self.idx_k_cache.ndim == 2 and self.idx_k_cache.shape[1] == self.d_idx
            s.idx_k_cache, s.idx_token_stride = _ptr(self.idx_k_cache), self.d_idx
        self.block_table = None
        if block_table is not None:
            self.block_table = _c(block_table, np.int32)
            assert self.block_table.ndim == 2 and self.block_table.shape[0] == self.B
            s.block_table = _ptr(self.block_table)
            s.block_size, s.max_blocks_per_seq = int(block_size), int(self.block_table.shape[1])
        self._s = s

    @property
    def max_seq_len(self) -> int:
        return int(self.seq_len.max())

    def visible(self, b: int, t: int) -> int:
        return int(lib().oracle_visible(ctypes.byref(self._s), b, t))

    # Eq. 3, scores -----------------------------------------------------------------------
    def index_scores(self, q_idx, score_stride=None) -> np.ndarray:
        """float64 [B, T, score_stride]; positions that are not visible hold NaN."""
        q_idx = _c(q_idx, np.uint16).reshape(self.B, self.T, self.d_idx)
        stride = int(score_stride or self.max_seq_len)
        scores = np.full((self.B, self.T, stride), np.nan, dtype=np.float64)
        lib().oracle_index_scores(ctypes.byref(self._s), _ptr(q_idx), _ptr(scores), ctypes.c_int64(stride))
        return scores

    # Eq. 3, TopK -------------------------------------------------------------------------
    def topk(self, scores, selector: str = "sort"):
        """(idx int32 [B,T,k] with -1 tail, count int32 [B,T]) from float64 scores [B,T,stride]."""
        scores = _c(scores, np.float64)
        assert scores.ndim == 3 and scores.shape[:2] == (self.B, self.T)
        idx = np.empty((self.B, self.T, self.k), dtype=np.int32)
        count = np.empty((self.B, self.T), dtype=np.int32)
        lib().oracle_topk(ctypes.byref(self._s), _ptr(scores), ctypes.c_int64(scores.shape[2]),
                          ctypes.c_int32({"sort": 0, "select": 1}[selector]), _ptr(idx), _ptr(count))
        return idx, count

    # Eq. 4 -------------------------------------------------------------------------------
    def sparse_attn(self, q, idx, count):
        """(out float64 [B,T,Hq,D], lse float64 [B,T,Hq]) for one layer's bf16 queries."""
        q = _c(q, np.uint16).reshape(self.B, self.T, self.Hq, self.D)
        idx = _c(idx, np.int32).reshape(self.B, self.T, self.k)
        count = _c(count, np.int32).reshape(self.B, self.T)
        out = np.empty((self.B, self.T, self.Hq, self.D), dtype=np.float64)
        lse = np.empty((self.B, self.T, self.Hq), dtype=np.float64)
        lib().oracle_sparse_attn(ctypes.byref(self._s), _ptr(q), _ptr(idx), _ptr(count), _ptr(out), _ptr(lse))
        return out, lse

    # Eq. 1 -------------------------------------------------------------------------------
    def dense_attn(self, q):
        q = _c(q, np.uint16).reshape(self.B, self.T, self.Hq, self.D)
        out = np.empty((self.B, self.T, self.Hq, self.D), dtype=np.float64)
        lse = np.empty((self.B, self.T, self.Hq), dtype=np.float64)
        lib().oracle_dense_attn(ctypes.byref(self._s), _ptr(q), _ptr(out), _ptr(lse))
        return out, lse

    # Eq. 2 + cache append ----------------------------------------------------------------
    def project_append(self, h, w_q_idx, w_k_idx, w_k=None, w_v=None) -> np.ndarray:
        """Projects the T newest tokens of every sequence (h: uint16 [B,T,d_model]; weights uint16 [n_out, d_model])
        and writes their K_idx (and, with w_k/w_v, K and V) rows into this problem's caches IN PLACE.
        Returns q_idx as uint16 [B,T,d_idx]."""
        h = _c(h, np.uint16)
        d_model = h.shape[-1]
        h = h.reshape(self.B, self.T, d_model)
        w_q_idx, w_k_idx = _c(w_q_idx, np.uint16), _c(w_k_idx, np.uint16)
        assert w_q_idx.shape == (self.d_idx, d_model) and w_k_idx.shape == (self.d_idx, d_model)
        assert self.idx_k_cache is not None and self.idx_k_cache.flags.writeable
        if w_k is not None:
            w_k, w_v = _c(w_k, np.uint16), _c(w_v, np.uint16)
            assert w_k.shape == (self.Hkv * self.D, d_model) and w_v.shape == w_k.shape
            assert self.k_cache is not None and self.k_cache.flags.writeable and self.v_cache.flags.writeable
        q_idx = np.empty((self.B, self.T, self.d_idx), dtype=np.uint16)
        lib().oracle_project_append(ctypes.byref(self._s), ctypes.c_int32(d_model), _ptr(h), _ptr(w_q_idx),
                                    _ptr(w_k_idx), _ptr(w_k), _ptr(w_v), _ptr(q_idx))
        return q_idx

    # whole step --------------------------------------------------------------------------
    def decode_step(self, q_idx, q_layers):
        """q_layers: uint16 [L,B,T,Hq,D]. Returns dict(scores, idx, count, out [L,...], lse [L,...])."""
        q_idx = _c(q_idx, np.uint16).reshape(self.B, self.T, self.d_idx)
        q_layers = _c(q_layers, np.uint16)
        L = q_layers.shape[0]
        assert q_layers.shape == (L, self.B, self.T, self.Hq, self.D)
        stride = self.max_seq_len
        scores = np.full((self.B, self.T, stride), np.nan, dtype=np.float64)
        idx = np.empty((self.B, self.T, self.k), dtype=np.int32)
        count = np.empty((self.B, self.T), dtype=np.int32)
        out = np.empty((L, self.B, self.T, self.Hq, self.D), dtype=np.float64)
        lse = np.empty((L, self.B, self.T, self.Hq), dtype=np.float64)
        lib().oracle_decode_step(ctypes.byref(self._s), ctypes.c_int32(L), _ptr(q_idx), _ptr(q_layers),
                                 _ptr(scores), ctypes.c_int64(stride), _ptr(idx), _ptr(count), _ptr(out), _ptr(lse))
        return {"scores": scores, "idx": idx, "count": count, "out": out, "lse": lse}


def problem_from_workload(w, k_cache=None, v_cache=None, idx_k_cache=None, block_table=None, block_size=0) -> Problem:
    """Problem for a `workloads.Workload` (duck-typed: only its cfg fields and packing are read)."""
    c = w.cfg
    return Problem(num_seqs=c.num_seqs, q_per_seq=c.q_per_seq, num_q_heads=c.num_q_heads,
                   num_kv_heads=c.num_kv_heads, head_dim=c.head_dim, idx_dim=c.idx_dim, top_k=c.top_k,
                   causal=c.causal, sm_scale=c.sm_scale, seq_start=w.seq_start, seq_len=w.seq_len,
                   k_cache=k_cache, v_cache=v_cache, idx_k_cache=idx_k_cache, block_table=block_table,
                   block_size=block_size)
