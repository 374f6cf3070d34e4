"""Python binding of the CLSA C-ABI library (`libclsa.so`, hand-written CUDA for sm_100a).

Argument marshalling only: every function below has the name and the argument order of its
`include/clsa.h` counterpart, takes torch CUDA tensors (or raw device addresses) and passes their
pointers through ctypes. No step of the path runs in Python or in torch; torch supplies device
memory and streams. There is no fallback: if the library has not been built, importing this
package raises.
"""
from __future__ import annotations

import ctypes
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libclsa.so")

CLSA_OK, CLSA_ERR_INVALID_ARG, CLSA_ERR_UNSUPPORTED, CLSA_ERR_WORKSPACE, CLSA_ERR_CUDA = range(5)
CLSA_DEV_BAD_INDEX, CLSA_DEV_BAD_SEQLEN, CLSA_DEV_BAD_COUNT, CLSA_DEV_TIMEOUT, CLSA_DEV_BAD_WORKSPACE = 1, 2, 4, 8, 16
CLSA_DEV_ROUTING_OVERFLOW = 32

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it first (python paper_2606_06467_b200/build.py, or "
        "__graft_entry__.build()). This package has no CPU or PyTorch fallback.")

_lib = ctypes.CDLL(LIB_PATH)


class clsa_params(ctypes.Structure):
    """Mirror of `clsa_params` in include/clsa.h (same field order and types)."""

    _fields_ = [
        ("num_seqs", ctypes.c_int32), ("q_per_seq", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("idx_dim", ctypes.c_int32),
        ("top_k", ctypes.c_int32), ("num_layers", ctypes.c_int32), ("causal", ctypes.c_int32),
        ("max_seq_len", ctypes.c_int32), ("sm_scale", ctypes.c_float),
        ("seq_start", ctypes.c_void_p), ("seq_len", ctypes.c_void_p),
        ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
        ("kv_token_stride", ctypes.c_int64), ("kv_head_stride", ctypes.c_int64),
        ("idx_k_cache", ctypes.c_void_p), ("idx_token_stride", ctypes.c_int64), ("num_cache_rows", ctypes.c_int64),
        ("block_table", ctypes.c_void_p), ("block_size", ctypes.c_int32), ("max_blocks_per_seq", ctypes.c_int32),
    ]


class clsa_attn_hints(ctypes.Structure):
    """Mirror of `clsa_attn_hints` in include/clsa.h."""

    _fields_ = [("reverse", ctypes.c_int32), ("shared_gpu", ctypes.c_int32), ("keep_rows", ctypes.c_int32),
                ("only_q_pending", ctypes.c_int32)]


_P = ctypes.POINTER(clsa_params)
_H = ctypes.POINTER(clsa_attn_hints)
_vp, _i64, _sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t
_lib.clsa_workspace_bytes.argtypes = [_P, ctypes.POINTER(_sz)]
_lib.clsa_index_scores.argtypes = [_P, _vp, _vp, _i64, _vp, _sz, _vp]
_lib.clsa_topk.argtypes = [_P, _vp, _i64, _vp, _vp, _vp, _sz, _vp]
_lib.clsa_index_topk.argtypes = [_P, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.clsa_sparse_attn.argtypes = [_P, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.clsa_sparse_attn_hinted.argtypes = [_P, _vp, _vp, _vp, _vp, _vp, _H, _vp, _sz, _vp]
_lib.clsa_gather_probe.argtypes = [_P, _vp, _vp, _H, _vp, _sz, _vp]
_lib.clsa_decode_step.argtypes = [_P, _vp, ctypes.POINTER(_vp), ctypes.POINTER(_vp), _vp, _vp, _vp, _sz, _vp]
_lib.clsa_decode_step_static.argtypes = [_P, _vp, ctypes.POINTER(_vp), ctypes.POINTER(_vp), _vp, _vp, _vp, _vp]
_lib.clsa_sparse_attn_layers.argtypes = [_P, ctypes.POINTER(_vp), _vp, _vp, ctypes.POINTER(_vp), _vp, _sz, _vp]
_lib.clsa_project_append.argtypes = [_P, ctypes.c_int32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.clsa_chain_plan.argtypes = [_P, ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
_lib.clsa_clear_status.argtypes = [_vp, _sz, _vp]
_lib.clsa_device_status.argtypes = [_vp, ctypes.POINTER(ctypes.c_uint32), _vp]
_lib.clsa_status_string.argtypes = [ctypes.c_int]
_lib.clsa_status_string.restype = ctypes.c_char_p
_lib.clsa_version.restype = ctypes.c_int
for _name in ("clsa_workspace_bytes", "clsa_index_scores", "clsa_topk", "clsa_index_topk", "clsa_sparse_attn", "clsa_sparse_attn_hinted",
              "clsa_gather_probe", "clsa_decode_step", "clsa_decode_step_static", "clsa_sparse_attn_layers",
              "clsa_project_append", "clsa_chain_plan", "clsa_clear_status", "clsa_device_status"):
    getattr(_lib, _name).restype = ctypes.c_int

EXPORTS = ("clsa_workspace_bytes", "clsa_index_scores", "clsa_topk", "clsa_index_topk", "clsa_sparse_attn", "clsa_sparse_attn_hinted",
           "clsa_gather_probe", "clsa_decode_step", "clsa_decode_step_static", "clsa_sparse_attn_layers",
           "clsa_project_append", "clsa_chain_plan", "clsa_clear_status", "clsa_device_status", "clsa_status_string",
           "clsa_version")


class ClsaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {clsa_status_string(status)} (status {status})")


def _check(status: int, where: str) -> None:
    if status != CLSA_OK:
        raise ClsaError(status, where)


def _ptr(x):
    """Device address of a torch tensor, or an int address, or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream(stream):
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _nbytes(ws, ws_bytes):
    if ws_bytes is not None:
        return ws_bytes
    return ws.numel() * ws.element_size()


def make_params(*, num_seqs, q_per_seq=1, num_q_heads, num_kv_heads, head_dim=128, idx_dim, top_k, num_layers=1,
                causal=0, max_seq_len, sm_scale, seq_start=None, seq_len=None, k_cache=None, v_cache=None,
                kv_token_stride=None, kv_head_stride=None, idx_k_cache=None, idx_token_stride=None,
                num_cache_rows=None, block_table=None, block_size=0, max_blocks_per_seq=None) -> clsa_params:
    """Fill a clsa_params. Tensor arguments contribute their device address (and, for the caches, their strides
    unless given); the caller keeps them alive while the struct is in use."""
    p = clsa_params()
    p.num_seqs, p.q_per_seq, p.num_q_heads, p.num_kv_heads = num_seqs, q_per_seq, num_q_heads, num_kv_heads
    p.head_dim, p.idx_dim, p.top_k, p.num_layers, p.causal = head_dim, idx_dim, top_k, num_layers, causal
    p.max_seq_len, p.sm_scale = max_seq_len, sm_scale
    p.seq_start, p.seq_len = _ptr(seq_start), _ptr(seq_len)
    p.k_cache, p.v_cache, p.idx_k_cache = _ptr(k_cache), _ptr(v_cache), _ptr(idx_k_cache)
    if kv_token_stride is None and k_cache is not None and not isinstance(k_cache, int):
        kv_token_stride, kv_head_stride = k_cache.stride(0), k_cache.stride(1)
    if idx_token_stride is None and idx_k_cache is not None and not isinstance(idx_k_cache, int):
        idx_token_stride = idx_k_cache.stride(0)
    p.kv_token_stride = kv_token_stride if kv_token_stride is not None else num_kv_heads * head_dim
    p.kv_head_stride = kv_head_stride if kv_head_stride is not None else head_dim
    p.idx_token_stride = idx_token_stride if idx_token_stride is not None else idx_dim
    if num_cache_rows is None and idx_k_cache is not None and not isinstance(idx_k_cache, int):
        num_cache_rows = idx_k_cache.shape[0]
    p.num_cache_rows = num_cache_rows or 0
    p.block_table = _ptr(block_table)
    p.block_size = block_size
    if max_blocks_per_seq is None and block_table is not None and not isinstance(block_table, int):
        max_blocks_per_seq = block_table.shape[1]
    p.max_blocks_per_seq = max_blocks_per_seq or 0
    return p


def clsa_workspace_bytes(p: clsa_params) -> int:
    n = _sz(0)
    _check(_lib.clsa_workspace_bytes(ctypes.byref(p), ctypes.byref(n)), "clsa_workspace_bytes")
    return int(n.value)


def clsa_index_scores(p, q_idx, scores, score_stride, workspace, workspace_bytes=None, stream=None) -> None:
    _check(_lib.clsa_index_scores(ctypes.byref(p), _ptr(q_idx), _ptr(scores), score_stride, _ptr(workspace),
                                  _nbytes(workspace, workspace_bytes), _stream(stream)), "clsa_index_scores")


def clsa_topk(p, scores, score_stride, idx, count, workspace, workspace_bytes=None, stream=None) -> None:
    _check(_lib.clsa_topk(ctypes.byref(p), _ptr(scores), score_stride, _ptr(idx), _ptr(count), _ptr(workspace),
                          _nbytes(workspace, workspace_bytes), _stream(stream)), "clsa_topk")


def clsa_index_topk(p, q_idx, idx, count, workspace, workspace_bytes=None, stream=None) -> None:
    """Eq. 3 in one call (scores + TopK); for a prefill chunk the score matrix is never materialised."""
    _check(_lib.clsa_index_topk(ctypes.byref(p), _ptr(q_idx), _ptr(idx), _ptr(count), _ptr(workspace),
                                _nbytes(workspace, workspace_bytes), _stream(stream)), "clsa_index_topk")


def clsa_sparse_attn(p, q, idx, count, out, lse, workspace, workspace_bytes=None, stream=None) -> None:
    _check(_lib.clsa_sparse_attn(ctypes.byref(p), _ptr(q), _ptr(idx), _ptr(count), _ptr(out), _ptr(lse),
                                 _ptr(workspace), _nbytes(workspace, workspace_bytes), _stream(stream)),
           "clsa_sparse_attn")


def make_hints(reverse=0, shared_gpu=0, keep_rows=0, only_q_pending=0) -> clsa_attn_hints:
    return clsa_attn_hints(int(reverse), int(shared_gpu), int(keep_rows), int(only_q_pending))


def clsa_sparse_attn_hinted(p, q, idx, count, out, lse, hints, workspace, workspace_bytes=None, stream=None) -> None:
    """clsa_sparse_attn with a clsa_attn_hints (or None): launch shape and access order, never the result."""
    _check(_lib.clsa_sparse_attn_hinted(ctypes.byref(p), _ptr(q), _ptr(idx), _ptr(count), _ptr(out), _ptr(lse),
                                        None if hints is None else ctypes.byref(hints), _ptr(workspace),
                                        _nbytes(workspace, workspace_bytes), _stream(stream)), "clsa_sparse_attn_hinted")


def clsa_gather_probe(p, idx, count, hints, workspace, workspace_bytes=None, stream=None) -> None:
    """Measurement aid: the memory accesses of one decode attention launch without its arithmetic."""
    _check(_lib.clsa_gather_probe(ctypes.byref(p), _ptr(idx), _ptr(count), None if hints is None else ctypes.byref(hints),
                                  _ptr(workspace), _nbytes(workspace, workspace_bytes), _stream(stream)), "clsa_gather_probe")


def clsa_decode_step(p, q_idx, q_layers, out_layers, idx, count, workspace, workspace_bytes=None, stream=None) -> None:
    """q_layers / out_layers: sequences of L tensors (or addresses), one per cross-decoder layer."""
    L = p.num_layers
    if len(q_layers) != L or len(out_layers) != L:
        raise ValueError("q_layers and out_layers must have num_layers entries")
    qs = (_vp * L)(*[_ptr(t) for t in q_layers])
    outs = (_vp * L)(*[_ptr(t) for t in out_layers])
    _check(_lib.clsa_decode_step(ctypes.byref(p), _ptr(q_idx), qs, outs, _ptr(idx), _ptr(count), _ptr(workspace),
                                 _nbytes(workspace, workspace_bytes), _stream(stream)), "clsa_decode_step")


def clsa_decode_step_static(p, q_idx, q_layers, out_layers, idx, count, dev_status=None, stream=None) -> None:
    """clsa_decode_step for callers that cannot allocate: its scratch (a whole workspace) is a fixed 16 MiB array
    inside the library, shared by every call on the GPU, so no workspace is passed. Shapes whose workspace would be
    larger raise ClsaError(CLSA_ERR_WORKSPACE). Calls must not overlap on the GPU; make the first
    call on a device outside stream capture. `dev_status`: optional caller-owned uint32 device tensor."""
    L = p.num_layers
    if len(q_layers) != L or len(out_layers) != L:
        raise ValueError("q_layers and out_layers must have num_layers entries")
    qs = (_vp * L)(*[_ptr(t) for t in q_layers])
    outs = (_vp * L)(*[_ptr(t) for t in out_layers])
    _check(_lib.clsa_decode_step_static(ctypes.byref(p), _ptr(q_idx), qs, outs, _ptr(idx), _ptr(count),
                                        _ptr(dev_status), _stream(stream)), "clsa_decode_step_static")


def clsa_sparse_attn_layers(p, q_layers, idx, count, out_layers, workspace, workspace_bytes=None, stream=None) -> None:
    """The L attention launches of clsa_decode_step on an index that already exists (idx, count from clsa_topk)."""
    L = p.num_layers
    if len(q_layers) != L or len(out_layers) != L:
        raise ValueError("q_layers and out_layers must have num_layers entries")
    qs = (_vp * L)(*[_ptr(t) for t in q_layers])
    outs = (_vp * L)(*[_ptr(t) for t in out_layers])
    _check(_lib.clsa_sparse_attn_layers(ctypes.byref(p), qs, _ptr(idx), _ptr(count), outs, _ptr(workspace),
                                        _nbytes(workspace, workspace_bytes), _stream(stream)), "clsa_sparse_attn_layers")


def clsa_project_append(p, d_model, h, w_q_idx, w_k_idx, w_k, w_v, q_idx_out, idx_k_cache_out, k_cache_out,
                        v_cache_out, workspace, workspace_bytes=None, stream=None) -> None:
    """Eq. 2 for the T newest tokens of every sequence and the append of their K_idx (and, with w_k/w_v, K and V)
    rows through the writable cache pointers `idx_k_cache_out`, `k_cache_out`, `v_cache_out` (the caches that `p`
    describes). Weights are [n_out][d_model]."""
    _check(_lib.clsa_project_append(ctypes.byref(p), int(d_model), _ptr(h), _ptr(w_q_idx), _ptr(w_k_idx), _ptr(w_k),
                                    _ptr(w_v), _ptr(q_idx_out), _ptr(idx_k_cache_out), _ptr(k_cache_out),
                                    _ptr(v_cache_out), _ptr(workspace), _nbytes(workspace, workspace_bytes),
                                    _stream(stream)), "clsa_project_append")


def clsa_chain_plan(p, sm_count, clock_khz):
    """(fine_layers, paired_layers): the trailing layers of an L-layer chain that use the finer launch shape, and the
    leading layers that are computed two per launch. Host only."""
    a, b = ctypes.c_int32(0), ctypes.c_int32(0)
    _check(_lib.clsa_chain_plan(ctypes.byref(p), int(sm_count), int(clock_khz), ctypes.byref(a), ctypes.byref(b)), "clsa_chain_plan")
    return int(a.value), int(b.value)


def clsa_clear_status(workspace, workspace_bytes=None, stream=None) -> None:
    _check(_lib.clsa_clear_status(_ptr(workspace), _nbytes(workspace, workspace_bytes), _stream(stream)),
           "clsa_clear_status")


def clsa_device_status(workspace, stream=None) -> int:
    bits = ctypes.c_uint32(0)
    _check(_lib.clsa_device_status(_ptr(workspace), ctypes.byref(bits), _stream(stream)), "clsa_device_status")
    return int(bits.value)


def clsa_status_string(status: int) -> str:
    return _lib.clsa_status_string(int(status)).decode()


def clsa_version() -> int:
    return int(_lib.clsa_version())


def raw():
    """The ctypes library handle (status codes returned, nothing raised) for tests of the error paths."""
    return _lib
