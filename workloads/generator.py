"""Seeded, counter-based synthetic inputs, bit-identical on the host (numpy) and on a GPU (torch).

Every tensor element is a pure function of (seed, tensor id, flat element index):

    value = QTABLE[ mix64(stream_base(seed, tensor_id) + element * GOLDEN) >> 48 ]

`mix64` is the splitmix64 finaliser (integer only) and `QTABLE` holds the 65 536 bf16 values
bf16(Phi^-1((i + 1/2) / 65536)), i.e. an N(0,1) sample quantised to 16 bits of probability.
Because only integer arithmetic and one table look-up are involved, the host can synthesise any
single row of a multi-gigabyte cache without materialising the rest, and a GPU fill of the whole
tensor produces exactly the same bits.

This module holds no arithmetic of the method under test (no dot products, no selection, no
softmax): it only produces inputs. Both the CPU oracle's tests and the CUDA path's tests feed
from it.
"""
from __future__ import annotations

import numpy as np

_M64 = (1 << 64) - 1
GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB


def mix64_int(x: int) -> int:
    """splitmix64 finaliser on a Python int (reference form of the two vector versions below)."""
    x &= _M64
    x ^= x >> 30
    x = (x * _C1) & _M64
    x ^= x >> 27
    x = (x * _C2) & _M64
    x ^= x >> 31
    return x


def stream_base(seed: int, tensor_id: int) -> int:
    """64-bit base of the counter stream of one tensor."""
    return mix64_int((seed & _M64) ^ mix64_int((tensor_id + 1) * GOLDEN))


def mix64_np(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on a uint64 array (wrapping arithmetic)."""
    x = x.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        x ^= x >> np.uint64(30)
        x *= np.uint64(_C1)
        x ^= x >> np.uint64(27)
        x *= np.uint64(_C2)
        x ^= x >> np.uint64(31)
    return x


def hash_np(base: int, counters: np.ndarray) -> np.ndarray:
    """mix64(base + counter * GOLDEN) for a uint64/int64 counter array."""
    c = counters.astype(np.uint64, copy=False)
    with np.errstate(over="ignore"):
        return mix64_np(c * np.uint64(GOLDEN) + np.uint64(base))


def _signed(c: int) -> int:
    c &= _M64
    return c - (1 << 64) if c >= (1 << 63) else c


def mix64_torch(x):
    """splitmix64 finaliser on an int64 torch tensor; logical shifts are emulated with masks."""
    x = x ^ ((x >> 30) & ((1 << 34) - 1))
    x = x * _signed(_C1)
    x = x ^ ((x >> 27) & ((1 << 37) - 1))
    x = x * _signed(_C2)
    x = x ^ ((x >> 31) & ((1 << 33) - 1))
    return x


def hash_torch(base: int, counters):
    """mix64(base + counter * GOLDEN) for an int64 torch tensor (two's-complement wrap-around)."""
    return mix64_torch(counters * _signed(GOLDEN) + _signed(base))


# ----------------------------------------------------------------------------- bf16 helpers
def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float64 -> float32 -> bf16 (both round-to-nearest-even); returns uint16 bit patterns."""
    f32 = np.asarray(x, dtype=np.float64).astype(np.float32)
    bits = f32.view(np.uint32).astype(np.uint64)
    rounded = (bits + np.uint64(0x7FFF) + ((bits >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


_QTABLE = None


def qtable() -> np.ndarray:
    """65 536 bf16 bit patterns: bf16(Phi^-1((i + 1/2)/65536)), built once in float64."""
    global _QTABLE
    if _QTABLE is None:
        from scipy.special import ndtri

        p = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
        _QTABLE = f64_to_bf16_bits(ndtri(p))
        _QTABLE.setflags(write=False)
    return _QTABLE


_QTABLE_DEV = {}


def qtable_torch(device):
    import torch

    key = str(device)
    if key not in _QTABLE_DEV:
        t = torch.from_numpy(qtable().astype(np.int16, copy=True).copy())
        _QTABLE_DEV[key] = t.to(device)
    return _QTABLE_DEV[key]


# ----------------------------------------------------------------------------- element streams
class Stream:
    """The infinite bf16 element stream of one (seed, tensor id)."""

    def __init__(self, seed: int, tensor_id: int):
        self.seed = seed
        self.tensor_id = tensor_id
        self.base = stream_base(seed, tensor_id)

    # host ------------------------------------------------------------------
    def host_elements(self, elements: np.ndarray) -> np.ndarray:
        """bf16 bit patterns (uint16) of arbitrary flat element indices."""
        h = hash_np(self.base, np.asarray(elements))
        return qtable()[(h >> np.uint64(48)).astype(np.int64)]

    def host_range(self, start: int, count: int) -> np.ndarray:
        return self.host_elements(np.arange(start, start + count, dtype=np.uint64))

    def host_rows(self, rows: np.ndarray, row_elems: int) -> np.ndarray:
        """Rows `rows` (any order, any repeats) of the stream viewed as [*, row_elems]."""
        rows = np.asarray(rows, dtype=np.uint64).reshape(-1)
        out = np.empty((rows.size, row_elems), dtype=np.uint16)
        step = max(1, (1 << 22) // max(1, row_elems))
        cols = np.arange(row_elems, dtype=np.uint64)[None, :]
        for i in range(0, rows.size, step):
            r = rows[i : i + step, None]
            out[i : i + step] = self.host_elements(r * np.uint64(row_elems) + cols)
        return out

    # device ----------------------------------------------------------------
    def device_fill(self, out, row_source=None, row_elems: int = 0, chunk: int = 1 << 25):
        """Fill the contiguous bf16 torch tensor `out` with stream elements 0..numel-1.

        If `row_source` (int64 tensor, one entry per row of `row_elems` elements) is given, row r of
        `out` takes the stream's row row_source[r] instead of row r.
        """
        import torch

        assert out.is_contiguous() and out.dtype == torch.bfloat16
        flat = out.view(-1).view(torch.int16)
        table = qtable_torch(out.device)
        n = flat.numel()
        for s in range(0, n, chunk):
            e = min(n, s + chunk)
            el = torch.arange(s, e, dtype=torch.int64, device=out.device)
            if row_source is not None:
                r = torch.div(el, row_elems, rounding_mode="floor")
                el = row_source[r] * row_elems + (el - r * row_elems)
            h = hash_torch(self.base, el)
            flat[s:e] = table[(h >> 48) & 0xFFFF]
        return out


def hash_u64(seed: int, tensor_id: int, counters: np.ndarray) -> np.ndarray:
    """Raw 64-bit hashes, for integer draws (lengths, positions, duplicate sources)."""
    return hash_np(stream_base(seed, tensor_id), np.asarray(counters))
