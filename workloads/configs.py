"""The five benchmark workloads as data, plus host/device materialisation of their tensors.

Shapes follow the paper's long-context decoding set-up (128K context, 2048 selected tokens, 16
cross-decoder layers sharing one KV cache and one index, head_dim 128, GQA); contents are seeded
synthetic values from `workloads.generator`. Nothing here computes scores, selections or attention.
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass

import numpy as np

from . import generator as g

TID_Q_IDX, TID_K_IDX, TID_K, TID_V = 0, 1, 2, 3
TID_LEN, TID_DUP_FLAG, TID_DUP_SRC, TID_PLANT = 4, 5, 6, 7
TID_BLOCK_PERM = 8
TID_H, TID_W_QIDX, TID_W_KIDX, TID_W_K, TID_W_V = 9, 10, 11, 12, 13
WEIGHT_SHIFT = 6  # projection weights are table values times 2^-6 (about 1/sqrt(d_model)): exact in bf16
TID_Q_LAYER0 = 16


@dataclass(frozen=True)
class Config:
    name: str
    seed: int
    num_seqs: int
    ctx: int                 # context length n (max over sequences when ragged), incl. the T query tokens
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    idx_dim: int
    top_k: int
    num_layers: int
    q_per_seq: int = 1       # T
    causal: int = 0
    ragged_min: int = 0      # >0: lengths uniform in [ragged_min, ctx]
    num_short: int = 0       # that many sequences forced into [ragged_min, top_k - 1]
    planted: int = 0         # planted high-score tokens per sequence (decode only)
    plant_boost: float = 4.0
    dup_frac: float = 0.0    # fraction of indexer-key rows that are exact copies of an earlier row
    d_model: int = 2560      # hidden size of the states the projections read (the paper's 4B-scale model)

    def replace(self, **kw) -> "Config":
        return dataclasses.replace(self, **kw)

    @property
    def sm_scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)


_SEED0 = 0xC15A0000

TINY = Config("tiny", _SEED0 + 1, 1, 4096, 8, 1, 128, 64, 256, 4)
MID = Config("mid", _SEED0 + 2, 8, 32768, 32, 8, 128, 128, 2048, 16)
HEADLINE = Config("headline128k", _SEED0 + 3, 16, 131072, 32, 8, 128, 128, 2048, 16, planted=64)
RAGGED = Config("ragged", _SEED0 + 4, 64, 131072, 32, 8, 128, 128, 2048, 16,
                ragged_min=1024, num_short=4, dup_frac=0.05)
PREFILL = Config("prefill_chunk", _SEED0 + 5, 1, 131072 + 4096, 32, 8, 128, 128, 2048, 16,
                 q_per_seq=4096, causal=1)

# a scaled-down prefill chunk (scores 285 MB, caches 142 MB: beyond L2, small enough to profile)
PREFILL_SMALL = PREFILL.replace(name="prefill_small", ctx=32768 + 2048, q_per_seq=2048, num_layers=2)

CONFIGS = {c.name: c for c in (TINY, MID, HEADLINE, RAGGED, PREFILL, PREFILL_SMALL)}


class Workload:
    """Lengths, packing and tensor contents of one Config."""

    def __init__(self, cfg: Config):
        self.cfg = cfg
        B = cfg.num_seqs
        if cfg.ragged_min > 0:
            h = g.hash_u64(cfg.seed, TID_LEN, np.arange(B, dtype=np.uint64))
            span = np.uint64(cfg.ctx - cfg.ragged_min + 1)
            lens = (h % span).astype(np.int64) + cfg.ragged_min
            if cfg.num_short > 0:
                # the first num_short picks of a hashed permutation become shorter than top_k
                order = np.argsort(g.hash_u64(cfg.seed, TID_LEN, np.arange(B, 2 * B, dtype=np.uint64)), kind="stable")
                hs = g.hash_u64(cfg.seed, TID_LEN, np.arange(2 * B, 2 * B + cfg.num_short, dtype=np.uint64))
                short_span = np.uint64(max(1, cfg.top_k - cfg.ragged_min))
                lens[order[: cfg.num_short]] = (hs % short_span).astype(np.int64) + cfg.ragged_min
            lens = np.maximum(lens, cfg.q_per_seq)
            starts = np.zeros(B, dtype=np.int64)
            acc = 0
            for b in range(B):
                starts[b] = acc
                acc += (int(lens[b]) + 63) // 64 * 64
            self.total_rows = acc
        else:
            lens = np.full(B, cfg.ctx, dtype=np.int64)
            starts = np.arange(B, dtype=np.int64) * cfg.ctx
            self.total_rows = B * cfg.ctx
        self.seq_len = lens.astype(np.int32)
        self.seq_start = starts
        self.max_seq_len = int(lens.max())
        self._s_qidx = g.Stream(cfg.seed, TID_Q_IDX)
        self._s_kidx = g.Stream(cfg.seed, TID_K_IDX)
        self._s_k = g.Stream(cfg.seed, TID_K)
        self._s_v = g.Stream(cfg.seed, TID_V)
        self._row_source = None

    # ------------------------------------------------------------------ sizes
    @property
    def kv_row_elems(self) -> int:
        return self.cfg.num_kv_heads * self.cfg.head_dim

    def visible(self, b: int, t: int) -> int:
        n = int(self.seq_len[b])
        return n - self.cfg.q_per_seq + t + 1 if self.cfg.causal else n

    def selected_counts(self) -> np.ndarray:
        c = self.cfg
        out = np.empty((c.num_seqs, c.q_per_seq), dtype=np.int64)
        for b in range(c.num_seqs):
            for t in range(c.q_per_seq):
                out[b, t] = min(c.top_k, self.visible(b, t))
        return out

    def algorithmic_bytes(self) -> int:
        """Indexer-key bytes + L * (selected rows * Hkv * D * 2 bytes * {K,V})."""
        c = self.cfg
        idx_bytes = int(self.seq_len.astype(np.int64).sum()) * c.idx_dim * 2
        gathered = int(self.selected_counts().sum()) * c.num_kv_heads * c.head_dim * 2 * 2
        return idx_bytes + c.num_layers * gathered

    # ------------------------------------------------------------------ indexer-key row sources
    def row_source(self) -> np.ndarray:
        """For every cache row, the stream row its indexer key is taken from (itself unless duplicated)."""
        if self._row_source is None:
            src = np.arange(self.total_rows, dtype=np.int64)
            c = self.cfg
            if c.dup_frac > 0.0:
                thr = int(c.dup_frac * (1 << 24))
                for b in range(c.num_seqs):
                    n, s0 = int(self.seq_len[b]), int(self.seq_start[b])
                    rows = np.arange(s0, s0 + n, dtype=np.uint64)
                    flag = (g.hash_u64(c.seed, TID_DUP_FLAG, rows) >> np.uint64(40)).astype(np.int64) < thr
                    pos = np.arange(n, dtype=np.uint64)
                    pick = g.hash_u64(c.seed, TID_DUP_SRC, rows) % np.maximum(pos, np.uint64(1))
                    flag[0] = False
                    src[s0 : s0 + n] = np.where(flag, s0 + pick.astype(np.int64), src[s0 : s0 + n])
            self._row_source = src
        return self._row_source

    def planted_positions(self, b: int) -> np.ndarray:
        c = self.cfg
        if c.planted == 0:
            return np.zeros(0, dtype=np.int64)
        n = int(self.seq_len[b])
        want = min(c.planted, n)
        seen, out, i = set(), [], 0
        while len(out) < want:
            h = int(g.hash_u64(c.seed, TID_PLANT, np.array([b * 65536 + i], dtype=np.uint64))[0])
            p = h % n
            i += 1
            if p not in seen:
                seen.add(p)
                out.append(p)
        return np.array(sorted(out), dtype=np.int64)

    def _planted_rows(self, b: int):
        """(positions, bf16 rows) of the boosted indexer keys: bf16(K_idx[p] + boost * q/|q|)."""
        c = self.cfg
        pos = self.planted_positions(b)
        if pos.size == 0:
            return pos, np.zeros((0, c.idx_dim), dtype=np.uint16)
        q = g.bf16_bits_to_f64(self.q_idx_bits()[b, 0])
        qhat = q / np.linalg.norm(q)
        base = g.bf16_bits_to_f64(self._s_kidx.host_rows(self.row_source()[self.seq_start[b] + pos], c.idx_dim))
        return pos, g.f64_to_bf16_bits(base + c.plant_boost * qhat[None, :])

    # ------------------------------------------------------------------ host tensors (uint16 bf16 bits)
    def q_idx_bits(self) -> np.ndarray:
        c = self.cfg
        return self._s_qidx.host_range(0, c.num_seqs * c.q_per_seq * c.idx_dim).reshape(
            c.num_seqs, c.q_per_seq, c.idx_dim)

    def kidx_bits(self, b: int) -> np.ndarray:
        """[n_b, idx_dim] indexer keys of sequence b."""
        c = self.cfg
        n, s0 = int(self.seq_len[b]), int(self.seq_start[b])
        rows = self._s_kidx.host_rows(self.row_source()[s0 : s0 + n], c.idx_dim)
        pos, boosted = self._planted_rows(b)
        if pos.size:
            rows[pos] = boosted
        return rows

    def kv_rows_bits(self, which: str, global_rows: np.ndarray) -> np.ndarray:
        s = self._s_k if which == "k" else self._s_v
        return s.host_rows(global_rows, self.kv_row_elems)

    def q_layer_bits(self, layer: int) -> np.ndarray:
        c = self.cfg
        n = c.num_seqs * c.q_per_seq * c.num_q_heads * c.head_dim
        return g.Stream(c.seed, TID_Q_LAYER0 + layer).host_range(0, n).reshape(
            c.num_seqs, c.q_per_seq, c.num_q_heads, c.head_dim)

    # ------------------------------------------------------------------ projection inputs (Eq. 2)
    def weight_shape(self, which: str):
        c = self.cfg
        return (c.idx_dim if which in ("q_idx", "k_idx") else c.num_kv_heads * c.head_dim, c.d_model)

    def hidden_bits(self) -> np.ndarray:
        """[B, T, d_model] hidden states of the query tokens, N(0,1)."""
        c = self.cfg
        return g.Stream(c.seed, TID_H).host_range(0, c.num_seqs * c.q_per_seq * c.d_model).reshape(
            c.num_seqs, c.q_per_seq, c.d_model)

    def weight_bits(self, which: str) -> np.ndarray:
        """[n_out, d_model] projection weights (one output feature per row), N(0,1) * 2^-WEIGHT_SHIFT."""
        tid = {"q_idx": TID_W_QIDX, "k_idx": TID_W_KIDX, "k": TID_W_K, "v": TID_W_V}[which]
        n_out, d = self.weight_shape(which)
        raw = g.Stream(self.cfg.seed, tid).host_range(0, n_out * d).reshape(n_out, d)
        return g.f64_to_bf16_bits(g.bf16_bits_to_f64(raw) * 2.0 ** -WEIGHT_SHIFT)

    def projection_to_device(self, device="cuda"):
        """dict(h, w_q_idx, w_k_idx, w_k, w_v) as bf16 torch tensors, bit-identical to the host versions."""
        import torch

        c = self.cfg
        dev = torch.device(device)
        out = {}
        h = torch.empty((c.num_seqs, c.q_per_seq, c.d_model), dtype=torch.bfloat16, device=dev)
        g.Stream(c.seed, TID_H).device_fill(h)
        out["h"] = h
        for which, tid in (("q_idx", TID_W_QIDX), ("k_idx", TID_W_KIDX), ("k", TID_W_K), ("v", TID_W_V)):
            t = torch.empty(self.weight_shape(which), dtype=torch.bfloat16, device=dev)
            g.Stream(c.seed, tid).device_fill(t)
            out["w_" + which] = t.mul_(2.0 ** -WEIGHT_SHIFT)  # a power of two: exact
        return out

    def host_kidx_cache(self) -> np.ndarray:
        """Full [total_rows, idx_dim] indexer-key cache on the host."""
        c = self.cfg
        out = np.zeros((self.total_rows, c.idx_dim), dtype=np.uint16)
        for b in range(c.num_seqs):
            s0, n = int(self.seq_start[b]), int(self.seq_len[b])
            out[s0 : s0 + n] = self.kidx_bits(b)
        return out

    def host_kv_sparse(self, idx: np.ndarray, count: np.ndarray):
        """Full-size zero-initialised host K and V caches with only the rows named by (idx, count) filled.

        The arrays are calloc-backed, so untouched rows cost no physical memory; an 8 GiB cache of
        which 32 768 rows are touched occupies a few hundred MiB. `idx` is [B, T, k] sequence-local.
        """
        c = self.cfg
        k = np.zeros((self.total_rows, c.num_kv_heads, c.head_dim), dtype=np.uint16)
        v = np.zeros((self.total_rows, c.num_kv_heads, c.head_dim), dtype=np.uint16)
        for b in range(c.num_seqs):
            sel = [idx[b, t, : int(count[b, t])] for t in range(c.q_per_seq)]
            rows = np.unique(np.concatenate(sel).astype(np.int64)) + int(self.seq_start[b])
            if rows.size == 0:
                continue
            k[rows] = self.kv_rows_bits("k", rows).reshape(-1, c.num_kv_heads, c.head_dim)
            v[rows] = self.kv_rows_bits("v", rows).reshape(-1, c.num_kv_heads, c.head_dim)
        return k, v

    def host_kv_full(self):
        """Whole K and V caches on the host (small configs only)."""
        c = self.cfg
        rows = np.arange(self.total_rows, dtype=np.int64)
        k = self.kv_rows_bits("k", rows).reshape(-1, c.num_kv_heads, c.head_dim)
        v = self.kv_rows_bits("v", rows).reshape(-1, c.num_kv_heads, c.head_dim)
        return k, v

    # ------------------------------------------------------------------ paged layout
    def block_table(self, block_size: int):
        """(table int32 [B, max_blocks], num_blocks): a hashed permutation scatters the blocks of all sequences over
        the cache, as a block allocator under churn would."""
        B = self.cfg.num_seqs
        per_seq = [(int(n) + block_size - 1) // block_size for n in self.seq_len]
        total = sum(per_seq)
        order = np.argsort(g.hash_u64(self.cfg.seed, TID_BLOCK_PERM, np.arange(total, dtype=np.uint64)), kind="stable")
        table = np.zeros((B, max(per_seq)), dtype=np.int32)
        pos = 0
        for b in range(B):
            table[b, : per_seq[b]] = order[pos: pos + per_seq[b]]
            pos += per_seq[b]
        return table, total

    def paged_rows(self, block_size: int):
        """(src, num_rows): src[r] = contiguous-layout row whose contents sit in paged row r (-1 for padding)."""
        table, total = self.block_table(block_size)
        src = np.full(total * block_size, -1, dtype=np.int64)
        for b in range(self.cfg.num_seqs):
            n, s0 = int(self.seq_len[b]), int(self.seq_start[b])
            s = np.arange(n, dtype=np.int64)
            rows = table[b, s // block_size].astype(np.int64) * block_size + s % block_size
            src[rows] = s0 + s
        return src, total * block_size

    def paginate_host(self, arr: np.ndarray, block_size: int) -> np.ndarray:
        """Rearrange a host cache [total_rows, ...] (contiguous sequences) into the paged layout."""
        src, nrows = self.paged_rows(block_size)
        out = np.zeros((nrows,) + arr.shape[1:], dtype=arr.dtype)
        ok = src >= 0
        out[ok] = arr[src[ok]]
        return out

    def paginate_device(self, tensors: dict, block_size: int) -> dict:
        """Paged copies of the device caches in `tensors` plus the block table (torch)."""
        import torch

        src, nrows = self.paged_rows(block_size)
        dev = tensors["k_cache"].device
        src_t = torch.from_numpy(np.where(src >= 0, src, 0)).to(dev)
        ok = torch.from_numpy(src >= 0).to(dev)
        out = dict(tensors)
        for name in ("k_cache", "v_cache", "idx_k_cache"):
            t = tensors[name][src_t]
            t[~ok] = 0
            out[name] = t.contiguous()
        table, _ = self.block_table(block_size)
        out["block_table"] = torch.from_numpy(table).to(dev)
        return out

    # ------------------------------------------------------------------ device tensors
    def to_device(self, device="cuda", layers=None):
        """Materialise everything on `device` as bf16/int torch tensors (dict)."""
        import torch

        c = self.cfg
        L = c.num_layers if layers is None else layers
        dev = torch.device(device)
        out = {}
        out["seq_start"] = torch.from_numpy(self.seq_start.copy()).to(dev)
        out["seq_len"] = torch.from_numpy(self.seq_len.copy()).to(dev)
        q_idx = torch.empty((c.num_seqs, c.q_per_seq, c.idx_dim), dtype=torch.bfloat16, device=dev)
        self._s_qidx.device_fill(q_idx)
        out["q_idx"] = q_idx
        kidx = torch.empty((self.total_rows, c.idx_dim), dtype=torch.bfloat16, device=dev)
        src = None
        if c.dup_frac > 0.0:
            src = torch.from_numpy(self.row_source().copy()).to(dev)
        self._s_kidx.device_fill(kidx, row_source=src, row_elems=c.idx_dim)
        for b in range(c.num_seqs):
            pos, boosted = self._planted_rows(b)
            if pos.size:
                rows = torch.from_numpy(pos + int(self.seq_start[b])).to(dev)
                kidx.view(torch.int16)[rows] = torch.from_numpy(boosted.view(np.int16).copy()).to(dev)
        out["idx_k_cache"] = kidx
        for name, s in (("k_cache", self._s_k), ("v_cache", self._s_v)):
            t = torch.empty((self.total_rows, c.num_kv_heads, c.head_dim), dtype=torch.bfloat16, device=dev)
            s.device_fill(t)
            out[name] = t
        q_layers = torch.empty((L, c.num_seqs, c.q_per_seq, c.num_q_heads, c.head_dim),
                               dtype=torch.bfloat16, device=dev)
        for l in range(L):
            g.Stream(c.seed, TID_Q_LAYER0 + l).device_fill(q_layers[l])
        out["q_layers"] = q_layers
        return out
