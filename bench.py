#!/usr/bin/env python
"""Benchmark of the CLSA decode hot path: index scores + top-k + L sparse-attention layers per step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

A step is one pass of the whole path (all through the C ABI) over one batch of seeded synthetic input that is
already resident in HBM. Two ways of issuing the L layers are timed, each step bracketed by its own CUDA events on
the launch stream, with the L2 flushed (and cleaned) between steps:

  dependent    clsa_index_scores, clsa_topk, then one clsa_sparse_attn_hinted per layer, every launch waiting for
               its predecessor -- what a decoder can run whose layer l+1 queries depend on layer l's output (the
               cross-decoder has an FFN between its attention layers). This is the headline: `value`, `step_us`.
  independent  clsa_decode_step: all L query tensors are handed over up front, the layers do not wait for one
               another, several are in flight at once and share the selected rows through L2. Legal for this ABI,
               but not an HBM rate: reported beside the headline under "modes".

`value` = algorithmic bytes per step (indexer-key bytes + L * selected rows * Hkv * D * 2 B * {K,V}) divided by the
median step time, summed over ranks. With --gpus N > 1 (launched by torchrun) every rank runs an independent replica
of the workload: the path has no exchange step, so there is no collective on the data path ("replicas only").

--impl reference times the CPU oracle on the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode step algorithmic GB/s (index+top-k+L-layer sparse attn, layers issued one by one)"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="headline128k")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--num-seqs", type=int, default=0, help="override the workload's batch size")
    ap.add_argument("--ctx", type=int, default=0, help="override the workload's context length")
    ap.add_argument("--top-k", type=int, default=0, help="override the workload's k")
    ap.add_argument("--q-heads", type=int, default=0, help="override the number of query heads")
    ap.add_argument("--kv-heads", type=int, default=0, help="override the number of KV heads")
    ap.add_argument("--layers", type=int, default=0, help="override the number of cross-decoder layers")
    ap.add_argument("--graph", action="store_true",
                    help="capture the independent-layers step once into a CUDA graph and time replays (removes host "
                         "launch gaps; matters for small, launch-bound workloads)")
    ap.add_argument("--compare", action="store_true",
                    help="also time, on the same inputs, dense attention over the whole cache (Eq. 1) and routing "
                         "repeated in every layer, and print them as a second JSON line")
    ap.add_argument("--project", action="store_true",
                    help="also time the upstream step (Eq. 2 projections of the new tokens + cache append, "
                         "clsa_project_append) on the same workload; reported under \"projection\", not part of the step")
    ap.add_argument("--block-size", type=int, default=0, help="page the caches into scattered blocks of this many rows")
    ap.add_argument("--e2e-group", type=int, default=2, help="--e2e-out streamed: layers per device-to-host copy")
    ap.add_argument("--e2e-out", default="auto", choices=["auto", "mapped", "copy", "streamed"],
                    help="end-to-end legs, how the L outputs reach the host: the layers store them straight into pinned "
                         "host memory (mapped), into HBM followed by one device-to-host copy (copy), or into HBM with each "
                         "layer's output copied on a second stream while the next layers run (streamed; layers one by one "
                         "only). auto: streamed for the layers-one-by-one mode, mapped for clsa_decode_step")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
    ap.add_argument("--no-breakdown", action="store_true", help="skip the per-kernel instrumented loop and the gather ceilings")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the short runs of the other benchmark configs (mid, ragged, tiny, prefill chunk)")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def profiled_traffic(workload: str, kernel: str):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) recorded from an ncu capture, from
    profiles/traffic.txt ("workload kernel bytes ..." lines); None if that capture has not been recorded."""
    path = os.path.join(ROOT, "profiles", "traffic.txt")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        for line in f:
            parts = line.split()
            if len(parts) >= 3 and not line.startswith("#") and parts[0] == workload and parts[1] == kernel:
                return float(parts[2])
    return None


def spread(xs):
    """median / min / max / mean of a list of per-step times."""
    return {"median": statistics.median(xs), "min": min(xs), "max": max(xs), "mean": sum(xs) / len(xs)}


def spread_us(ms_list):
    return {k: v * 1e3 for k, v in spread(ms_list).items()}


class ClockSampler(threading.Thread):
    """Polls NVML (read-only) for SM clock and clock-event reasons while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop_evt = threading.Event()
        self._active = threading.Event()   # samples are taken only while a timed region runs
        self.ok = False
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            if not self._active.is_set():
                time.sleep(0.001)
                continue
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                try:
                    r = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in self.REASONS.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.001)

    def pause(self):
        self._active.clear()

    def resume(self):
        self._active.set()

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        med = sorted(self.samples)[len(self.samples) // 2] if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(ms: float, dist, device) -> float:
    """Step time of the job = the slowest rank's (all_reduce MAX); identity on one rank."""
    if dist is None:
        return ms
    import torch

    tt = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def aggregate_value(world: int, bytes_per_rank_step: int, ms_per_step: float) -> float:
    """Whole-job GB/s: every rank moves `bytes_per_rank_step` algorithmic bytes per step."""
    return world * bytes_per_rank_step / (ms_per_step * 1e-3) / 1e9


def pick_config(args):
    """The named workload, with any command-line overrides applied (the name then says so)."""
    from workloads import CONFIGS

    c = CONFIGS[args.config]
    over = {}
    for field, val in (("num_seqs", args.num_seqs), ("ctx", args.ctx), ("top_k", args.top_k),
                       ("num_q_heads", args.q_heads), ("num_kv_heads", args.kv_heads), ("num_layers", args.layers)):
        if val:
            over[field] = val
    if over:
        c = c.replace(name=c.name + "+" + ",".join(f"{k}={v}" for k, v in sorted(over.items())), **over)
    return c


def config_dict(c, w, args, world=1):
    """`config` of the JSON line; both arms print the same keys and values, so that the two lines compare equal."""
    return {"workload": c.name, "num_seqs": c.num_seqs, "context": c.ctx, "top_k": c.top_k, "layers": c.num_layers,
            "q_heads": c.num_q_heads, "kv_heads": c.num_kv_heads, "idx_dim": c.idx_dim,
            "algorithmic_bytes_per_step": w.algorithmic_bytes(),
            "cache_layout": f"paged, {args.block_size}-row blocks" if args.block_size else "contiguous sequences",
            "parallelism": "replicas only" if world > 1 else "single GPU",
            "l2": "GPU arm: flushed between steps (512 MiB rewrite, then 256 MiB read so that no dirty lines remain); "
                  "CPU arm: host caches as the previous pass leaves them",
            "statistic": "median of the timed steps"}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# --------------------------------------------------------------------------------------- oracle legs
def set_omp_threads(n: int) -> bool:
    """Thread count of the OpenMP runtime the oracle library is linked against (the oracle itself is not touched)."""
    try:
        ctypes.CDLL("libgomp.so.1").omp_set_num_threads(int(n))
        return True
    except Exception:
        return False


class OracleSample:
    """The oracle, as it stands, on sequences `seqs` and `layers` layers of workload `w`.

    Input synthesis happens once here and is never timed (the K/V rows the selection will touch are found by one
    untimed routing pass); `run()` then times Eq. 3's scores, the TopK -- with the oracle's partition selector, the
    one meant for timing (its full sort is the checker) -- and every layer's attention (Eq. 4)."""

    def __init__(self, w, seqs, layers):
        import numpy as np

        import oracle
        from workloads import Workload

        c = w.cfg
        self.layers = layers
        sub = Workload(c.replace(num_seqs=len(seqs), num_layers=layers))
        sub.seq_len = w.seq_len[seqs].copy()          # same lengths, keys and queries as the parent's sequences
        sub.max_seq_len = int(sub.seq_len.max())
        starts, acc = [], 0
        for n in sub.seq_len:
            starts.append(acc)
            acc += int(n)
        sub.seq_start = np.array(starts, dtype=np.int64)
        sub.total_rows = acc
        kidx = np.concatenate([w.kidx_bits(int(b)) for b in seqs])
        self.q_idx = w.q_idx_bits()[seqs]
        route = oracle.problem_from_workload(sub, idx_k_cache=kidx)
        idx, cnt = route.topk(route.index_scores(self.q_idx), selector="select")
        kc = np.zeros((sub.total_rows, c.num_kv_heads, c.head_dim), dtype=np.uint16)
        vc = np.zeros_like(kc)
        for i, b in enumerate(seqs):
            for t in range(c.q_per_seq):
                loc = idx[i, t, : cnt[i, t]].astype(np.int64)
                rows = int(w.seq_start[b]) + loc
                kc[sub.seq_start[i] + loc] = w.kv_rows_bits("k", rows).reshape(-1, c.num_kv_heads, c.head_dim)
                vc[sub.seq_start[i] + loc] = w.kv_rows_bits("v", rows).reshape(-1, c.num_kv_heads, c.head_dim)
        self.prob = oracle.problem_from_workload(sub, k_cache=kc, v_cache=vc, idx_k_cache=kidx)
        self.qs = [w.q_layer_bits(l)[seqs] for l in range(layers)]
        self.nbytes = (int(sub.seq_len.astype(np.int64).sum()) * c.idx_dim * 2
                       + layers * int(cnt.sum()) * c.num_kv_heads * c.head_dim * 4)
        self.threads = oracle.num_threads()

    def run(self) -> float:
        t0 = time.perf_counter()
        scores = self.prob.index_scores(self.q_idx)
        idx, cnt = self.prob.topk(scores, selector="select")
        for q in self.qs:
            self.prob.sparse_attn(q, idx, cnt)
        return time.perf_counter() - t0


def oracle_sample_for(w):
    """The bounded sample both oracle timings use: up to 16 sequences of the workload, all layers, whole context."""
    c = w.cfg
    seqs = list(range(c.num_seqs)) if c.num_seqs <= 16 else list(range(0, c.num_seqs, c.num_seqs // 16))[:16]
    return OracleSample(w, seqs, c.num_layers), f"{len(seqs)} of {c.num_seqs} sequences, all {c.num_layers} layers, whole context"


def single_thread_oracle(w):
    """GB/s of the oracle on one thread, on one sequence and up to four layers (a few seconds at most)."""
    import oracle

    c = w.cfg
    threads = oracle.num_threads()
    if not set_omp_threads(1):
        return None
    try:
        smp = OracleSample(w, [0], min(4, c.num_layers))
        secs = smp.run()
        return {"value": smp.nbytes / secs / 1e9, "unit": "GB/s", "cores": 1,
                "sample": f"sequence 0, {smp.layers} layers, one pass ({secs:.1f} s)"}
    finally:
        set_omp_threads(threads)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from workloads import Workload

    oracle.build()
    w = Workload(pick_config(args))
    c = w.cfg
    smp, sample = oracle_sample_for(w)
    for _ in range(max(1, min(args.warmup, 2))):
        smp.run()
    times = [smp.run() for _ in range(args.steps)]
    med = statistics.median(times)
    val = smp.nbytes / med / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": med * 1e3, "step_ms": spread([t * 1e3 for t in times]),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(c, w, args),
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": smp.threads, "kind": "oracle",
                         "sample": sample + ", per step; input synthesis not timed; TopK by the oracle's partition selector",
                         "single_thread": single_thread_oracle(w)},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------------------- CUDA arm
class Problem:
    """Device tensors, params and buffers of one workload, and the ways of issuing its step."""

    def __init__(self, clsa, torch, w, dev, block_size=0):
        self.clsa, self.torch, self.w, self.dev = clsa, torch, w, dev
        c = self.c = w.cfg
        T = self.T = c.q_per_seq
        t = w.to_device(dev)
        if block_size:
            t = w.paginate_device(t, block_size)
        self.t = t
        L = self.L = c.num_layers
        self.p = clsa.make_params(num_seqs=c.num_seqs, num_q_heads=c.num_q_heads, num_kv_heads=c.num_kv_heads,
                                  head_dim=c.head_dim, idx_dim=c.idx_dim, top_k=c.top_k, num_layers=L,
                                  max_seq_len=w.max_seq_len, sm_scale=c.sm_scale, seq_start=t["seq_start"],
                                  seq_len=t["seq_len"], k_cache=t["k_cache"], v_cache=t["v_cache"],
                                  idx_k_cache=t["idx_k_cache"], q_per_seq=T, causal=c.causal,
                                  block_table=t.get("block_table"), block_size=block_size)
        self.ws = torch.zeros(clsa.clsa_workspace_bytes(self.p), dtype=torch.uint8, device=dev)
        self.idx = torch.empty((c.num_seqs, T, c.top_k), dtype=torch.int32, device=dev)
        self.cnt = torch.empty((c.num_seqs, T), dtype=torch.int32, device=dev)
        self.q_layers = [t["q_layers"][l] for l in range(L)]
        self.outs = [torch.empty((c.num_seqs, T, c.num_q_heads, c.head_dim), dtype=torch.bfloat16, device=dev) for _ in range(L)]
        self.stride = (w.max_seq_len + 63) // 64 * 64
        self.scores = torch.empty((c.num_seqs, T, self.stride), dtype=torch.float32, device=dev) if T == 1 else None
        self.alg_bytes = w.algorithmic_bytes()
        self.key_bytes = int(w.seq_len.astype("int64").sum()) * c.idx_dim * 2
        self.gathered_per_layer = int(w.selected_counts().sum()) * c.num_kv_heads * c.head_dim * 4

    def layer_hints(self, l):
        """A decoder that issues its layers one by one: alternate the walking direction, say that the rows are read
        again by the next layer, and -- from the second layer on -- that only the queries are still pending."""
        return self.clsa.make_hints(reverse=l & 1, keep_rows=l + 1 < self.L, only_q_pending=l > 0)

    def routing(self, q_idx=None):
        """Eq. 3. Decoding: the two public calls (scores in a buffer of the caller's). A prefill chunk: clsa_index_topk,
        which never materialises the T x n score matrix."""
        clsa = self.clsa
        q_idx = self.t["q_idx"] if q_idx is None else q_idx
        if self.T > 1:
            clsa.clsa_index_topk(self.p, q_idx, self.idx, self.cnt, self.ws)
            return
        clsa.clsa_index_scores(self.p, q_idx, self.scores, self.stride, self.ws)
        clsa.clsa_topk(self.p, self.scores, self.stride, self.idx, self.cnt, self.ws)

    def layers_one_by_one(self, q_list=None, out_list=None, between=None):
        q_list = self.q_layers if q_list is None else q_list
        out_list = self.outs if out_list is None else out_list
        for l in range(self.L):
            self.clsa.clsa_sparse_attn_hinted(self.p, q_list[l], self.idx, self.cnt, out_list[l], None, self.layer_hints(l), self.ws)
            if between is not None and l + 1 < self.L:
                between()

    def dependent_step(self, between=None):
        """Routing, then the layers one by one, each waiting for its predecessor (the public calls a decoder with a
        layer-to-layer dependency makes). `between`: called between two layers (a stand-in for the layer's FFN)."""
        self.routing()
        self.layers_one_by_one(between=between)

    def independent_step(self, q_idx=None, q_list=None, out_list=None):
        """clsa_decode_step (T = 1): the layers do not wait for one another. A prefill chunk (T > 1): the scores (a
        GEMM), the top-k, and the layers as one call."""
        clsa = self.clsa
        q_idx = self.t["q_idx"] if q_idx is None else q_idx
        q_list = self.q_layers if q_list is None else q_list
        out_list = self.outs if out_list is None else out_list
        if self.T == 1:
            clsa.clsa_decode_step(self.p, q_idx, q_list, out_list, self.idx, self.cnt, self.ws)
        else:
            self.routing(q_idx)
            clsa.clsa_sparse_attn_layers(self.p, q_list, self.idx, self.cnt, out_list, self.ws)


class Timer:
    """Event-timed steps on torch's current stream, each behind an L2 flush."""

    def __init__(self, torch, dev):
        self.torch, self.dev = torch, dev
        self.stream = torch.cuda.current_stream()
        self.flush_w = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
        self.flush_r = torch.zeros(64 << 20, dtype=torch.float32, device=dev)   # 256 MiB

    def flush(self):
        """Cold AND clean L2 before a timed step: rewrite 512 MiB (evicts everything), then stream 256 MiB of
        reads, which pushes the rewrite's dirty lines out to HBM so that their write-back is not charged to the
        step that follows."""
        self.flush_w.zero_()
        self.torch.sum(self.flush_r)

    def steps(self, fn, k, warmup=0, flush=True):
        """Per-step milliseconds of k calls of fn()."""
        torch = self.torch
        for _ in range(warmup):
            if flush:
                self.flush()
            fn()
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(k)]
        for a, b in ev:
            if flush:
                self.flush()
            a.record(self.stream)
            fn()
            b.record(self.stream)
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in ev]


def probe_us(clsa, torch, p, idx, cnt, hints, ws):
    """Device-side duration of one clsa_gather_probe launch (the probe leaves its earliest start and latest end, in
    nanoseconds of the GPU's global timer, in the workspace header)."""
    clsa.clsa_clear_status(ws)
    clsa.clsa_gather_probe(p, idx, cnt, hints, ws)
    torch.cuda.synchronize()
    words = ws[:32].view(torch.int64).cpu().numpy().view("uint64")
    start, end = int(~words[1]) & 0xFFFFFFFFFFFFFFFF, int(words[2])
    return (end - start) / 1e3


def gather_ceilings(clsa, torch, timer, pr):
    """What the memory system delivers to the attention kernel's access pattern, measured with clsa_gather_probe
    (the same split over the SMs, the same 16-byte asynchronous copies into the same shared-memory ring, no
    arithmetic), as bytes over the launch's own device-side duration: from DRAM, a launch over the workload's whole
    selected set right after an L2 flush; from L2, launches over a subset of the sequences whose selected rows fit
    in L2, repeated until resident."""
    c = pr.c
    cold = []
    for _ in range(5):
        timer.flush()
        cold.append(probe_us(clsa, torch, pr.p, pr.idx, pr.cnt, None, pr.ws))
    med = statistics.median(cold)
    out = {"dram_gather_ceiling": {"GBps": pr.gathered_per_layer / (med * 1e-6) / 1e9, "us_per_launch": med,
                                   "bytes": pr.gathered_per_layer,
                                   "how": "one probe launch over the whole selected set behind an L2 flush; device-side duration "
                                          "(first warp's start to last warp's end), ramp included"}}
    # From L2: a launch of the same size whose rows are resident. Every sequence of the probe's batch is pointed at
    # one of the first `nsrc` sequences' cache rows and index rows (round robin), so that the launch gathers as many
    # bytes as a real layer from a footprint that fits in L2 several times over.
    l2_bytes = torch.cuda.get_device_properties(pr.dev).L2_cache_size
    per_seq = pr.gathered_per_layer / c.num_seqs
    nsrc = max(1, min(c.num_seqs, int(0.25 * l2_bytes / per_seq)))
    src = torch.arange(c.num_seqs, device=pr.dev) % nsrc
    seq_start2 = pr.t["seq_start"][src].contiguous() if pr.t.get("block_table") is None else pr.t["seq_start"]
    seq_len2 = pr.t["seq_len"][src].contiguous()
    table2 = pr.t["block_table"][src].contiguous() if pr.t.get("block_table") is not None else None
    idx2, cnt2 = pr.idx[src].contiguous(), pr.cnt[src].contiguous()
    p2 = clsa.make_params(num_seqs=c.num_seqs, num_q_heads=c.num_q_heads, num_kv_heads=c.num_kv_heads, head_dim=c.head_dim,
                          idx_dim=c.idx_dim, top_k=c.top_k, num_layers=c.num_layers, max_seq_len=pr.w.max_seq_len,
                          sm_scale=c.sm_scale, seq_start=seq_start2, seq_len=seq_len2,
                          k_cache=pr.t["k_cache"], v_cache=pr.t["v_cache"], idx_k_cache=pr.t["idx_k_cache"],
                          block_table=table2, block_size=pr.p.block_size)
    ws2 = torch.zeros(clsa.clsa_workspace_bytes(p2), dtype=torch.uint8, device=pr.dev)
    hint = clsa.make_hints(keep_rows=1)
    warm = [probe_us(clsa, torch, p2, idx2, cnt2, hint, ws2) for _ in range(8)][3:]
    med = statistics.median(warm)
    bytes2 = int(cnt2.sum().item()) * c.num_kv_heads * c.head_dim * 4
    out["l2_gather_ceiling"] = {"GBps": bytes2 / (med * 1e-6) / 1e9, "us_per_launch": med, "bytes": bytes2,
                                "footprint_bytes": int(cnt2[:nsrc].sum().item()) * c.num_kv_heads * c.head_dim * 4,
                                "how": f"probe launches of a whole layer's size whose sequences all point at the first {nsrc} "
                                       "sequences' rows (resident in L2 after the first launches); device-side duration, ramp "
                                       "included"}
    return out


def breakdown(clsa, torch, timer, pr, nb):
    """Per-kernel microseconds of the dependent step: the same launches with events between the segments."""
    stream, L = timer.stream, pr.L
    acc = {"index_scores": [], "topk": [], "first_layer_cold": [], "other_layers": []}
    for i in range(nb + 2):
        timer.flush()
        m = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
        m[0].record(stream)
        clsa.clsa_index_scores(pr.p, pr.t["q_idx"], pr.scores, pr.stride, pr.ws)
        m[1].record(stream)
        clsa.clsa_topk(pr.p, pr.scores, pr.stride, pr.idx, pr.cnt, pr.ws)
        m[2].record(stream)
        clsa.clsa_sparse_attn_hinted(pr.p, pr.q_layers[0], pr.idx, pr.cnt, pr.outs[0], None, pr.layer_hints(0), pr.ws)
        m[3].record(stream)
        for l in range(1, L):           # L - 1 public calls back to back, no event between them
            clsa.clsa_sparse_attn_hinted(pr.p, pr.q_layers[l], pr.idx, pr.cnt, pr.outs[l], None, pr.layer_hints(l), pr.ws)
        m[4].record(stream)
        torch.cuda.synchronize()
        if i >= 2:
            for j, k in enumerate(acc):
                acc[k].append(m[j].elapsed_time(m[j + 1]) * 1e3)
    out = {k: statistics.median(v) for k, v in acc.items()}
    out["steady_layer"] = out.pop("other_layers") / (L - 1) if L > 1 else None
    out["note"] = "each segment between its own events (an event pair costs a few microseconds, which every segment carries)"
    return out


def chunk_breakdown(clsa, torch, timer, pr, nb):
    """Per-call microseconds of a prefill chunk's step: the fused routing (clsa_index_topk) and the L layers; and, for
    comparison, the routing as the two materialising calls (a T x n fp32 score matrix written and read back)."""
    stream = timer.stream
    acc = {"index_topk_fused": [], "sparse_attn": []}
    for i in range(nb + 1):
        timer.flush()
        m = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        m[0].record(stream)
        clsa.clsa_index_topk(pr.p, pr.t["q_idx"], pr.idx, pr.cnt, pr.ws)
        m[1].record(stream)
        clsa.clsa_sparse_attn_layers(pr.p, pr.q_layers, pr.idx, pr.cnt, pr.outs, pr.ws)
        m[2].record(stream)
        torch.cuda.synchronize()
        if i >= 1:
            for j, k in enumerate(acc):
                acc[k].append(m[j].elapsed_time(m[j + 1]) * 1e3)
    out = {k: statistics.median(v) for k, v in acc.items()}
    out["sparse_attn_per_layer"] = out["sparse_attn"] / pr.L
    scores = torch.empty((pr.c.num_seqs, pr.T, pr.stride), dtype=torch.float32, device=pr.dev)
    idx2, cnt2 = torch.empty_like(pr.idx), torch.empty_like(pr.cnt)
    pair = {"index_scores": [], "topk": []}
    for i in range(3):
        timer.flush()
        m = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        m[0].record(stream)
        clsa.clsa_index_scores(pr.p, pr.t["q_idx"], scores, pr.stride, pr.ws)
        m[1].record(stream)
        clsa.clsa_topk(pr.p, scores, pr.stride, idx2, cnt2, pr.ws)
        m[2].record(stream)
        torch.cuda.synchronize()
        if i >= 1:
            for j, k in enumerate(pair):
                pair[k].append(m[j].elapsed_time(m[j + 1]) * 1e3)
    out["materialising_pair"] = {k: statistics.median(v) for k, v in pair.items()}
    assert torch.equal(idx2, pr.idx) and torch.equal(cnt2, pr.cnt), "fused routing differs from the materialising pair"
    return out


def short_run(clsa, torch, timer, name, peak, steps=5, graph=False):
    """A few steps of another benchmark config: step time in both modes, algorithmic GB/s, per-kernel breakdown."""
    from workloads import CONFIGS, Workload

    pr = Problem(clsa, torch, Workload(CONFIGS[name]), timer.dev)
    out = {"num_seqs": pr.c.num_seqs, "q_per_seq": pr.T, "context": pr.c.ctx, "layers": pr.L,
           "algorithmic_bytes_per_step": pr.alg_bytes}
    ind = pr.independent_step
    if graph:
        ind()
        torch.cuda.synchronize()
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            pr.independent_step()
        ind = gr.replay
        out["launch"] = "CUDA graph replay of the independent-layers step"
    ms_ind = timer.steps(ind, steps, warmup=3)
    out["independent"] = {"step_us": spread_us(ms_ind),
                          "algorithmic_GBps": pr.alg_bytes / (statistics.median(ms_ind) * 1e-3) / 1e9}
    if pr.T == 1 and not graph:
        ms_dep = timer.steps(pr.dependent_step, steps, warmup=3)
        gbs = pr.alg_bytes / (statistics.median(ms_dep) * 1e-3) / 1e9
        out["dependent"] = {"step_us": spread_us(ms_dep), "algorithmic_GBps": gbs, "frac_of_hbm_peak": gbs / peak}
        out["breakdown_us"] = breakdown(clsa, torch, timer, pr, min(steps, 4))
    elif not graph:
        out["breakdown_us"] = chunk_breakdown(clsa, torch, timer, pr, min(steps, 3))
    assert clsa.clsa_device_status(pr.ws) == 0, f"{name}: device status word is not clean"
    return out


def time_projection(clsa, torch, pr):
    """clsa_project_append alone: the weights of Eq. 2 (and of the shared K/V rows) streamed once against the
    B*T newest hidden states. One launch lasts a few microseconds, below what a pair of events resolves, so 8
    launches are captured in a CUDA graph, once back to back (weights stay in L2: warm) and once each behind an
    L2 flush, with the flushes alone timed the same way and subtracted (cold)."""
    c, w, t, dev = pr.c, pr.w, pr.t, pr.dev
    proj = w.projection_to_device(dev)
    q = torch.empty((c.num_seqs, c.q_per_seq, c.idx_dim), dtype=torch.bfloat16, device=dev)
    scrub = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def call():
        clsa.clsa_project_append(pr.p, c.d_model, proj["h"], proj["w_q_idx"], proj["w_k_idx"], proj["w_k"], proj["w_v"], q,
                                 t["idx_k_cache"], t["k_cache"], t["v_cache"], pr.ws)

    def flush():
        scrub.fill_(1)

    call()
    torch.cuda.synchronize()
    reps = 8
    side = torch.cuda.Stream()
    graphs = {}
    with torch.cuda.stream(side):
        for name, body in (("warm", (call,)), ("flush", (flush,)), ("cold", (flush, call))):
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr, stream=side):
                for _ in range(reps):
                    for f in body:
                        f()
            graphs[name] = gr
        us = {}
        for name, gr in graphs.items():
            gr.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(side)
            for _ in range(10):
                gr.replay()
            e1.record(side)
            torch.cuda.synchronize()
            us[name] = e0.elapsed_time(e1) * 1e3 / (10 * reps)
    weight_bytes = 2 * c.d_model * (2 * c.idx_dim + 2 * c.num_kv_heads * c.head_dim)
    cold = us["cold"] - us["flush"]
    peak, peak_kind = measured_peaks()
    return {"kernel": "project_append_kernel", "rows": c.num_seqs * c.q_per_seq, "d_model": c.d_model,
            "weight_bytes": weight_bytes, "us_cold_l2": cold, "us_warm_l2": us["warm"],
            "weights_GBs_cold": weight_bytes / cold / 1e3, "frac_of_hbm_peak": weight_bytes / cold / 1e3 / peak,
            "peak_kind": peak_kind, "gpu_launches": 10 * reps * 2 + 1,
            "note": "a stream of 11.8 MB lasts 1.8 us at the HBM peak, less than a kernel launch and one memory round "
                    "trip: the op is latency-bound at decode batch sizes"}


def compare_baselines(clsa, torch, timer, pr, sparse_ms):
    """Two comparison points on the same inputs and kernels (context for the shared-routing design, Sec. 2.3):
    (a) routing recomputed in every layer (index scores + top-k + attention, L times), as a per-layer token-sparse
        design would do; (b) dense cross attention over the whole cache (Eq. 1), run as the k = n case of the same
        attention kernel with an index row that lists every position."""
    c, t, p = pr.c, pr.t, pr.p
    L, B, n = c.num_layers, c.num_seqs, pr.w.max_seq_len

    def per_layer_routing():
        for l in range(L):
            pr.routing()
            clsa.clsa_sparse_attn_hinted(p, pr.q_layers[l], pr.idx, pr.cnt, pr.outs[l], None, clsa.make_hints(reverse=l & 1), pr.ws)

    unamortised_ms = statistics.median(timer.steps(per_layer_routing, 5, warmup=1))
    pd = clsa.make_params(num_seqs=B, num_q_heads=c.num_q_heads, num_kv_heads=c.num_kv_heads, head_dim=c.head_dim,
                          idx_dim=c.idx_dim, top_k=n, num_layers=L, max_seq_len=n, sm_scale=c.sm_scale,
                          seq_start=t["seq_start"], seq_len=t["seq_len"], k_cache=t["k_cache"], v_cache=t["v_cache"],
                          idx_k_cache=t["idx_k_cache"], block_table=t.get("block_table"), block_size=p.block_size)
    ws_dense = torch.zeros(clsa.clsa_workspace_bytes(pd), dtype=torch.uint8, device=pr.dev)
    all_idx = torch.arange(n, dtype=torch.int32, device=pr.dev).repeat(B, 1).reshape(B, 1, n)
    all_idx = torch.where(all_idx < t["seq_len"].reshape(B, 1, 1), all_idx, torch.full_like(all_idx, -1))
    all_cnt = t["seq_len"].reshape(B, 1).to(torch.int32).contiguous()

    def dense_layers():
        for l in range(L):
            clsa.clsa_sparse_attn_hinted(pd, pr.q_layers[l], all_idx, all_cnt, pr.outs[l], None, clsa.make_hints(reverse=l & 1), ws_dense)

    dense_ms = statistics.median(timer.steps(dense_layers, 2, warmup=1))
    return {
        "comparison": "same inputs, same kernels, one GPU, layers issued one by one; context only",
        "workload": c.name,
        "clsa_step_us": sparse_ms * 1e3,
        "routing_in_every_layer_step_us": unamortised_ms * 1e3,
        "dense_cross_attention_L_layers_us": dense_ms * 1e3,
        "dense_per_layer_us": dense_ms * 1e3 / L,
        "dense_GBps": L * int(t["seq_len"].sum().item()) * c.num_kv_heads * c.head_dim * 4 / (dense_ms * 1e-3) / 1e9,
        "speedup_vs_dense_attention": dense_ms / sparse_ms,
        "speedup_vs_routing_in_every_layer": unamortised_ms / sparse_ms,
    }


def run_ours(args):
    import torch

    import __graft_entry__ as entry

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        entry._load_build_module().build()
    if dist is not None:
        dist.barrier()   # nobody loads the library before rank 0 has (re)built it
    import paper_2606_06467_b200 as clsa
    from workloads import Workload

    dev = torch.device("cuda", local)
    w = Workload(pick_config(args))
    c = w.cfg
    pr = Problem(clsa, torch, w, dev, args.block_size)
    T, L = pr.T, pr.L
    alg_bytes, gathered = pr.alg_bytes, pr.gathered_per_layer
    timer = Timer(torch, dev)
    stream = timer.stream
    peak, peak_kind = measured_peaks()
    K, W = args.steps, max(3, args.warmup)
    solo = rank == 0 and world == 1   # the legs that only a single-GPU run carries

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- independent layers (clsa_decode_step), device-resident -------------------------------------------
    independent = pr.independent_step
    if args.graph:
        independent()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):   # the binding launches on torch's current stream: the capture stream here
            pr.independent_step()
        independent = graph.replay
    sync_all()
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    sampler.resume()
    ind_ms = timer.steps(independent, K, warmup=W)
    sync_all()
    sampler.pause()
    ind_outs = [o.clone() for o in pr.outs]
    ind_med = max_over_ranks(statistics.median(ind_ms), dist, dev)

    # ---- dependent layers, device-resident: the headline ---------------------------------------------------
    decode = T == 1
    if decode:
        sync_all()
        sampler.resume()
        dep_ms = timer.steps(pr.dependent_step, K, warmup=W)
        sync_all()
        sampler.pause()
        dep_med = max_over_ranks(statistics.median(dep_ms), dist, dev)
        for l in range(L):   # the two modes split the selected set differently: the same result to rounding
            err = (pr.outs[l].float() - ind_outs[l].float()).abs().max().item()
            assert err <= 2e-2, f"layer {l}: the two modes differ by {err}"
    else:                    # a prefill chunk has one way of issuing its layers
        dep_ms, dep_med = ind_ms, ind_med
    del ind_outs
    assert clsa.clsa_device_status(pr.ws) == 0, "device status word is not clean"
    value = aggregate_value(world, alg_bytes, dep_med)

    # ---- end to end: per-step inputs from pinned host memory, per-step results back to the host --------
    # One pinned staging buffer each way: [q_idx | Q^(0) .. Q^(L-1)] up, [O^(0) .. O^(L-1)] down. q_idx goes up first
    # on the launch stream; the L query tensors follow on a second stream while the routing runs, and the launch
    # stream waits for them just before the first layer. The outputs come back in one of three ways (--e2e-out): the
    # layers store them straight into the pinned host buffer (any address the device can reach serves as an output),
    # one copy behind the last layer, or one copy per layer on a second stream while the layers behind it run.
    n_qidx = pr.t["q_idx"].numel()
    n_q = pr.q_layers[0].numel()
    h_in = torch.empty(n_qidx + L * n_q, dtype=torch.bfloat16).pin_memory()
    h_in[:n_qidx].copy_(pr.t["q_idx"].reshape(-1).cpu())
    for l in range(L):
        h_in[n_qidx + l * n_q: n_qidx + (l + 1) * n_q].copy_(pr.q_layers[l].reshape(-1).cpu())
    d_in = torch.empty_like(h_in, device=dev)
    d_qidx = d_in[:n_qidx].view(pr.t["q_idx"].shape)
    d_q = [d_in[n_qidx + l * n_q: n_qidx + (l + 1) * n_q].view(pr.q_layers[l].shape) for l in range(L)]
    d_out = torch.empty((L,) + tuple(pr.outs[0].shape), dtype=torch.bfloat16, device=dev)
    h_out = torch.empty(d_out.shape, dtype=torch.bfloat16).pin_memory()
    out_mode = {True: args.e2e_out, False: args.e2e_out}   # keyed by "layers one by one"
    if args.e2e_out == "auto":
        out_mode = {True: "streamed", False: "mapped"}
    if out_mode[False] == "streamed":
        out_mode[False] = "copy"
    if not decode:
        out_mode = {True: "copy", False: "copy"}
    copy_stream = torch.cuda.Stream(device=dev)
    out_stream = torch.cuda.Stream(device=dev)
    q_ready = torch.cuda.Event()
    step_start = torch.cuda.Event()
    layer_done = [torch.cuda.Event() for _ in range(L)]
    outs_home = torch.cuda.Event()
    kGroup = args.e2e_group

    def e2e_step(one_by_one):
        if not decode:  # a prefill chunk: one upload, the three calls, one download
            d_in.copy_(h_in, non_blocking=True)
            pr.independent_step(d_qidx, d_q, [d_out[l] for l in range(L)])
            h_out.copy_(d_out, non_blocking=True)
            return
        mode = out_mode[one_by_one]
        targets = [(h_out if mode == "mapped" else d_out)[l] for l in range(L)]
        d_in[:n_qidx].copy_(h_in[:n_qidx], non_blocking=True)
        step_start.record(stream)
        with torch.cuda.stream(copy_stream):
            # The upload belongs to this step, and it goes behind q_idx's: released at the same moment, the two copies
            # are taken in either order by the copy engine, and every other step the 4 KB that the first kernel waits
            # for queued behind the 2 MB that nobody needs yet.
            copy_stream.wait_event(step_start)
            d_in[n_qidx:].copy_(h_in[n_qidx:], non_blocking=True)
            q_ready.record(copy_stream)
        pr.routing(d_qidx)
        stream.wait_event(q_ready)
        if one_by_one and mode == "streamed":
            # a layer's output goes home on a second stream while the layers behind it run
            # (in groups of kGroup layers: a copy per layer costs the host more than it saves the device)
            for l in range(L):
                clsa.clsa_sparse_attn_hinted(pr.p, d_q[l], pr.idx, pr.cnt, targets[l], None, pr.layer_hints(l), pr.ws)
                if (l + 1) % kGroup == 0 or l == L - 1:
                    first = l - l % kGroup
                    layer_done[l].record(stream)
                    with torch.cuda.stream(out_stream):
                        out_stream.wait_event(layer_done[l])
                        h_out[first:l + 1].copy_(d_out[first:l + 1], non_blocking=True)
            with torch.cuda.stream(out_stream):
                outs_home.record(out_stream)
            stream.wait_event(outs_home)             # the step ends when the last output has reached the host
            return
        if one_by_one:
            pr.layers_one_by_one(d_q, targets)
        else:
            clsa.clsa_sparse_attn_layers(pr.p, d_q, pr.idx, pr.cnt, targets, pr.ws)
        if mode != "mapped":
            h_out.copy_(d_out, non_blocking=True)

    sampler.resume()
    e2e_ms = timer.steps(lambda: e2e_step(decode), K, warmup=3)
    sync_all()
    for l in range(L):  # the host copy of the last end-to-end step equals the device-resident step's outputs
        assert torch.equal(h_out[l].view(torch.int16), pr.outs[l].cpu().view(torch.int16)), f"end-to-end output {l} differs"
    e2e_ind_ms = timer.steps(lambda: e2e_step(False), K, warmup=3) if decode else e2e_ms
    sync_all()
    clocks = sampler.stop()   # sampled across every timed region above
    e2e_med = max_over_ranks(statistics.median(e2e_ms), dist, dev)
    h2d, d2h = h_in.numel() * 2, h_out.numel() * 2

    # ---- the same step with an FFN-sized read between the layers ----------------------------------------
    # In the model each layer's FFN weights (about 118 MB in bf16 at the paper's 2560 x 7680 width, three matrices)
    # pass through L2 between two attention launches, so the rows a layer leaves in L2 are not all there for the
    # next one. A plain read of that many bytes stands in for the FFN; its own time is measured alone and taken off.
    dep_ffn = None
    if decode and solo and L > 1:
        ffn = torch.zeros((3 * 2560 * 7680 * 2) // 4, dtype=torch.int32, device=dev)

        def ffn_read():
            torch.sum(ffn)

        def ffn_only():
            for _ in range(L - 1):
                ffn_read()

        kk = min(K, 10)
        with_ffn = statistics.median(timer.steps(lambda: pr.dependent_step(between=ffn_read), kk, warmup=2))
        alone = statistics.median(timer.steps(ffn_only, kk, warmup=2))
        gbs = alg_bytes / ((with_ffn - alone) * 1e-3) / 1e9
        dep_ffn = {"step_us": (with_ffn - alone) * 1e3, "ffn_reads_alone_us": alone * 1e3, "ffn_bytes_per_layer": ffn.numel() * 4,
                   "algorithmic_GBps": gbs, "frac_of_hbm_peak": gbs / peak,
                   "what": "the dependent step with a 118 MB read (a stand-in for a layer's FFN weights) between consecutive "
                           "layers; the reads' own time, measured alone in the same loop, is taken off"}
        del ffn

    # ---- per-kernel durations and the gather ceilings -----------------------------------------------------
    bd = ceilings = None
    if not args.no_breakdown:
        if decode:
            bd = breakdown(clsa, torch, timer, pr, min(K, 20))
            if solo:
                ceilings = gather_ceilings(clsa, torch, timer, pr)
        else:
            bd = chunk_breakdown(clsa, torch, timer, pr, min(K, 6))

    # ---- roofline of the dominant kernel of the timed (dependent) configuration ------------------------------
    roofline = None
    if bd is not None and decode:
        cold_us = bd["first_layer_cold"]
        steady_us = bd["steady_layer"] or cold_us
        rate = lambda us: gathered / (us * 1e-6) / 1e9
        roofline = {
            "bound": "hbm",
            "kernel": "sparse attention, one layer = one launch that waits for its predecessor (L launches per step)",
            "achieved": rate(steady_us), "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": rate(steady_us) / peak,
            "algorithmic_bytes_per_launch": gathered,
            "steady_layer": {"us": steady_us, "GBps": rate(steady_us), "frac_of_hbm_peak": rate(steady_us) / peak},
            "cold_first_layer": {"us": cold_us, "GBps": rate(cold_us), "frac_of_hbm_peak": rate(cold_us) / peak,
                                 "traffic": profiled_traffic(c.name, "sparse_attn_kernel_cold")},
            "traffic": profiled_traffic(c.name, "sparse_attn_kernel"),
            "traffic_note": "DRAM bytes read by one steady layer (cold_first_layer.traffic: by the first layer), from a "
                            "one-pass ncu capture of this workload with the cache state carried from launch to launch "
                            "(profiles/launch_list_headline128k.md; for other workloads one launch behind an L2 flush); "
                            "recorded in profiles/traffic.txt, not measured in this run",
            "note": "achieved/frac: algorithmic (gathered) bytes of one layer over the steady layer's time (layers 2..L of the "
                    "dependent step, event-timed as a group). A steady layer finds part of its rows in L2, where its "
                    "predecessor left them, so this is a rate of algorithmic bytes and HBM traffic stays below it; the cold "
                    "first layer reads every row from DRAM",
        }
        for key, name in (("steady_layer", "sparse_attn_kernel"), ("cold_first_layer", "sparse_attn_kernel_cold")):
            t = profiled_traffic(c.name, name)   # DRAM bytes of that launch as recorded from the one-pass ncu capture
            if t is not None:
                roofline[key]["traffic"] = t
                roofline[key]["dram_GBps"] = t / (roofline[key]["us"] * 1e-6) / 1e9
                roofline[key]["dram_frac_of_hbm_peak"] = roofline[key]["dram_GBps"] / peak
        if ceilings is not None:
            roofline.update(ceilings)
            for key in ("steady_layer", "cold_first_layer"):
                roofline[key]["frac_of_dram_gather_ceiling"] = roofline[key]["GBps"] / ceilings["dram_gather_ceiling"]["GBps"]
        key_gbs = pr.key_bytes / (bd["index_scores"] * 1e-6) / 1e9
        roofline["others"] = [
            {"kernel": "index_scores_decode_kernel (one event-timed call)", "bound": "hbm",
             "algorithmic_bytes_per_launch": pr.key_bytes, "us": bd["index_scores"], "achieved": key_gbs, "frac": key_gbs / peak,
             "traffic": profiled_traffic(c.name, "index_scores_decode_kernel"),
             "traffic_note": "scaled from an ncu capture of the mid workload by the keys streamed; not measured in this run"},
            {"kernel": "topk_radix_kernel", "bound": "latency", "us": bd["topk"],
             "note": "cluster barriers and dependent sweeps, not bytes"}]

    # ---- the modes side by side ------------------------------------------------------------------------------------
    def mode(ms_list, med, e2e_list):
        gbs = world * alg_bytes / (med * 1e-3) / 1e9
        return {"step_us": spread_us(ms_list), "algorithmic_GBps": gbs, "frac_of_hbm_peak": gbs / world / peak,
                "frac_of_nominal_8TBps": gbs / world / 8000.0, "e2e_step_us": spread_us(e2e_list),
                "e2e_algorithmic_GBps": world * alg_bytes / (statistics.median(e2e_list) * 1e-3) / 1e9}

    modes = {}
    if decode:
        modes["dependent"] = mode(dep_ms, dep_med, e2e_ms)
        modes["dependent"]["what"] = ("clsa_index_scores, clsa_topk, then one clsa_sparse_attn_hinted per layer, each launch waiting "
                                      "for its predecessor: what a decoder with a layer-to-layer dependency runs (the headline)")
        if dep_ffn is not None:
            modes["dependent_with_ffn_reads"] = dep_ffn
    modes["independent"] = mode(ind_ms, ind_med, e2e_ind_ms)
    modes["independent"]["what"] = ("clsa_decode_step: every layer's queries are handed over up front, the layers do not wait for "
                                    "one another, go two per launch (the rows are copied from L2 once for both) and share the "
                                    "selected rows through L2 -- a rate of algorithmic bytes above the HBM peak is L2 reuse, not "
                                    "HBM bandwidth" if decode else
                                    "a prefill chunk: clsa_index_scores (tensor-core GEMM), clsa_topk, clsa_sparse_attn_layers")
    if decode and bd is not None and ceilings is not None:
        per_layer = (ind_med * 1e3 - bd["index_scores"] - bd["topk"]) / L
        modes["independent"]["attention_per_layer_us"] = per_layer
        modes["independent"]["attention_frac_of_l2_gather_ceiling"] = (gathered / (per_layer * 1e-6) / 1e9) / ceilings["l2_gather_ceiling"]["GBps"]
        modes["independent"]["attention_note"] = ("gathered bytes per layer over the step's attention time per layer, against the rate at "
                                                  "which one launch copies that many bytes from L2; above 1 where two layers share a "
                                                  "launch, because the pair copies its rows once")

    cpu_baseline = None
    if solo and not args.no_cpu_baseline:
        import oracle

        oracle.build()
        smp, sample = oracle_sample_for(w)
        secs, nbytes, passes = 0.0, 0, 0
        while secs < 10.0 and passes < 200:
            secs += smp.run()
            nbytes += smp.nbytes
            passes += 1
        cpu_baseline = {"value": nbytes / secs / 1e9, "unit": "GB/s", "cores": smp.threads, "kind": "oracle",
                        "sample": f"{sample}, {passes} passes ({secs:.1f} s of oracle time; input synthesis not timed; TopK by "
                                  "the oracle's partition selector)",
                        "single_thread": single_thread_oracle(w)}
        del smp

    comparison = None
    if args.compare and solo and decode:
        comparison = compare_baselines(clsa, torch, timer, pr, dep_med)

    projection = None
    if args.project and solo:   # it overwrites the newest rows of the caches: nothing of this workload runs after it
        projection = time_projection(clsa, torch, pr)

    other = None
    if solo and not args.no_other_configs and args.config == "headline128k" and not args.block_size:
        del pr, d_in, d_q, d_qidx, d_out
        torch.cuda.empty_cache()
        other = {}
        for name, graph in (("mid", False), ("ragged", False), ("tiny", False), ("tiny", True), ("prefill_chunk", False)):
            key = name + ("_graph" if graph else "")
            try:
                other[key] = short_run(clsa, torch, timer, name, peak, steps=5, graph=graph)
            except Exception as e:  # one config failing must not lose the headline line
                other[key] = {"error": f"{type(e).__name__}: {e}"}
            torch.cuda.empty_cache()

    if rank == 0:
        cfg = config_dict(c, w, args, world)
        modes["independent"]["launch"] = "CUDA graph replay" if args.graph else "stream launches"
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": dep_med, "step_us": dep_med * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": cfg,
            "frac_of_hbm_peak": value / world / peak, "frac_of_nominal_8TBps": value / world / 8000.0,
            "modes": modes, "clocks": clocks, "roofline": roofline, "breakdown_us": bd, "cpu_baseline": cpu_baseline,
            "e2e": {"value": aggregate_value(world, alg_bytes, e2e_med), "unit": "GB/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_med,
                    "note": "the headline's mode with per-step inputs from pinned host memory (q_idx on the launch stream, the L "
                            "query tensors on a second stream while the routing runs) and all L outputs back ("
                            + {"mapped": "stored by the layers straight into pinned host memory", "copy": "one copy behind the last layer",
                               "streamed": f"the outputs of each {kGroup} layers copied on a second stream while the next layers run"}[out_mode[decode]]
                            + "); the KV "
                            "and indexer-key caches are decoder state and stay resident"},
            "gpu_launches": K * (2 + L),
        }
        if other is not None:
            line["other_configs"] = other
        if projection is not None:
            line["projection"] = projection
        print(json.dumps(line))
        if comparison is not None:
            print(json.dumps(comparison))
    if dist is not None:
        dist.destroy_process_group()


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
