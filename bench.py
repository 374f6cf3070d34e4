#!/usr/bin/env python
"""Benchmark of the CLSA decode hot path: index scores + top-k + L sparse-attention layers per step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

A step is one `clsa_decode_step` call (through the C ABI) over one batch of seeded synthetic input
that is already resident in HBM. Each timed step is bracketed by its own CUDA events on the launch
stream; between steps a 512 MiB buffer is rewritten so every step starts with a cold L2 (the reuse
of gathered rows between the layers of one step is part of the method and is kept).
`value` = algorithmic bytes per step (indexer-key bytes + L * selected rows * Hkv * D * 2 B * {K,V})
divided by the mean step time, summed over ranks. With --gpus N > 1 (launched by torchrun) every rank
runs an independent replica of the workload: the path has no exchange step, so there is no collective
on the data path ("replicas only").

--impl reference times the CPU oracle on the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode step HBM GB/s (index+top-k+L-layer sparse attn)"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
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
                    help="capture the step once into a CUDA graph and time replays (removes host launch gaps; matters "
                         "for small, launch-bound workloads)")
    ap.add_argument("--compare", action="store_true",
                    help="also time, on the same inputs, dense attention over the whole cache (Eq. 1) and routing "
                         "repeated in every layer, and print them as a second JSON line")
    ap.add_argument("--project", action="store_true",
                    help="also time the upstream step (Eq. 2 projections of the new tokens + cache append, "
                         "clsa_project_append) on the same workload; reported under \"projection\", not part of the step")
    ap.add_argument("--block-size", type=int, default=0, help="page the caches into scattered blocks of this many rows")
    ap.add_argument("--e2e-out", default="mapped", choices=["mapped", "copy"],
                    help="end-to-end leg, decode: the layers store their outputs straight into pinned host memory "
                         "(mapped) or into HBM followed by one device-to-host copy (copy)")
    ap.add_argument("--profile-range", action="store_true",
                    help="bracket one extra step (after the warm-up, L2 flushed first) with cudaProfilerStart/Stop, so "
                         "that a profiler in range mode sees the whole chained step with its layers in flight together")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
    ap.add_argument("--no-breakdown", action="store_true", help="skip the per-kernel instrumented loop")
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


class ClockSampler(threading.Thread):
    """Polls NVML (read-only) for SM clock and clock-event reasons while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop_evt = threading.Event()
        self._active = threading.Event()   # samples are taken only while a timed region runs
        self._active.set()
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


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# --------------------------------------------------------------------------------------- oracle legs
class OracleSample:
    """The oracle, as it stands, on sequences `seqs` and `layers` layers of workload `w`.

    Input synthesis happens once here and is never timed (the K/V rows the selection will touch are found
    by one untimed routing pass); `run()` then times scores + top-k + every layer's attention."""

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
        idx, cnt = route.topk(route.index_scores(self.q_idx))
        kc = np.zeros((sub.total_rows, c.num_kv_heads, c.head_dim), dtype=np.uint16)
        vc = np.zeros_like(kc)
        for i, b in enumerate(seqs):
            for t in range(c.q_per_seq):
                loc = idx[i, t, : cnt[i, t]].astype(np.int64)
                rows = int(w.seq_start[b]) + loc
                kc[sub.seq_start[i] + loc] = w.kv_rows_bits("k", rows).reshape(-1, c.num_kv_heads, c.head_dim)
                vc[sub.seq_start[i] + loc] = w.kv_rows_bits("v", rows).reshape(-1, c.num_kv_heads, c.head_dim)
        self.prob = oracle.problem_from_workload(sub, k_cache=kc, v_cache=vc, idx_k_cache=kidx)
        self.qs = np.stack([w.q_layer_bits(l)[seqs] for l in range(layers)])
        self.nbytes = (int(sub.seq_len.astype(np.int64).sum()) * c.idx_dim * 2
                       + layers * int(cnt.sum()) * c.num_kv_heads * c.head_dim * 4)
        self.threads = oracle.num_threads()

    def run(self) -> float:
        t0 = time.perf_counter()
        self.prob.decode_step(self.q_idx, self.qs)
        return time.perf_counter() - t0


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from workloads import CONFIGS, Workload

    oracle.build()
    w = Workload(pick_config(args))
    c = w.cfg
    seqs = [0]
    sample = f"sequence 0 of {c.num_seqs}, all {c.num_layers} layers, whole context, per step"
    smp = OracleSample(w, seqs, c.num_layers)
    threads = smp.threads
    for _ in range(max(1, min(args.warmup, 3))):
        smp.run()
    tot_s, tot_b = 0.0, 0
    for _ in range(args.steps):
        tot_s += smp.run()
        tot_b += smp.nbytes
    val = tot_b / tot_s / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": tot_s / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": c.name, "num_seqs": c.num_seqs, "context": c.ctx, "top_k": c.top_k,
                   "layers": c.num_layers, "q_heads": c.num_q_heads, "kv_heads": c.num_kv_heads, "idx_dim": c.idx_dim},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def compare_baselines(clsa, torch, w, t, p, ws, idx, cnt, q_layers, outs, flush, stream, sparse_ms):
    """Two comparison points on the same inputs and kernels (context for the shared-routing design, Sec. 2.3):
    (a) routing recomputed in every layer (index scores + top-k + attention, L times), as a per-layer token-sparse
        design would do; (b) dense cross attention over the whole cache (Eq. 1), run as the k = n case of the same
        attention kernel with an index row that lists every position."""
    c = w.cfg
    L, B, n = c.num_layers, c.num_seqs, w.max_seq_len
    stride = (n + 63) // 64 * 64
    scores = torch.empty((B, 1, stride), dtype=torch.float32, device=idx.device)

    def timed(fn, reps=5):
        fn()
        torch.cuda.synchronize()
        tot = 0.0
        for _ in range(reps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            fn()
            e1.record(stream)
            torch.cuda.synchronize()
            tot += e0.elapsed_time(e1)
        return tot / reps

    def per_layer_routing():
        for l in range(L):
            clsa.clsa_index_scores(p, t["q_idx"], scores, stride, ws, stream=stream)
            clsa.clsa_topk(p, scores, stride, idx, cnt, ws, stream=stream)
            clsa.clsa_sparse_attn_hinted(p, q_layers[l], idx, cnt, outs[l], None, clsa.make_hints(reverse=l & 1), ws, stream=stream)

    unamortised_ms = timed(per_layer_routing)
    # dense: every position selected
    pd = clsa.make_params(num_seqs=B, num_q_heads=c.num_q_heads, num_kv_heads=c.num_kv_heads, head_dim=c.head_dim,
                          idx_dim=c.idx_dim, top_k=n, num_layers=L, max_seq_len=n, sm_scale=c.sm_scale,
                          seq_start=t["seq_start"], seq_len=t["seq_len"], k_cache=t["k_cache"], v_cache=t["v_cache"],
                          idx_k_cache=t["idx_k_cache"], block_table=t.get("block_table"), block_size=p.block_size)
    all_idx = torch.arange(n, dtype=torch.int32, device=idx.device).repeat(B, 1).reshape(B, 1, n)
    all_idx = torch.where(all_idx < t["seq_len"].reshape(B, 1, 1), all_idx, torch.full_like(all_idx, -1))
    all_cnt = t["seq_len"].reshape(B, 1).to(torch.int32).contiguous()
    ws_dense = torch.zeros(clsa.clsa_workspace_bytes(pd), dtype=torch.uint8, device=idx.device)

    def dense_layers():
        for l in range(L):
            clsa.clsa_sparse_attn_hinted(pd, q_layers[l], all_idx, all_cnt, outs[l], None, clsa.make_hints(reverse=l & 1), ws_dense, stream=stream)

    dense_ms = timed(dense_layers, reps=2)
    return {
        "comparison": "same inputs, same kernels, one GPU; context only",
        "workload": c.name,
        "clsa_step_us": sparse_ms * 1e3,
        "routing_in_every_layer_step_us": unamortised_ms * 1e3,
        "dense_cross_attention_L_layers_us": dense_ms * 1e3,
        "dense_per_layer_us": dense_ms * 1e3 / L,
        "dense_GBps": L * int(t["seq_len"].sum().item()) * c.num_kv_heads * c.head_dim * 4 / (dense_ms * 1e-3) / 1e9,
        "speedup_vs_dense_attention": dense_ms / sparse_ms,
        "speedup_vs_routing_in_every_layer": unamortised_ms / sparse_ms,
    }


# --------------------------------------------------------------------------------------- CUDA arm
def time_projection(clsa, torch, w, t, p, ws, dev):
    """clsa_project_append alone: the weights of Eq. 2 (and of the shared K/V rows) streamed once against the
    B*T newest hidden states. One launch lasts a few microseconds, below what a pair of events resolves, so 8
    launches are captured in a CUDA graph, once back to back (weights stay in L2: warm) and once each behind an
    L2 flush, with the flushes alone timed the same way and subtracted (cold)."""
    c = w.cfg
    proj = w.projection_to_device(dev)
    q = torch.empty((c.num_seqs, c.q_per_seq, c.idx_dim), dtype=torch.bfloat16, device=dev)
    scrub = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def call():
        clsa.clsa_project_append(p, c.d_model, proj["h"], proj["w_q_idx"], proj["w_k_idx"], proj["w_k"], proj["w_v"], q,
                                 t["idx_k_cache"], t["k_cache"], t["v_cache"], ws)

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
    from workloads import CONFIGS, Workload

    dev = torch.device("cuda", local)
    w = Workload(pick_config(args))
    c = w.cfg
    T = c.q_per_seq
    t = w.to_device(dev)
    if args.block_size:
        t = w.paginate_device(t, args.block_size)
    L = c.num_layers
    p = clsa.make_params(num_seqs=c.num_seqs, num_q_heads=c.num_q_heads, num_kv_heads=c.num_kv_heads,
                         head_dim=c.head_dim, idx_dim=c.idx_dim, top_k=c.top_k, num_layers=L, max_seq_len=w.max_seq_len,
                         sm_scale=c.sm_scale, seq_start=t["seq_start"], seq_len=t["seq_len"], k_cache=t["k_cache"],
                         v_cache=t["v_cache"], idx_k_cache=t["idx_k_cache"], q_per_seq=T, causal=c.causal,
                         block_table=t.get("block_table"), block_size=args.block_size)
    ws = torch.zeros(clsa.clsa_workspace_bytes(p), dtype=torch.uint8, device=dev)
    idx = torch.empty((c.num_seqs, T, c.top_k), dtype=torch.int32, device=dev)
    cnt = torch.empty((c.num_seqs, T), dtype=torch.int32, device=dev)
    q_layers = [t["q_layers"][l] for l in range(L)]
    outs = [torch.empty((c.num_seqs, T, c.num_q_heads, c.head_dim), dtype=torch.bfloat16, device=dev) for _ in range(L)]
    stride = (w.max_seq_len + 63) // 64 * 64
    chunk_scores = torch.empty((c.num_seqs, T, stride), dtype=torch.float32, device=dev) if T > 1 else None
    flush_w = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    flush_r = torch.zeros(64 << 20, dtype=torch.float32, device=dev)   # 256 MiB

    class _Flush:
        """Cold AND clean L2 before a timed step: rewrite 512 MiB (evicts everything), then stream 256 MiB of
        reads, which pushes the rewrite's dirty lines out to HBM so that their write-back is not charged to
        the step that follows."""

        @staticmethod
        def zero_():
            flush_w.zero_()
            torch.sum(flush_r)

    flush = _Flush
    alg_bytes = w.algorithmic_bytes()
    stream = torch.cuda.current_stream()

    def run_step(q_idx_t, q_list, out_list=None):
        out_list = outs if out_list is None else out_list
        if T == 1:
            clsa.clsa_decode_step(p, q_idx_t, q_list, out_list, idx, cnt, ws, stream=None)
        else:  # a prefill chunk: the scores (a GEMM here), the top-k, and the layers as one call
            clsa.clsa_index_scores(p, q_idx_t, chunk_scores, stride, ws, stream=None)
            clsa.clsa_topk(p, chunk_scores, stride, idx, cnt, ws, stream=None)
            clsa.clsa_sparse_attn_layers(p, q_list, idx, cnt, out_list, ws, stream=None)

    def step():
        run_step(t["q_idx"], q_layers)

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        flush.zero_()
        step()
    sync_all()
    if args.graph:
        eager_step = step
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):   # the binding launches on torch's current stream: the capture stream here
            eager_step()

        def step():  # noqa: F811
            graph.replay()

        for _ in range(3):
            flush.zero_()
            step()
        sync_all()
    if args.profile_range:
        flush.zero_()
        sync_all()
        torch.cuda.profiler.start()
        step()
        torch.cuda.synchronize()
        torch.cuda.profiler.stop()
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    K = args.steps
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for i in range(K):
        flush.zero_()
        ev[i][0].record(stream)
        step()
        ev[i][1].record(stream)
    sync_all()
    sampler.pause()
    total_ms = sum(a.elapsed_time(b) for a, b in ev)
    assert clsa.clsa_device_status(ws) == 0, "device status word is not clean"
    total_ms = max_over_ranks(total_ms, dist, dev)
    ms_per_step = total_ms / K
    value = aggregate_value(world, alg_bytes, ms_per_step)

    # ---- end to end: per-step inputs from pinned host memory, per-step results back to the host --------
    # One pinned staging buffer each way: [q_idx | Q^(0) .. Q^(L-1)] up, [O^(0) .. O^(L-1)] down.
    n_qidx = t["q_idx"].numel()
    n_q = q_layers[0].numel()
    h_in = torch.empty(n_qidx + L * n_q, dtype=torch.bfloat16).pin_memory()
    h_in[:n_qidx].copy_(t["q_idx"].reshape(-1).cpu())
    for l in range(L):
        h_in[n_qidx + l * n_q: n_qidx + (l + 1) * n_q].copy_(q_layers[l].reshape(-1).cpu())
    d_in = torch.empty_like(h_in, device=dev)
    d_qidx = d_in[:n_qidx].view(t["q_idx"].shape)
    d_q = [d_in[n_qidx + l * n_q: n_qidx + (l + 1) * n_q].view(q_layers[l].shape) for l in range(L)]
    d_out = torch.empty((L,) + tuple(outs[0].shape), dtype=torch.bfloat16, device=dev)
    h_out = torch.empty(d_out.shape, dtype=torch.bfloat16).pin_memory()
    # A decode step's outputs are small (L x B x H x D bf16): the attention kernels can store them straight into the
    # pinned host buffer, which the device addresses through the unified address space, instead of into HBM followed
    # by a copy. The bytes that cross to the host are the same; the copy's launch and its wait for the last layer go.
    mapped_out = T == 1 and args.e2e_out == "mapped"
    e2e_outs = [(h_out if mapped_out else d_out)[l] for l in range(L)]

    # The routing needs only q_idx (a few KB). It goes up first on the launch stream; the L query tensors follow on a
    # second stream while the index scores and the top-k run, and the launch stream waits for them just before the
    # attention layers (the public calls clsa_index_scores, clsa_topk, clsa_sparse_attn_layers: together they are
    # clsa_decode_step, bit for bit). The outputs come back in one copy after the last layer.
    copy_stream = torch.cuda.Stream(device=dev)
    q_ready = torch.cuda.Event()
    step_start = torch.cuda.Event()
    e2e_scores = torch.empty((c.num_seqs, 1, stride), dtype=torch.float32, device=dev) if T == 1 else None

    def e2e_step():
        if T > 1:  # a prefill chunk: one upload, the three calls, one download
            d_in.copy_(h_in, non_blocking=True)
            run_step(d_qidx, d_q, e2e_outs)
            h_out.copy_(d_out, non_blocking=True)
            return
        step_start.record(stream)
        d_in[:n_qidx].copy_(h_in[:n_qidx], non_blocking=True)
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(step_start)       # the upload belongs to this step: it may not start earlier
            d_in[n_qidx:].copy_(h_in[n_qidx:], non_blocking=True)
            q_ready.record(copy_stream)
        clsa.clsa_index_scores(p, d_qidx, e2e_scores, stride, ws, stream=None)
        clsa.clsa_topk(p, e2e_scores, stride, idx, cnt, ws, stream=None)
        stream.wait_event(q_ready)
        clsa.clsa_sparse_attn_layers(p, d_q, idx, cnt, e2e_outs, ws, stream=None)
        if not mapped_out:
            h_out.copy_(d_out, non_blocking=True)

    for _ in range(3):
        flush.zero_()
        e2e_step()
    sync_all()
    ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    sampler.resume()
    for i in range(K):
        flush.zero_()
        ev2[i][0].record(stream)
        e2e_step()
        ev2[i][1].record(stream)
    sync_all()
    clocks = sampler.stop()   # sampled across both timed regions (device-resident and end-to-end)
    e2e_ms = sum(a.elapsed_time(b) for a, b in ev2)
    e2e_ms = max_over_ranks(e2e_ms, dist, dev)
    e2e_value = aggregate_value(world, alg_bytes, e2e_ms / K)
    h2d = h_in.numel() * 2
    d2h = h_out.numel() * 2
    for l in range(L):  # the host copy of the last end-to-end step equals the device-resident step's outputs
        assert torch.equal(h_out[l].view(torch.int16), outs[l].cpu().view(torch.int16)), f"end-to-end output {l} differs"

    # ---- per-kernel durations: the same launches issued as separate ABI calls with events between -------
    breakdown = None
    attn_us = None
    if not args.no_breakdown:
        scores = chunk_scores if T > 1 else torch.empty((c.num_seqs, 1, stride), dtype=torch.float32, device=dev)
        nb = min(K, 20)
        acc = {"index_scores": 0.0, "topk": 0.0, "sparse_attn": 0.0}
        for i in range(nb + 2):
            flush.zero_()
            marks = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            marks[0].record(stream)
            clsa.clsa_index_scores(p, t["q_idx"], scores, stride, ws, stream=stream)
            marks[1].record(stream)
            clsa.clsa_topk(p, scores, stride, idx, cnt, ws, stream=stream)
            marks[2].record(stream)
            for l in range(L):           # L public calls back to back, no event between them
                clsa.clsa_sparse_attn_hinted(p, q_layers[l], idx, cnt, outs[l], None,
                                             clsa.make_hints(reverse=l & 1, keep_rows=l + 1 < L, only_q_pending=l > 0), ws, stream=stream)
            marks[3].record(stream)
            torch.cuda.synchronize()
            if i >= 2:
                acc["index_scores"] += marks[0].elapsed_time(marks[1])
                acc["topk"] += marks[1].elapsed_time(marks[2])
                acc["sparse_attn"] += marks[2].elapsed_time(marks[3])
        breakdown = {k: v / nb * 1e3 for k, v in acc.items()}  # microseconds per step
        attn_us = breakdown["sparse_attn"] / L
        breakdown["sparse_attn_per_layer"] = attn_us
        # inside clsa_decode_step the layers overlap head to tail; what is left of the step after the two
        # routing kernels, per layer:
        breakdown["sparse_attn_per_layer_in_step"] = (ms_per_step * 1e3 - breakdown["index_scores"] - breakdown["topk"]) / L

    peak, peak_kind = measured_peaks()
    gathered_per_layer = int(w.selected_counts().sum()) * c.num_kv_heads * c.head_dim * 4
    roofline = {
        "bound": "hbm", "kernel": "sparse_attn_kernel, one layer (one launch)",
        "achieved": (gathered_per_layer / (attn_us * 1e-6) / 1e9) if attn_us else None,
        "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
        "frac": (gathered_per_layer / (attn_us * 1e-6) / 1e9 / peak) if attn_us else None,
        "traffic": None,
        "algorithmic_bytes_per_launch": gathered_per_layer,
        "step_frac": value / world / peak,
        "note": "achieved/frac: one attention launch on its own (whole-GPU launch shape, event-timed back to back, "
                "each launch waiting for its predecessor). In the chained step the layers do not wait for one another: "
                "several are in flight at once over the same selected rows and share them through L2, which is why "
                "step_frac (whole step, all algorithmic bytes / step time / peak) can exceed 1.",
    }
    if breakdown is not None:
        in_step_us = breakdown["sparse_attn_per_layer_in_step"]
        roofline["achieved_in_step"] = gathered_per_layer / (in_step_us * 1e-6) / 1e9
        roofline["frac_in_step"] = roofline["achieved_in_step"] / peak
    roofline["traffic"] = profiled_traffic(c.name, "sparse_attn_kernel")
    if breakdown is not None and T == 1:
        # the step's other streaming kernel, as one event-timed public call (launch latency included)
        key_bytes = int(w.seq_len.astype("int64").sum()) * c.idx_dim * 2
        idx_gbs = key_bytes / (breakdown["index_scores"] * 1e-6) / 1e9
        roofline["others"] = [{"kernel": "index_scores_decode_kernel (one event-timed call)", "bound": "hbm",
                               "algorithmic_bytes_per_launch": key_bytes, "achieved": idx_gbs, "frac": idx_gbs / peak,
                               "traffic": profiled_traffic(c.name, "index_scores_decode_kernel")},
                              {"kernel": "topk_radix_kernel", "bound": "latency",
                               "us": breakdown["topk"], "note": "cluster barriers and dependent sweeps, not bytes"}]

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle

        oracle.build()
        seqs = list(range(c.num_seqs)) if c.num_seqs <= 16 else list(range(0, c.num_seqs, c.num_seqs // 16))[:16]
        smp = OracleSample(w, seqs, L)
        threads = smp.threads
        secs, nbytes, passes = 0.0, 0, 0
        while secs < 10.0 and passes < 200:
            secs += smp.run()
            nbytes += smp.nbytes
            passes += 1
        cpu_baseline = {"value": nbytes / secs / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
                        "sample": f"{len(seqs)} of {c.num_seqs} sequences, all {L} layers, {passes} passes "
                                  f"({secs:.1f} s of oracle time; input synthesis not timed)"}

    comparison = None
    if args.compare and rank == 0 and world == 1 and T == 1:
        comparison = compare_baselines(clsa, torch, w, t, p, ws, idx, cnt, q_layers, outs, flush, stream, ms_per_step)

    projection = None
    if args.project and rank == 0 and world == 1:   # last: it overwrites the newest rows of the caches
        projection = time_projection(clsa, torch, w, t, p, ws, dev)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": max(3, args.warmup),
            "ms_per_step": ms_per_step, "step_us": ms_per_step * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": c.name, "num_seqs": c.num_seqs, "context": c.ctx, "top_k": c.top_k, "layers": L,
                       "q_heads": c.num_q_heads, "kv_heads": c.num_kv_heads, "idx_dim": c.idx_dim,
                       "algorithmic_bytes_per_step": alg_bytes, "l2": "flushed between steps (512 MiB rewrite, then 256 MiB read so no dirty lines remain)",
                       "parallelism": "replicas only" if world > 1 else "single GPU",
                       "cache_layout": f"paged, {args.block_size}-row blocks" if args.block_size else "contiguous sequences",
                       "launch": "CUDA graph replay" if args.graph else "stream launches"},
            "clocks": clocks, "roofline": roofline, "breakdown_us": breakdown, "cpu_baseline": cpu_baseline,
            "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms / K,
                    "note": "per-step inputs from pinned host memory (q_idx on the launch stream, the L query tensors on a "
                            "second stream while the routing runs) and all L outputs back ("
                            + ("stored by the layers straight into pinned host memory" if mapped_out else "one copy") + "), through "
                            "clsa_index_scores + clsa_topk + clsa_sparse_attn_layers; the KV and indexer-key caches are "
                            "decoder state and stay resident"},
            "gpu_launches": K * (2 + L),
        }
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
