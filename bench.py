#!/usr/bin/env python
"""Benchmark of the delta-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = one pass of the prefill hot path (delta construction, sparsity counters, fused
hybrid attention, decode hand-off) over the Llama-3.2-1B attention-layer workload
(batch 1, 32 query / 8 KV heads, head_dim 64, T = 1024, bf16, block window 64) with the
threshold that gives about 60 % delta sparsity on the synthetic AR(1) streams.  The decode
step (cache prefilled to 2048 tokens, 256 steps, batch 1 and 16) is a different workload and
is timed in its own region of the same run; it is reported under "decode".

Rank 0 prints one JSON line.  With N > 1 every rank runs an independent replica of the
workload (different seed): the path shards over (batch, KV-head group, layer) with no
exchange step, so there is no collective on the data path ("scaling": "weak").
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2507_19608_b200 import workloads as WL

HEADLINE_THETA = 0.3          # S_m ~ 0.60 on the Llama-shape AR(1) workload
FLUSH_BYTES = 256 << 20       # > 126 MB of L2, written between timed iterations
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
                  "sm_max_mhz": 1965.0}
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "hybrid_attn_dram_traffic.txt")
KERNEL_SOURCES = {2: "k2_hybrid_attn_tcq.cu", 1: "k2_hybrid_attn_tc.cu", 0: "k2_hybrid_attn_generic.cu"}


def kernel_source_digest(kernel: int) -> str:
    import hashlib
    path = os.path.join(ROOT, "paper_2507_19608_b200", "csrc", KERNEL_SOURCES[kernel])
    with open(path, "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()[:16]


def measured_traffic(kernel: int, workload: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the hybrid-attention kernel, as the
    ncu capture summarised under profiles/ recorded it: lines `kernel workload source-digest bytes`.
    None when there is no capture of this workload, or the kernel source has changed since."""
    try:
        for line in open(TRAFFIC_FILE):
            f = line.split()
            if len(f) == 4 and not line.startswith("#") and int(f[0]) == kernel and f[1] == workload:
                return int(f[3]) if f[2] == kernel_source_digest(kernel) else None
    except (OSError, ValueError):
        pass
    return None


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, f"/tmp/delta_bench_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100", "-i", str(self.index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()          # the exact child started above
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                p = [x.strip() for x in line.split(",")]
                if len(p) < 7:
                    continue
                try:
                    sm.append(float(p[0])); mx.append(float(p[1]))
                except ValueError:
                    continue
                for nme, val in zip(names, p[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(nme)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# --------------------------------------------------------------------------- reference arm
def host_cores() -> int:
    """Cores this process may run on (the scheduler's affinity mask, not the machine's count)."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return min(max(n) if n else 1, host_cores())
    except Exception:
        return 1


class blas_limit:
    """Pins the BLAS pool the oracle's matrix products use to n threads (its Python loops are
    single-threaded whatever the pool is)."""

    def __init__(self, n):
        self.n, self.ctx = n, None

    def __enter__(self):
        try:
            from threadpoolctl import threadpool_limits
            self.ctx = threadpool_limits(limits=self.n, user_api="blas")
            self.ctx.__enter__()
        except Exception:
            self.ctx = None
        return self

    def __exit__(self, *a):
        if self.ctx is not None:
            self.ctx.__exit__(*a)


def oracle_prefill_sample(w, tensors, theta, heads):
    """The oracle, as it stands, on a few heads of the workload; returns seconds."""
    from oracle import delta_oracle as O
    g = w.H // w.H_kv
    t0 = time.perf_counter()
    for h in heads:
        O.prefill_head(tensors["q"][0, h], tensors["k"][0, h // g], tensors["v"][0, h // g], theta,
                       w.window, "block")
    return time.perf_counter() - t0


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = WL.WORKLOADS[args.workload]
    tensors = WL.make_qkv(w, n_decode=0)
    heads = list(range(0, w.H, max(1, w.H // args.ref_heads)))[:args.ref_heads]
    for _ in range(args.warmup):
        oracle_prefill_sample(w, tensors, args.theta, heads[:1])
    times = [oracle_prefill_sample(w, tensors, args.theta, heads) for _ in range(args.steps)]
    per_head = statistics.mean(times) / len(heads)
    step_s = per_head * w.H * w.B           # extrapolated to every head of the layer
    value = w.B * w.T / step_s
    cores = blas_threads()
    sample = (f"{len(heads)} of {w.H} heads per step (heads {heads}), full T={w.T}; "
              f"layer time extrapolated by head count; BLAS pool of {cores} threads on {host_cores()} "
              f"available cores, the oracle's row loops are single-threaded")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_dict(w, args.theta),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


METRIC = "delta-attn prefill tokens/s at Llama-3.2-1B layer shape (decode us/step alongside)"


def config_dict(w, theta):
    return {"workload": w.name, "B": w.B, "H": w.H, "H_kv": w.H_kv, "T": w.T, "d": w.d,
            "dtype": w.dtype, "theta": theta, "window": w.window, "window_shape": "block",
            "source": "query", "l2": f"flushed between timed iterations ({FLUSH_BYTES >> 20} MiB write)"}


# --------------------------------------------------------------------------- our arm
def to_dev(x, dtype, torch):
    if dtype == "bf16":
        return torch.from_numpy(WL.bf16_bits(x).view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


KERNEL_NAMES = {0: "generic (FP32 pipes)", 1: "tcgen05 + FP32 delta path", 2: "tcgen05 telescoped"}


def flop_model(w, stats, kernel):
    """Flops of one hybrid-attention launch, from the library's own counters.

    method: what the method itself has to do (Eq. 4 + Eq. 1): 2 x the executed multiply-adds of the
      score stage (d per in-window pair, nnz(dq_i) per out-of-window pair: the library's macs_done)
      plus 2 d per causal pair for P.V.  This is the figure the roofline fraction is taken from.
    executed: what the selected kernel really runs.  Kernel 2 (telescoped) multiplies q_hat.k
      densely, d multiply-adds for every pair, on the tensor cores and skips nothing; kernel 1
      runs the sparse products (plus one dense seed row per 128-row query tile) on the FP32 pipes;
      kernel 0 runs everything on the FP32 pipes.
    dense_equiv: 4 d per causal pair, what dense attention would be credited with."""
    BH = w.B * w.H
    N_c = w.T * (w.T + 1) // 2
    pv = 2.0 * w.d * N_c * BH                                   # P.V over every causal pair
    qk = 2.0 * stats["macs_done"]                               # exact in-window + fired out-of-window
    full, rem = divmod(w.T, w.window) if w.window > 0 else (0, 0)
    n_in = (full * w.window * (w.window + 1) // 2 + rem * (rem + 1) // 2) if w.window > 0 else 0
    qk_in = 2.0 * w.d * n_in * BH
    seeds = 2.0 * w.d * (N_c - n_in) * BH / 128.0               # one dense row per 128-row query tile
    dense_equiv = 4.0 * w.d * N_c * BH
    method = qk + pv
    if kernel == 2:
        return dict(method=method, executed=dense_equiv, alu=0.0, tensor=dense_equiv, dense_equiv=dense_equiv)
    if kernel == 1:
        return dict(method=method, executed=qk + seeds + pv, alu=(qk - qk_in) + seeds, tensor=qk_in + pv,
                    dense_equiv=dense_equiv)
    return dict(method=method, executed=qk + seeds + pv, alu=qk + seeds + pv, tensor=0.0, dense_equiv=dense_equiv)


def k2_roofline(w, stats, kernel, k2_ms, peaks, n_sm, sustained=False):
    """Roofline of the hybrid-attention kernel.  `achieved` and `frac` count the method's own flops
    (2 x executed multiply-adds of the score stage + 2 d N_c for P.V); the flops the kernel really
    executed and the dense-equivalent figure stand beside them under their own keys."""
    fm = flop_model(w, stats, kernel)
    sm_max = float(peaks.get("sm_max_mhz", 1965.0))
    alu_peak = n_sm * 128 * 2 * sm_max * 1e6 / 1e12          # TFLOP/s: SMs x FP32 lanes x FMA x clock
    t = k2_ms * 1e-3
    common = {"kernel": KERNEL_NAMES[kernel], "kernel_ms": k2_ms,
              "method_gflop_per_launch": fm["method"] / 1e9, "executed_gflop_per_launch": fm["executed"] / 1e9,
              "method_tflops": fm["method"] / t / 1e12, "executed_tflops": fm["executed"] / t / 1e12,
              "dense_equiv_tflops": fm["dense_equiv"] / t / 1e12, "traffic": measured_traffic(kernel, w.name)}
    if kernel == 2:
        key = "bf16_tflops_sustained" if sustained and "bf16_tflops_sustained" in peaks else "bf16_tflops"
        peak = float(peaks[key])
        a = fm["method"] / t / 1e12
        return {**common, "bound": "tensor", "achieved": a, "peak": peak, "unit": "TFLOP/s", "frac": a / peak,
                "executed_frac": fm["executed"] / t / 1e12 / peak,
                "peak_source": f"{peaks['_source']} cuBLAS bf16 {'sustained' if key.endswith('sustained') else 'burst'}",
                "note": "achieved = the method's flops (the kernel multiplies q_hat.k densely and skips nothing: "
                        "executed_tflops = dense_equiv_tflops)"}
    a = fm["alu"] / t / 1e12
    return {**common, "bound": "alu", "achieved": a, "peak": alu_peak, "unit": "TFLOP/s", "frac": a / alu_peak,
            "peak_source": f"derived: {n_sm} SMs x 128 FP32 lanes x 2 x {sm_max:.0f} MHz",
            "tensor_tflops": fm["tensor"] / t / 1e12}



def replica_layer(rank: int) -> int:
    """Input stream of a rank: every rank is an independent replica with its own seeds
    (workloads.make_qkv's `layer` argument), so N ranks do N times the work."""
    return rank


def max_over_ranks(total_ms: float, dist, device) -> float:
    """The slowest rank's device time (the job is as slow as its slowest replica)."""
    if dist is None:
        return float(total_ms)
    import torch
    t = torch.tensor([total_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(n_ranks: int, tokens_per_rank_step: int, ms_per_step: float) -> float:
    """Whole-job tokens/s: the tokens all ranks processed in a step over the slowest rank's step time."""
    return n_ranks * tokens_per_rank_step / (ms_per_step * 1e-3)


def run_ours(args):
    import torch
    from paper_2507_19608_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = load_peaks()
    props = torch.cuda.get_device_properties(local)
    n_sm = props.multi_processor_count

    w = WL.WORKLOADS[args.workload]
    theta = args.theta
    tens = WL.make_qkv(w, layer=replica_layer(rank), n_decode=0)          # each rank: an independent replica
    q, k, v = (to_dev(tens[n], w.dtype, torch) for n in ("q", "k", "v"))
    out = torch.empty_like(q)
    cfg = B.make_config(w.B, w.H, w.H_kv, w.d, w.T, w.dtype)
    st = B.delta_state_init(cfg)
    if args.kernel >= 0:
        B.delta_state_set_prefill_kernel(st, args.kernel)
    kernel = B.delta_state_prefill_kernel(st)
    flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    def step():
        B.delta_state_reset(st)
        B.delta_attn_prefill(st, q, k, v, out, w.T, w.H, w.H_kv, w.d, theta, w.window)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    # ---- timed region: K steps, device time by CUDA events, L2 flushed before each step
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = B.delta_launch_count()
    evs = []
    barrier()
    for _ in range(args.steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.delta_state_reset(st)                 # the memset a fresh sequence needs is part of the step
        B.delta_attn_prefill(st, q, k, v, out, w.T, w.H, w.H_kv, w.d, theta, w.window)
        e1.record()
        evs.append((e0, e1))
    barrier()
    launches = B.delta_launch_count() - launches0
    step_ms = [a.elapsed_time(b) for a, b in evs]
    total_ms = sum(step_ms)
    total_ms = max_over_ranks(total_ms, dist, "cuda")
    ms_per_step = total_ms / args.steps
    stats = B.delta_sparsity_stats(st)["prefill"]

    # ---- the same steps with per-kernel events (roofline of the dominant kernel)
    B.delta_state_enable_profiling(st, True)
    kms = []
    for _ in range(args.steps):
        flush.zero_()
        B.delta_state_reset(st)
        B.delta_attn_prefill(st, q, k, v, out, w.T, w.H, w.H_kv, w.d, theta, w.window)
        kms.append(B.delta_state_prefill_kernel_ms(st))
    B.delta_state_enable_profiling(st, False)
    clocks = sampler.stop() if rank == 0 else None
    kmean = [statistics.mean(x[i] for x in kms) for i in range(4)]
    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    roofline = k2_roofline(w, stats, kernel, kmean[2], peaks, n_sm)
    # K1 is a streaming pass: report it against the HBM copy bandwidth as well
    es = 2 if w.dtype == "bf16" else 4
    # chain kernel (query deltas): reads Q, writes the reference in front of every 8-row block
    k1_bytes = w.B * w.H * w.T * (w.d * es + w.d * 4 // 8)
    k1 = {"kernel": "delta_chain", "bound": "hbm", "kernel_ms": kmean[0],
          "achieved": k1_bytes / (kmean[0] * 1e-3) / 1e9, "peak": float(peaks["hbm_gbs"]), "unit": "GB/s",
          "frac": k1_bytes / (kmean[0] * 1e-3) / 1e9 / float(peaks["hbm_gbs"]),
          "note": f"{w.B * w.H * w.d} token-sequential chains of {w.T} steps: latency-bound at this size"}

    line = {
        "metric": METRIC, "value": job_value(args.gpus, w.B * w.T, ms_per_step), "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if w.dtype == "f32" else "bf16 in, f32 accumulate", "data": "synthetic",
        "config": config_dict(w, theta), "impl": "ours",
        "ms_per_step_median": statistics.median(step_ms), "ms_per_step_min": min(step_ms),
        "prefill_kernel": KERNEL_NAMES[kernel],
        "gpu_launches": int(launches),
        "kernel_ms": {"delta_chain": kmean[0], "delta_finish": kmean[1], "hybrid_attn": kmean[2]},
        "sparsity": {"S_m": stats["S_m"], "S_c_eq6": stats["S_c_eq6"], "S_c_exact": stats["S_c_exact"],
                     "paper_context": "paper: ~60% prefill, ~57% prefill+decode (key deltas, real activations, A100)"},
        "roofline": roofline, "roofline_delta_construct": k1, "clocks": clocks,
        "peaks": {k_: peaks[k_] for k_ in ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained") if k_ in peaks}
        | {"source": peaks["_source"]},
    }

    if not args.quick:
        line["kernel_variants"] = run_variants(args, B, torch, w, q, k, v, out, flush, theta, peaks, n_sm, kernel)
        line["e2e"] = run_e2e(args, B, torch, w, tens, theta)
        line["theta_sweep"] = run_sweep(args, B, torch, w, q, k, v, out, st, flush)
        line["decode"] = run_decode(args, B, torch, peaks)
        line["key_deltas"] = run_key_deltas(args, B, torch, w, tens, theta, flush, peaks)
        line["strategies"] = run_strategy_errors(B, torch, w, tens, theta)
        line["window_grid"] = run_window_grid(B, torch, flush, theta)
        line["delta_pass_large"] = run_delta_pass_large(B, torch, peaks, flush, n_sm)
        line["configs"] = {
            "single_head_fp32": run_config_leg(args, B, torch, "single_head_fp32", (0.1,), flush, peaks, n_sm),
            "bitnet_2b_prefill": run_config_leg(args, B, torch, "bitnet_2b_prefill",
                                                WL.WORKLOADS["bitnet_2b_prefill"].thetas, flush, peaks, n_sm),
            "llama32_1b_stack": run_stack_layer(args, B, torch, peaks, flush, n_sm),
        }
        d16 = line["decode"].get("batch16") or {}
        if d16.get("roofline_l2_flushed"):
            line["roofline_decode"] = {**d16["roofline_l2_flushed"], "workload": "llama32_1b_decode_b16",
                                       "us_per_step": d16["us_per_step_l2_flushed"],
                                       "us_per_step_l2_flushed_by_read": d16["us_per_step_l2_flushed_by_read"],
                                       "us_per_step_graph_l2_warm": d16["us_per_step_graph"],
                                       "algorithmic_bytes_per_step": d16["algorithmic_bytes_per_step"],
                                       "note": "L2 flushed (256 MiB write) before every step, each step timed alone by events"}
        line["cpu_baseline"] = run_cpu_baseline(args, w, tens, theta)
    print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def time_prefill(B, torch, st, q, k, v, out, w, theta, window, flush, iters, warm=2, T=None):
    """Device time of `iters` prefill steps (state reset + delta_attn_prefill, both inside the
    events; L2 flushed before each step); returns the list of milliseconds."""
    T = w.T if T is None else T
    ms = []
    for i in range(warm + iters):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.delta_state_reset(st)
        B.delta_attn_prefill(st, q, k, v, out, T, w.H, w.H_kv, w.d, theta, window)
        e1.record()
        torch.cuda.synchronize()
        if i >= warm:
            ms.append(e0.elapsed_time(e1))
    return ms


def run_variants(args, B, torch, w, q, k, v, out, flush, theta, peaks, n_sm, default_kernel):
    """The other prefill kernels on the same inputs (same step, L2 flushed): step time, the
    hybrid-attention kernel's time and its roofline."""
    res = []
    for kern in (1, 2, 0):
        if kern == default_kernel:
            continue
        cfg = B.make_config(w.B, w.H, w.H_kv, w.d, w.T, w.dtype)
        st = B.delta_state_init(cfg)
        try:
            B.delta_state_set_prefill_kernel(st, kern)
        except B.DeltaError:
            continue
        B.delta_state_enable_profiling(st, True)
        kms, steps = [], []
        for i in range(3 + min(args.steps, 10)):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            B.delta_state_reset(st)
            B.delta_attn_prefill(st, q, k, v, out, w.T, w.H, w.H_kv, w.d, theta, w.window)
            e1.record()
            torch.cuda.synchronize()
            if i >= 3:
                kms.append(B.delta_state_prefill_kernel_ms(st)); steps.append(e0.elapsed_time(e1))
        stats = B.delta_sparsity_stats(st)["prefill"]
        k2 = statistics.mean(x[2] for x in kms)
        res.append({"prefill_kernel": KERNEL_NAMES[kern], "ms_per_step": statistics.mean(steps),
                    "tokens_per_s": w.B * w.T / (statistics.mean(steps) * 1e-3),
                    "roofline": k2_roofline(w, stats, kern, k2, peaks, n_sm)})
    return res


def run_e2e(args, B, torch, w, tens, theta):
    """Same metric through delta_attn_prefill_host: pinned host buffers in, host buffer out."""
    cfg = B.make_config(w.B, w.H, w.H_kv, w.d, w.T, w.dtype)
    st = B.delta_state_init(cfg)
    staging = torch.empty(B.delta_prefill_staging_bytes(cfg, w.T), dtype=torch.uint8, device="cuda")

    def host(x):
        if w.dtype == "bf16":
            return torch.from_numpy(WL.bf16_bits(x).view(np.int16)).pin_memory()
        return torch.from_numpy(np.ascontiguousarray(x)).pin_memory()
    hq, hk, hv = host(tens["q"]), host(tens["k"]), host(tens["v"])
    ho = torch.empty_like(hq).pin_memory()
    times = []
    for i in range(3 + args.steps):
        B.delta_state_reset(st)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        B.delta_attn_prefill_host(st, hq, hk, hv, ho, staging, w.T, theta, w.window)   # synchronises
        t1 = time.perf_counter()
        if i >= 3:
            times.append(t1 - t0)
    s = statistics.mean(times)
    h2d = (hq.numel() + hk.numel() + hv.numel()) * hq.element_size()
    return {"value": w.B * w.T / s, "unit": "tokens/s", "ms_per_step": s * 1e3,
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(ho.numel() * ho.element_size()),
            "api": "delta_attn_prefill_host (pinned host buffers, wall clock around the synchronous call)"}


def run_sweep(args, B, torch, w, q, k, v, out, st, flush):
    res = []
    for th in w.thetas:
        ms = time_prefill(B, torch, st, q, k, v, out, w, th, w.window, flush, min(args.steps, 10))
        s = B.delta_sparsity_stats(st)["prefill"]
        res.append({"theta": th, "ms_per_step": statistics.mean(ms),
                    "tokens_per_s": w.B * w.T / (statistics.mean(ms) * 1e-3), "S_m": s["S_m"],
                    "S_c_exact": s["S_c_exact"]})
    return res


def run_decode(args, B, torch, peaks, source="query", names=("llama32_1b_decode_b1", "llama32_1b_decode_b16"),
               packed=False):
    """Decode leg: cache prefilled to 2048 tokens, then 256 steps; batch 1 and 16.
    source="key": the paper's adopted strategy (3) (key deltas; the carried state is the reference key)."""
    res = {}
    key = source == "key"
    for name in names:
        w = WL.WORKLOADS[name]
        theta = w.thetas[0]
        tens = WL.make_qkv(w)
        cfg = B.make_config(w.B, w.H, w.H_kv, w.d, w.T_max, w.dtype, prefill_window=B.DELTA_WIN_SLIDING,
                            source=B.DELTA_SRC_KEY if key else B.DELTA_SRC_QUERY)
        st = B.delta_state_init(cfg)
        if packed:
            B.delta_state_set_key_cache(st, True)     # decode from the compressed key-delta cache
        q = to_dev(tens["q"], w.dtype, torch)

        def cache(x):
            full = np.zeros((w.B, w.H_kv, w.T_max, w.d), np.float32)
            full[:, :, :w.T] = x
            return to_dev(full, w.dtype, torch)
        kc, vc = cache(tens["k"]), cache(tens["v"])
        out_p = torch.empty_like(q)
        qd = to_dev(np.ascontiguousarray(tens["q_dec"].transpose(2, 0, 1, 3)), w.dtype, torch)
        kd = to_dev(np.ascontiguousarray(tens["k_dec"].transpose(2, 0, 1, 3)), w.dtype, torch)
        vd = to_dev(np.ascontiguousarray(tens["v_dec"].transpose(2, 0, 1, 3)), w.dtype, torch)
        od = torch.empty_like(qd)

        def prefill():
            B.delta_state_reset(st)
            B.delta_attn_prefill(st, q, kc, vc, out_p, w.T, w.H, w.H_kv, w.d, theta, w.window)

        def steps():
            for s in range(w.n_decode):
                B.delta_attn_decode_step(st, qd[s], kd[s], vd[s], kc, vc, od[s], theta, w.window)

        eager = []
        for i in range(3):
            prefill()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); steps(); e1.record()
            torch.cuda.synchronize()
            eager.append(e0.elapsed_time(e1) * 1e3 / w.n_decode)
        od_eager = od.clone()
        dstats = B.delta_sparsity_stats(st)
        cache_bytes = None
        if packed:
            pb, db = B.delta_key_cache_bytes(st)
            cache_bytes = {"packed": pb, "dense_reference_keys": db, "ratio": pb / db}
        # the same 256 launches replayed from a CUDA graph (removes the host launch path)
        graph_us, graph_ok = None, None
        try:
            prefill()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                steps()
            reps = []
            for i in range(4):
                prefill()
                od.zero_()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); g.replay(); e1.record()
                torch.cuda.synchronize()
                reps.append(e0.elapsed_time(e1) * 1e3 / w.n_decode)
            graph_us = statistics.median(reps[1:])
            graph_ok = bool(torch.equal(od, od_eager))
        except Exception as ex:  # graph capture is an optimisation of the bench, not of the library
            graph_ok = f"capture failed: {type(ex).__name__}"
        es = 2
        n_avg = w.T + (w.n_decode - 1) / 2.0
        # K (or reference-key) and V rows once per KV head; query deltas also write the score row R
        # (and read it, where the step runs on the FP32 pipes: the tensor-core form recomputes it)
        r_passes = 0 if key else (1 if B.delta_state_decode_kernel(st) == 1 else 2)
        bytes_step = w.B * (2 * w.H_kv * n_avg * w.d * es + r_passes * w.H * n_avg * 4)
        if packed:      # values + V rows: the key side is the encoding, not dense rows
            bytes_step = w.B * w.H_kv * n_avg * w.d * es * (1.0 + cache_bytes["ratio"])
        # the same steps with L2 flushed before each one (in a model every layer's cache passes
        # through L2 between two steps of the same layer, so a step finds its cache in HBM):
        # device time of each step alone, by events
        # two ways of emptying L2: overwriting a 256 MiB buffer leaves L2 full of dirty lines, whose
        # write-back then shares HBM with the step's reads; reading the buffer leaves clean lines
        # (what a preceding weight-streaming GEMM leaves behind)
        flushed_us = flushed_read_us = None
        try:
            flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda")
            flush.zero_()
            flush64 = flush.view(torch.int64)
            sink = torch.zeros((), dtype=torch.int64, device="cuda")

            def flushed(evict):
                prefill()
                evs = []
                for s in range(min(w.n_decode, 64)):
                    evict()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    B.delta_attn_decode_step(st, qd[s], kd[s], vd[s], kc, vc, od[s], theta, w.window)
                    e1.record()
                    evs.append((e0, e1))
                torch.cuda.synchronize()
                return statistics.mean(a.elapsed_time(b) * 1e3 for a, b in evs[4:])

            flushed_us = flushed(lambda: flush.zero_())
            flushed_read_us = flushed(lambda: sink.copy_(flush64.sum()))
            del flush, flush64, sink
        except Exception as ex:
            pass
        best = graph_us if graph_us else min(eager)
        gbs = bytes_step / (best * 1e-6) / 1e9
        gbs_flushed = bytes_step / (flushed_us * 1e-6) / 1e9 if flushed_us else None
        res[f"batch{w.B}"] = {
            "us_per_step_eager": statistics.median(eager), "us_per_step_graph": graph_us,
            "us_per_step_l2_flushed": flushed_us, "us_per_step_l2_flushed_by_read": flushed_read_us,
            "graph_matches_eager": graph_ok, "steps": w.n_decode,
            "decode_kernel": ("FP32 pipes, compressed key-delta cache" if packed else
                              "tensor-core scores" if B.delta_state_decode_kernel(st) == 1 else "FP32 pipes"),
            "key_cache_bytes": cache_bytes, "cache_tokens": w.T, "theta": theta,
            "window": w.window, "algorithmic_bytes_per_step": bytes_step,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": float(peaks["hbm_gbs"]), "unit": "GB/s",
                         "frac": gbs / float(peaks["hbm_gbs"]),
                         "note": "batch 1 moves ~5 MB per step: launch latency, not bandwidth, sets the time"
                         if w.B == 1 else "the step re-reads the same cache every step and 71 MB fit the 126 MB L2: "
                         "the fraction compares with the HBM copy rate, the data comes largely from L2"},
            "roofline_l2_flushed": ({"bound": "hbm", "achieved": gbs_flushed, "peak": float(peaks["hbm_gbs"]),
                                     "unit": "GB/s", "frac": gbs_flushed / float(peaks["hbm_gbs"])}
                                    if gbs_flushed else None),
            "S_m_decode": dstats["decode"]["S_m"], "S_c_exact_decode": dstats["decode"]["S_c_exact"],
            "S_c_exact_combined": dstats["combined"]["S_c_exact"],
        }
        del st, q, kc, vc, qd, kd, vd, od
        torch.cuda.empty_cache()
    return res


def run_key_deltas(args, B, torch, w, tens, theta, flush, peaks):
    """The paper's adopted strategy (3) on the same inputs: key stream thresholded per KV head."""
    q, k, v = (to_dev(tens[n], w.dtype, torch) for n in ("q", "k", "v"))
    out = torch.empty_like(q)
    st = B.delta_state_init(B.make_config(w.B, w.H, w.H_kv, w.d, w.T, w.dtype, source=B.DELTA_SRC_KEY))
    ms = time_prefill(B, torch, st, q, k, v, out, w, theta, w.window, flush, min(args.steps, 20), warm=3)
    stt = B.delta_sparsity_stats(st)["prefill"]
    return {"prefill": {"theta": theta, "ms_per_step": statistics.mean(ms),
                        "tokens_per_s": w.B * w.T / (statistics.mean(ms) * 1e-3), "S_m": stt["S_m"],
                        "S_c_exact": stt["S_c_exact"]},
            "decode": run_decode(args, B, torch, peaks, source="key", names=("llama32_1b_decode_b16",)),
            "decode_packed_cache": run_decode(args, B, torch, peaks, source="key", names=("llama32_1b_decode_b16",),
                                              packed=True)}



def run_strategy_errors(B, torch, w, tens, theta):
    """Section III-A's three construction strategies on the same inputs: output error against
    dense attention (the library itself with a window that covers the sequence) and the delta
    sparsity each one reaches.  (1) query deltas top-down, (2) query deltas bottom-up, (3) key
    deltas; same theta and window for all three."""
    q, k, v = (to_dev(tens[n], w.dtype, torch) for n in ("q", "k", "v"))

    def run(source, window):
        st = B.delta_state_init(B.make_config(w.B, w.H, w.H_kv, w.d, w.T, w.dtype, source=source))
        out = torch.empty_like(q)
        B.delta_attn_prefill(st, q, k, v, out, w.T, w.H, w.H_kv, w.d, theta, window)
        torch.cuda.synchronize()
        return out.float(), B.delta_sparsity_stats(st)["prefill"]
    dense, _ = run(B.DELTA_SRC_QUERY, w.T)
    res = {"theta": theta, "window": w.window, "reference": "dense attention (window = T) by the same library"}
    for name, src in (("query_top_down", B.DELTA_SRC_QUERY), ("query_bottom_up", B.DELTA_SRC_QUERY_BOTTOM_UP),
                      ("key", B.DELTA_SRC_KEY)):
        out, stt = run(src, w.window)
        err = (out - dense).abs()
        res[name] = {"mean_abs_err": float(err.mean()), "max_abs_err": float(err.max()),
                     "rel_rms_err": float((err.pow(2).mean().sqrt() / dense.pow(2).mean().sqrt())),
                     # rows in the first / last quarter of the sequence: where each strategy's basis row sits
                     "mean_abs_err_first_quarter": float(err[:, :, : w.T // 4].mean()),
                     "mean_abs_err_last_quarter": float(err[:, :, -(w.T // 4):].mean()),
                     "S_m": stt["S_m"], "S_c_exact": stt["S_c_exact"]}
    return res



def run_window_grid(B, torch, flush, theta):
    """Eq. 5: the prefill window follows the input length, W = min(floor(gamma n), W_max).  One
    sequence of every length at the Llama-3.2-1B layer shape, the paper's gamma grid, and its
    decode window W_d = 4 (64 steps after the longest prefill): delta sparsity, computational
    sparsity (Eq. 6 and exact) and time per call."""
    base = WL.WORKLOADS["llama32_1b_prefill"]
    W_MAX = 256
    rows = []
    for n in (128, 256, 512, 1024, 2048, 4096):
        tens = WL.make_qkv(base, T=n, n_decode=0)
        q, k, v = (to_dev(tens[x], base.dtype, torch) for x in ("q", "k", "v"))
        out = torch.empty_like(q)
        st = B.delta_state_init(B.make_config(base.B, base.H, base.H_kv, base.d, n, base.dtype))
        for gamma in (0.02, 0.05, 0.1):
            W = B.delta_window_from_gamma(n, gamma, W_MAX)
            ms = time_prefill(B, torch, st, q, k, v, out, base, theta, W, flush, 4, T=n)
            s_ = B.delta_sparsity_stats(st)["prefill"]
            rows.append({"n": n, "gamma": gamma, "W": W, "ms": statistics.mean(ms), "S_m": s_["S_m"],
                         "S_c_eq6": s_["S_c_eq6"], "S_c_exact": s_["S_c_exact"]})
    # the same lengths as ONE ragged batch per gamma (delta_attn_prefill_varlen): every sequence
    # with its own window, Eq. 6 aggregated over the batch
    lengths = (128, 256, 512, 1024, 2048, 4096)
    seqs = [WL.make_qkv(base, layer=7 + i, T=n, n_decode=0) for i, n in enumerate(lengths)]
    T_max = max(lengths)
    st = B.delta_state_init(B.make_config(len(lengths), base.H, base.H_kv, base.d, T_max, base.dtype))
    qp = to_dev(np.concatenate([x["q"][0].reshape(-1) for x in seqs]), base.dtype, torch)
    kc = np.zeros((len(lengths), base.H_kv, T_max, base.d), np.float32)
    vc = np.zeros_like(kc)
    for b_, (x, n) in enumerate(zip(seqs, lengths)):
        kc[b_, :, :n] = x["k"][0]
        vc[b_, :, :n] = x["v"][0]
    kcd, vcd = to_dev(kc, base.dtype, torch), to_dev(vc, base.dtype, torch)
    outp = torch.empty_like(qp)
    ragged = []
    for gamma in (0.02, 0.05, 0.1):
        wins = [B.delta_window_from_gamma(n, gamma, W_MAX) for n in lengths]
        ms = []
        for i in range(5):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            B.delta_state_reset(st)
            B.delta_attn_prefill_varlen(st, qp, kcd, vcd, outp, lengths, wins, theta)
            e1.record()
            torch.cuda.synchronize()
            if i >= 2:
                ms.append(e0.elapsed_time(e1))
        s_ = B.delta_sparsity_stats(st)["prefill"]
        ragged.append({"gamma": gamma, "lengths": list(lengths), "windows": wins, "ms_per_call": statistics.mean(ms),
                       "tokens_per_s": sum(lengths) / (statistics.mean(ms) * 1e-3), "S_m": s_["S_m"],
                       "S_c_eq6": s_["S_c_eq6"], "S_c_exact": s_["S_c_exact"]})
    del st, qp, kcd, vcd, outp
    # decode with the paper's W_d = 4 behind a prefill with gamma = 0.05
    w = WL.WORKLOADS["llama32_1b_decode_b1"]
    steps = 64
    tens = WL.make_qkv(w, n_decode=steps)
    st = B.delta_state_init(B.make_config(w.B, w.H, w.H_kv, w.d, w.T + steps, w.dtype,
                                          prefill_window=B.DELTA_WIN_BLOCK))
    q = to_dev(tens["q"], w.dtype, torch)

    def cache(x):
        full = np.zeros((w.B, w.H_kv, w.T + steps, w.d), np.float32)
        full[:, :, :w.T] = x
        return to_dev(full, w.dtype, torch)
    kc, vc = cache(tens["k"]), cache(tens["v"])
    out = torch.empty_like(q)
    W = B.delta_window_from_gamma(w.T, 0.05, W_MAX)
    B.delta_attn_prefill(st, q, kc, vc, out, w.T, w.H, w.H_kv, w.d, theta, W)
    qd, kd, vd = (to_dev(np.ascontiguousarray(tens[x].transpose(2, 0, 1, 3)), w.dtype, torch)
                  for x in ("q_dec", "k_dec", "v_dec"))
    od = torch.empty_like(qd)
    for s in range(steps):
        B.delta_attn_decode_step(st, qd[s], kd[s], vd[s], kc, vc, od[s], theta, 4)
    torch.cuda.synchronize()
    st_all = B.delta_sparsity_stats(st)
    return {"theta": theta, "W_max": W_MAX, "prefill": rows, "ragged_batch": ragged,
            "prefill_plus_decode": {"n": w.T, "gamma": 0.05, "W": W, "W_d": 4, "decode_steps": steps,
                                    "S_c_exact_prefill": st_all["prefill"]["S_c_exact"],
                                    "S_c_exact_decode": st_all["decode"]["S_c_exact"],
                                    "S_c_exact_combined": st_all["combined"]["S_c_exact"],
                                    "S_c_eq6_combined": st_all["combined"]["S_c_eq6"]}}


def run_delta_pass_large(B, torch, peaks, flush, n_sm=148):
    """Delta construction at the size of one layer of the 16-layer stack configuration
    (batch 8, T = 4096: 16384 chains per mask word), where the pass is bandwidth- rather than
    latency-bound: chain and finish kernel times and their algorithmic HBM rates."""
    w = WL.WORKLOADS["llama32_1b_stack_layer"]
    theta = 0.2
    tens = WL.make_qkv(w, n_decode=0)
    q, k, v = (to_dev(tens[n], w.dtype, torch) for n in ("q", "k", "v"))
    out = torch.empty_like(q)
    st = B.delta_state_init(B.make_config(w.B, w.H, w.H_kv, w.d, w.T, w.dtype))
    B.delta_state_enable_profiling(st, True)
    kms, steps = [], []
    for i in range(5):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.delta_state_reset(st)
        B.delta_attn_prefill(st, q, k, v, out, w.T, w.H, w.H_kv, w.d, theta, w.window)
        e1.record()
        torch.cuda.synchronize()
        if i >= 2:
            kms.append(B.delta_state_prefill_kernel_ms(st)); steps.append(e0.elapsed_time(e1))
    stt = B.delta_sparsity_stats(st)["prefill"]
    n = w.B * w.H * w.T
    chain_b = n * (w.d * 2 + w.d * 4 // 8)                               # Q read, 8-row checkpoints written
    # Q and checkpoints read; delta values, mask words, indices, row counts written; K read, R written
    finish_b = n * (w.d * 2 + w.d * 4 // 8 + w.d * 4 + w.d // 8 + w.d + 2) + w.B * w.H_kv * w.T * w.d * 2 + n * 4
    hbm = float(peaks["hbm_gbs"])
    cm, fm = statistics.mean(x[0] for x in kms), statistics.mean(x[1] for x in kms)
    am = statistics.mean(x[2] for x in kms)
    N_c = w.T * (w.T + 1) // 2
    return {"workload": w.name, "theta": theta, "S_m": stt["S_m"], "ms_per_layer": statistics.mean(steps),
            "tokens_per_s": w.B * w.T / (statistics.mean(steps) * 1e-3),
            "delta_chain": {"ms": cm, "bound": "hbm", "achieved": chain_b / (cm * 1e-3) / 1e9, "peak": hbm,
                            "unit": "GB/s", "frac": chain_b / (cm * 1e-3) / 1e9 / hbm},
            "delta_finish": {"ms": fm, "bound": "hbm", "achieved": finish_b / (fm * 1e-3) / 1e9, "peak": hbm,
                             "unit": "GB/s", "frac": finish_b / (fm * 1e-3) / 1e9 / hbm},
            "hybrid_attn": k2_roofline(w, stt, B.delta_state_prefill_kernel(st), am, peaks, n_sm, sustained=True)}


def run_cpu_baseline(args, w, tens, theta):
    """The oracle, as it stands, on a bounded head sample: once with the BLAS pool pinned to one
    thread, once with the pool it gets by default on the cores this process may use."""
    heads = list(range(0, w.H, max(1, w.H // 8)))[:8]
    oracle_prefill_sample(w, tens, theta, heads[:1])     # warm-up

    def timed(budget_s):
        reps, t_used = [], 0.0
        while t_used < budget_s and len(reps) < 6:
            t = oracle_prefill_sample(w, tens, theta, heads)
            reps.append(t); t_used += t
        per_head = statistics.mean(reps) / len(heads)
        return w.B * w.T / (per_head * w.H * w.B), len(reps)
    with blas_limit(1):
        v1, n1 = timed(6.0)
    vall, nall = timed(6.0)
    pool = blas_threads()
    best, cores = (vall, pool) if vall >= v1 else (v1, 1)
    return {"value": best, "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "single_thread": {"value": v1, "cores": 1}, "all_cores": {"value": vall, "cores": pool},
            "available_cores": host_cores(),
            "sample": f"{len(heads)} of {w.H} heads x {n1}+{nall} repeats, full T={w.T}; extrapolated by head "
                      f"count; the oracle's row loops are single-threaded, only its matrix products use the BLAS pool"}


def run_config_leg(args, B, torch, name, thetas, flush, peaks, n_sm, iters=10):
    """One of the named workloads besides the headline: step time (reset + prefill, L2
    flushed), tokens/s, per-kernel times and the hybrid-attention roofline, per theta."""
    w = WL.WORKLOADS[name]
    tens = WL.make_qkv(w, n_decode=0)
    q, k, v = (to_dev(tens[n], w.dtype, torch) for n in ("q", "k", "v"))
    out = torch.empty_like(q)
    st = B.delta_state_init(B.make_config(w.B, w.H, w.H_kv, w.d, w.T, w.dtype))
    kernel = B.delta_state_prefill_kernel(st)
    rows = []
    for th in thetas:
        ms = time_prefill(B, torch, st, q, k, v, out, w, th, w.window, flush, iters)
        B.delta_state_enable_profiling(st, True)
        kms = []
        for i in range(4):
            flush.zero_()
            B.delta_state_reset(st)
            B.delta_attn_prefill(st, q, k, v, out, w.T, w.H, w.H_kv, w.d, th, w.window)
            if i >= 1:
                kms.append(B.delta_state_prefill_kernel_ms(st))
        B.delta_state_enable_profiling(st, False)
        stt = B.delta_sparsity_stats(st)["prefill"]
        km = [statistics.mean(x[i] for x in kms) for i in range(3)]
        rows.append({"theta": th, "ms_per_step": statistics.mean(ms), "ms_per_step_min": min(ms),
                     "tokens_per_s": w.B * w.T / (statistics.mean(ms) * 1e-3), "S_m": stt["S_m"],
                     "S_c_exact": stt["S_c_exact"],
                     "kernel_ms": {"delta_chain": km[0], "delta_finish": km[1], "hybrid_attn": km[2]},
                     "roofline": k2_roofline(w, stt, kernel, km[2], peaks, n_sm)})
    return {"workload": name, "config": config_dict(w, list(thetas)), "prefill_kernel": KERNEL_NAMES[kernel], "runs": rows}


def run_stack_layer(args, B, torch, peaks, flush, n_sm):
    """One layer of the 16-layer stack configuration (batch 8, T = 4096, window 256): prefill at
    each theta of the sweep, then the 128 decode steps (n = 4096 .. 4223) with L2 flushed before
    every step.  The layers are independent draws of the same shape, so the 16-layer figures are
    16 x one layer."""
    w = WL.WORKLOADS["llama32_1b_stack_layer"]
    tens = WL.make_qkv(w)
    cfg = B.make_config(w.B, w.H, w.H_kv, w.d, w.T_max, w.dtype)
    st = B.delta_state_init(cfg)
    q = to_dev(tens["q"], w.dtype, torch)

    def cache(x):
        full = np.zeros((w.B, w.H_kv, w.T_max, w.d), np.float32)
        full[:, :, :w.T] = x
        return to_dev(full, w.dtype, torch)
    kc, vc = cache(tens["k"]), cache(tens["v"])
    out = torch.empty_like(q)
    kernel = B.delta_state_prefill_kernel(st)
    pre = []
    for th in w.thetas:
        ms = time_prefill(B, torch, st, q, kc, vc, out, w, th, w.window, flush, 3, warm=1)
        B.delta_state_enable_profiling(st, True)
        flush.zero_()
        B.delta_state_reset(st)
        B.delta_attn_prefill(st, q, kc, vc, out, w.T, w.H, w.H_kv, w.d, th, w.window)
        km = B.delta_state_prefill_kernel_ms(st)
        B.delta_state_enable_profiling(st, False)
        stt = B.delta_sparsity_stats(st)["prefill"]
        pre.append({"theta": th, "ms_per_layer": statistics.mean(ms), "ms_16_layers": 16 * statistics.mean(ms),
                    "tokens_per_s": w.B * w.T / (statistics.mean(ms) * 1e-3), "S_m": stt["S_m"],
                    "S_c_exact": stt["S_c_exact"],
                    "kernel_ms": {"delta_chain": km[0], "delta_finish": km[1], "hybrid_attn": km[2]},
                    "roofline": k2_roofline(w, stt, kernel, km[2], peaks, n_sm, sustained=True)})
    # decode: the state the last prefill left (theta = the sweep's last value), 128 steps
    theta = w.thetas[-1]
    qd, kd, vd = (to_dev(np.ascontiguousarray(tens[x].transpose(2, 0, 1, 3)), w.dtype, torch)
                  for x in ("q_dec", "k_dec", "v_dec"))
    od = torch.empty_like(qd)
    evs = []
    for s_ in range(w.n_decode):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.delta_attn_decode_step(st, qd[s_], kd[s_], vd[s_], kc, vc, od[s_], theta, w.window)
        e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    us = [a.elapsed_time(b) * 1e3 for a, b in evs[4:]]
    n_avg = w.T + (w.n_decode - 1) / 2.0
    r_passes = 1 if B.delta_state_decode_kernel(st) == 1 else 2
    bytes_step = w.B * (2 * w.H_kv * n_avg * w.d * 2 + r_passes * w.H * n_avg * 4)
    gbs = bytes_step / (statistics.mean(us) * 1e-6) / 1e9
    dec = {"theta": theta, "steps": w.n_decode, "us_per_step_l2_flushed": statistics.mean(us),
           "us_per_step_16_layers": 16 * statistics.mean(us), "algorithmic_bytes_per_step": bytes_step,
           "roofline": {"bound": "hbm", "achieved": gbs, "peak": float(peaks["hbm_gbs"]), "unit": "GB/s",
                        "frac": gbs / float(peaks["hbm_gbs"])},
           "S_c_exact_combined": B.delta_sparsity_stats(st)["combined"]["S_c_exact"]}
    return {"workload": w.name, "config": config_dict(w, list(w.thetas)), "layers": 16,
            "note": "one layer measured; layers are independent draws of one shape: 16-layer figures = 16 x one layer",
            "prefill": pre, "decode": dec}


def run_only(args):
    """One secondary leg alone: the decode leg at one batch size, or one prefill of the stack-layer shape."""
    import torch
    from paper_2507_19608_b200 import binding as B
    torch.cuda.set_device(0)
    peaks = load_peaks()
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    if args.only in ("stack", "bitnet"):
        flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda")
        res = (run_stack_layer(args, B, torch, peaks, flush, n_sm) if args.only == "stack" else
               run_config_leg(args, B, torch, "bitnet_2b_prefill", WL.WORKLOADS["bitnet_2b_prefill"].thetas, flush,
                              peaks, n_sm))
    elif args.only == "stack_layer":
        flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda")
        res = run_delta_pass_large(B, torch, peaks, flush, torch.cuda.get_device_properties(0).multi_processor_count)
    else:
        res = run_decode(args, B, torch, peaks, names=("llama32_1b_" + args.only,))
    print(json.dumps({"only": args.only, "result": res}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama32_1b_prefill")
    ap.add_argument("--theta", type=float, default=HEADLINE_THETA)
    ap.add_argument("--kernel", type=int, default=-1, help="-1 auto, 0 generic, 1 tcgen05 + FP32 delta path, 2 tcgen05 telescoped")
    ap.add_argument("--quick", action="store_true", help="prefill timing only (used for ncu launch lists)")
    ap.add_argument("--only", default="", choices=["", "decode_b1", "decode_b16", "stack_layer", "stack", "bitnet"],
                    help="run one secondary leg alone on one GPU (small ncu captures of its kernels)")
    ap.add_argument("--ref-heads", type=int, default=4, help="heads per reference step")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.only:
        run_only(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
