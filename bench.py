#!/usr/bin/env python
"""Benchmark of the SEA attention layer (estimate -> top-k mask -> sparse attention) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one sea_attention call (all stages) over one synthetic batch of the workload's shape.
The default workload is the OPT-1.3B-shaped causal bf16 configuration, on which the headline
metric is quoted.  One JSON line is printed by rank 0.

  value      tokens/s (B*T per step, all ranks) with inputs resident in HBM: mean of K per-step CUDA
             event pairs, L2 flushed between steps, max over ranks; `ms_stats` adds median and min.
  e2e        the same through sea_attention_host: pinned host Q, K, V, omega, W_dec in, O out.
  clocks     nvidia-smi samples taken while the K timed steps and an untimed continuation of the
             same steps run (the K steps alone last a few milliseconds, less than one sample).
  stages_ms  per-stage milliseconds from a second pass that calls the three stage entry points
             with events between them (same kernels as the fused call).
  roofline   the sparse-attention kernel, against the resource that binds the kernel that ran.  The
             tile kernel forms the masked products as dense tiles on the tensor cores: achieved =
             the FLOPs it executes / its time, peak = the measured dense bf16 rate.  The per-row
             kernels gather: achieved = Q + O + every row's gathered K/V bytes / time against the
             measured HBM copy bandwidth.  `gather_model` always gives that byte figure (the
             benchmark definition's) without calling it a fraction of anything when the kernel
             gathers nothing; `bounds_ms` lists the time each resource alone would need.
  roofline_estimate, roofline_mask
             the other two stages against HBM: their compulsory bytes / stage time.
  lean       the fused call asked for O and the CSR mask only (the estimate and the probabilities are
             never written out); per-rank, not part of `value`.
  grouped, causal_aware
             the same step with the causal-per-batch grouping (sea_attention_grouped) and with the
             causal-aware per-query selection (sea_attention_causal_aware) on this rank, and their
             selection and sparse stages; per-rank, not part of `value`.
  structured_mask
             the mask and sparse stages when the caller gives a banded estimate (the structure of
             trained SEA masks): the tile kernel skips the key tiles nothing was selected in.
  decoder_head  the layer with the paper's estimator head (MLPs + three-layer CNN, random-init
             weights) and output mixing through sea_attention_decoder, MLPs and convolutions on
             tcgen05 (timed by default up to T = 2048; longer shapes with --decoder).
  cpu_baseline  the fp64 oracle on a bounded sample of heads, one head per host core at a time.

With N > 1 (torchrun) every rank runs an independent replica of the workload (the path has no
exchange step between GPUs); value sums the ranks' tokens over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "SEA attention-layer tokens/s on 1 B200 (all stages)"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
SM_COUNT = 148
XU_PER_CLK_PER_SM = 16  # ex2 results per clock and SM
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_traffic.json")
KERNEL_SOURCES = {
    "sparse_attn_tiles_tc_kernel": "sea_sparse_tc.cu",
    "sparse_attn_blocks_tma_kernel": "sea_sparse_tma.cu",
    "sparse_attn_rows_mma_kernel": "sea_sparse.cu",
    "sparse_attn_rows_kernel": "sea_sparse.cu",
}


def measured_peaks():
    """(HBM GB/s, dense bf16 TFLOP/s for a kernel timed alone, 'measured' | 'fallback')."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            j = json.load(f)
        return float(j["hbm_gbs"]), float(j["bf16_tflops"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


def ncu_traffic(workload: str, kernel: str):
    """DRAM bytes of one launch of `kernel` on `workload` from the tracked ncu record, or None when
    there is none or the kernel's source file has changed since the capture."""
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f).get(workload, {}).get(kernel)
        if rec is None:
            return None
        src = os.path.join(ROOT, "paper_2310_01777_b200", "csrc", KERNEL_SOURCES[kernel])
        with open(src, "rb") as f:
            if hashlib.sha256(f.read()).hexdigest() != rec["source_sha256"]:
                return None
        return float(rec["dram_bytes_read"]) + float(rec["dram_bytes_write"])
    except Exception:
        return None


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_uuid: str):
        self.rows = []
        self.proc = None
        self.uuid = gpu_uuid

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for row in self.rows:
            parts = [p.strip() for p in row.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_min_mhz": sm[0], "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


# ---- the CPU oracle, timed ---------------------------------------------------------------------
def _oracle_heads(job):
    """Worker: the fp64 oracle, as it stands, on heads [lo, hi) of the workload; returns seconds."""
    name, lo, hi = job
    import numpy as np
    import torch
    from threadpoolctl import threadpool_limits

    from oracle import sea_oracle as orc
    from paper_2310_01777_b200.inputs import WORKLOADS, make_inputs

    w = WORKLOADS[name]
    torch.set_num_threads(1)
    small = w.scaled(B=1, H=hi)
    host = make_inputs(small)
    f64 = lambda t: t.to(dtype=torch.float64).numpy()
    given = "A_hat" in host  # workloads without an estimator stage bring the estimate along
    om, wd = (None, None) if given else (f64(host["omega"]), f64(host["W_dec"]))
    scale = 1.0 / np.sqrt(w.d)
    with threadpool_limits(limits=1):
        t0 = time.perf_counter()
        for h in range(lo, hi):
            orc.sea_attention_head(f64(host["Q"][0, h]), f64(host["K"][0, h]), f64(host["V"][0, h]), w.k_hat,
                                   w.Kc, w.causal, scale, A_hat=f64(host["A_hat"][0, h]) if given else None,
                                   omega=om, W_dec=wd)
        return time.perf_counter() - t0


def oracle_tokens_per_s(w, n_heads: int, cores: int):
    """Oracle throughput on the first n_heads (b, h) units, the heads dealt out to `cores` worker
    processes (each one runs the unchanged single-threaded oracle).  Returns (tokens/s, seconds,
    workers used).  Must run before this process initialises CUDA (the workers are forked)."""
    import multiprocessing as mp

    cores = max(1, min(cores, n_heads))
    per = (n_heads + cores - 1) // cores
    jobs = [(w.name, lo, min(lo + per, n_heads)) for lo in range(0, n_heads, per)]
    if len(jobs) == 1:
        secs = [_oracle_heads(jobs[0])]
    else:
        with mp.get_context("fork").Pool(len(jobs)) as pool:
            secs = pool.map(_oracle_heads, jobs)
    wall = max(secs)  # the workers run side by side; input generation is not part of the oracle
    tokens = n_heads * w.T / w.H  # a token passes through all H heads of the layer
    return tokens / wall, wall, len(jobs)


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def cpu_baseline(w, n_heads: int, max_cores: int):
    cores = min(host_cores(), max_cores)
    v, dt, used = oracle_tokens_per_s(w, n_heads, cores)
    return {"value": v, "unit": "tokens/s", "cores": used, "kind": "oracle",
            "sample": f"first {n_heads} of {w.B * w.H} heads of {w.name}, fp64 numpy oracle, {dt:.1f} s wall, "
                      f"{used} worker processes of one thread each"}


def run_reference(args, w):
    """The base contract's reference arm: the CPU oracle on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_heads = args.ref_heads
    cores = min(host_cores(), args.cpu_cores, n_heads)
    for _ in range(args.warmup):
        oracle_tokens_per_s(w, 1, 1)
    times, used = [], 1
    for _ in range(args.steps):
        _, dt, used = oracle_tokens_per_s(w, n_heads, cores)
        times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = (n_heads * w.T / w.H) / (ms / 1e3)
    sample = (f"{n_heads} of {w.B * w.H} heads of {w.name} per step, fp64 numpy oracle, {used} worker processes of "
              "one thread each")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": used, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of timings over all ranks: the job is as slow as its slowest
    replica.  Without a process group (one GPU) the values come back unchanged."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def workload_config(w):
    return {"workload": f"{w.name}: B={w.B} H={w.H} T={w.T} d={w.d} m={w.m} Kc={w.Kc} k_hat={w.k_hat} "
                        f"causal={int(w.causal)} io={w.dtype}",
            "io_dtype": w.dtype, "accumulate": "f32", "l2": "flushed between steps (256 MiB write)",
            "outputs": "O, A_hat, sel, row_ptr, col_idx and P all materialised"}


def ms_stats(ms):
    return {"mean": sum(ms) / len(ms), "median": statistics.median(ms), "min": min(ms), "n": len(ms)}


def sparse_roofline(w, kernel, exec_flops, nnz, sparse_ms, peaks, clocks):
    """Roofline block of the sparse-attention stage (see the module docstring)."""
    hbm_peak, tc_peak, kind = peaks
    elem = 2 if w.dtype == "bf16" else 4
    t = sparse_ms / 1e3
    gather_bytes = 2 * w.rows * w.d * elem + 2 * nnz * w.d * elem  # Q + O + every row's gathered K and V
    useful_flops = 4 * nnz * w.d
    # bytes that must cross HBM whatever the kernel: Q, K, V in, O and P out, sel and row_ptr in
    compulsory = 4 * w.rows * w.d * elem + nnz * elem + w.rows * w.k_hat * 4 + (w.rows + 1) * 4
    block = {"kernel": kernel, "ms": sparse_ms, "useful_flops": useful_flops,
             "sparse_stage_tokens_per_s": w.B * w.T / t,
             "gather_model": {"algorithmic_gather_bytes": gather_bytes, "gbs": gather_bytes / t / 1e9,
                              "frac_of_gather_model": gather_bytes / t / 1e9 / hbm_peak,
                              "note": "Q + O + gathered K/V of every row over the HBM copy bandwidth; the tile kernel "
                                      "gathers nothing, so this is not a fraction of a resource it uses"},
             "compulsory_hbm_bytes": compulsory, "compulsory_hbm_gbs": compulsory / t / 1e9,
             "traffic": ncu_traffic(w.name, kernel),
             "traffic_source": "profiles/ncu_traffic.json (one ncu capture; null when the kernel's source changed since)"}
    bounds = {"hbm_compulsory": compulsory / (hbm_peak * 1e9) * 1e3}
    if kernel == "sparse_attn_tiles_tc_kernel" and exec_flops:
        mhz = (clocks or {}).get("sm_mhz") or 1965.0
        nq = w.T // 128
        n_ex2 = w.B * w.H * (nq * (nq + 1) // 2 if w.causal else nq * nq) * 128 * 128  # one per entry of every score tile
        bounds["tensor"] = exec_flops / (tc_peak * 1e12) * 1e3
        bounds["xu_ex2"] = n_ex2 / (XU_PER_CLK_PER_SM * SM_COUNT * mhz * 1e6) * 1e3
        achieved = exec_flops / t / 1e12
        block.update({"bound": "tensor", "achieved": achieved, "peak": tc_peak, "unit": "TFLOP/s",
                      "frac": achieved / tc_peak, "peak_source": f"{kind} dense bf16 (burst)",
                      "executed_flops": exec_flops, "useful_over_executed": useful_flops / exec_flops})
    else:
        achieved = gather_bytes / t / 1e9
        block.update({"bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                      "frac": achieved / hbm_peak, "peak_source": f"{kind} HBM copy bandwidth",
                      "note": "K and V of a head stay in L2 between the rows that gather them, so the gathered bytes "
                              "mostly never cross HBM and this figure can exceed 1"})
    block["bounds_ms"] = bounds
    block["frac_of_tightest_bound"] = max(bounds.values()) / sparse_ms
    return block


def hbm_roofline(kernels, nbytes, ms, peaks, what):
    hbm_peak, _, kind = peaks
    achieved = nbytes / (ms / 1e3) / 1e9
    return {"kernels": kernels, "bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
            "frac": achieved / hbm_peak, "peak_source": f"{kind} HBM copy bandwidth", "algorithmic_bytes": nbytes,
            "ms": ms, "bytes": what}


# Latencies the paper reports for its own implementation on one RTX 2080 Ti (App. Tables A.1 / A.2:
# bidirectional, K = 128, random inputs; batch and head counts not stated): context, not a target.
PAPER_SWEEP_MS = {32: {4096: 1.45, 8192: 3.07, 16384: 6.21, 32768: 12.00, 65536: 25.74, 131072: 50.89},
                  64: {4096: 1.77, 8192: 3.69, 16384: 7.40, 32768: 13.46, 65536: 28.74, 131072: 56.46},
                  128: {4096: 2.39, 8192: 4.89, 16384: 9.81, 32768: 16.49, 65536: 37.94, 131072: 72.59}}


def run_capped_sweep(args):
    """The paper's long-sequence setting with a fixed compressed width: K = 128, k in {32, 64, 128},
    T = 4096 .. 131072, not causal; k_hat = max(1, round(k K / T)) and every selected column keeps
    k* = min(k, ceil(T / K)) uniformly spaced keys (sea_attention_capped).  One JSON line."""
    import torch

    import paper_2310_01777_b200 as sea
    from paper_2310_01777_b200.inputs import Workload, make_inputs

    dev = torch.device("cuda", 0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    rows_out = []
    for k in (32, 64, 128):
        for T in (4096, 8192, 16384, 32768, 65536, 131072):
            Kc = 128
            k_hat = max(1, round(k * Kc / T))  # Sec. 3.1; Python rounds halves to even
            k_star = min(k, -(-T // Kc))
            w = Workload(f"sweep_T{T}_k{k}", args.sweep_B, args.sweep_H, T, 64, 128, Kc, k_hat, False, "bf16", 0)
            host = make_inputs(w)
            d = {n: v.to(dev) for n, v in host.items()}
            shape = sea.make_shape(w)
            ws = torch.empty(sea.sea_workspace_bytes_capped(shape, k_star), dtype=torch.uint8, device=dev)
            ws[:256].zero_()
            cap = w.rows * k_hat * min(k_star, T // Kc)
            O = torch.empty_like(d["Q"])
            col = torch.empty((cap,), dtype=torch.int32, device=dev)
            P = torch.empty((cap,), dtype=torch.bfloat16, device=dev)
            rp = torch.empty((w.rows + 1,), dtype=torch.int32, device=dev)

            def step():
                sea.sea_attention_capped(shape, k_star, d["Q"], d["K"], d["V"], d["omega"], d["W_dec"], O, ws, col,
                                         row_ptr=rp, P=P)

            for _ in range(3):
                step()
            torch.cuda.synchronize(dev)
            ms = []
            for _ in range(args.steps if args.steps <= 10 else 10):
                flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); step(); b.record()
                torch.cuda.synchronize(dev)
                ms.append(a.elapsed_time(b))
            if sea.sea_device_status(ws) != 0:
                raise SystemExit("device status word set in the capped sweep")
            rows_out.append({"T": T, "k": k, "k_hat": k_hat, "k_star": k_star, "nnz": int(rp[-1]), "ms": ms_stats(ms),
                             "tokens_per_s": w.B * T / (statistics.median(ms) / 1e3), "paper_2080ti_ms": PAPER_SWEEP_MS[k][T]})
            del d, ws, O, col, P, rp
            torch.cuda.empty_cache()
    print(json.dumps({"metric": "SEA attention latency on the paper's long-sequence sweep (all stages, with P)",
                      "unit": "ms", "config": {"workload": f"B={args.sweep_B} H={args.sweep_H} d=64 m=128 K=128 not causal bf16, "
                                                           "capped replication (App. Sparse Interpolation)",
                                               "l2": "flushed between steps (256 MiB write)"},
                      "note": "paper_2080ti_ms: the paper's own figures on its hardware, batch and heads unstated; context only",
                      "sweep": rows_out}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="opt_1p3b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-heads", type=int, default=16, help="heads per step of the reference arm")
    ap.add_argument("--cpu-heads", type=int, default=64, help="heads in the cpu_baseline sample")
    ap.add_argument("--cpu-cores", type=int, default=32, help="most worker processes the oracle is dealt out to")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-modes", action="store_true", help="skip the grouped / causal-aware / lean regions")
    ap.add_argument("--soak-s", type=float, default=1.2, help="seconds of steps the clock sampler watches")
    ap.add_argument("--decoder", action="store_true",
                    help="time the paper's MLP + CNN estimator head (a few ms per step) even with --no-modes; without "
                         "--no-modes it is timed anyway on the workloads of up to 2048 tokens per sequence")
    ap.add_argument("--no-decoder", action="store_true", help="skip the estimator-head region")
    ap.add_argument("--capped-sweep", action="store_true", help="time the paper's long-sequence sweep shape instead")
    ap.add_argument("--sweep-B", type=int, default=1)
    ap.add_argument("--sweep-H", type=int, default=12)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2310_01777_b200.inputs import WORKLOADS, make_inputs, torch_dtype

    w = WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return

    if args.capped_sweep:
        run_capped_sweep(args)
        return

    if w.m == 0:
        raise SystemExit(f"bench.py times workloads that start at the estimator; {w.name} is a parity-test case")

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    # the oracle's worker processes are forked, which has to happen before CUDA is initialised
    cpu_line = None
    if rank == 0 and not args.no_cpu_baseline:
        cpu_line = cpu_baseline(w, min(args.cpu_heads, w.B * w.H), args.cpu_cores)

    import torch
    import torch.distributed as dist

    import paper_2310_01777_b200 as sea

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libsea has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    sea.binding.load_library()

    def barrier():
        if world > 1:
            dist.barrier()

    host = make_inputs(w.scaled(seed=w.seed + rank))
    d = {k: v.to(dev) for k, v in host.items()}
    shape = sea.make_shape(w)
    io = torch_dtype(w.dtype)
    ws = sea.new_workspace(shape, dev, host_staging=True)
    O = torch.empty((w.B, w.H, w.T, w.d), dtype=io, device=dev)
    A_hat = torch.empty((w.B, w.H, w.T, w.Kc), dtype=torch.float32, device=dev)
    sel = torch.empty((w.rows, w.k_hat), dtype=torch.int32, device=dev)
    row_ptr = torch.empty((w.rows + 1,), dtype=torch.int32, device=dev)
    col_idx = torch.empty((w.nnz_cap,), dtype=torch.int32, device=dev)
    P = torch.empty((w.nnz_cap,), dtype=io, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def timed(fn, steps):
        """Per-step milliseconds of `steps` calls of fn, each bracketed by its own event pair on the
        launching stream, the L2 flushed before each."""
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in ev:
            flush.zero_()
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize(dev)
        return [a.elapsed_time(b) for a, b in ev]

    def step():
        sea.sea_attention(shape, d["Q"], d["K"], d["V"], d["omega"], d["W_dec"], O, ws, A_hat=A_hat, sel=sel,
                          row_ptr=row_ptr, col_idx=col_idx, P=P)

    for _ in range(args.warmup):
        flush.zero_()
        step()
    torch.cuda.synchronize(dev)
    launches_per_step = sea.sea_last_launch_count()
    if sea.sea_device_status(ws) != 0:
        raise SystemExit("device status word set during warm-up")

    sampler = ClockSampler(_gpu_index(local_rank))
    # ---- timed region 1: the fused call ------------------------------------------------
    barrier()
    torch.cuda.synchronize(dev)
    if rank == 0:
        sampler.start()
    step_ms = timed(step, args.steps)
    barrier()
    # The K steps above are the measurement.  They last milliseconds, less than one nvidia-smi sample,
    # so the same steps go on untimed until the sampler has seen the GPU under this load for a while.
    soak_steps = 0
    if rank == 0:
        t_end = time.perf_counter() + 8.0
        t_soak = time.perf_counter() + args.soak_s
        while (time.perf_counter() < t_soak or len(sampler.rows) < 12) and time.perf_counter() < t_end:
            for _ in range(50):
                flush.zero_()
                step()
            torch.cuda.synchronize(dev)
            soak_steps += 50
    clocks = sampler.stop() if rank == 0 else None
    if clocks is not None:
        clocks["watched"] = f"the {args.steps} timed steps and {soak_steps} more untimed ones of the same call"
    barrier()

    # ---- timed region 2: stage by stage (for the rooflines) ----------------------------
    for _ in range(2):  # the stage entry points launch kernels the fused call does not: load them first
        sea.sea_estimate(shape, d["Q"], d["K"], d["V"], d["omega"], d["W_dec"], A_hat, ws)
        sea.sea_topk_mask(shape, A_hat, sel, row_ptr, col_idx, ws)
        sea.sea_sparse_attn(shape, d["Q"], d["K"], d["V"], row_ptr, col_idx, sel, O, P, ws)
    torch.cuda.synchronize(dev)
    sparse_kernel = sea.sea_last_sparse_kernel()
    sparse_flops = sea.sea_last_sparse_flops()
    sparse_launches = sea.sea_last_launch_count()
    sev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    for e in sev:
        flush.zero_()
        e[0].record()
        sea.sea_estimate(shape, d["Q"], d["K"], d["V"], d["omega"], d["W_dec"], A_hat, ws)
        e[1].record()
        sea.sea_topk_mask(shape, A_hat, sel, row_ptr, col_idx, ws)
        e[2].record()
        sea.sea_sparse_attn(shape, d["Q"], d["K"], d["V"], row_ptr, col_idx, sel, O, P, ws)
        e[3].record()
    torch.cuda.synchronize(dev)
    stage_all = [[e[i].elapsed_time(e[i + 1]) for e in sev] for i in range(3)]
    stage_ms = [sum(x) / len(x) for x in stage_all]
    nnz = int(row_ptr[-1])

    # ---- timed region 3: end to end from pinned host memory ---------------------------
    hp = {k: v.pin_memory() for k, v in host.items()}
    hO = torch.empty((w.B, w.H, w.T, w.d), dtype=io).pin_memory()
    e2e_steps = max(3, min(args.steps, 20))

    def host_step():
        sea.sea_attention_host(shape, hp["Q"], hp["K"], hp["V"], hp["omega"], hp["W_dec"], hO, ws)

    for _ in range(2):
        host_step()
    barrier()
    torch.cuda.synchronize(dev)
    e2e_all = timed(host_step, e2e_steps)
    barrier()
    e2e_ms = sum(e2e_all) / e2e_steps
    if not torch.equal(hO, O.cpu()):
        raise SystemExit("host entry point and device entry point disagree")

    lean = grouped = causal_aware = None
    if not args.no_modes:
        # ---- timed region 3b: the fused call with the required outputs only (O and the CSR mask) ------
        O_lean = torch.empty_like(O)
        rp_lean = torch.empty_like(row_ptr)

        def lean_step():
            sea.sea_attention(shape, d["Q"], d["K"], d["V"], d["omega"], d["W_dec"], O_lean, ws, row_ptr=rp_lean,
                              col_idx=col_idx)

        for _ in range(3):
            flush.zero_()
            lean_step()
        lean_launches = sea.sea_last_launch_count()
        torch.cuda.synchronize(dev)
        lean_all = timed(lean_step, args.steps)
        lean_ms = sum(lean_all) / args.steps
        if not (torch.equal(O_lean, O) and torch.equal(rp_lean, row_ptr)):
            raise SystemExit("the call without the optional outputs gives a different O or row_ptr")
        lean = {"outputs": "O, row_ptr and col_idx only (no A_hat, sel, P)", "ms_per_step": lean_ms,
                "ms_stats": ms_stats(lean_all), "value": w.B * w.T / (lean_ms / 1e3), "unit": "tokens/s",
                "gpu_launches_per_step": lean_launches}

        # ---- timed region 4: the selections that leave as bit masks (fused call, then the stages) ----
        def time_bits_mode(label, fused_fn, topk_fn):
            bits = torch.empty((w.rows, (w.Kc + 31) // 32), dtype=torch.int32, device=dev)

            def gstep():
                fused_fn(shape, d["Q"], d["K"], d["V"], d["omega"], d["W_dec"], O, ws, A_hat=A_hat, mask_bits=bits,
                         row_ptr=row_ptr, col_idx=col_idx, P=P)

            for _ in range(3):
                flush.zero_()
                gstep()
            g_launches = sea.sea_last_launch_count()
            torch.cuda.synchronize(dev)
            g_all = timed(gstep, args.steps)
            g_ms = sum(g_all) / args.steps
            for _ in range(2):
                topk_fn(shape, A_hat, bits, row_ptr, col_idx, ws)
                sea.sea_sparse_attn_masked(shape, d["Q"], d["K"], d["V"], row_ptr, col_idx, bits, O, P, ws)
            torch.cuda.synchronize(dev)
            gsev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
            for e in gsev:
                flush.zero_()
                e[0].record()
                topk_fn(shape, A_hat, bits, row_ptr, col_idx, ws)
                e[1].record()
                sea.sea_sparse_attn_masked(shape, d["Q"], d["K"], d["V"], row_ptr, col_idx, bits, O, P, ws)
                e[2].record()
            torch.cuda.synchronize(dev)
            if sea.sea_device_status(ws) != 0:
                raise SystemExit(f"device status word set by the {label} path")
            return {"selection": label, "ms_per_step": g_ms, "ms_stats": ms_stats(g_all),
                    "value": w.B * w.T / (g_ms / 1e3), "unit": "tokens/s", "gpu_launches_per_step": g_launches,
                    "stages_ms": {"topk_mask": sum(e[0].elapsed_time(e[1]) for e in gsev) / args.steps,
                                  "sparse_attn_masked": sum(e[1].elapsed_time(e[2]) for e in gsev) / args.steps},
                    "nnz": int(row_ptr[-1])}

        if w.Kc % 4 == 0 and w.H * ((w.Kc + 31) // 32 + 1) <= 12288:
            grouped = time_bits_mode("causal-per-batch", sea.sea_attention_grouped, sea.sea_topk_mask_grouped)
        if w.causal:
            causal_aware = time_bits_mode("causal-aware per-query", sea.sea_attention_causal_aware,
                                          sea.sea_topk_mask_causal_aware)

    structured = None
    if not args.no_modes:
        # ---- timed region 5: a structured (banded + sink column) estimate given by the caller -------
        # Trained SEA masks are banded; the random decoder's are not.  The mask and sparse stages on such a
        # mask, by the tile kernel (which leaves out the key tiles no row of a query tile selected) and by
        # the per-row kernels.
        from paper_2310_01777_b200.inputs import banded_estimate

        A_band = banded_estimate(w).to(dev)

        def band_step():
            sea.sea_attention(shape, d["Q"], d["K"], d["V"], None, None, O, ws, A_hat_in=A_band, sel=sel, row_ptr=row_ptr,
                              col_idx=col_idx, P=P)

        for _ in range(3):
            flush.zero_()
            band_step()
        torch.cuda.synchronize(dev)
        band_all = timed(band_step, args.steps)
        band_kernel = sea.sea_last_sparse_kernel()
        band_nnz = int(row_ptr[-1])
        tile_all = timed(lambda: sea.sea_sparse_attn(shape, d["Q"], d["K"], d["V"], row_ptr, col_idx, sel, O, P, ws), args.steps)
        rows_all = timed(lambda: sea.sea_sparse_attn(shape, d["Q"], d["K"], d["V"], row_ptr, col_idx, sel, O, P, ws[:256]),
                         args.steps)
        rows_kernel = sea.sea_last_sparse_kernel()
        structured = {"estimate": "given: band of about 2 compressed columns around the diagonal plus column 0, noise 0.05",
                      "mask_and_sparse_ms": ms_stats(band_all), "nnz": band_nnz,
                      "sparse_attn_ms": {band_kernel: ms_stats(tile_all), rows_kernel: ms_stats(rows_all)}}
        step()  # the outputs of the benchmark workload again, for what follows
        torch.cuda.synchronize(dev)

    decoder = None
    # the estimator head's buffers grow with T * Kc per head and channel: the long-context shapes only on request
    if (args.decoder or (not args.no_modes and w.T <= 2048)) and not args.no_decoder:
        # ---- timed region 6: the paper's estimator head (MLPs + three-layer CNN) with random-init weights ----
        from paper_2310_01777_b200.inputs import make_decoder_params

        d_hidden, c_s, c_h = 64, 2, 4
        dp = {k: v.to(dev) for k, v in make_decoder_params(w, d_hidden, c_s, c_h).items()}
        dec = sea.make_decoder(dp, d_hidden, c_s, c_h, w.causal)
        dws = torch.empty(sea.sea_workspace_bytes_decoder(shape, dec), dtype=torch.uint8, device=dev)
        dws[:256].zero_()
        Zb = torch.empty((w.B, w.H, w.T, d_hidden), dtype=torch.float32, device=dev)

        def dstep():
            sea.sea_attention_decoder(shape, dec, d["Q"], d["K"], d["V"], d["omega"], O, dws, A_hat=A_hat, sel=sel,
                                      row_ptr=row_ptr, col_idx=col_idx, P=P)

        for _ in range(2):
            dstep()
        d_launches = sea.sea_last_launch_count()
        torch.cuda.synchronize(dev)
        n_d = max(3, min(args.steps, 5))
        d_all = timed(dstep, n_d)
        e_all = timed(lambda: sea.sea_estimate_decoder(shape, dec, d["Q"], d["K"], d["V"], d["omega"], A_hat, Zb, dws), n_d)
        C = w.H * c_h
        conv_flops = 2 * 9 * w.B * (2 * C * C * w.T * (w.Kc // c_s) // (1 if w.causal else c_s) + C * w.H * w.T * w.Kc)
        if not w.causal:  # the second layer also runs at the reduced height; the first writes it
            conv_flops = 2 * 9 * w.B * (2 * C * C * (w.T // c_s) * (w.Kc // c_s) + C * w.H * w.T * w.Kc)
        if sea.sea_device_status(dws) != 0:
            raise SystemExit("device status word set by the decoder path")
        d_ms = sum(d_all) / n_d
        decoder = {"head": f"d_hidden={d_hidden} c_s={c_s} c_h={c_h}: V_cat, mu, nu, 3-layer CNN over {C} channels, softmax; "
                           "s_prob, s_mix, C_avg mixing; random-init weights; MLPs and convolutions on tcgen05 "
                           "(bf16 head/remainder operands, three products per step, fp32 accumulators)",
                   "ms_per_step": d_ms, "ms_stats": ms_stats(d_all), "value": w.B * w.T / (d_ms / 1e3), "unit": "tokens/s",
                   "gpu_launches_per_step": d_launches, "estimate_decoder_ms": ms_stats(e_all),
                   "conv_flops": conv_flops, "conv_tflops_if_all_time_were_conv": conv_flops / (sum(e_all) / n_d / 1e3) / 1e12}
        step()
        torch.cuda.synchronize(dev)
        del dws, Zb

    ms_per_step, e2e_ms = max_over_ranks([sum(step_ms) / args.steps, e2e_ms], dev)
    tokens = w.B * w.T * world
    elem = 2 if w.dtype == "bf16" else 4
    h2d = sum(host[k].numel() * host[k].element_size() for k in ("Q", "K", "V", "omega", "W_dec"))
    d2h = O.numel() * O.element_size()

    if rank == 0:
        peaks = measured_peaks()
        qkv_bytes = 3 * w.rows * w.d * elem
        a_hat_bytes = w.rows * w.Kc * 4
        mask_out = w.rows * w.k_hat * 4 + (w.rows + 1) * 4 + nnz * 4
        line = {
            "metric": METRIC, "value": tokens / (ms_per_step / 1e3), "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "ms_stats": ms_stats(step_ms),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": workload_config(w),
            "e2e": {"value": tokens / (e2e_ms / 1e3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "ms_stats": ms_stats(e2e_all)},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks,
            "clock_x_time": None if not clocks or not clocks.get("sm_mhz") else
            {"mhz_ms_per_step": clocks["sm_mhz"] * ms_per_step, "note": "median SM MHz x ms per step"},
            "stages_ms": {"estimate": stage_ms[0], "topk_mask": stage_ms[1], "sparse_attn": stage_ms[2]},
            "stages_ms_stats": {"estimate": ms_stats(stage_all[0]), "topk_mask": ms_stats(stage_all[1]),
                                "sparse_attn": ms_stats(stage_all[2])},
            "nnz": nnz,
            "lean": lean,
            "grouped": grouped,
            "causal_aware": causal_aware,
            "structured_mask": structured,
            "decoder_head": decoder,
            "roofline": sparse_roofline(w, sparse_kernel, sparse_flops, nnz, stage_ms[2], peaks, clocks),
            "roofline_estimate": hbm_roofline("favor_prep_tc / favor_state_tc / favor_scan_tc / favor_output_tc",
                                              qkv_bytes + a_hat_bytes, stage_ms[0], peaks,
                                              "Q, K, V in, A_hat (fp32) out"),
            "roofline_mask": hbm_roofline("top-k selection, row_ptr scan, fill_col_idx", a_hat_bytes + mask_out,
                                          stage_ms[1], peaks, "A_hat in; sel, row_ptr, col_idx out"),
        }
        line["roofline"]["launches_in_timed_call"] = sparse_launches
        if cpu_line is not None:
            line["cpu_baseline"] = cpu_line
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def _gpu_index(local_rank: int) -> str:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        ids = [x.strip() for x in vis.split(",") if x.strip()]
        if local_rank < len(ids):
            return ids[local_rank]
    return str(local_rank)


if __name__ == "__main__":
    main()
