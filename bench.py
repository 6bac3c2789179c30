#!/usr/bin/env python
"""Benchmark of the SEA attention layer (estimate -> top-k mask -> sparse attention) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one sea_attention call (all stages) over one synthetic batch of the workload's shape.
The default workload is the OPT-1.3B-shaped causal bf16 configuration, on which the headline
metric is quoted.  One JSON line is printed by rank 0.

  value      tokens/s (B*T per step, all ranks) with inputs resident in HBM, CUDA events per step,
             L2 flushed between steps, max over ranks.
  e2e        the same through sea_attention_host: pinned host Q, K, V, omega, W_dec in, O out.
  roofline   the sparse-attention kernel: algorithmic bytes (Q + O + every row's gathered K/V)
             over its CUDA-event time, against the measured HBM copy bandwidth.  The kernel forms
             the masked products as dense tiles on the tensor cores and gathers nothing, so this
             figure exceeds 1; `tensor` inside it gives the FLOPs the kernel really executes
             (every key tile a query tile may see, Q K^T twice and P V as head + remainder)
             against the measured dense bf16 peak.
  stages     per-stage milliseconds from a second pass that calls the three stage entry points
             with events between them (same kernels as the fused call).
  lean       the fused call asked for O and the CSR mask only (the estimate and the probabilities are
             never written out); per-rank, not part of `value`.
  grouped, causal_aware
             the same step with the causal-per-batch grouping (sea_attention_grouped) and with the
             causal-aware per-query selection (sea_attention_causal_aware) on this rank, and their
             selection and sparse stages; per-rank, not part of `value`.
  cpu_baseline  the fp64 oracle on a bounded sample of heads, on this machine's host cores.

With N > 1 (torchrun) every rank runs an independent replica of the workload (the path has no
exchange step between GPUs); value sums the ranks' tokens over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
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
# dram__bytes_read.sum + dram__bytes_write.sum of one sparse-attention launch, from the ncu capture
# summarised in profiles/sparse_attn_tiles_tc_opt_1p3b.md (one launch covers the whole workload; 290.6 MB
# read + 200.7 MB written).
NCU_TRAFFIC_BYTES = {"opt_1p3b": 491.3e6}


def measured_peaks():
    """(HBM GB/s, dense bf16 TFLOP/s for a kernel timed alone, 'measured' | 'fallback')."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            j = json.load(f)
        return float(j["hbm_gbs"]), float(j["bf16_tflops"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


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
        time.sleep(0.15)
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
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_tokens_per_s(w, n_heads: int, repeats: int = 1):
    """The fp64 oracle, as it stands, on the first n_heads (b, h) units of the workload."""
    import numpy as np
    from threadpoolctl import threadpool_limits

    from oracle import sea_oracle as orc
    from paper_2310_01777_b200.inputs import make_inputs

    small = w.scaled(B=1, H=n_heads)
    host = make_inputs(small)
    f64 = lambda t: t.to(dtype=__import__("torch").float64).numpy()
    given = "A_hat" in host  # workloads without an estimator stage bring the estimate along
    om, wd = (None, None) if given else (f64(host["omega"]), f64(host["W_dec"]))
    scale = 1.0 / np.sqrt(w.d)
    best = None
    with threadpool_limits(limits=1):
        for _ in range(repeats):
            t0 = time.perf_counter()
            for h in range(n_heads):
                orc.sea_attention_head(f64(host["Q"][0, h]), f64(host["K"][0, h]), f64(host["V"][0, h]), w.k_hat,
                                       w.Kc, w.causal, scale, A_hat=f64(host["A_hat"][0, h]) if given else None,
                                       omega=om, W_dec=wd)
            dt = time.perf_counter() - t0
            best = dt if best is None else min(best, dt)
    tokens = n_heads * w.T / w.H  # a token passes through all H heads of the layer
    return tokens / best, best


def run_reference(args, w):
    """The base contract's reference arm: the CPU oracle on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_heads = args.ref_heads
    for _ in range(args.warmup):
        oracle_tokens_per_s(w, 1)
    times = []
    for _ in range(args.steps):
        _, dt = oracle_tokens_per_s(w, n_heads)
        times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = (n_heads * w.T / w.H) / (ms / 1e3)
    sample = f"{n_heads} of {w.B * w.H} heads of {w.name} per step, fp64 numpy oracle, BLAS threads limited to 1"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w),
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": 1, "kind": "oracle", "sample": sample},
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="opt_1p3b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-heads", type=int, default=8, help="heads per step of the reference arm")
    ap.add_argument("--cpu-heads", type=int, default=64, help="heads in the cpu_baseline sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2310_01777_b200.inputs import WORKLOADS, make_inputs, torch_dtype

    w = WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return

    if w.m == 0:
        raise SystemExit(f"bench.py times workloads that start at the estimator; {w.name} is a parity-test case")

    import torch
    import torch.distributed as dist

    import paper_2310_01777_b200 as sea

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
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
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    torch.cuda.synchronize(dev)
    if rank == 0:
        sampler.start()
    for a, b in ev:
        flush.zero_()
        a.record()
        step()
        b.record()
    torch.cuda.synchronize(dev)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = sum(a.elapsed_time(b) for a, b in ev)

    # ---- timed region 2: stage by stage (for the roofline of the dominant kernel) -------
    for _ in range(2):  # the stage entry points launch kernels the fused call does not: load them first
        sea.sea_estimate(shape, d["Q"], d["K"], d["V"], d["omega"], d["W_dec"], A_hat, ws)
        sea.sea_topk_mask(shape, A_hat, sel, row_ptr, col_idx, ws)
        sea.sea_sparse_attn(shape, d["Q"], d["K"], d["V"], row_ptr, col_idx, sel, O, P, ws)
    torch.cuda.synchronize(dev)
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
    stage_ms = [sum(e[i].elapsed_time(e[i + 1]) for e in sev) / args.steps for i in range(3)]
    nnz = int(row_ptr[-1])

    # ---- timed region 3: end to end from pinned host memory ---------------------------
    hp = {k: v.pin_memory() for k, v in host.items()}
    hO = torch.empty((w.B, w.H, w.T, w.d), dtype=io).pin_memory()
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(2):
        sea.sea_attention_host(shape, hp["Q"], hp["K"], hp["V"], hp["omega"], hp["W_dec"], hO, ws)
    eev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(e2e_steps)]
    barrier()
    torch.cuda.synchronize(dev)
    for a, b in eev:
        flush.zero_()
        a.record()
        sea.sea_attention_host(shape, hp["Q"], hp["K"], hp["V"], hp["omega"], hp["W_dec"], hO, ws)
        b.record()
    torch.cuda.synchronize(dev)
    barrier()
    e2e_ms = sum(a.elapsed_time(b) for a, b in eev) / e2e_steps
    if not torch.equal(hO, O.cpu()):
        raise SystemExit("host entry point and device entry point disagree")

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
    lev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    torch.cuda.synchronize(dev)
    for a, b in lev:
        flush.zero_()
        a.record()
        lean_step()
        b.record()
    torch.cuda.synchronize(dev)
    lean_ms = sum(a.elapsed_time(b) for a, b in lev) / args.steps
    if not (torch.equal(O_lean, O) and torch.equal(rp_lean, row_ptr)):
        raise SystemExit("the call without the optional outputs gives a different O or row_ptr")
    lean = {"outputs": "O, row_ptr and col_idx only (no A_hat, sel, P)", "ms_per_step": lean_ms,
            "value": w.B * w.T / (lean_ms / 1e3), "unit": "tokens/s", "gpu_launches_per_step": lean_launches}

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
        gev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        torch.cuda.synchronize(dev)
        for a, b in gev:
            flush.zero_()
            a.record()
            gstep()
            b.record()
        torch.cuda.synchronize(dev)
        g_ms = sum(a.elapsed_time(b) for a, b in gev) / args.steps
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
        return {"selection": label, "ms_per_step": g_ms, "value": w.B * w.T / (g_ms / 1e3), "unit": "tokens/s",
                "gpu_launches_per_step": g_launches,
                "stages_ms": {"topk_mask": sum(e[0].elapsed_time(e[1]) for e in gsev) / args.steps,
                              "sparse_attn_masked": sum(e[1].elapsed_time(e[2]) for e in gsev) / args.steps},
                "nnz": int(row_ptr[-1])}

    grouped = None
    if w.Kc % 4 == 0 and w.H * w.Kc <= 32768:
        grouped = time_bits_mode("causal-per-batch", sea.sea_attention_grouped, sea.sea_topk_mask_grouped)
    causal_aware = None
    if w.causal:
        causal_aware = time_bits_mode("causal-aware per-query", sea.sea_attention_causal_aware,
                                      sea.sea_topk_mask_causal_aware)

    ms_per_step, e2e_ms = max_over_ranks([total_ms / args.steps, e2e_ms], dev)
    tokens = w.B * w.T * world
    elem = 2 if w.dtype == "bf16" else 4
    h2d = sum(host[k].numel() * host[k].element_size() for k in ("Q", "K", "V", "omega", "W_dec"))
    d2h = O.numel() * O.element_size()

    if rank == 0:
        peak, tc_peak, peak_kind = measured_peaks()
        alg_bytes = 2 * w.rows * w.d * elem + 2 * nnz * w.d * elem  # Q + O + gathered K and V
        # what the tile kernel executes: per (query tile, key tile) pair S = Q K^T in both passes and
        # P V with P as bf16 head + remainder, 2 * 128 * 128 * 64 FLOPs each
        r = w.T // w.Kc
        tiled = w.dtype == "bf16" and w.T % 128 == 0 and r >= 4 and r & (r - 1) == 0 and w.k_hat * 40 >= w.Kc
        nq = w.T // 128
        pairs = w.B * w.H * (nq * (nq + 1) // 2 if w.causal else nq * nq)
        exec_flops = pairs * 4 * (2 * 128 * 128 * w.d) if tiled else None
        sparse_s = stage_ms[2] / 1e3
        unique_bytes = 4 * w.rows * w.d * elem + nnz * elem + w.rows * w.k_hat * 4 + (w.rows + 1) * 4
        achieved = alg_bytes / sparse_s / 1e9
        line = {
            "metric": METRIC, "value": tokens / (ms_per_step / 1e3), "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": workload_config(w),
            "e2e": {"value": tokens / (e2e_ms / 1e3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks,
            "stages_ms": {"estimate": stage_ms[0], "topk_mask": stage_ms[1], "sparse_attn": stage_ms[2]},
            "nnz": nnz,
            "lean": lean,
            "grouped": grouped,
            "causal_aware": causal_aware,
            "roofline": {"kernel": "sparse_attn_tiles_tc_kernel" if tiled else "sparse_attn_blocks_tma_kernel",
                         "bound": "hbm", "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": achieved / peak, "peak_source": f"{peak_kind} HBM copy bandwidth",
                         "algorithmic_bytes": alg_bytes, "traffic": NCU_TRAFFIC_BYTES.get(w.name) if tiled else None,
                         "ms": stage_ms[2], "sparse_stage_tokens_per_s": w.B * w.T / sparse_s,
                         "tensor": None if not tiled else {
                             "executed_flops": exec_flops, "achieved": exec_flops / sparse_s / 1e12, "peak": tc_peak,
                             "unit": "TFLOP/s", "frac": exec_flops / sparse_s / 1e12 / tc_peak,
                             "peak_source": f"{peak_kind} dense bf16 (burst)"},
                         # K and V of every head fit the L2 together, so the bytes that must cross HBM are
                         # far fewer than the algorithmic ones: Q, K, V once, O and P once, sel and row_ptr
                         "compulsory_hbm_bytes": unique_bytes,
                         "compulsory_hbm_gbs": unique_bytes / sparse_s / 1e9},
        }
        if not args.no_cpu_baseline and world == 1:
            n = min(args.cpu_heads, w.B * w.H)
            v, dt = oracle_tokens_per_s(w, n)
            line["cpu_baseline"] = {"value": v, "unit": "tokens/s", "cores": 1, "kind": "oracle",
                                    "sample": f"first {n} of {w.B * w.H} heads, fp64 numpy oracle, {dt:.1f} s, "
                                              "BLAS threads limited to 1"}
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
