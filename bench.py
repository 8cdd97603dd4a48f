#!/usr/bin/env python
"""Benchmark of the HDQT quantized training GEMM hot path on B200.

One "step" = one pass of the whole path over one synthetic batch:
  calibration maximum + FWHT + quantize of both operands -> tiled int8 tensor-core GEMM with
  8-bit per-tile accumulators -> wide tile sum -> dequantising epilogue.
Workload = one shape of the roofline sweep (dgrad layout: A K-contiguous with stochastic
rounding, B K-contiguous with nearest rounding), operands Student-t(3) with 0.1 % outliers x50.

Prints ONE JSON line (see README for the keys).  `--impl reference` times the CPU
oracle on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "hdqt_gemm_int_tops"
UNIT = "TOPS"
SEED = 1234
# dram__bytes_read.sum + dram__bytes_write.sum of the GEMM kernels of one step at M=N=K=8192 (pair kernel + fix-up),
# from the ncu capture summarised in profiles/gemm_i8_tiled_kernel_sweep.md
GEMM_DRAM_BYTES_8192 = 301.8e6 + 241.0e6 + 36.5e6 + 0.3e6


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="hdqt", choices=["hdqt", "reference"])
    ap.add_argument("--size", type=int, default=8192, help="M = N = K of the sweep shape")
    ap.add_argument("--layout", default="dgrad", choices=["dgrad", "wgrad"],
                    help="dgrad: both operands K-contiguous, A stochastic / B nearest; "
                         "wgrad: both operands K-strided (transposed reads), both stochastic")
    ap.add_argument("--workload", default="sweep", choices=["sweep", "mlp"],
                    help="sweep: the GEMM roofline shape (default, the headline line); mlp: training steps/s of the "
                         "synthetic 1152-512-256-12 MLP, batch 256 (a secondary report)")
    ap.add_argument("--acc-tile", type=int, default=32, help="accumulator tile length s along K (0 = whole K)")
    ap.add_argument("--acc-bits", type=int, default=8, help="accumulator bit width b_a")
    ap.add_argument("--no-merge", action="store_true", help="disable merging of provably clamp-free tiles")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true")
    return ap.parse_args()


def workload_config(size: int, merge: bool, layout: str = "dgrad", acc_tile: int = 32, acc_bits: int = 8):
    return {
        "workload": f"roofline-sweep {layout}-layout HDQT GEMM M=N=K={size} (Student-t(3), 0.1% outliers x50)",
        "M": size, "N": size, "K": size,
        "in_bits": 4, "acc_bits": acc_bits, "acc_tile": acc_tile, "had_block": 32, "acc_shift": 0,
        "rounding": "A stochastic (Philox4x32-10), B nearest" if layout == "dgrad" else "A and B stochastic (Philox4x32-10)",
        "clamp_free_tile_merging": bool(merge),
        "l2": "inputs_exceed_l2" if size * size * 4 > 126 * 2 ** 20 else "inputs_within_l2_not_flushed",
        "parallelism": "replicas",
    }


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
# CPU oracle arm (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------

def oracle_sample_run(size: int, rows_a: int, rows_b: int, seed: int, layout: str = "dgrad"):
    """One pass of the oracle over a slice of the workload: rows_a rows of A, rows_b rows of B, full K.
    Returns (seconds, equivalent integer ops)."""
    from oracle import hdqt_oracle as O
    from paper_2310_03675_b200 import inputs
    A = inputs.heavy_tailed(rows_a, size, seed)
    B = inputs.heavy_tailed(rows_b, size, seed + 1)
    t0 = time.perf_counter()
    if layout == "wgrad":
        O.gemm_wgrad(np.ascontiguousarray(A.T), np.ascontiguousarray(B.T), O.wgrad_desc(seed=seed))
    else:
        O.gemm_dgrad(A, B, O.dgrad_desc(seed=seed))
    dt = time.perf_counter() - t0
    return dt, 2.0 * rows_a * rows_b * size


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(size: int, layout: str = "dgrad"):
    rows_a, rows_b = min(size, 1024), min(size, 2048)
    dt, ops = oracle_sample_run(size, rows_a, rows_b, SEED, layout)
    return {"value": ops / dt / 1e12, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "seconds": dt,
            "sample": f"{rows_a} rows of A x {rows_b} rows of B, full K={size} (whole path: FWHT, quantize, "
                      f"tiled GEMM, dequant); ops counted as 2*rows_a*rows_b*K"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    size = args.size
    rows_a, rows_b = min(size, 256), min(size, 512)
    for _ in range(min(args.warmup, 1)):
        oracle_sample_run(size, rows_a, rows_b, SEED, args.layout)
    total_t, total_ops = 0.0, 0.0
    for i in range(args.steps):
        dt, ops = oracle_sample_run(size, rows_a, rows_b, SEED + i, args.layout)
        total_t += dt
        total_ops += ops
    value = total_ops / total_t / 1e12
    sample = f"each step: {rows_a} rows of A x {rows_b} rows of B, full K={size}, whole path on the CPU oracle"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_t / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8/f32", "data": "synthetic",
        "config": workload_config(size, not args.no_merge, args.layout, args.acc_tile, args.acc_bits),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------

def launches_per_step(M, N, merge, wgrad, acc_bits, sms=148):
    """Kernels of this library launched by one step (what the host layer does, restated for the report):
    2 calibration + 2 quantize kernels, the tile-norm reduction for K-contiguous operands when merging, and the
    GEMM: one kernel, or - at >= 8 output blocks per SM with merging - classify, compact, pair kernel, fix-up and
    general kernel (the pair kernel alone when the accumulators are too wide to clamp)."""
    n = 4 + (2 if (merge and not wgrad) else 0)
    blocks = ((M + 127) // 128) * ((N + 255) // 256)
    if merge and blocks >= 8 * sms:
        n += 1 if acc_bits >= 13 else 5
    else:
        n += 1
    return n


def max_over_ranks(values, device, world):
    """Element-wise maximum of per-rank timings over all ranks (every rank gets the result)."""
    if world <= 1:
        return list(values)
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_tops(world, steps, ops_per_step, elapsed_ms):
    """Aggregate throughput of `world` replicas that each ran `steps` steps in `elapsed_ms` (max over ranks)."""
    return world * steps * ops_per_step / (elapsed_ms * 1e-3) / 1e12


def run_hdqt(args):
    import torch
    import torch.distributed as dist
    from paper_2310_03675_b200 import hdqt, inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    size = args.size
    M = N = K = size
    merge = not args.no_merge
    flags = 0 if merge else hdqt.FLAG_NO_MERGE
    wgrad = args.layout == "wgrad"
    desc = hdqt.default_desc("wgrad" if wgrad else "dgrad", seed=SEED, flags=flags, acc_tile=args.acc_tile,
                             acc_bits=args.acc_bits)

    # every rank works on its own operands (independent problems: no data-path collective)
    A = inputs.heavy_tailed_torch(M, K, SEED + 10 * rank, dev)
    B = inputs.heavy_tailed_torch(N, K, SEED + 10 * rank + 1, dev)
    if wgrad:
        # dW = X^T G: the operands are stored [K, M] and [K, N] (contraction index strided)
        Xs, Gs = A.t().contiguous(), B.t().contiguous()
        A, B = Xs.t(), Gs.t()          # logical [M, K] / [N, K] views with stride (1, M) / (1, N)
    out = torch.empty((M, N), dtype=torch.float32, device=dev)
    status = hdqt.new_status(dev)
    Kp = hdqt.padded_k(K)

    # stage-level buffers (the same launches the composite call makes, with events between stages)
    def qbufs(rows):
        return (torch.empty((rows, Kp), dtype=torch.int8, device=dev), torch.empty(1, device=dev),
                torch.empty(((rows + 127) // 128, Kp // 32), dtype=torch.int32, device=dev) if merge else None,
                torch.empty(hdqt.lib.hdqt_quantize_workspace_bytes(rows, K, 32), dtype=torch.uint8, device=dev))
    bufA, bufB = qbufs(M), qbufs(N)
    stream = torch.cuda.current_stream()

    def step(ev=None):
        if ev:
            ev[0].record(stream)
        hdqt.quantize_hadamard(A, 32, desc.in_bits, desc.clip_a, desc.round_a, desc.seed, desc.tag_a,
                               want_norms=merge, dev_status=status, out=bufA)
        hdqt.quantize_hadamard(B, 32, desc.in_bits, desc.clip_b, desc.round_b, desc.seed, desc.tag_b,
                               want_norms=merge, dev_status=status, out=bufB)
        if ev:
            ev[1].record(stream)
        hdqt.gemm_i8_tiled(bufA[0], bufB[0], bufA[1], bufB[1], desc.acc_bits, desc.acc_tile, desc.acc_shift,
                           desc.had_block, norms_a=bufA[2], norms_b=bufB[2], flags=flags, dev_status=status, out=out)
        if ev:
            ev[2].record(stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    hdqt.check_device_status(status, "warm-up")

    events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for i in range(args.steps):
        step(events[i])
    t_end.record(stream)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    hdqt.check_device_status(status, "timed region")
    elapsed_ms = t_start.elapsed_time(t_end)
    quant_ms = sum(e[0].elapsed_time(e[1]) for e in events) / args.steps
    gemm_ms = sum(e[1].elapsed_time(e[2]) for e in events) / args.steps

    # end to end through the public call with host buffers: H2D of both operands, D2H of the result
    e2e = None
    if not args.skip_e2e:
        srcA, srcB = (Xs, Gs) if wgrad else (A, B)
        hA = torch.empty(tuple(srcA.shape), dtype=torch.float32).pin_memory()
        hB = torch.empty(tuple(srcB.shape), dtype=torch.float32).pin_memory()
        hA.copy_(srcA)
        hB.copy_(srcB)
        hOut = torch.empty((M, N), dtype=torch.float32).pin_memory()
        dA, dB = torch.empty_like(srcA), torch.empty_like(srcB)
        ws = hdqt.Workspace(desc, M, N, K, dev)
        e2e_steps = max(3, min(args.steps, 5))
        public_call = hdqt.gemm_wgrad if wgrad else hdqt.gemm_dgrad

        def e2e_step():
            dA.copy_(hA, non_blocking=True)
            dB.copy_(hB, non_blocking=True)
            public_call(dA, dB, desc=desc, workspace=ws, dev_status=status, out=out)
            hOut.copy_(out, non_blocking=True)

        e2e_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1)
        e2e_ms = max_over_ranks([e2e_ms], dev, world)[0]
        e2e = {"value": whole_job_tops(world, e2e_steps, 2.0 * M * N * K, e2e_ms), "unit": UNIT,
               "h2d_bytes_per_step": hA.numel() * 4 + hB.numel() * 4, "d2h_bytes_per_step": hOut.numel() * 4,
               "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps}
        hdqt.check_device_status(status, "e2e")

    elapsed_ms, quant_ms, gemm_ms = max_over_ranks([elapsed_ms, quant_ms, gemm_ms], dev, world)

    certified = None
    if merge and bufA[2] is not None and desc.acc_tile == 32 and rank == 0:
        # fraction of (128x256 output block, K tile) pairs whose Cauchy-Schwarz bound proves "no clamp"
        na = bufA[2].to(torch.int64)                                    # [M/128, T]
        nb = bufB[2].to(torch.int64)
        if nb.shape[0] % 2:
            nb = torch.cat([nb, torch.zeros_like(nb[:1])])
        nb = nb.view(-1, 2, nb.shape[1]).amax(1)                        # [N/256, T]
        hi = (1 << (desc.acc_bits - 1)) - 1
        cert = 0
        for i in range(na.shape[0]):
            cert += int(((na[i][None, :] * nb) <= hi * hi).sum().item())
        certified = cert / float(na.shape[0] * nb.shape[0] * nb.shape[1])

    if rank == 0:
        peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
        if os.path.exists(peaks_path):
            peaks = json.load(open(peaks_path))
            bf16_sustained = peaks.get("bf16_tflops_sustained", peaks.get("bf16_tflops"))
            hbm = peaks["hbm_gbs"]
            peak_src = "measured bf16 sustained x2 (nominal int8:bf16 ratio)"
        else:
            bf16_sustained, hbm = 1400.0, 6650.0
            peak_src = "fallback bf16 sustained x2 (nominal int8:bf16 ratio)"
        int8_peak = 2.0 * bf16_sustained
        ops = 2.0 * M * N * K
        gemm_tops = ops / (gemm_ms * 1e-3) / 1e12
        quant_bytes = 9.0 * (M * K + N * K)      # 4 B calibration read + 4 B read + 1 B code written, per element
        line = {
            "metric": METRIC, "value": whole_job_tops(world, args.steps, ops, elapsed_ms), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": elapsed_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8/f32",
            "data": "synthetic", "config": workload_config(size, merge, args.layout, args.acc_tile, args.acc_bits),
            "roofline": {"bound": "tensor", "kernel": "hdqt_gemm_i8_tiled (pair kernel + fix-up + general kernel)", "achieved": gemm_tops,
                         "peak": int8_peak, "unit": "TOP/s", "frac": gemm_tops / int8_peak, "peak_source": peak_src,
                         "traffic": GEMM_DRAM_BYTES_8192 if (size == 8192 and merge and not wgrad) else None,
                         "traffic_unit": "bytes per launch (ncu dram read+write, profiles/gemm_i8_tiled_kernel_sweep.md)",
                         "algorithmic_bytes": float(M * K + N * K + 4 * M * N),
                         "ms_per_launch": gemm_ms, "certified_clamp_free_tile_fraction": certified},
            "quantize": {"ms_per_step": quant_ms, "algorithmic_gb_per_step": quant_bytes / 1e9,
                         "gbs": quant_bytes / (quant_ms * 1e-3) / 1e9, "hbm_peak_gbs": hbm,
                         "frac": quant_bytes / (quant_ms * 1e-3) / 1e9 / hbm,
                         "note": "both operands: calibration pass (4 B/elt) + FWHT/quantize pass (5 B/elt)"},
            "clocks": clocks, "gpu_launches": args.steps * launches_per_step(M, N, merge, wgrad, desc.acc_bits),
        }
        if e2e is not None:
            line["e2e"] = e2e
        if not args.skip_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(size, args.layout)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_mlp(args):
    """Training steps/s of the synthetic MLP step (every matmul through the library), with the fp32 torch
    step of the same model as context. Secondary report: one JSON line of its own."""
    import torch
    from paper_2310_03675_b200 import nn as hnn
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    x, labels = hnn.sensor_window_batch(256, 1152, 12, seed=SEED, device=dev)
    out = {}
    for name, quantized in (("hdqt", True), ("fp32_torch", False)):
        torch.manual_seed(0)
        model = hnn.Mlp(quantized=quantized).to(dev)
        opt = torch.optim.SGD(model.parameters(), lr=0.01, momentum=0.9)
        for i in range(max(args.warmup, 3)):
            hnn.train_step(model, opt, x, labels, i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(args.steps):
            loss = hnn.train_step(model, opt, x, labels, 1000 + i)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / args.steps
        out[name] = {"steps_per_s": 1e3 / ms, "ms_per_step": ms, "final_loss": float(loss.item())}
    print(json.dumps({"metric": "hdqt_mlp_train_steps_per_s", "value": out["hdqt"]["steps_per_s"], "unit": "steps/s",
                      "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3),
                      "ms_per_step": out["hdqt"]["ms_per_step"], "higher_is_better": True, "data": "synthetic",
                      "config": {"workload": "MLP 1152-512-256-12, batch 256, SGD momentum 0.9, 4-bit inputs, "
                                             "8-bit accumulators, Hadamard block 32"},
                      "fp32_torch": out["fp32_torch"], "hdqt": out["hdqt"]}))


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "mlp":
        run_mlp(args)
    else:
        run_hdqt(args)


if __name__ == "__main__":
    main()
