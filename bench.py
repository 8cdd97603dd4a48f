#!/usr/bin/env python
"""Benchmark of the HDQT quantized training GEMM hot path on B200.

One "step" = one pass of the whole path over one synthetic batch:
  calibration maximum + FWHT + quantize of both operands -> tiled int8 tensor-core GEMM with
  8-bit per-tile accumulators -> wide tile sum -> dequantising epilogue.
Headline workload = the largest shape of the roofline sweep (dgrad layout: A K-contiguous with
stochastic rounding, B K-contiguous with nearest rounding, M = N = K = 16384), operands Student-t(3)
with 0.1 % outliers x50.

Prints ONE JSON line.  Besides the contract keys it carries:
  roofline             GEMM kernels of the headline shape against 2 x the measured bf16 burst rate
  roofline_clamp_path  the same shape with every tile through the 8-bit accumulator epilogue (merging off)
  quantize, quantize_supplied_max   transform/quantize passes against the measured copy bandwidth
  sustained            the same step looped for seconds, with the clocks and power sampled meanwhile
  sweep                the other corners of the sweep (8192 / 16384, dgrad / wgrad layouts)
  train_steps_per_s    MLP, CNN and class-incremental steps per second, fp32 torch beside each
  e2e, cpu_baseline, clocks, gpu_launches
`--impl reference` times the CPU oracle on a bounded sample of the same workload instead.
`--workload mlp|cnn|cil` prints a training report of its own (cil: the full incremental run with accuracies).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
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
DATASHEET_INT8_TOPS = 4500.0      # dense int8, B200 (context only)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="hdqt", choices=["hdqt", "reference"])
    ap.add_argument("--size", type=int, default=16384, help="M = N = K of the headline sweep shape")
    ap.add_argument("--layout", default="dgrad", choices=["dgrad", "wgrad"],
                    help="dgrad: both operands K-contiguous, A stochastic / B nearest; "
                         "wgrad: both operands K-strided (transposed reads), both stochastic")
    ap.add_argument("--workload", default="sweep", choices=["sweep", "mlp", "cnn", "cil"],
                    help="sweep: the GEMM roofline line (default); mlp / cnn: training steps per second of the "
                         "synthetic models; cil: the full class-incremental run with final accuracies")
    ap.add_argument("--acc-tile", type=int, default=32, help="accumulator tile length s along K (0 = whole K)")
    ap.add_argument("--acc-bits", type=int, default=8, help="accumulator bit width b_a")
    ap.add_argument("--no-merge", action="store_true", help="disable merging of provably clamp-free tiles")
    ap.add_argument("--sustained-seconds", type=float, default=3.0)
    ap.add_argument("--steps-per-task", type=int, default=1000, help="cil workload: training steps per task")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-extras", action="store_true",
                    help="headline measurement only (no clamp-path, sustained, sweep and training records)")
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

    def __init__(self, gpu_index: int, period_ms: int = 50):
        self.gpu_index = gpu_index
        self.period_ms = period_ms
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms",
                 str(self.period_ms), "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL,
                text=True)
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
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
                power.append(float(parts[3]))
            except ValueError:
                continue
            for n, v in zip(names, parts[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_median": statistics.median(power) if power else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


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
    """The oracle as it stands on a bounded sample, once with the BLAS pool limited to one thread and once with
    all its threads (everything outside the per-tile matrix product is single-threaded numpy either way)."""
    rows_a, rows_b = min(size, 768), min(size, 1536)
    sample = (f"{rows_a} rows of A x {rows_b} rows of B, full K={size} (whole path: FWHT, quantize, tiled GEMM, "
              f"dequant); ops counted as 2*rows_a*rows_b*K")
    single = None
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            dt1, ops = oracle_sample_run(size, rows_a, rows_b, SEED, layout)
        single = {"value": ops / dt1 / 1e12, "seconds": dt1, "cores": 1}
    except Exception:
        pass
    dt, ops = oracle_sample_run(size, rows_a, rows_b, SEED, layout)
    return {"value": ops / dt / 1e12, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "seconds": dt,
            "single_thread": single, "sample": sample}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    size = args.size
    rows_a, rows_b = min(size, 256), min(size, 512)
    steps = min(args.steps, 20)
    for _ in range(min(args.warmup, 1)):
        oracle_sample_run(size, rows_a, rows_b, SEED, args.layout)
    total_t, total_ops = 0.0, 0.0
    for i in range(steps):
        dt, ops = oracle_sample_run(size, rows_a, rows_b, SEED + i, args.layout)
        total_t += dt
        total_ops += ops
    value = total_ops / total_t / 1e12
    sample = (f"each step: {rows_a} rows of A x {rows_b} rows of B, full K={size}, whole path on the CPU oracle "
              f"({steps} steps timed)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": args.warmup, "ms_per_step": total_t / steps * 1e3,
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

def launches_per_step(M, N, merge, acc_bits, sms=148):
    """Kernels of this library launched by one step of the stage-timed loop (what the host layer does, restated
    for the report): per operand one calibration and one quantize kernel, and the GEMM: one kernel, or - at >= 8
    output blocks per SM with merging - classify, compact, pair kernel, fix-up and general kernel (the pair
    kernel alone when the accumulators are too wide to clamp)."""
    n = 4
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


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        peaks = json.load(open(path))
        return {"bf16_burst": peaks.get("bf16_tflops"), "bf16_sustained": peaks.get("bf16_tflops_sustained"),
                "hbm": peaks["hbm_gbs"], "source": "measured"}
    return {"bf16_burst": 1590.0, "bf16_sustained": 1400.0, "hbm": 6650.0, "source": "fallback"}


class SweepCase:
    """Operands and buffers of one sweep shape, and the stage-timed step over them."""

    def __init__(self, hdqt, inputs, torch, dev, size, layout, merge, acc_tile, acc_bits, seed_shift=0):
        self.hdqt, self.torch, self.dev = hdqt, torch, dev
        self.M = self.N = self.K = size
        self.layout, self.merge = layout, merge
        self.flags = 0 if merge else hdqt.FLAG_NO_MERGE
        wgrad = layout == "wgrad"
        self.desc = hdqt.default_desc("wgrad" if wgrad else "dgrad", seed=SEED, flags=self.flags, acc_tile=acc_tile,
                                      acc_bits=acc_bits)
        A = inputs.heavy_tailed_torch(size, size, SEED + seed_shift, dev)
        B = inputs.heavy_tailed_torch(size, size, SEED + seed_shift + 1, dev)
        self.stored = (A, B)
        if wgrad:
            # dW = X^T G: the operands are stored [K, M] and [K, N] (contraction index strided)
            Xs, Gs = A.t().contiguous(), B.t().contiguous()
            del A, B
            self.stored = (Xs, Gs)
            A, B = Xs.t(), Gs.t()      # logical [M, K] / [N, K] views with stride (1, M) / (1, N)
        self.A, self.B = A, B
        self.out = torch.empty((size, size), dtype=torch.float32, device=dev)
        self.status = hdqt.new_status(dev)
        Kp = hdqt.padded_k(size)

        def qbufs(rows):
            return (torch.empty((rows, Kp), dtype=torch.int8, device=dev), torch.empty(1, device=dev),
                    torch.empty(((rows + 127) // 128, Kp // 32), dtype=torch.int32, device=dev) if merge else None,
                    torch.empty(hdqt.lib.hdqt_quantize_workspace_bytes(rows, size, 32), dtype=torch.uint8, device=dev))
        self.bufA, self.bufB = qbufs(size), qbufs(size)
        self.stream = torch.cuda.current_stream()

    def step(self, ev=None, amax=(None, None)):
        h, d = self.hdqt, self.desc
        if ev:
            ev[0].record(self.stream)
        h.quantize_hadamard(self.A, 32, d.in_bits, d.clip_a, d.round_a, d.seed, d.tag_a, amax=amax[0],
                            want_norms=self.merge, dev_status=self.status, out=self.bufA)
        h.quantize_hadamard(self.B, 32, d.in_bits, d.clip_b, d.round_b, d.seed, d.tag_b, amax=amax[1],
                            want_norms=self.merge, dev_status=self.status, out=self.bufB)
        if ev:
            ev[1].record(self.stream)
        h.gemm_i8_tiled(self.bufA[0], self.bufB[0], self.bufA[1], self.bufB[1], d.acc_bits, d.acc_tile, d.acc_shift,
                        d.had_block, norms_a=self.bufA[2], norms_b=self.bufB[2], flags=self.flags,
                        dev_status=self.status, out=self.out)
        if ev:
            ev[2].record(self.stream)

    def timed(self, steps, warmup, barrier=None, amax=(None, None)):
        """Returns (elapsed_ms, quant_ms_per_step, gemm_ms_per_step) over `steps` steps."""
        torch = self.torch
        for _ in range(max(warmup, 3)):
            self.step(amax=amax)
        torch.cuda.synchronize()
        self.hdqt.check_device_status(self.status, "warm-up")
        events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
        if barrier:
            barrier()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(self.stream)
        for i in range(steps):
            self.step(events[i], amax=amax)
        t1.record(self.stream)
        if barrier:
            barrier()
        else:
            torch.cuda.synchronize()
        self.hdqt.check_device_status(self.status, "timed region")
        quant_ms = sum(e[0].elapsed_time(e[1]) for e in events) / steps
        gemm_ms = sum(e[1].elapsed_time(e[2]) for e in events) / steps
        return t0.elapsed_time(t1), quant_ms, gemm_ms

    def certified_fraction(self):
        """Fraction of (128x256 output block, K tile) pairs whose Cauchy-Schwarz bound proves "no clamp"."""
        torch = self.torch
        if not self.merge or self.bufA[2] is None or self.desc.acc_tile != 32:
            return None
        na = self.bufA[2].to(torch.int64)
        nb = self.bufB[2].to(torch.int64)
        if nb.shape[0] % 2:
            nb = torch.cat([nb, torch.zeros_like(nb[:1])])
        nb = nb.view(-1, 2, nb.shape[1]).amax(1)
        hi = (1 << (self.desc.acc_bits - 1)) - 1
        cert = 0
        for i in range(na.shape[0]):
            cert += int(((na[i][None, :] * nb) <= hi * hi).sum().item())
        return cert / float(na.shape[0] * nb.shape[0] * nb.shape[1])


def shape_record(case, steps, warmup, peaks):
    elapsed, quant_ms, gemm_ms = case.timed(steps, warmup)
    ops = 2.0 * case.M * case.N * case.K
    qbytes = 9.0 * (case.M * case.K + case.N * case.K)
    peak = 2.0 * peaks["bf16_burst"]
    gemm_tops = ops / (gemm_ms * 1e-3) / 1e12
    return {"layout": case.layout, "M": case.M, "N": case.N, "K": case.K, "merging": case.merge,
            "value": ops * steps / (elapsed * 1e-3) / 1e12, "ms_per_step": elapsed / steps,
            "gemm_tops": gemm_tops, "gemm_frac": gemm_tops / peak, "gemm_ms": gemm_ms,
            "quantize_gbs": qbytes / (quant_ms * 1e-3) / 1e9, "quantize_frac": qbytes / (quant_ms * 1e-3) / 1e9 / peaks["hbm"],
            "quantize_ms": quant_ms, "certified_clamp_free_tile_fraction": case.certified_fraction()}


def train_steps_records(torch, dev, steps=20):
    """Training steps per second of the synthetic MLP and CNN workloads and of a class-incremental batch mix
    (new-task samples + replayed exemplars, grown head), every matmul through the library (with measured maxima,
    and with delayed scaling: maxima carried from the previous step, no calibration pass); the fp32 torch step of
    the same model beside each, and every variant once more as a step replayed from CUDA graphs.  Accuracy needs
    the long run (`--workload cil`)."""
    from paper_2310_03675_b200 import nn as hnn
    out = {}

    def time_steps(fn, n):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(n):
            fn(100 + i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    x, labels = hnn.sensor_window_batch(256, 1152, 12, seed=SEED, device=dev)
    rec = {}
    for name, quantized, over in (("hdqt", True, {}), ("hdqt_delayed_scaling", True, {"delayed": True}),
                                  ("fp32_torch", False, {})):
        torch.manual_seed(0)
        hnn.reset_delayed_scaling()
        model = hnn.Mlp(quantized=quantized, **over).to(dev)
        opt = torch.optim.SGD(model.parameters(), lr=0.01, momentum=0.9)
        ms = time_steps(lambda i: hnn.train_step(model, opt, x, labels, i), 5 * steps)
        rec[name] = {"steps_per_s": 1e3 / ms, "ms_per_step": ms}
        # the same step replayed from CUDA graphs (random stream advanced by a device-side word)
        stepper = hnn.GraphedTrainStep(model, opt, x, labels)
        ms = time_steps(lambda i: stepper(x, labels), 5 * steps)
        rec[name + "_cuda_graph"] = {"steps_per_s": 1e3 / ms, "ms_per_step": ms}
        del stepper
    out["mlp_1152_512_256_12_batch256"] = rec

    patterns = hnn.class_patterns(100, seed=SEED, device=dev)
    g = torch.Generator(device=dev)
    g.manual_seed(SEED)
    labels = torch.randint(0, 100, (128,), generator=g, device=dev)
    x = hnn.synthetic_images(labels, patterns, seed=SEED)
    rec = {}
    for name, quantized, over in (("hdqt", True, {}), ("hdqt_delayed_scaling", True, {"delayed": True}),
                                  ("fp32_torch", False, {})):
        torch.manual_seed(0)
        hnn.reset_delayed_scaling()
        model = hnn.ResNet18Width(100, quantized=quantized, **over).to(dev)
        opt = torch.optim.SGD(model.parameters(), lr=0.05, momentum=0.9, weight_decay=2e-4)
        ms = time_steps(lambda i: hnn.cnn_train_step(model, opt, x, labels, i), steps)
        rec[name] = {"steps_per_s": 1e3 / ms, "ms_per_step": ms}
        stepper = hnn.GraphedTrainStep(model, opt, x, labels)
        ms = time_steps(lambda i: stepper(x, labels), steps)
        rec[name + "_cuda_graph"] = {"steps_per_s": 1e3 / ms, "ms_per_step": ms}
        del stepper
        # class-incremental batch: second task, 64 new samples (classes 20..39) + 64 replayed, head of 40 neurons
        labels_cil = torch.cat([torch.randint(20, 40, (64,), generator=g, device=dev),
                                torch.randint(0, 20, (64,), generator=g, device=dev)])
        x_cil = hnn.synthetic_images(labels_cil, patterns, seed=SEED + 1)
        ms = time_steps(lambda i: hnn.cnn_train_step(model, opt, x_cil, labels_cil, i, n_seen=40), steps)
        out.setdefault("class_incremental_resnet18w_batch64new_64replay", {})[name] = \
            {"steps_per_s": 1e3 / ms, "ms_per_step": ms}
        del model, opt
    hnn.reset_delayed_scaling()
    out["cnn_resnet18w_32x32_batch128"] = rec
    return out


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
    merge = not args.no_merge
    peaks = load_peaks()
    extras = (not args.skip_extras) and world == 1

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # every rank works on its own operands (independent problems: no data-path collective)
    case = SweepCase(hdqt, inputs, torch, dev, size, args.layout, merge, args.acc_tile, args.acc_bits,
                     seed_shift=10 * rank)
    M = N = K = size
    sampler = ClockSampler(local_rank)
    for _ in range(max(args.warmup, 3)):
        case.step()
    torch.cuda.synchronize()
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    elapsed_ms, quant_ms, gemm_ms = case.timed(args.steps, args.warmup, barrier)
    clocks = sampler.stop() if rank == 0 else None

    # end to end through the public call with host buffers: H2D of both operands, D2H of the result
    e2e = None
    if not args.skip_e2e:
        wgrad = args.layout == "wgrad"
        srcA, srcB = case.stored
        hA = torch.empty(tuple(srcA.shape), dtype=torch.float32).pin_memory()
        hB = torch.empty(tuple(srcB.shape), dtype=torch.float32).pin_memory()
        hA.copy_(srcA)
        hB.copy_(srcB)
        hOut = torch.empty((M, N), dtype=torch.float32).pin_memory()
        dA, dB = torch.empty_like(srcA), torch.empty_like(srcB)
        ws = hdqt.Workspace(case.desc, M, N, K, dev)
        e2e_steps = 3
        public_call = hdqt.gemm_wgrad if wgrad else hdqt.gemm_dgrad

        def e2e_step():
            dA.copy_(hA, non_blocking=True)
            dB.copy_(hB, non_blocking=True)
            public_call(dA, dB, desc=case.desc, workspace=ws, dev_status=case.status, out=case.out)
            hOut.copy_(case.out, non_blocking=True)

        e2e_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(case.stream)
        for _ in range(e2e_steps):
            e2e_step()
        e1.record(case.stream)
        barrier()
        e2e_ms = max_over_ranks([e0.elapsed_time(e1)], dev, world)[0]
        e2e = {"value": whole_job_tops(world, e2e_steps, 2.0 * M * N * K, e2e_ms), "unit": UNIT,
               "h2d_bytes_per_step": hA.numel() * 4 + hB.numel() * 4, "d2h_bytes_per_step": hOut.numel() * 4,
               "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps}
        hdqt.check_device_status(case.status, "e2e")
        del hA, hB, hOut, dA, dB, ws

    elapsed_ms, quant_ms, gemm_ms = max_over_ranks([elapsed_ms, quant_ms, gemm_ms], dev, world)
    certified = case.certified_fraction() if rank == 0 else None
    # in-run yardstick: MMA-only loop of the GEMM's instruction shape on every SM (no loads, no epilogue)
    mma_probe_tops = hdqt.mma_rate_tops(dev_status=case.status) if rank == 0 else None

    sustained = clamp = supplied = None
    sweep, training = [], None
    if extras:
        # (ii) the same step looped for seconds, clocks and power sampled over the loop only
        s2 = ClockSampler(local_rank, period_ms=100)
        s2.start()
        time.sleep(0.2)
        n_loop = max(10, int(args.sustained_seconds * 1e3 / (elapsed_ms / args.steps)))
        el, q_ms, g_ms = case.timed(n_loop, 3)
        c2 = s2.stop()
        ops = 2.0 * M * N * K
        g_tops = ops / (g_ms * 1e-3) / 1e12
        sustained = {"seconds": el * 1e-3, "steps": n_loop, "value": ops * n_loop / (el * 1e-3) / 1e12,
                     "gemm_tops": g_tops, "gemm_frac_of_2x_bf16_sustained": g_tops / (2.0 * peaks["bf16_sustained"]),
                     "quantize_gbs": 9.0 * (M * K + N * K) / (q_ms * 1e-3) / 1e9, "clocks": c2,
                     "gemm_tops_scaled_to_max_clock": (g_tops * c2["sm_max_mhz"] / c2["sm_mhz"]) if c2.get("sm_mhz") else None}
        # 5 B/element mode: calibration maxima supplied by the caller (here: those just measured)
        amaxA = hdqt.absmax_hadamard(case.A)
        amaxB = hdqt.absmax_hadamard(case.B)
        _, q5_ms, _ = case.timed(min(args.steps, 30), 3, amax=(amaxA, amaxB))
        supplied = {"ms_per_step": q5_ms, "algorithmic_gb_per_step": 5.0 * (M * K + N * K) / 1e9,
                    "gbs": 5.0 * (M * K + N * K) / (q5_ms * 1e-3) / 1e9,
                    "frac": 5.0 * (M * K + N * K) / (q5_ms * 1e-3) / 1e9 / peaks["hbm"],
                    "note": "both operands with caller-supplied calibration maxima: FWHT/quantize pass only (5 B/elt)"}
        del case
        torch.cuda.empty_cache()
        # (iii) every tile through the 8-bit accumulator epilogue: what operands without clamp-free certificates get
        if merge:
            c = SweepCase(hdqt, inputs, torch, dev, size, args.layout, False, args.acc_tile, args.acc_bits)
            r = shape_record(c, max(3, min(args.steps, 10)), 3, peaks)
            clamp = {"bound": "tensor", "kernel": "gemm_i8_tiled_kernel (every tile through the accumulator epilogue)",
                     "achieved": r["gemm_tops"], "peak": 2.0 * peaks["bf16_burst"], "unit": "TOP/s",
                     "frac": r["gemm_frac"], "ms_per_launch": r["gemm_ms"], "whole_path_tops": r["value"],
                     "note": "same operands and shape as the headline, merging of certified tiles disabled"}
            del c
            torch.cuda.empty_cache()
        # (iv) the other corners of the sweep
        other = [(s, l) for s in (8192, 16384) for l in ("dgrad", "wgrad") if (s, l) != (size, args.layout)]
        for s_, l_ in other:
            c = SweepCase(hdqt, inputs, torch, dev, s_, l_, merge, args.acc_tile, args.acc_bits)
            sweep.append(shape_record(c, 30 if s_ <= 8192 else 12, 3, peaks))
            del c
            torch.cuda.empty_cache()
        training = train_steps_records(torch, dev)

    if rank == 0:
        int8_peak = 2.0 * peaks["bf16_burst"]
        peak_src = f"{peaks['source']} bf16 burst x2 (nominal int8:bf16 ratio); the kernel is timed by CUDA events in a short region"
        ops = 2.0 * M * N * K
        gemm_tops = ops / (gemm_ms * 1e-3) / 1e12
        quant_bytes = 9.0 * (M * K + N * K)      # 4 B calibration read + 4 B read + 1 B code written, per element
        line = {
            "metric": METRIC, "value": whole_job_tops(world, args.steps, ops, elapsed_ms), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": elapsed_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8/f32",
            "data": "synthetic", "config": workload_config(size, merge, args.layout, args.acc_tile, args.acc_bits),
            "roofline": {"bound": "tensor", "kernel": "hdqt_gemm_i8_tiled (pair kernel + fix-up + general kernel)",
                         "achieved": gemm_tops, "peak": int8_peak, "unit": "TOP/s", "frac": gemm_tops / int8_peak,
                         "peak_source": peak_src, "frac_of_datasheet_dense_int8": gemm_tops / DATASHEET_INT8_TOPS,
                         "mma_only_probe_tops": mma_probe_tops,
                         "frac_of_mma_only_probe": (gemm_tops / mma_probe_tops) if mma_probe_tops else None,
                         "traffic": None,
                         "traffic_note": "DRAM bytes of the GEMM kernels are captured with ncu on smaller shapes "
                                         "and do not scale linearly with the shape; they are listed per shape in "
                                         "the profile summaries, not pasted here",
                         "algorithmic_bytes": float(M * K + N * K + 4 * M * N),
                         "ms_per_launch": gemm_ms, "certified_clamp_free_tile_fraction": certified,
                         "depends_on_data": "tiles with a clamp-free certificate are merged on the tensor core; "
                                            "see roofline_clamp_path for operands without certificates"},
            "quantize": {"ms_per_step": quant_ms, "algorithmic_gb_per_step": quant_bytes / 1e9,
                         "gbs": quant_bytes / (quant_ms * 1e-3) / 1e9, "hbm_peak_gbs": peaks["hbm"],
                         "frac": quant_bytes / (quant_ms * 1e-3) / 1e9 / peaks["hbm"],
                         "note": "both operands: calibration pass (4 B/elt) + FWHT/quantize pass (5 B/elt)"},
            "clocks": clocks, "gpu_launches": args.steps * launches_per_step(M, N, merge, args.acc_bits),
        }
        if clamp is not None:
            line["roofline_clamp_path"] = clamp
        if supplied is not None:
            line["quantize_supplied_max"] = supplied
        if sustained is not None:
            line["sustained"] = sustained
        if sweep:
            line["sweep"] = sweep
        if training is not None:
            line["train_steps_per_s"] = training
        if e2e is not None:
            line["e2e"] = e2e
        if not args.skip_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(size, args.layout)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_training_report(args):
    """Training report of its own: `mlp` / `cnn` steps per second, `cil` the full class-incremental run (5 tasks x
    20 classes, replay memory 2000, 64 new + 64 replayed samples per batch) for the quantized path and for fp32
    torch from the same seed, with the accuracy after every task."""
    import torch
    from paper_2310_03675_b200 import nn as hnn
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    if args.workload in ("mlp", "cnn"):
        rec = train_steps_records(torch, dev, steps=max(10, min(args.steps, 50)))
        key = "mlp_1152_512_256_12_batch256" if args.workload == "mlp" else "cnn_resnet18w_32x32_batch128"
        print(json.dumps({"metric": f"hdqt_{args.workload}_train_steps_per_s", "value": rec[key]["hdqt"]["steps_per_s"],
                          "unit": "steps/s", "n_gpus": 1, "higher_is_better": True, "data": "synthetic",
                          "config": {"workload": key}, "train_steps_per_s": rec}))
        return
    out = {}
    for name, quantized, extra in (("hdqt", True, {}),
                                   ("hdqt_cuda_graph_delayed_scaling", True, {"graphed": True, "delayed": True}),
                                   ("fp32_torch", False, {})):
        hnn.reset_delayed_scaling()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        res = hnn.class_incremental_run(quantized, dev, steps_per_task=args.steps_per_task, seed=0,
                                        log=lambda m, n=name: print(f"[{n}] {m}", file=sys.stderr), **extra)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        res["steps_per_s_end_to_end"] = res["steps"] / dt
        res["seconds"] = dt
        out[name] = res
    print(json.dumps({"metric": "hdqt_class_incremental_steps_per_s", "value": out["hdqt"]["steps_per_s_end_to_end"],
                      "unit": "steps/s", "n_gpus": 1, "higher_is_better": True, "data": "synthetic",
                      "config": {"workload": "class-incremental ResNet-18-width: 5 tasks x 20 synthetic classes, "
                                             f"{args.steps_per_task} steps per task, replay memory 2000, batch 64 new + 64 "
                                             "replayed, SGD lr 0.05 momentum 0.9 wd 2e-4, 4-bit inputs / 8-bit accumulators"},
                      "hdqt": out["hdqt"], "hdqt_cuda_graph_delayed_scaling": out["hdqt_cuda_graph_delayed_scaling"],
                      "fp32_torch": out["fp32_torch"]}))


def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def main():
    args = parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # plain `python bench.py --gpus N`: start the N replica processes ourselves
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    if args.impl == "reference":
        run_reference(args)
    elif args.workload != "sweep":
        run_training_report(args)
    else:
        run_hdqt(args)


if __name__ == "__main__":
    main()
