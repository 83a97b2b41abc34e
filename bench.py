#!/usr/bin/env python
"""Benchmark of the W4A4 + low-rank linear forward on synthetic DiT-shaped inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload attn_proj|ffn_up|ffn_down|tiny]
                    [--impl ours|reference]

A step is one pass of the whole layer (activation kernel + GEMM kernel) over one batch of M tokens.
`value` is effective TOPS = 2*M*K*N / step time with the inputs already resident in HBM; `e2e` is the
same metric with the activations starting in pinned host memory and the output read back, copies inside
the timed region.  Rank 0 prints exactly one JSON line.  With N > 1 every rank runs an independent
replica on its own GPU (token rows are independent; there is no data-path collective).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import generator as gen  # noqa: E402

METRIC = "w4a4_lowrank_linear_effective_tops"
UNIT = "TOPS"
NOMINAL_INT8_TOPS = 4500.0
NOMINAL_HBM_GBS = 7700.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch, each from one single-launch ncu capture of the kernel as
# it stands (summaries under profiles/); None where no capture exists for that kernel and workload.
NCU_TRAFFIC_BYTES = {("gemm", "attn_proj"): 545.9e6, ("quantize", "attn_proj"): 503.3e6}


def max_over_ranks(ms: float, dist, device="cpu") -> float:
    """Device time of the slowest rank (the whole job is as slow as its slowest replica)."""
    if dist is None:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tops(ops_per_step_per_rank: float, world: int, ms_per_step: float) -> float:
    """Aggregate effective TOPS of `world` independent replicas that each do ops_per_step_per_rank per step."""
    return world * ops_per_step_per_rank / (ms_per_step * 1e-3) / 1e12


def dit_step_layers(blocks: int = 40, qkv_packed: bool = False):
    """(K, N, r) of the quantized linears of one denoising step: per block q, k, v, o, cross q, cross o, ffn up,
    ffn down at r = 32.  With qkv_packed the self-attention q, k and v (one input, one smoothing vector, one clip entry)
    are one layer 5120 -> 15360 of joint rank 96 whose L2 is block-diagonal: one activation pass instead of three."""
    if qkv_packed:
        per_block = [(5120, 15360, 96)] + [(5120, 5120, 32)] * 3 + [(5120, 13824, 32), (13824, 5120, 32)]
    else:
        per_block = [(5120, 5120, 32)] * 6 + [(5120, 13824, 32), (13824, 5120, 32)]
    return per_block * blocks


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_burst=float(p["bf16_tflops"]),
                    bf16_sustained=float(p["bf16_tflops_sustained"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


def _time_loop(fn, stream, seconds: float):
    """(best single-call ms over 10 calls, mean ms of calls issued back to back for about `seconds`)."""
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    best = float("inf")
    for _ in range(10):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        fn()
        e1.record(stream)
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    reps = max(10, int(seconds * 1e3 / best))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(reps):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return best, e0.elapsed_time(e1) / reps


def measure_tensor_peaks(dev, seconds: float = 3.0):
    """Dense 8-bit tensor-core peaks of this GPU from library GEMMs (8192^3), taken the way MEASURED_PEAKS.json's
    BF16 figures were: best of 10 calls (burst) and a seconds-long back-to-back loop (sustained).  Library calls are
    fine for a peak probe; nothing here is on the layer's path or inside a timed region of it."""
    n = 8192
    ops = 2.0 * n ** 3
    stream = torch.cuda.current_stream()
    out = {}
    try:
        a = torch.randn(n, n, device=dev).to(torch.float8_e4m3fn)
        b = torch.randn(n, n, device=dev).to(torch.float8_e4m3fn).t()
        one = torch.ones((), device=dev, dtype=torch.float32)
        best, mean = _time_loop(lambda: torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16), stream, seconds)
        out["fp8_tops_burst"], out["fp8_tops_sustained"] = ops / (best * 1e-3) / 1e12, ops / (mean * 1e-3) / 1e12
        del a, b
    except Exception as e:  # noqa: BLE001
        out["fp8_error"] = repr(e)[:200]
    try:
        a = torch.randint(-8, 8, (n, n), device=dev, dtype=torch.int8)
        b = torch.randint(-8, 8, (n, n), device=dev, dtype=torch.int8).t().contiguous().t()
        best, mean = _time_loop(lambda: torch._int_mm(a, b), stream, seconds)
        out["int8_tops_burst"], out["int8_tops_sustained"] = ops / (best * 1e-3) / 1e12, ops / (mean * 1e-3) / 1e12
        del a, b
    except Exception as e:  # noqa: BLE001
        out["int8_error"] = repr(e)[:200]
    out["how"] = "torch._scaled_mm (E4M3) and torch._int_mm (INT8) at 8192^3: best of 10 and a %.0f s back-to-back loop" % seconds
    torch.cuda.empty_cache()
    return out


def tensor_roofline(gemm_tops: float, timed_seconds: float, peaks: dict, tp: dict, fp4: bool = False) -> dict:
    """Fractions of the dense tensor peak of the contraction's own type.  8-bit (the INT4-exact path runs on the FP8
    pipe): the FP8 figures measured in this run when they exist, else 2 x the measured BF16 figures (nominal ratio).
    FP4 (the MXFP4 variant): no library FP4 GEMM is timed, so 2 x the 8-bit figure (nominal ratio 9 : 4.5).  The burst
    figure serves a timed region shorter than a second, the sustained one a longer region."""
    if tp and "fp8_tops_burst" in tp:
        burst, sustained, src = tp["fp8_tops_burst"], tp["fp8_tops_sustained"], "library FP8 GEMM 8192^3 measured in this run"
    else:
        burst, sustained = 2.0 * peaks["bf16_burst"], 2.0 * peaks["bf16_sustained"]
        src = f"{peaks['source']} BF16 figures x 2 (nominal 8-bit : BF16 ratio; no 8-bit library GEMM was timed in this run)"
    nominal = NOMINAL_INT8_TOPS
    if fp4:
        burst, sustained, nominal, src = 2.0 * burst, 2.0 * sustained, 2.0 * NOMINAL_INT8_TOPS, src + ", x 2 (nominal FP4 : 8-bit ratio)"
    use_burst = timed_seconds < 1.0
    peak = burst if use_burst else sustained
    out = dict(bound="tensor", achieved=gemm_tops, peak=peak, unit="TOP/s", frac=gemm_tops / peak,
               peak_kind="burst" if use_burst else "sustained", peak_source=src,
               frac_burst=gemm_tops / burst, frac_sustained=gemm_tops / sustained)
    out["frac_of_nominal_%d" % nominal] = gemm_tops / nominal
    return out


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except Exception:
                pass
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except Exception:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        busy = [c for c in sm if c > 500] or sm
        return dict(sm_mhz=statistics.median(busy) if busy else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def workload_inputs(name: str, device, n_buffers: int):
    shp = gen.CONFIG_SHAPES[name]
    M, K, N, r = shp["M"], shp["K"], shp["N"], shp["r"]
    num_bins = 8 if name != "tiny" else 1
    if name == "tiny":
        idx = gen.outlier_channels(K, 0, 0, count=4)
        xs = [gen.make_activations(M, K, outlier_idx=idx, outlier_gain=40.0, seed=s, device=device) for s in range(n_buffers)]
        layer = gen.make_layer_svd(K, N, r, xs[0], seed=1, device=device, keep_float64=False)
        clip = torch.full((1, 1, 1), 0.9, dtype=torch.float32)
        bins = [0] * n_buffers
    else:
        dist = "gelu" if name == "ffn_down" else "normal"
        gain = 80.0 if name == "ffn_down" else 50.0
        idx = gen.outlier_channels(K, 0.01, 2)
        bins = [b % num_bins for b in range(n_buffers)]
        sig = (lambda b: 1.0) if dist == "gelu" else gen.sigma_for_bin
        calib = gen.make_activations(1024, K, sigma=sig(0), outlier_idx=idx, outlier_gain=gain, dist=dist, seed=2000,
                                     device=device)
        layer = gen.make_layer_svd(K, N, r, calib, seed=2001, bias_std=0.01, device=device, exact_svd=False,
                                   keep_float64=False)
        xs = [gen.make_activations(M, K, sigma=sig(b), outlier_idx=idx, outlier_gain=gain, dist=dist, seed=2002 + i,
                                   device=device) for i, b in enumerate(bins)]
        clip = gen.make_clip_table(1, 1, num_bins, [(0.6, 1.0)], seed=2)
    return dict(M=M, K=K, N=N, r=r, xs=xs, bins=bins, layer=layer, clip=clip, num_bins=num_bins)


def bits(t):
    return gen.bf16_bits(t.cpu()).numpy().view(np.uint16)


def oracle_time_rows(w, n_rows: int, seed: int = 0):
    """Times the CPU oracle (as it stands, one thread) on n_rows sampled rows.  Returns seconds."""
    import oracle  # test infrastructure; allowed here for the CPU-baseline / reference leg only

    lay = w["layer"]
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(w["M"], size=min(n_rows, w["M"]), replace=False))
    x = w["xs"][0][torch.from_numpy(rows).to(w["xs"][0].device)].cpu()
    rho = float(w["clip"][0, 0, w["bins"][0]])
    args = (bits(x), np.arange(len(rows), dtype=np.int32), lay.lam.cpu().numpy(), rho,
            bits(lay.L1) if lay.r > 0 else None, bits(lay.L2) if lay.r > 0 else None, lay.qweight.cpu().numpy(),
            lay.wscale.cpu().numpy(), None if lay.bias is None else lay.bias.cpu().numpy())
    t0 = time.perf_counter()
    oracle.forward_rows(*args)
    return time.perf_counter() - t0, len(rows)


def cpu_baseline(w, target_seconds: float = 12.0):
    t_probe, n_probe = oracle_time_rows(w, 4)
    per_row = t_probe / n_probe
    n = int(max(4, min(w["M"], target_seconds / max(per_row, 1e-9))))
    t, n = oracle_time_rows(w, n, seed=1)
    tops = 2.0 * n * w["K"] * w["N"] / t / 1e12
    return dict(value=tops, unit=UNIT, cores=1, kind="oracle",
                sample=f"{n} sampled token rows of the same workload, all {w['N']} output columns, "
                       f"{t:.1f} s single thread ({t / n * 1e3:.2f} ms/row; whole batch extrapolates to "
                       f"{t / n * w['M']:.0f} s)",
                host_cores=os.cpu_count())


def run_reference(args, rank):
    """--impl reference: the CPU oracle timed on host cores; each step is a bounded row sample."""
    if rank != 0:
        return
    if args.workload.startswith("gptq"):
        run_reference_gptq(args)
        return
    if args.workload not in gen.CONFIG_SHAPES:
        print(json.dumps(dict(impl="reference", unavailable="the reference arm (the CPU oracle) covers the single-layer "
                              "workloads and gptq*; %s has no oracle-timed counterpart" % args.workload)), flush=True)
        return
    w = workload_inputs(args.workload, "cpu" if not torch.cuda.is_available() else "cuda:0", 1)
    t_probe, n_probe = oracle_time_rows(w, 2)
    budget = 90.0 / max(1, args.steps + args.warmup)
    n = int(max(1, min(w["M"], budget / max(t_probe / n_probe, 1e-9))))
    for i in range(args.warmup):
        oracle_time_rows(w, n, seed=100 + i)
    times = [oracle_time_rows(w, n, seed=200 + i)[0] for i in range(args.steps)]
    total = sum(times)
    value = 2.0 * n * w["K"] * w["N"] * args.steps / total / 1e12
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=total / args.steps * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic", impl="reference",
                config=dict(workload=args.workload, M=w["M"], K=w["K"], N=w["N"], r=w["r"], group=64,
                            rows_per_step=n),
                cpu_baseline=dict(value=value, unit=UNIT, cores=1, kind="oracle",
                                  sample=f"{n} sampled token rows per step, all output columns"),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line), flush=True)


def run_reference_gptq(args):
    """--impl reference for the gptq workloads: the FP64 oracle on host cores.  A step is the full statistic, its
    inverse and Cholesky factor, and the sweep on a sample of 32 output channels (the sweep over all of them would take
    minutes; the part that does not depend on the output channels is done in full)."""
    import oracle  # test infrastructure; allowed here for the reference leg only

    K, N = {"gptq": (5120, 5120), "gptq_mx": (5120, 5120), "gptq_ffn_up": (5120, 13824),
            "gptq_ffn_down": (13824, 5120)}[args.workload]
    M_cal = 2048
    sweep = oracle.gptq_quantize_mx if args.workload == "gptq_mx" else oracle.gptq_quantize
    R, xhat = gen.make_gptq_inputs(K, N, M_cal, seed=7)
    cols = list(range(0, N, N // 32))[:32]
    Rs, xb = R[:, cols].double().numpy(), bits(xhat)
    steps, warmup = max(1, min(args.steps, 5)), min(args.warmup, 1)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        sweep(Rs, oracle.gptq_hessian(xb))
        if i >= warmup:
            times.append((time.perf_counter() - t0) * 1e3)
    ms = statistics.median(times)
    sample = "the full statistic and its inverse, the sweep on 32 of the %d output channels" % N
    print(json.dumps(dict(
        metric="gptq_layer_time", value=ms, unit="ms", n_gpus=args.gpus, steps=steps, warmup=warmup, ms_per_step=ms,
        higher_is_better=False, scaling="weak", vs_baseline=None, dtype="f64", data="synthetic", impl="reference",
        config=dict(workload=args.workload, K=K, N=N, calibration_tokens=M_cal, group=64, percdamp=0.01),
        cpu_baseline=dict(value=ms, unit="ms", cores=torch.get_num_threads(), kind="oracle", sample=sample),
        e2e=dict(value=ms, unit="ms", h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)), flush=True)


def time_layer(w4, layer, xs, bins, expert, clip, Y, M, iters, warmup, stream):
    """Mean (quantize ms, gemm ms) of one layer over `iters` forwards, CUDA events on `stream`."""
    for i in range(warmup):
        w4.w4a4_linear_forward(layer.ptr, xs[i % len(xs)], M, expert, bins[i % len(xs)], clip, Y, stream)
    torch.cuda.synchronize()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(iters)]
    for i in range(iters):
        b = i % len(xs)
        ev[i][0].record(stream)
        w4.w4a4_quantize_activations(layer.ptr, xs[b], M, expert, bins[b], clip, stream)
        ev[i][1].record(stream)
        w4.w4a4_gemm_from_workspace(layer.ptr, M, expert, Y, stream)
        ev[i][2].record(stream)
    torch.cuda.synchronize()
    return (statistics.mean(e[0].elapsed_time(e[1]) for e in ev), statistics.mean(e[1].elapsed_time(e[2]) for e in ev))


def measure_dit_step(w4, dev, local_rank, steps, warmup, blocks, dist=None, qkv_packed=False):
    """One denoising step's quantized linears of a `blocks`-block, 5120-hidden DiT at M = 32760, r = 32, with both
    experts' weight sets resident; step s uses expert (s >= 20) and timestep bin s // 5 (40-step schedule).
    Returns this rank's device time per step and what the step holds."""
    M, r, bins, experts = 32760, 32, 8, 2
    shapes = dit_step_layers(blocks, qkv_packed)
    L = len(shapes)
    ctx = w4.Context(local_rank, M, 13824, 96 if qkv_packed else r)
    layers = []
    for li, (K, N, rl) in enumerate(shapes):
        ex = [gen.make_layer_direct(K, N, rl, seed=4000 + 2 * li + e, device=dev) for e in range(experts)]
        if rl == 96:  # three projections side by side: each reads only its own 32 columns of T
            for lay in ex:
                for i in range(3):
                    for j in range(3):
                        if i != j:
                            lay.L2[32 * i:32 * (i + 1), 5120 * j:5120 * (j + 1)] = 0
        layers.append(w4.Layer(ctx, ex, num_bins=bins, num_layers=L, layer_id=li))
        del ex
    weight_bytes = sum(w4.w4a4_handle_bytes(l.ptr) for l in layers)
    clip = gen.make_clip_table(experts, L, bins, [(0.6, 1.0), (0.8, 1.0)], seed=4).to(dev)
    idx = {K: gen.outlier_channels(K, 0.01, 40 + K) for K in (5120, 13824)}
    xs = {5120: [gen.make_activations(M, 5120, sigma=1.0, outlier_idx=idx[5120], outlier_gain=50.0, seed=4100 + i,
                                      device=dev) for i in range(3)],
          13824: [gen.make_activations(M, 13824, dist="gelu", outlier_idx=idx[13824], outlier_gain=80.0, seed=4200 + i,
                                       device=dev) for i in range(3)]}
    Y = {n: torch.empty(M, n, dtype=torch.bfloat16, device=dev) for n in (5120, 13824, 15360)[:3 if qkv_packed else 2]}
    stream = torch.cuda.current_stream()

    def step(s):
        expert, b = (1 if (s % 40) >= 20 else 0), (s % 40) // 5
        for li, (K, N, _) in enumerate(shapes):
            w4.w4a4_linear_forward(layers[li].ptr, xs[K][(s + li) % 3], M, expert, b, clip, Y[N], stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for s in range(warmup):
        step(s)
    barrier()
    ctx.check()
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for s in range(steps):
        step(18 + s)  # straddles the expert switch at step 20
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    ctx.check()
    total_ms = e0.elapsed_time(e1)
    for l in layers:
        l.close()
    ctx.close()
    del xs, Y
    torch.cuda.empty_cache()
    return dict(total_ms=total_ms, ops=sum(2.0 * M * K * N for (K, N, _) in shapes), M=M, r=r, experts=experts, bins=bins,
                linears=L, weight_bytes=weight_bytes, clocks=clocks, qkv_packed=qkv_packed)


def run_dit_step(args, w4, dev, local_rank, rank, world, dist, peaks, tp):
    d = measure_dit_step(w4, dev, local_rank, args.steps, args.warmup, args.blocks, dist, args.qkv_packed)
    total_ms = max_over_ranks(d["total_ms"], dist, dev)
    ms_per_step = total_ms / args.steps
    if rank == 0:
        tops = whole_job_tops(d["ops"], world, ms_per_step)
        roof = tensor_roofline(tops / world, total_ms * 1e-3, peaks, tp)
        roof.update(traffic=None, kernel="quantize + expand + gemm of every layer, whole step")
        line = dict(metric=METRIC, value=tops, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                    ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="e4m3",
                    data="synthetic",
                    config=dict(workload="dit_step", M=d["M"], r=d["r"], group=64, blocks=args.blocks, linears=d["linears"],
                                qkv="one packed layer 5120 -> 15360, joint rank 96" if d["qkv_packed"] else "three layers",
                                experts=d["experts"], bins=d["bins"], resident_weight_gb=d["weight_bytes"] / 1e9,
                                tera_ops_per_step=d["ops"] / 1e12,
                                l2="inputs larger than L2: 3 rotating activation buffers per shape (335 / 906 MB)",
                                parallelism="replicas" if world > 1 else "single"),
                    ms_per_dit_step=ms_per_step, roofline=roof, tensor_peaks=tp,
                    gpu_launches=3 * d["linears"] * args.steps, clocks=d["clocks"])
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def measure_single_layer(w4, dev, local_rank, name, iters, warmup):
    """Mean kernel times of one of the single-layer workloads (used for the second shape the performance target names)."""
    w = workload_inputs(name, dev, 3)
    M, K, N, r = w["M"], w["K"], w["N"], w["r"]
    ctx = w4.Context(local_rank, M, K, r)
    layer = w4.Layer(ctx, [w["layer"]], num_bins=w["num_bins"])
    clip = w["clip"].to(dev)
    Y = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
    tq, tg = time_layer(w4, layer, w["xs"], w["bins"], 0, clip, Y, M, iters, warmup, torch.cuda.current_stream())
    ctx.check()
    layer.close()
    ctx.close()
    del w, Y
    torch.cuda.empty_cache()
    return dict(M=M, K=K, N=N, r=r, quantize_ms=tq, gemm_ms=tg, iters=iters)


def run_sweep(args, w4, dev, local_rank, rank, peaks, tp):
    """Shape sweep: M x (K, N) x r x outlier fraction x clip ratio, TOPS and roofline fractions per point."""
    if rank != 0:
        return
    int8_peak = tp.get("fp8_tops_sustained", 2.0 * peaks["bf16_sustained"])   # hours of back-to-back kernels: the sustained figure
    rows = []
    stream = torch.cuda.current_stream()
    for (K, N) in ((5120, 5120), (5120, 13824), (13824, 5120)):
        for r in (0, 16, 32, 64):
            for M in (1560, 32760, 75600):
                ctx = w4.Context(local_rank, M, K, r)
                layer = w4.Layer(ctx, [gen.make_layer_direct(K, N, r, seed=5000 + r + K // 64, device=dev)], num_bins=2)
                clip = torch.tensor([[[0.7, 1.0]]], dtype=torch.float32, device=dev)
                Y = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
                for frac in (0.0, 0.01, 0.05):
                    n_x = 2 if M * K * 2 > 64e6 else 4
                    xs = [gen.make_activations(M, K, outlier_idx=gen.outlier_channels(K, frac, 50 + i), outlier_gain=50.0,
                                               seed=5100 + i, device=dev) for i in range(n_x)]
                    for b, alpha in ((0, 0.7), (1, 1.0)):
                        tq, tg = time_layer(w4, layer, xs, [b] * n_x, 0, clip, Y, M, args.steps, max(3, args.warmup), stream)
                        ops = 2.0 * M * K * N
                        qb = M * (2.5625 * K + 2.0 * r)   # X, 4-bit codes, FP32 scales, BF16 T: the bytes the step needs, not the layout's
                        rows.append(dict(M=M, K=K, N=N, r=r, outlier_fraction=frac, alpha=alpha, quantize_ms=tq, gemm_ms=tg,
                                         layer_tops=ops / ((tq + tg) * 1e-3) / 1e12, gemm_tops=ops / (tg * 1e-3) / 1e12,
                                         gemm_frac=ops / (tg * 1e-3) / 1e12 / int8_peak,
                                         quantize_gbs=qb / (tq * 1e-3) / 1e9, quantize_frac=qb / (tq * 1e-3) / 1e9 / peaks["hbm_gbs"]))
                    del xs
                ctx.check()
                layer.close()
                ctx.close()
                del Y
                torch.cuda.empty_cache()
    out = args.out or os.path.join(ROOT, "bench_out", "sweep.json")
    os.makedirs(os.path.dirname(out), exist_ok=True)
    with open(out, "w") as f:
        json.dump(rows, f)
    best = max(rows, key=lambda x: x["gemm_tops"])
    print(json.dumps(dict(metric=METRIC, unit=UNIT, value=statistics.mean(x["layer_tops"] for x in rows), n_gpus=1,
                          steps=args.steps, warmup=args.warmup, higher_is_better=True, scaling="weak", vs_baseline=None,
                          dtype="e4m3", data="synthetic", config=dict(workload="sweep", points=len(rows), table=out),
                          best_point=best, gpu_launches=3 * args.steps * len(rows))), flush=True)


def run_mxfp4(args, w4, dev, local_rank, rank, peaks, tp):
    """The MXFP4 variant of the layer (E2M1 elements, E8M0 block scales applied inside the tensor core) on the
    shape of one of the single-layer workloads: `--workload mxfp4_attn_proj | mxfp4_ffn_up | mxfp4_ffn_down`."""
    if rank != 0:
        return
    name = args.workload[len("mxfp4_"):]
    shp = gen.CONFIG_SHAPES[name]
    M, K, N, r = shp["M"], shp["K"], shp["N"], shp["r"]
    num_bins, n_buf = 8, 4
    dist = "gelu" if name == "ffn_down" else "normal"
    gain = 80.0 if name == "ffn_down" else 50.0
    idx = gen.outlier_channels(K, 0.01, 2)
    sig = (lambda b: 1.0) if dist == "gelu" else gen.sigma_for_bin
    lay = gen.make_layer_mx_direct(K, N, r, seed=2001, device=dev)
    bins = [b % num_bins for b in range(n_buf)]
    xs = [gen.make_activations(M, K, sigma=sig(b), outlier_idx=idx, outlier_gain=gain, dist=dist, seed=2002 + i, device=dev)
          for i, b in enumerate(bins)]
    clip = gen.make_clip_table(1, 1, num_bins, [(0.6, 1.0)], seed=2).to(dev)
    ctx = w4.Context(local_rank, M, K, r)
    layer = w4.MxLayer(ctx, [lay], num_bins=num_bins)
    Y = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.current_stream()
    for i in range(max(3, args.warmup)):
        w4.w4a4_mx_linear_forward(layer.ptr, xs[i % n_buf], M, 0, bins[i % n_buf], clip, Y, stream)
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        w4.w4a4_mx_linear_forward(layer.ptr, xs[i % n_buf], M, 0, bins[i % n_buf], clip, Y, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(min(args.steps, 50))]
    for i, e in enumerate(ev):
        e[0].record(stream)
        w4.w4a4_mx_quantize_activations(layer.ptr, xs[i % n_buf], M, 0, bins[i % n_buf], clip, stream)
        e[1].record(stream)
        w4.w4a4_mx_gemm_from_workspace(layer.ptr, M, 0, Y, stream)
        e[2].record(stream)
    torch.cuda.synchronize()
    ctx.check()
    tq = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    tg = statistics.mean(e[1].elapsed_time(e[2]) for e in ev)
    ops = 2.0 * M * K * N
    gemm_tops = ops / (tg * 1e-3) / 1e12
    roof = tensor_roofline(gemm_tops, tg * 1e-3 * len(ev), peaks, tp, fp4=True)
    roof.update(traffic=None, kernel="mx_gemm2_kernel (CTA pairs; mx_gemm_kernel when M <= 128)", ms=tg)
    q_bytes = M * (2.0 * K + K / 2.0 + K / 32.0 + 4.0 * r)  # X read, packed codes, scale bytes, T hi | lo
    print(json.dumps(dict(
        metric=METRIC, value=ops / (ms * 1e-3) / 1e12, unit=UNIT, n_gpus=1, steps=args.steps, warmup=args.warmup,
        ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="e2m1 x e8m0 (mxfp4)",
        data="synthetic",
        config=dict(workload=args.workload, M=M, K=K, N=N, r=r, block=32, experts=1, bins=num_bins,
                    l2="inputs larger than L2: 4 rotating activation buffers of %.0f MB" % (M * K * 2 / 1e6)),
        roofline=roof,
        roofline_quantize=dict(bound="hbm", achieved=q_bytes / (tq * 1e-3) / 1e9, peak=peaks["hbm_gbs"], unit="GB/s",
                               frac=q_bytes / (tq * 1e-3) / 1e9 / peaks["hbm_gbs"], kernel="quantize_kernel (MXFP4 format)",
                               ms=tq, algorithmic_bytes=q_bytes, peak_source=peaks["source"]),
        kernel_ms=dict(quantize_mean=tq, gemm_mean=tg), e2e=None, gpu_launches=2 * args.steps, clocks=clocks)), flush=True)
    layer.close()
    ctx.close()


def run_mxfp4_ffn(args, w4, dev, local_rank, rank, peaks, tp):
    """The FFN of the MXFP4 variant, 5120 -> 13824 (GELU) -> 5120 at M = 32760: the fused call (the up-projection's
    epilogue quantizes for the down-projection; the hidden activation never reaches memory) against the same two
    layers as two calls (`--workload mxfp4_ffn`)."""
    if rank != 0:
        return
    up_s, dn_s = gen.CONFIG_SHAPES["ffn_up"], gen.CONFIG_SHAPES["ffn_down"]
    M, K, H, N, r = up_s["M"], up_s["K"], up_s["N"], dn_s["N"], up_s["r"]
    num_bins, n_buf = 8, 4
    idx = gen.outlier_channels(K, 0.01, 2)
    up = gen.make_layer_mx_direct(K, H, r, seed=2101, device=dev)
    down = gen.make_layer_mx_direct(H, N, r, seed=2102, device=dev)
    bins = [b % num_bins for b in range(n_buf)]
    xs = [gen.make_activations(M, K, sigma=gen.sigma_for_bin(b), outlier_idx=idx, outlier_gain=50.0, seed=2103 + i, device=dev)
          for i, b in enumerate(bins)]
    clip = gen.make_clip_table(1, 2, num_bins, [(0.6, 1.0)], seed=2).to(dev)
    ctx = w4.Context(local_rank, M, max(K, H), r)
    l_up = w4.MxLayer(ctx, [up], num_bins=num_bins, num_layers=2, layer_id=0, output_activation=w4.ACT_GELU_TANH)
    l_dn = w4.MxLayer(ctx, [down], num_bins=num_bins, num_layers=2, layer_id=1)
    hidden = torch.empty(M, H, dtype=torch.bfloat16, device=dev)
    Y = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.current_stream()

    def fused(i):
        w4.w4a4_mx_ffn_forward(l_up.ptr, l_dn.ptr, xs[i % n_buf], M, 0, bins[i % n_buf], clip, Y, stream)

    def two_calls(i):
        w4.w4a4_mx_linear_forward(l_up.ptr, xs[i % n_buf], M, 0, bins[i % n_buf], clip, hidden, stream)
        w4.w4a4_mx_linear_forward(l_dn.ptr, hidden, M, 0, bins[i % n_buf], clip, Y, stream)

    def timed(fn):
        for i in range(max(3, args.warmup)):
            fn(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(args.steps):
            fn(i)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.steps

    ms_two = timed(two_calls)
    sampler = ClockSampler(local_rank)
    sampler.start()
    ms = timed(fused)
    clocks = sampler.stop()
    ctx.check()
    ops = 2.0 * M * K * H + 2.0 * M * H * N
    roof = tensor_roofline(ops / (ms * 1e-3) / 1e12, ms * 1e-3 * args.steps, peaks, tp, fp4=True)
    roof.update(traffic=None, kernel="whole fused call: quantize, mx_gemm2_kernel<fused epilogue>, T finish, mx_gemm2_kernel")
    print(json.dumps(dict(
        metric=METRIC, value=ops / (ms * 1e-3) / 1e12, unit=UNIT, n_gpus=1, steps=args.steps, warmup=args.warmup,
        ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="e2m1 x e8m0 (mxfp4)",
        data="synthetic",
        config=dict(workload=args.workload, M=M, K=K, hidden=H, N=N, r=r, block=32, activation="gelu_tanh",
                    l2="inputs larger than L2: 4 rotating activation buffers of %.0f MB" % (M * K * 2 / 1e6)),
        roofline=roof,
        two_calls=dict(ms_per_step=ms_two, value=ops / (ms_two * 1e-3) / 1e12, unit=UNIT,
                       note="same layers as w4a4_mx_linear_forward twice (hidden activation stored and re-read)"),
        e2e=None, gpu_launches=5 * args.steps, clocks=clocks)), flush=True)
    l_up.close()
    l_dn.close()
    ctx.close()


def mxfp4_context(w4, ctx, w, clip, Y, stream, iters: int = 20):
    """The same layer shape through the MXFP4 variant (E2M1 elements, E8M0 block scales applied inside the tensor
    core), timed on the buffers of the main run: a different quantizer, reported for context, never part of `value`."""
    M, K, N, r = w["M"], w["K"], w["N"], w["r"]
    lay = w4.MxLayer(ctx, [gen.make_layer_mx_direct(K, N, r, seed=2001, device=Y.device)], num_bins=w["num_bins"])
    xs, bins = w["xs"], w["bins"]
    for i in range(3):
        w4.w4a4_mx_linear_forward(lay.ptr, xs[i % len(xs)], M, 0, bins[i % len(xs)], clip, Y, stream)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for i in range(iters):
        w4.w4a4_mx_linear_forward(lay.ptr, xs[i % len(xs)], M, 0, bins[i % len(xs)], clip, Y, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    ctx.check()
    ms = e0.elapsed_time(e1) / iters
    lay.close()
    return dict(value=2.0 * M * K * N / (ms * 1e-3) / 1e12, unit=UNIT, ms_per_step=ms, steps=iters,
                note="MXFP4 variant of the same layer shape (w4a4_mx_linear_forward): a different quantizer, for context only")


def run_clip_search(args, w4, dev, local_rank, rank, peaks):
    """Clipping-ratio search (Eq. 10) at the attention-projection shape: six candidates, two calibration samples
    per search; every candidate runs the real forward with the squared error fused into the GEMM epilogue."""
    if rank != 0:
        return
    shape = gen.CONFIG_SHAPES["attn_proj"]
    M, K, N, r = shape["M"], shape["K"], shape["N"], shape["r"]
    cands = [0.5, 0.6, 0.7, 0.8, 0.9, 1.0]
    n_samples = 2
    lay = gen.make_layer_direct(K, N, r, seed=7000, device=dev)
    idx = gen.outlier_channels(K, 0.01, 7001)
    xs = [gen.make_activations(M, K, sigma=gen.sigma_for_bin(3), outlier_idx=idx, outlier_gain=50.0, seed=7002 + i, device=dev)
          for i in range(n_samples)]
    ys = [gen.reference_output(x, lay) for x in xs]
    ctx = w4.Context(local_rank, M, K, r)
    layer = w4.Layer(ctx, [lay], num_bins=8)
    table = torch.ones((1, 1, 8), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    for _ in range(max(1, min(args.warmup, 2))):
        w4.w4a4_clip_search(layer.ptr, xs, ys, M, 0, 3, cands, table)
    searches = max(1, min(args.steps, 5))
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(searches):
        best, errs = w4.w4a4_clip_search(layer.ptr, xs, ys, M, 0, 3, cands, table)
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / searches
    forwards = len(cands) * n_samples
    ctx.check()
    print(json.dumps(dict(
        metric=METRIC, value=2.0 * M * K * N * forwards / (ms * 1e-3) / 1e12, unit=UNIT, n_gpus=1, steps=searches,
        warmup=args.warmup, ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="e4m3",
        data="synthetic",
        config=dict(workload="clip_search", M=M, K=K, N=N, r=r, candidates=cands, samples=n_samples,
                    l2="inputs larger than L2: activations and reference outputs of %.0f MB each" % (M * K * 2 / 1e6)),
        ms_per_forward=ms / forwards, best_candidate=cands[best], objective=errs,
        gpu_launches=(2 * forwards + 2) * searches, clocks=clocks)), flush=True)
    layer.close()
    ctx.close()


def gptq_launch_count(K: int, nb: int = 64, band: int = 512, lazy: int = 256) -> int:
    """Kernel launches of one w4a4_gptq_quantize call with calibration activations: the library's loop structure
    (conversion, statistic, diagonal fix-ups, weight copy; banded factorization; banded triangular inverse; sweep in
    lazy batches), counting only launches that have work."""
    n = 5
    hi = K
    while hi > 0:                                   # H = V V^T
        lo = max(0, hi - band)
        for j0 in range(hi - nb, lo - 1, -nb):
            n += 1                                  # diagonal block
            if j0 == 0:
                break
            n += 1 + (1 if j0 > lo else 0)          # panel, in-band update
        n += 1 if lo > 0 else 0
        hi = lo
    hi = K
    while hi > 0:                                   # U = V^-1
        lo = max(0, hi - band)
        n += 1                                      # the band's diagonal inverses
        n += 2 * len(range(hi - 2 * nb, lo - 1, -nb))
        n += 2 if K - hi > 0 else 0
        hi = lo
    for b0 in range(0, K, lazy):                    # sweep
        b1 = min(K, b0 + lazy)
        for k0 in range(b0, b1, nb):
            n += 1 + (1 if b1 - k0 - nb > 0 else 0)
        if b1 < K:
            b2 = min(K, b1 + lazy)
            n += 1 + (1 if K - b2 > 0 else 0)       # next batch's rows, then the rest
    return n


def run_gptq(args, w4, dev, local_rank, rank, peaks):
    """GPTQ on the residual branch (Sec. III-B) for one attention-projection layer: statistic from 2048 calibration
    tokens, factorization, triangular inverse and the sweep, all FP64 on the device.  An offline step: the number is a
    time per layer, with the FP64 rate it amounts to."""
    if rank != 0:
        return
    K, N = {"gptq": (5120, 5120), "gptq_mx": (5120, 5120), "gptq_ffn_up": (5120, 13824),
            "gptq_ffn_down": (13824, 5120)}[args.workload]
    M_cal = 2048
    mx = args.workload == "gptq_mx"                 # the MX variant's grid: E2M1 codes, E8M0 exponents per 32 channels
    quantize = w4.w4a4_mx_gptq_quantize if mx else w4.w4a4_gptq_quantize
    R, xhat = gen.make_gptq_inputs(K, N, M_cal, seed=7)
    Rd, xd = R.to(dev), xhat.to(dev)
    codes = torch.empty((K, N), dtype=torch.uint8 if mx else torch.int8, device=dev)
    scales = (torch.empty((K // 32, N), dtype=torch.uint8, device=dev) if mx
              else torch.empty((K // 64, N), dtype=torch.float32, device=dev))
    ws = torch.empty(w4.w4a4_gptq_workspace_bytes(K, N, M_cal), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    for _ in range(2):
        quantize(Rd, codes, scales, Xhat=xd, workspace=ws)
    runs = max(1, min(args.steps, 9))
    sampler = ClockSampler(local_rank)
    sampler.start()
    per_call = []
    torch.cuda.synchronize()
    for _ in range(runs):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        quantize(Rd, codes, scales, Xhat=xd, workspace=ws)
        e1.record(stream)
        torch.cuda.synchronize()
        per_call.append(e0.elapsed_time(e1))
    clocks = sampler.stop()
    # A call is some 600 short launches from one host thread; when the host is disturbed a call takes up to twice
    # as long with the same kernels.  The median says what the device does, the mean is reported beside it.
    ms = statistics.median(per_call)
    # FP64 operations the algorithm needs: upper triangle of X^T X, H = V V^T, U = V^-1, the error propagation
    flops = M_cal * K * K + K ** 3 / 3 + K ** 3 / 3 + float(K) * K * N
    sm_mhz = clocks.get("sm_max_mhz") or 1965
    peak = 148 * 64 * 2 * sm_mhz * 1e6 / 1e12      # 64 FP64 fused multiply-adds per SM and clock
    cpu = None
    if not args.no_cpu_baseline:
        import oracle  # test infrastructure; allowed here for the CPU-baseline leg only

        cols = list(range(0, N, N // 32))[:32]   # (the statistic's inverse dominates: minutes at K = 13824)
        t0 = time.perf_counter()
        H = oracle.gptq_hessian(bits(xhat))
        (oracle.gptq_quantize_mx if mx else oracle.gptq_quantize)(R[:, cols].double().numpy(), H)
        cpu = dict(value=(time.perf_counter() - t0) * 1e3, unit="ms", cores=torch.get_num_threads(), kind="oracle",
                   sample="the full statistic and its inverse, the sweep on 32 of the %d output channels" % N)
    print(json.dumps(dict(
        metric="gptq_layer_time", value=ms, unit="ms", n_gpus=1, steps=runs, warmup=2, ms_per_step=ms,
        higher_is_better=False, scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
        config=dict(workload=args.workload, K=K, N=N, calibration_tokens=M_cal, group=64, percdamp=0.01,
                    l2="working set of %.0f MB, larger than L2" % ((2 * K * K + K * N) * 8 / 1e6)),
        ms_per_call=dict(median=ms, mean=statistics.mean(per_call), min=min(per_call), max=max(per_call)),
        roofline=dict(bound="alu", achieved=flops / (ms * 1e-3) / 1e12, peak=peak, unit="TFLOP/s",
                      frac=flops / (ms * 1e-3) / 1e12 / peak, traffic=None,
                      note="peak = 148 SMs x 64 FP64 FMA per clock x 2 x max SM clock (nominal unit count)"),
        cpu_baseline=cpu, gpu_launches=gptq_launch_count(K) * runs, clocks=clocks)), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="attn_proj", choices=sorted(gen.CONFIG_SHAPES) + ["dit_step", "sweep", "clip_search", "mxfp4_attn_proj", "mxfp4_ffn_up",
                                                            "mxfp4_ffn_down", "mxfp4_ffn", "gptq", "gptq_mx", "gptq_ffn_up", "gptq_ffn_down"])
    ap.add_argument("--chunk-rows", type=int, default=4096, help="token rows per chunk of the host-buffer forward (e2e)")
    ap.add_argument("--blocks", type=int, default=40, help="DiT blocks for --workload dit_step")
    ap.add_argument("--qkv-packed", action="store_true",
                    help="dit_step: self-attention q, k, v as one layer packed along N (one activation pass for the three)")
    ap.add_argument("--out", default=None, help="file for the per-point table of --workload sweep")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the library peak probe, the second target shape and the short DiT-step run (profiling runs)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import paper_2605_27003_b200 as w4  # fails loudly when the CUDA library is missing
    from paper_2605_27003_b200 import build as pkg_build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the layer has no CPU path")
    if not os.path.exists(w4.LIB_PATH):
        pkg_build.build()
    w4.load_library()
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device(dev))

    peaks = load_peaks()
    # Library 8-bit GEMM peaks of this GPU, before (and outside) every timed region of the layer.
    tp = {} if (args.no_extras or args.workload.startswith("gptq") or args.workload == "tiny") else measure_tensor_peaks(dev)
    if args.workload == "dit_step":
        run_dit_step(args, w4, dev, local_rank, rank, world, dist, peaks, tp)
        return
    if args.workload == "sweep":
        run_sweep(args, w4, dev, local_rank, rank, peaks, tp)
        return
    if args.workload == "mxfp4_ffn":
        run_mxfp4_ffn(args, w4, dev, local_rank, rank, peaks, tp)
        return
    if args.workload.startswith("mxfp4_"):
        run_mxfp4(args, w4, dev, local_rank, rank, peaks, tp)
        return
    if args.workload == "clip_search":
        run_clip_search(args, w4, dev, local_rank, rank, peaks)
        return
    if args.workload.startswith("gptq"):
        run_gptq(args, w4, dev, local_rank, rank, peaks)
        return
    n_buf = 4
    w = workload_inputs(args.workload, dev, n_buf)
    M, K, N, r = w["M"], w["K"], w["N"], w["r"]
    ctx = w4.Context(local_rank, M, K, r)
    layer = w4.Layer(ctx, [w["layer"]], num_bins=w["num_bins"])
    clip = w["clip"].to(dev)
    Y = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.current_stream()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # -------------------------------------------------------------- device-resident timing
    for i in range(args.warmup):
        w4.w4a4_linear_forward(layer.ptr, w["xs"][i % n_buf], M, 0, w["bins"][i % n_buf], clip, Y, stream)
    barrier()
    ctx.check()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    sampler.start()
    barrier()
    for i in range(args.steps):
        b = i % n_buf
        ev[i][0].record(stream)
        w4.w4a4_quantize_activations(layer.ptr, w["xs"][b], M, 0, w["bins"][b], clip, stream)
        ev[i][1].record(stream)
        w4.w4a4_gemm_from_workspace(layer.ptr, M, 0, Y, stream)
        ev[i][2].record(stream)
    barrier()
    clocks = sampler.stop()
    ctx.check()
    total_ms = max_over_ranks(ev[0][0].elapsed_time(ev[-1][2]), dist, dev)
    t_q = [e[0].elapsed_time(e[1]) for e in ev]
    t_g = [e[1].elapsed_time(e[2]) for e in ev]
    ms_per_step = total_ms / args.steps
    ops = 2.0 * M * K * N
    value = whole_job_tops(ops, world, ms_per_step)

    # -------------------------------------------------------------- end to end from pinned host memory
    e2e_steps = max(1, min(args.e2e_steps, args.steps))
    xh = [torch.empty(M, K, dtype=torch.bfloat16).pin_memory().copy_(w["xs"][i]) for i in range(2)]
    yh = torch.empty(M, N, dtype=torch.bfloat16).pin_memory()
    chunk_rows = min(M, args.chunk_rows)
    w4.w4a4_ctx_enable_host_io(ctx.ptr, chunk_rows, N)

    def e2e_step(i):
        # Host buffers in, host buffers out, through the C ABI: chunked H2D / kernels / D2H on three streams.
        w4.w4a4_linear_forward_host(layer.ptr, xh[i % 2], M, 0, w["bins"][i % 2], clip, yh, stream)

    for i in range(2):
        e2e_step(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(e2e_steps):
        e2e_step(i)
    e1.record(stream)
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), dist, dev)
    e2e_value = whole_job_tops(ops, world, e2e_ms / e2e_steps)
    ctx.check()

    mx_ctx = mxfp4_context(w4, ctx, w, clip, Y, stream) if (rank == 0 and args.workload != "tiny") else None
    layer.close()
    ctx.close()
    w_small = dict(M=M, K=K, N=N, r=r, num_bins=w["num_bins"], xs=w["xs"][:1], bins=w["bins"][:1], layer=w["layer"], clip=w["clip"])
    del w, Y, xh, yh
    torch.cuda.empty_cache()

    if rank == 0:
        tq, tg = statistics.mean(t_q), statistics.mean(t_g)
        gemm_tops = ops / (tg * 1e-3) / 1e12
        roof = tensor_roofline(gemm_tops, total_ms * 1e-3, peaks, tp)
        roof.update(traffic=NCU_TRAFFIC_BYTES.get(("gemm", args.workload)),
                    kernel="gemm_w4a4_kernel (with the 9 us expand_weight_kernel in front of it)", ms=tg)
        # Bytes the activation step needs by its definition (X read; 4-bit codes, FP32 group scales and BF16 T written)
        # and bytes this layout moves (one E4M3 byte per code, FP32 scales plus the 8-byte scale operand of the GEMM's
        # scale MMA per (token, group), T as a BF16 high | low pair).
        q_alg = M * (2.0 * K + 0.5 * K + 4.0 * K / 64.0 + 2.0 * r)
        q_layout = M * (2.0 * K + 1.0 * K + 4.0 * K / 64.0 + 8.0 * K / 64.0 + 4.0 * r)
        q_gbs = q_alg / (tq * 1e-3) / 1e9
        line = dict(
            metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
            ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="e4m3",
            data="synthetic",
            config=dict(workload=args.workload, M=M, K=K, N=N, r=r, group=64, experts=1, bins=w_small["num_bins"],
                        l2="inputs larger than L2: 4 rotating activation buffers of %.0f MB" % (M * K * 2 / 1e6),
                        parallelism="replicas" if world > 1 else "single"),
            roofline=roof,
            roofline_quantize=dict(bound="hbm", achieved=q_gbs, peak=peaks["hbm_gbs"], unit="GB/s",
                                   frac=q_gbs / peaks["hbm_gbs"], traffic=NCU_TRAFFIC_BYTES.get(("quantize", args.workload)),
                                   kernel="quantize_kernel", ms=tq, algorithmic_bytes=q_alg,
                                   bytes_note="algorithmic = X + 4-bit codes + FP32 scales + BF16 T (13,184 B per token at K = 5120, r = 32)",
                                   layout_bytes=q_layout, frac_of_layout_bytes=q_layout / (tq * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                   frac_of_nominal_7700=q_gbs / NOMINAL_HBM_GBS, peak_source=peaks["source"]),
            kernel_ms=dict(quantize_mean=tq, quantize_min=min(t_q), gemm_mean=tg, gemm_min=min(t_g)),
            e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=M * K * 2, d2h_bytes_per_step=M * N * 2,
                     ms_per_step=e2e_ms / e2e_steps, steps=e2e_steps,
                     path="w4a4_linear_forward_host: pinned host X -> %d-row chunks over 3 streams -> pinned host Y"
                          % chunk_rows),
            gpu_launches=3 * args.steps, clocks=clocks, tensor_peaks=tp)
        if mx_ctx is not None:
            line["mxfp4_variant"] = mx_ctx
        if not args.no_extras and args.workload == "attn_proj" and world == 1:
            # The second shape of the performance target and a short run of one denoising step's 320 linears.
            up = measure_single_layer(w4, dev, local_rank, "ffn_up", 20, 3)
            up_tops = 2.0 * up["M"] * up["K"] * up["N"] / (up["gemm_ms"] * 1e-3) / 1e12
            up["roofline"] = tensor_roofline(up_tops, up["gemm_ms"] * 1e-3 * up["iters"], peaks, tp)
            up["layer_tops"] = 2.0 * up["M"] * up["K"] * up["N"] / ((up["gemm_ms"] + up["quantize_ms"]) * 1e-3) / 1e12
            line["ffn_up"] = up
            d = measure_dit_step(w4, dev, local_rank, 3, 3, 40)
            d_ms = d["total_ms"] / 3
            d_tops = d["ops"] / (d_ms * 1e-3) / 1e12
            line["dit_step"] = dict(ms_per_dit_step=d_ms, steps=3, warmup=3, value=d_tops, unit=UNIT, linears=d["linears"],
                                    tera_ops_per_step=d["ops"] / 1e12, resident_weight_gb=d["weight_bytes"] / 1e9,
                                    roofline=tensor_roofline(d_tops, d["total_ms"] * 1e-3, peaks, tp), clocks=d["clocks"])
        if not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(w_small)
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
