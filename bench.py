#!/usr/bin/env python
"""Benchmark of the PEQA quantized-linear hot path on B200.

Headline workload: one LLaMA-65B decoder layer, 3-bit weights in groups of 64
(q, k, v, o 8192x8192; gate, up 22016x8192; down 8192x22016; 4096 tokens).
One step runs, for the seven linears in layer order, the whole path through the
C ABI: RTN quantize+pack of the fp32 weight, forward, dX, dS with the AdamW
step on the scales applied in the same launch, and an M=1 decode.  The headline
value counts only the 6*T*N*K flop of forward + backward against the time of
the whole step.

The same JSON line carries sub-records (each with its own clock record): the
LLaMA-7B attention projection (3-bit g128, 2048 tokens) and SwiGLU MLP shapes
(4-bit per-channel, 4096 tokens), decode at M in {1, 4, 16} on the three
LLaMA-65B shapes with a bare-read ceiling beside each, and the per-channel dS
from the stored output.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
  python bench.py --render-md LINE.json     # markdown tables of a saved line

Prints exactly one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD = "c5"
WORKLOAD_TEXT = ("c5: one LLaMA-65B decoder layer, seven linears in layer order (q,k,v,o 8192x8192; "
                 "gate,up 22016x8192; down 8192x22016), 3-bit, group 64, T=4096 tokens")
METRIC = "qlinear fwd+bwd TFLOP/s (% bf16 peak); 3-bit decode GB/s (% HBM peak)"
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
LR, BETA1, BETA2, EPS, WD = 1e-5, 0.9, 0.999, 1e-8, 0.0
STAGES = ("quantize_rtn", "qlinear_fwd", "qlinear_bwd_dx", "qlinear_bwd_ds", "qlinear_decode")
DECODE_SHAPES = (("attn_8192x8192", 8192, 8192), ("gate_up_22016x8192", 22016, 8192),
                 ("down_8192x22016", 8192, 22016))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return json.load(f), "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


SHARED_DEVICE_HEADERS = ("common.cuh", "dequant.cuh", "sm100_ptx.cuh", "tensor_map.cuh")


def device_sources_sha256(files):
    """Hash of the kernel sources a stage's counters depend on (its .cu file and the shared headers)."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2305_14152_b200", "csrc")
    for name in sorted(set(files) | set(SHARED_DEVICE_HEADERS)):
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def measured_traffic(stage_name):
    """DRAM bytes per launch of the dominant kernel from the committed ncu capture (scaled to the
    mean launch of the headline step as that file states), or None when the kernel's sources have
    changed since the counters were taken."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic_c5.json")) as f:
            doc = json.load(f)
        k = doc["kernels"][stage_name]
        if doc.get("workload") != WORKLOAD or device_sources_sha256(k["sources"]) != k["sources_sha256"]:
            return None
        return k["traffic_bytes_mean_launch"]
    except Exception:
        return None


# --------------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while a timed region runs."""

    def __init__(self, index, period=0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def physical_gpu_index(local_index):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


class Timed:
    """A timed region: CUDA events on the current stream, clocks sampled meanwhile."""

    def __init__(self, torch, min_seconds=0.0):
        self.torch = torch
        self.sampler = ClockSampler(physical_gpu_index(torch.cuda.current_device()))
        self.e0 = torch.cuda.Event(enable_timing=True)
        self.e1 = torch.cuda.Event(enable_timing=True)

    def __enter__(self):
        self.torch.cuda.synchronize()
        self.sampler.start()
        self.e0.record()
        return self

    def __exit__(self, *exc):
        self.e1.record()
        self.torch.cuda.synchronize()
        self.clocks = self.sampler.stop()
        self.ms = self.e0.elapsed_time(self.e1)
        return False


def aggregate_max(ms_local, dist_mod=None, device=None):
    """Max over ranks of a per-rank time in ms (identity without a process group)."""
    if dist_mod is None or not dist_mod.is_initialized():
        return ms_local
    import torch
    t = torch.tensor([ms_local], dtype=torch.float64, device=device or "cpu")
    dist_mod.all_reduce(t, op=dist_mod.ReduceOp.MAX)
    return float(t.item())


def peak_for_clock(peaks, clocks):
    """Burst or sustained bf16 denominator, chosen by the SM clock sampled during the region:
    a region that ran near the maximum clock is compared with the burst figure, one that ran
    power-capped with the sustained one."""
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    capped = (mhz is not None and mx and mhz < 0.85 * mx) or "sw_power_cap" in clocks.get("reasons", [])
    if capped:
        return peaks["bf16_tflops_sustained"], "sustained"
    return peaks["bf16_tflops"], "burst"


# --------------------------------------------------------------------------- oracle arm
def oracle_sample(spec, layer, n_tok=512, n_rows=512):
    """Times the CPU oracle on a bounded sample of one linear; returns (seconds, flop, text)."""
    import oracle
    t0 = time.perf_counter()
    codes, zeros, scales = oracle.quantize_rtn(layer["W"], spec.bits, spec.group_size)
    packed = oracle.pack(codes, spec.bits)
    tok = np.linspace(0, spec.T - 1, n_tok).astype(np.int32)
    rows = np.linspace(0, spec.N - 1, n_rows).astype(np.int32)
    oracle.fwd(layer["X"], packed, zeros, scales, spec.bits, spec.group_size, tokens=tok)
    oracle.bwd_dx(layer["dY"], packed, zeros, scales, spec.K, spec.bits, spec.group_size, tokens=tok)
    oracle.bwd_ds(layer["X"], layer["dY"], packed, zeros, spec.bits, spec.group_size, rows=rows)
    dt = time.perf_counter() - t0
    flop = 2.0 * n_tok * spec.N * spec.K * 2 + 2.0 * spec.T * spec.K * n_rows
    what = (f"linear '{spec.name}' ({spec.N}x{spec.K}) of the layer: quantize+pack of W, fwd and dX on "
            f"{n_tok} of {spec.T} tokens, dS on {n_rows} of {spec.N} rows; throughput by flop count, "
            f"the other six linears extrapolate at the same rate")
    return dt, flop, what


def first_layer_host():
    from paper_2305_14152_b200 import synth
    return next(synth.generate(WORKLOAD))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    layer = first_layer_host()
    spec = layer["spec"]
    for _ in range(min(args.warmup, 1)):
        oracle_sample(spec, layer, 16, 16)
    steps = max(1, min(args.steps, 3))
    total_t, total_f, what = 0.0, 0.0, ""
    for _ in range(steps):
        dt, fl, what = oracle_sample(spec, layer, 256, 256)
        total_t += dt
        total_f += fl
    val = total_f / total_t / 1e12
    out = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": total_t / steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT,
                   "note": "fp64 CPU oracle on a bounded sample per step"},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": oracle.num_threads(),
                         "kind": "oracle", "sample": what},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(out), flush=True)


# --------------------------------------------------------------------------- CUDA arm
class Linear:
    """Device buffers of one linear of a workload."""

    def __init__(self, torch, binding, dev, d, keep_w=True):
        spec = d["spec"]
        self.spec = spec
        self.N, self.K, self.T, self.bits, self.g = spec.N, spec.K, spec.T, spec.bits, spec.group_size
        self.G = self.K // self.g if self.g else 1
        self.flop = 2.0 * self.T * self.N * self.K

        def bf16(bits_arr):
            return torch.from_numpy(bits_arr.view(np.int16)).view(torch.bfloat16).to(dev)

        self.W = torch.from_numpy(d["W"]).to(dev)
        self.X = bf16(d["X"])
        self.dY = bf16(d["dY"]) if d["dY"] is not None else None
        self.qw = binding.quantize_rtn(self.W, self.bits, self.g)
        if not keep_w:
            self.W = None
        self.m = torch.zeros((self.N, self.G), dtype=torch.float32, device=dev)
        self.v = torch.zeros((self.N, self.G), dtype=torch.float32, device=dev)
        self.dS = torch.empty((self.N, self.G), dtype=torch.float32, device=dev)
        self.Yd = torch.empty((1, self.N), dtype=torch.bfloat16, device=dev)
        # Q is frozen (Sec. 3.3): the copy the decode kernel streams is prepared once, here
        self.prep = binding.decode_prepare(self.qw) if binding.decode_prepared_supported(self.qw) else None
        self.ws = binding.alloc_workspace(binding.OP_BWD, self.T, self.qw)


def load_workload(torch, binding, dev, name, keep_first_host=False):
    from paper_2305_14152_b200 import synth
    layers, first = [], None
    for d in synth.generate(name):
        layers.append(Linear(torch, binding, dev, d))
        if keep_first_host and first is None:
            first = d
    return layers, first


def run_stage(binding, L, k, Y, dX, step_no):
    if k == 0:
        binding.quantize_rtn(L.W, L.bits, L.g, out=L.qw)
    elif k == 1:
        binding.qlinear_fwd(L.qw, L.X, Y[:L.T * L.N].view(L.T, L.N))
    elif k == 2:
        binding.qlinear_bwd(L.qw, None, L.dY, dX=dX[:L.T * L.K].view(L.T, L.K), need_ds=False)
    elif k == 3:
        binding.qlinear_bwd_ds_adamw(L.qw, L.X, L.dY, L.m, L.v, LR, BETA1, BETA2, EPS, WD, step_no,
                                     dS=L.dS, workspace=L.ws)
    elif L.prep is not None:
        binding.qlinear_decode_prepared(L.qw, L.prep, L.X[:1], L.Yd)
    else:
        binding.qlinear_decode(L.qw, L.X[:1], L.Yd)


def time_layer_steps(torch, binding, layers, Y, dX, steps, warmup, dist=None, dev=None):
    """Times `steps` passes over `layers` (all five stages of every linear); returns the total ms
    (max over ranks), per-stage mean ms [linear][stage], and the clock record."""
    n = len(layers)
    for i in range(warmup):
        for L in layers:
            for k in range(len(STAGES)):
                run_stage(binding, L, k, Y, dX, i + 1)
    binding.check_status()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(n * len(STAGES) + 1)] for _ in range(steps)]
    if dist is not None:
        dist.barrier()
    with Timed(torch) as tm:
        for i in range(steps):
            e = evs[i]
            e[0].record()
            j = 0
            for L in layers:
                for k in range(len(STAGES)):
                    run_stage(binding, L, k, Y, dX, warmup + i + 1)
                    j += 1
                    e[j].record()
    if dist is not None:
        dist.barrier()
    binding.check_status()
    ms_total = aggregate_max(tm.ms, dist, dev)
    stage_ms = [[float(np.mean([evs[i][li * len(STAGES) + k].elapsed_time(evs[i][li * len(STAGES) + k + 1])
                                for i in range(steps)])) for k in range(len(STAGES))] for li in range(n)]
    return ms_total, stage_ms, tm.clocks


def launches_per_step(layers):
    """Kernels of this library per step: one per stage, plus the dS reduce kernel when a
    quantization group is wider than 128 columns."""
    return sum(len(STAGES) + (1 if L.ws is not None else 0) for L in layers)


def run_cuda(args):
    import torch
    from paper_2305_14152_b200 import binding, build
    build.build()
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    else:
        torch.cuda.set_device(0)
    dev = torch.device("cuda", torch.cuda.current_device())
    peaks, peak_src = load_peaks()

    if args.only_decode:
        print(json.dumps({"decode": bench_decode(torch, binding, dev, peaks, reps=min(args.steps, 30),
                                                 shapes=args.case)}), flush=True)
        return

    extras = rank == 0 and not args.only_step
    layers, first_host = load_workload(torch, binding, dev, WORKLOAD, keep_first_host=extras and world == 1)
    if args.case:
        layers = [L for L in layers if L.spec.name in args.case.split(",")]
    Y = torch.empty(max(L.T * L.N for L in layers), dtype=torch.bfloat16, device=dev)
    dX = torch.empty(max(L.T * L.K for L in layers), dtype=torch.bfloat16, device=dev)
    warmup = max(args.warmup, 3)
    ms_total, stage_ms, clocks = time_layer_steps(torch, binding, layers, Y, dX, args.steps, warmup, dist, dev)
    ms_step = ms_total / args.steps
    flop_step = 3.0 * sum(L.flop for L in layers)
    value = world * flop_step / (ms_step * 1e-3) / 1e12

    # ---- roofline of the dominant kernel: the contraction with the largest share of the step
    tot = {k: sum(stage_ms[li][k] for li in range(len(layers))) for k in (1, 2, 3)}
    dom = max(tot, key=tot.get)
    mean_flop = sum(L.flop for L in layers) / len(layers)
    mean_ms = tot[dom] / len(layers)
    ach = mean_flop / (mean_ms * 1e-3) / 1e12
    peak, which = peak_for_clock(peaks, clocks)
    roofline = {
        "bound": "tensor", "kernel": STAGES[dom], "achieved": ach, "peak": peak, "unit": "TFLOP/s",
        "frac": ach / peak, "traffic": measured_traffic(STAGES[dom]),
        "traffic_unit": "DRAM bytes per mean launch (ncu)",
        "peak_source": f"{peak_src} cuBLAS bf16 {which} (chosen by the sampled SM clock)",
        "launches_per_step": len(layers), "flop_per_mean_launch": mean_flop, "ms_per_mean_launch": mean_ms,
        "frac_of_measured_burst": ach / peaks["bf16_tflops"],
        "frac_of_measured_sustained": ach / peaks["bf16_tflops_sustained"],
        "frac_of_nominal_2250": ach / NOMINAL_BF16_TFLOPS,
        "target_60pct_of_nominal_met": bool(ach / NOMINAL_BF16_TFLOPS >= 0.60),
        "per_kernel_tflops": {STAGES[k]: sum(L.flop for L in layers) / (tot[k] * 1e-3) / 1e12 for k in (1, 2, 3)},
    }
    per_linear = {L.spec.name: {"N": L.N, "K": L.K,
                                **{STAGES[k] + "_ms": stage_ms[li][k] for k in range(len(STAGES))},
                                "fwd_dx_ds_tflops": 3.0 * L.flop / (sum(stage_ms[li][1:4]) * 1e-3) / 1e12}
                  for li, L in enumerate(layers)}

    out = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT + "; step = per linear: quantize+pack, fwd, dX, dS+AdamW (one "
                               "launch), decode(M=1)" + (f"; restricted to {args.case}" if args.case else ""),
                   "l2": "every linear's operands (X, dY, Y/dX, packed W: 0.3-0.6 GB) exceed the 126 MB L2 and "
                         "the seven linears use distinct buffers, so every launch starts cold; no flush kernel",
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "flop_per_step": flop_step},
        "clocks": clocks, "gpu_launches": launches_per_step(layers) * args.steps,
        "stage_ms": {STAGES[k]: sum(stage_ms[li][k] for li in range(len(layers))) for k in range(len(STAGES))},
        "per_linear": per_linear, "roofline": roofline,
        "value_frac_of_measured_burst": value / world / peaks["bf16_tflops"],
        "value_frac_of_measured_sustained": value / world / peaks["bf16_tflops_sustained"],
        "value_frac_of_nominal_2250": value / world / NOMINAL_BF16_TFLOPS,
    }

    # ---- the same fwd + dX + dS/AdamW of the seven linears as ONE library call per step
    if not args.only_step:
        out["layer_call"] = bench_layer_call(args, binding, torch, layers, peaks, warmup)

    # ---- end to end through the host-buffer entry point (pinned host memory both ways)
    out["e2e"] = None
    if not args.only_step:
        out["e2e"] = bench_e2e(args, binding, torch, layers, Y, dX, dist, dev, world, flop_step)

    if extras:
        del layers
        torch.cuda.empty_cache()
        out["c2"] = bench_small_workload(torch, binding, dev, peaks, "c2", steps=200, n_sets=4)
        out["c3"] = bench_small_workload(torch, binding, dev, peaks, "c3", steps=20, n_sets=2)
        out["decode"] = bench_decode(torch, binding, dev, peaks)
        out["ds_from_y"] = bench_ds_from_y(torch, binding, dev, peaks)
        if world == 1:
            import oracle
            dt, fl, what = oracle_sample(first_host["spec"], first_host)
            out["cpu_baseline"] = {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(),
                                   "kind": "oracle", "sample": what, "seconds": dt}
    if rank == 0:
        print(json.dumps(out), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def bench_layer_call(args, binding, torch, layers, peaks, warmup):
    """peqa_layer_train_step: forward, dX and dS with the AdamW step for all linears of the layer,
    enqueued by one call (no quantize or decode stage, no events between the kernels)."""
    dev = layers[0].X.device
    items = [binding.LayerLinear(w=L.qw, X=L.X, dY=L.dY,
                                 Y=torch.empty((L.T, L.N), dtype=torch.bfloat16, device=dev),
                                 dX=torch.empty((L.T, L.K), dtype=torch.bfloat16, device=dev),
                                 dS=L.dS, m=L.m, v=L.v, workspace=L.ws) for L in layers]
    for i in range(2):
        binding.layer_train_step(items, LR, BETA1, BETA2, EPS, WD, step=warmup + 1000 + i)
    binding.check_status()
    steps = args.steps
    with Timed(torch) as tm:
        for i in range(steps):
            binding.layer_train_step(items, LR, BETA1, BETA2, EPS, WD, step=warmup + 2000 + i)
    binding.check_status()
    ms = tm.ms / steps
    flop = 3.0 * sum(L.flop for L in layers)
    tf = flop / (ms * 1e-3) / 1e12
    peak, which = peak_for_clock(peaks, tm.clocks)
    return {"what": "peqa_layer_train_step: fwd, dX, dS+AdamW of the seven linears per call", "steps": steps,
            "ms_per_step": ms, "value": tf, "unit": "TFLOP/s", "clocks": tm.clocks, "peak": peak,
            "peak_kind": which, "frac_of_peak": tf / peak, "frac_of_nominal_2250": tf / NOMINAL_BF16_TFLOPS}


def host_linears(torch, binding, dev, layers):
    """Pinned host buffers and per-linear device staging buffers for peqa_layer_train_step_host."""
    hl = []
    for L in layers:
        hX = torch.empty((L.T, L.K), dtype=torch.bfloat16).pin_memory()
        hdY = torch.empty((L.T, L.N), dtype=torch.bfloat16).pin_memory()
        hX.copy_(L.X)
        hdY.copy_(L.dY)
        hl.append(binding.HostLinear(
            w=L.qw, h_X=hX, h_dY=hdY,
            h_Y=torch.empty((L.T, L.N), dtype=torch.bfloat16).pin_memory(),
            h_dX=torch.empty((L.T, L.K), dtype=torch.bfloat16).pin_memory(),
            h_dS=torch.empty((L.N, L.G), dtype=torch.float32).pin_memory(),
            d_X=torch.empty((L.T, L.K), dtype=torch.bfloat16, device=dev),
            d_dY=torch.empty((L.T, L.N), dtype=torch.bfloat16, device=dev),
            d_Y=torch.empty((L.T, L.N), dtype=torch.bfloat16, device=dev),
            d_dX=torch.empty((L.T, L.K), dtype=torch.bfloat16, device=dev),
            d_dS=L.dS, d_m=L.m, d_v=L.v, workspace=L.ws))
    return hl


def time_host_step(torch, binding, hl, steps, dist=None, dev=None):
    """ms per peqa_layer_train_step_host call (max over ranks), bytes copied each way, clocks."""
    binding.layer_train_step_host(hl, LR, step=1)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    with Timed(torch) as tm:
        for k in range(steps):
            binding.layer_train_step_host(hl, LR, step=k + 2)
    ms = aggregate_max(tm.ms / steps, dist, dev)
    return ms, {"h2d_bytes_per_step": int(sum(H.h_X.numel() * 2 + H.h_dY.numel() * 2 for H in hl)),
                "d2h_bytes_per_step": int(sum(H.h_Y.numel() * 2 + H.h_dX.numel() * 2 + H.h_dS.numel() * 4 for H in hl)),
                "ms_per_step": ms, "steps": steps, "clocks": tm.clocks}


def bench_e2e(args, binding, torch, layers, Y, dX, dist, dev, world, flop_step):
    """Same metric through peqa_layer_train_step_host, one call per step: every step copies each
    linear's X and dY from pinned host memory and returns Y, dX and dS to pinned host memory;
    every linear has device staging buffers of its own, so its copies overlap its neighbours'
    kernels."""
    hl = host_linears(torch, binding, dev, layers)
    ms, rec = time_host_step(torch, binding, hl, max(2, min(args.steps, 5)), dist, dev)
    out = {"value": world * flop_step / (ms * 1e-3) / 1e12, "unit": "TFLOP/s"}
    out.update(rec)
    out["what"] = ("peqa_layer_train_step_host, one call per step: per linear H2D X,dY; fwd, dX, dS+AdamW; "
                   "D2H Y,dX,dS; the copies of a linear overlap the kernels of its neighbours")
    return out


def bench_small_workload(torch, binding, dev, peaks, name, steps, n_sets):
    """The same five stages on another configured workload (a sub-record of the line): `n_sets`
    seeded draws of every linear rotate so that launches start cold in L2."""
    from paper_2305_14152_b200 import synth
    wl = synth.WORKLOADS[name]
    rng = np.random.Generator(np.random.PCG64(wl.seed))
    sets = [[Linear(torch, binding, dev, synth.draw_layer(rng, spec)) for spec in wl.layers]
            for _ in range(n_sets)]
    Y = torch.empty(max(L.T * L.N for L in sets[0]), dtype=torch.bfloat16, device=dev)
    dX = torch.empty(max(L.T * L.K for L in sets[0]), dtype=torch.bfloat16, device=dev)
    n = len(wl.layers)
    for i in range(3):
        for L in sets[i % n_sets]:
            for k in range(len(STAGES)):
                run_stage(binding, L, k, Y, dX, i + 1)
    binding.check_status()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(n * len(STAGES) + 1)] for _ in range(steps)]
    with Timed(torch) as tm:
        for i in range(steps):
            e = evs[i]
            e[0].record()
            j = 0
            for L in sets[i % n_sets]:
                for k in range(len(STAGES)):
                    run_stage(binding, L, k, Y, dX, 4 + i)
                    j += 1
                    e[j].record()
    binding.check_status()
    stage_ms = [[float(np.mean([evs[i][li * len(STAGES) + k].elapsed_time(evs[i][li * len(STAGES) + k + 1])
                                for i in range(steps)])) for k in range(len(STAGES))] for li in range(n)]
    layers = sets[0]
    flop_step = 3.0 * sum(L.flop for L in layers)
    ms_step = tm.ms / steps
    peak, which = peak_for_clock(peaks, tm.clocks)
    rec = {"workload": name, "steps": steps, "ms_per_step": ms_step,
           "value": flop_step / (ms_step * 1e-3) / 1e12, "unit": "TFLOP/s (6*T*N*K over the whole step)",
           "clocks": tm.clocks, "peak": peak, "peak_kind": which,
           "l2": f"{n_sets} rotating seeded draws of every linear", "per_linear": {}}
    for li, L in enumerate(layers):
        r = {"N": L.N, "K": L.K, "T": L.T, "bits": L.bits, "group": L.g}
        for k in range(len(STAGES)):
            r[STAGES[k] + "_ms"] = stage_ms[li][k]
        for k in (1, 2, 3):
            r[STAGES[k] + "_tflops"] = L.flop / (stage_ms[li][k] * 1e-3) / 1e12
        tf = 3.0 * L.flop / (sum(stage_ms[li][1:4]) * 1e-3) / 1e12
        r.update({"fwd_dx_ds_tflops": tf, "frac_of_peak": tf / peak, "frac_of_nominal_2250": tf / NOMINAL_BF16_TFLOPS})
        rec["per_linear"][L.spec.name] = r
    # the same workload end to end from pinned host buffers (copies both ways inside the time)
    hl = host_linears(torch, binding, dev, layers)
    ms, e2e = time_host_step(torch, binding, hl, max(5, steps // 10))
    e2e.update({"value": flop_step / (ms * 1e-3) / 1e12, "unit": "TFLOP/s"})
    rec["e2e"] = e2e
    del sets, hl
    torch.cuda.empty_cache()
    return rec


def bench_decode(torch, binding, dev, peaks, reps=30, shapes=None):
    """GB/s of decode at M in {1, 4, 16} on the three LLaMA-65B shapes (3-bit, one scale per
    channel), from the prepared weights (peqa_qlinear_decode_prepared, what a server runs) and
    from the canonical packed matrix (peqa_qlinear_decode); the weights rotate through enough
    distinct copies to exceed L2, so every launch streams from HBM.  Launches are back to back
    with no event between them.  Beside each shape: a kernel that only reads the same bytes."""
    res = {}
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    sink = torch.zeros(1024, dtype=torch.int32, device=dev)
    for name, N, K in DECODE_SHAPES:
        if shapes and name not in shapes.split(","):
            continue
        words = K * 3 // 32
        wbytes = N * words * 4
        copies = max(2, int(np.ceil(4 * 126e6 / wbytes)))
        qs = [torch.randint(-2 ** 31, 2 ** 31 - 1, (N, words), dtype=torch.int32, device=dev, generator=gen)
              for _ in range(copies)]
        z = torch.full((N, 1), 3, dtype=torch.uint8, device=dev)
        s = torch.full((N, 1), 0.01, dtype=torch.float32, device=dev)
        qws = [binding.QWeight(3, N, K, 0, q, z, s) for q in qs]
        rec = {"bytes_weights": wbytes, "copies": copies}

        def timed(fn):
            """Mean device time per launch: `reps` launches rotating through the weight copies are
            captured into one CUDA graph (the same C-ABI calls, recorded instead of run) and the
            graph is replayed, so host launch overhead is not what is measured.  Falls back to
            eager launches if the capture is refused."""
            for i in range(copies):
                fn(i)
            torch.cuda.synchronize()
            graph = None
            try:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    for i in range(reps):
                        fn(i % copies)
                graph = g
                graph.replay()
                torch.cuda.synchronize()
            except Exception:
                graph = None
                torch.cuda.synchronize()
            replays = 5
            with Timed(torch) as tm:
                for _ in range(replays):
                    if graph is not None:
                        graph.replay()
                    else:
                        for i in range(reps):
                            fn(i % copies)
            rec["launch_mode"] = "cuda graph replay" if graph is not None else "eager"
            return tm.ms / (reps * replays) * 1e3, tm.clocks

        us, clk = timed(lambda i: binding.probe_read(qs[i], sink))
        rec["bare_read"] = {"us": us, "GB/s": wbytes / (us * 1e-6) / 1e9,
                            "frac_measured_hbm": wbytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"], "clocks": clk}
        preps = [binding.decode_prepare(qw) for qw in qws]
        torch.cuda.synchronize()

        def time_both(qws_, M, G, into, prefix):
            X = torch.randn((M, K), device=dev, generator=gen).to(torch.bfloat16)
            Y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            ws = binding.alloc_workspace(binding.OP_DECODE, M, qws_[0])
            nbytes = wbytes + N * G * 5 + M * K * 2 + M * N * 2
            for key, fn in (("prepared", lambda i: binding.qlinear_decode_prepared(qws_[i], preps[i], X, Y)),
                            ("canonical", lambda i: binding.qlinear_decode(qws_[i], X, Y, workspace=ws))):
                us, clk = timed(fn)
                gbs = nbytes / (us * 1e-6) / 1e9
                into[f"{prefix}M{M}_{key}"] = {"us": us, "GB/s": gbs, "frac_measured_hbm": gbs / peaks["hbm_gbs"],
                                               "frac_nominal_8000": gbs / NOMINAL_HBM_GBS, "bytes": nbytes,
                                               "frac_of_bare_read_time": rec["bare_read"]["us"] / us, "clocks": clk}

        for M in (1, 4, 16):
            time_both(qws, M, 1, rec, "")
        # the same matrices with scales in groups of 64 columns (the LLaMA-65B layer workload's setting)
        G64 = K // 64
        z64 = torch.full((N, G64), 3, dtype=torch.uint8, device=dev)
        s64 = torch.full((N, G64), 0.01, dtype=torch.float32, device=dev)
        qws64 = [binding.QWeight(3, N, K, 64, q, z64, s64) for q in qs]
        for M in (1, 4):
            time_both(qws64, M, G64, rec, "g64_")
        del qws64, z64, s64
        del preps
        binding.check_status()
        res[name] = rec
        del qs, qws
    return res


def bench_ds_from_y(torch, binding, dev, peaks, reps=20):
    """GB/s of peqa_qlinear_bwd_ds_from_y on the LLaMA-7B MLP gate shape (N=11008, T=4096, 4-bit
    per-channel): two rotating (dY, Y) pairs of 180 MB each, so every launch streams from HBM."""
    N, K, T = 11008, 4096, 4096
    gen = torch.Generator(device=dev)
    gen.manual_seed(3)
    q = torch.zeros((N, K * 4 // 32), dtype=torch.int32, device=dev)
    z = torch.zeros((N, 1), dtype=torch.uint8, device=dev)
    s = torch.full((N, 1), 0.01, dtype=torch.float32, device=dev)
    qw = binding.QWeight(4, N, K, 0, q, z, s)
    pairs = [(torch.randn((T, N), device=dev, generator=gen).to(torch.bfloat16),
              torch.randn((T, N), device=dev, generator=gen).to(torch.bfloat16)) for _ in range(2)]
    dS = torch.empty((N, 1), dtype=torch.float32, device=dev)
    ws = binding.alloc_workspace(binding.OP_BWD_DS_FROM_Y, T, qw)
    for i in range(3):
        binding.qlinear_bwd_ds_from_y(qw, pairs[i % 2][0], pairs[i % 2][1], dS, ws)
    with Timed(torch) as tm:
        for i in range(reps):
            binding.qlinear_bwd_ds_from_y(qw, pairs[i % 2][0], pairs[i % 2][1], dS, ws)
    us = tm.ms / reps * 1e3
    nbytes = 4 * T * N + 8 * N
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"workload": "N=11008, T=4096 (c3 gate), bf16 dY and Y", "us": us, "GB/s": gbs,
            "frac_measured_hbm": gbs / peaks["hbm_gbs"], "bytes": nbytes, "clocks": tm.clocks,
            "replaces": "the dS contraction of the same layer (2*T*N*K flop)"}


# --------------------------------------------------------------------------- rendering
def render_md(path):
    """Markdown tables of a saved JSON line (the tables of the results write-up are made this way)."""
    with open(path) as f:
        text = f.read()
    doc = None
    for line in text.splitlines():
        line = line.strip()
        if line.startswith("{") and '"metric"' in line:
            doc = json.loads(line)
    if doc is None:
        doc = json.loads(text)
        doc = doc.get("parsed", doc)
    o = []
    c, r = doc["clocks"], doc["roofline"]
    o.append(f"Headline ({doc['config']['workload']}): **{doc['value']:.0f} TFLOP/s**, {doc['ms_per_step']:.3f} ms "
             f"per step over {doc['steps']} steps; SM clock median {c['sm_mhz']} of {c['sm_max_mhz']} MHz, "
             f"reasons {c['reasons']}.  Of the measured cuBLAS burst {doc['value_frac_of_measured_burst']:.2f}, "
             f"of the measured sustained {doc['value_frac_of_measured_sustained']:.2f}, of the nominal 2250 "
             f"{doc['value_frac_of_nominal_2250']:.2f}.")
    o.append(f"Dominant kernel `{r['kernel']}`: {r['achieved']:.0f} TFLOP/s = {r['frac']:.2f} of {r['peak_source']} "
             f"({r['frac_of_measured_burst']:.2f} burst / {r['frac_of_measured_sustained']:.2f} sustained / "
             f"{r['frac_of_nominal_2250']:.2f} nominal; 60 % of nominal met: {r['target_60pct_of_nominal_met']}).")
    o.append("")
    o.append("| workload | linear | fwd ms | dX ms | dS+AdamW ms | quantize ms | decode M=1 ms | fwd+dX+dS TFLOP/s | of nominal 2250 |")
    o.append("|---|---|---|---|---|---|---|---|---|")
    for name, p in doc["per_linear"].items():
        o.append(f"| c5 | {name} {p['N']}x{p['K']} | {p['qlinear_fwd_ms']:.3f} | {p['qlinear_bwd_dx_ms']:.3f} | "
                 f"{p['qlinear_bwd_ds_ms']:.3f} | {p['quantize_rtn_ms']:.3f} | {p['qlinear_decode_ms']:.3f} | "
                 f"{p['fwd_dx_ds_tflops']:.0f} | {p['fwd_dx_ds_tflops'] / NOMINAL_BF16_TFLOPS:.2f} |")
    for key in ("c2", "c3"):
        sub = doc.get(key)
        if not sub:
            continue
        for name, p in sub["per_linear"].items():
            o.append(f"| {key} (clock {sub['clocks']['sm_mhz']} MHz, {sub['peak_kind']}) | {name} {p['N']}x{p['K']} T={p['T']} | "
                     f"{p['qlinear_fwd_ms']:.4f} | {p['qlinear_bwd_dx_ms']:.4f} | {p['qlinear_bwd_ds_ms']:.4f} | "
                     f"{p['quantize_rtn_ms']:.4f} | {p['qlinear_decode_ms']:.4f} | {p['fwd_dx_ds_tflops']:.0f} | "
                     f"{p['frac_of_nominal_2250']:.2f} |")
    if doc.get("layer_call"):
        lc = doc["layer_call"]
        o.append("")
        o.append(f"One call per layer ({lc['what']}): {lc['value']:.0f} TFLOP/s, {lc['ms_per_step']:.3f} ms per step; "
                 f"clock {lc['clocks']['sm_mhz']} MHz, {lc['frac_of_peak']:.2f} of the measured {lc['peak_kind']} "
                 f"peak, {lc['frac_of_nominal_2250']:.2f} of nominal.")
    if doc.get("e2e"):
        e = doc["e2e"]
        o.append("")
        o.append(f"End to end ({e['what']}): {e['value']:.0f} TFLOP/s, {e['ms_per_step']:.2f} ms per step, "
                 f"{e['h2d_bytes_per_step'] / 1e6:.0f} MB in and {e['d2h_bytes_per_step'] / 1e6:.0f} MB out per step.")
    for key in ("c2", "c3"):
        e = (doc.get(key) or {}).get("e2e")
        if e:
            o.append(f"End to end, {key}: {e['value']:.0f} TFLOP/s, {e['ms_per_step']:.3f} ms per step, "
                     f"{e['h2d_bytes_per_step'] / 1e6:.1f} MB in and {e['d2h_bytes_per_step'] / 1e6:.1f} MB out per step "
                     f"({(e['h2d_bytes_per_step'] + e['d2h_bytes_per_step']) / e['ms_per_step'] / 1e6:.0f} GB/s over the link, both directions).")
    if doc.get("decode"):
        o.append("")
        o.append("| decode shape | bare read us (GB/s) | M | us | GB/s | of measured copy | of 8 TB/s | bare read / kernel |")
        o.append("|---|---|---|---|---|---|---|---|")
        for name, rec in doc["decode"].items():
            b = rec["bare_read"]
            for key, v in rec.items():
                if not (key.startswith("M") or key.startswith("g64_M")):
                    continue
                grp = "g64 " if key.startswith("g64_") else ""
                key = key[4:] if key.startswith("g64_") else key
                o.append(f"| {name} {grp}{key.split('_')[1]} | {b['us']:.1f} ({b['GB/s']:.0f}) | {key[1:].split('_')[0]} | {v['us']:.1f} | "
                         f"{v['GB/s']:.0f} | {v['frac_measured_hbm']:.2f} | {v['frac_nominal_8000']:.2f} | "
                         f"{v['frac_of_bare_read_time']:.2f} |")
    if doc.get("cpu_baseline"):
        cb = doc["cpu_baseline"]
        o.append("")
        o.append(f"CPU oracle: {cb['value']:.4f} TFLOP/s on {cb['cores']} threads ({cb['sample']}).")
    print("\n".join(o))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--only-decode", action="store_true",
                    help="run only the decode section (with --case: a comma list of its shape names)")
    ap.add_argument("--only-step", action="store_true",
                    help="time the step only: skip the e2e, sub-record and CPU-baseline sections "
                         "(lean runs under a profiler)")
    ap.add_argument("--case", default=None,
                    help="restrict the step to these linears of the layer (comma list: q,k,v,o,gate,up,down)")
    ap.add_argument("--render-md", default=None, help="print markdown tables of a saved JSON line")
    args = ap.parse_args()
    if args.render_md:
        render_md(args.render_md)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
