#!/usr/bin/env python
"""Benchmark of the PEQA quantized-linear hot path on B200.

One step = one pass of the whole path over one batch of the LLaMA-7B attention
projection workload (4096x4096, 3-bit, groups of 128, 2048 tokens): RTN
quantize+pack of the fp32 weight, forward, dX, dS, AdamW on the scales and an
M=1 decode.  The headline value counts only the 6*T*N*K flop of forward +
backward against the time of the whole step.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

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

WORKLOAD = "c2"
METRIC = "qlinear fwd+bwd TFLOP/s (% bf16 peak); 3-bit decode GB/s (% HBM peak)"
N_SETS = 4                       # rotating input sets: ~135 MB each, together > L2 (126 MB)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return json.load(f), "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def measured_traffic(kernel_name):
    """DRAM bytes per launch from the committed ncu capture, or None when the kernel sources
    have changed since the counters were taken."""
    import hashlib
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic_c2.json")) as f:
            doc = json.load(f)
        h = hashlib.sha256()
        csrc = os.path.join(ROOT, "paper_2305_14152_b200", "csrc")
        for name in sorted(os.listdir(csrc)):
            with open(os.path.join(csrc, name), "rb") as f:
                text = f.read()
            if name.endswith(".cuh") or b"__global__" in text:      # device code only
                h.update(text)
        if h.hexdigest() != doc["kernel_sources_sha256"] or doc.get("workload") != WORKLOAD:
            return None
        return doc["kernels"][kernel_name]["traffic_bytes"]
    except Exception:
        return None


def draw_sets(n_sets):
    """Set 0 is the canonical workload draw; further sets continue the same seeded stream."""
    from paper_2305_14152_b200 import synth
    wl = synth.WORKLOADS[WORKLOAD]
    spec = wl.layers[0]
    rng = np.random.Generator(np.random.PCG64(wl.seed))
    return spec, [synth.draw_layer(rng, spec) for _ in range(n_sets)]


# --------------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index, period=0.02):
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


# --------------------------------------------------------------------------- oracle arm
def oracle_sample(spec, layer, n_tok=512, n_rows=1024):
    """Times the CPU oracle on a bounded sample of the workload; returns (seconds, flop)."""
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
    return dt, flop, f"quantize+pack of W, fwd and dX on {n_tok} of {spec.T} tokens, dS on {n_rows} of {spec.N} rows"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    spec, sets = draw_sets(1)
    for _ in range(min(args.warmup, 1)):
        oracle_sample(spec, sets[0], 64, 64)
    steps = max(1, min(args.steps, 5))
    total_t, total_f, what = 0.0, 0.0, ""
    for _ in range(steps):
        dt, fl, what = oracle_sample(spec, sets[0], 256, 512)
        total_t += dt
        total_f += fl
    val = total_f / total_t / 1e12
    out = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": total_t / steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": f"{WORKLOAD}: LLaMA-7B attention projection 4096x4096, 3-bit g128, T=2048",
                   "note": "fp64 CPU oracle on a bounded sample per step"},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": oracle.num_threads(),
                         "kind": "oracle", "sample": what},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(out), flush=True)


# --------------------------------------------------------------------------- CUDA arm
def aggregate_max(ms_local, dist_mod=None, device=None):
    """Max over ranks of a per-rank time in ms (identity without a process group)."""
    if dist_mod is None or not dist_mod.is_initialized():
        return ms_local
    import torch
    t = torch.tensor([ms_local], dtype=torch.float64, device=device or "cpu")
    dist_mod.all_reduce(t, op=dist_mod.ReduceOp.MAX)
    return float(t.item())


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
        # the decode section alone (what the decode ncu summaries under profiles/ were taken on)
        print(json.dumps({"decode": bench_decode(binding, dev, peaks, reps=args.steps if args.steps < 30 else 30)}),
              flush=True)
        return

    spec, sets = draw_sets(N_SETS)
    N, K, T, bits, g = spec.N, spec.K, spec.T, spec.bits, spec.group_size
    G = K // g if g else 1

    def bf16(bits_arr):
        return torch.from_numpy(bits_arr.view(np.int16)).view(torch.bfloat16).to(dev)

    Ws = [torch.from_numpy(s["W"]).to(dev) for s in sets]
    Xs = [bf16(s["X"]) for s in sets]
    dYs = [bf16(s["dY"]) for s in sets]
    qws = [binding.quantize_rtn(W, bits, g) for W in Ws]
    Y = torch.empty((T, N), dtype=torch.bfloat16, device=dev)
    dX = torch.empty((T, K), dtype=torch.bfloat16, device=dev)
    dS = torch.empty((N, G), dtype=torch.float32, device=dev)
    m = torch.zeros((N, G), dtype=torch.float32, device=dev)
    v = torch.zeros((N, G), dtype=torch.float32, device=dev)
    Yd = torch.empty((1, N), dtype=torch.bfloat16, device=dev)
    ws = binding.alloc_workspace(binding.OP_BWD, T, qws[0])
    lr = 1e-5
    # dS and the AdamW step on the scales are one launch (the step is applied where each dS
    # value becomes final), so the step has five stages
    stage_names = ["quantize_rtn", "qlinear_fwd", "qlinear_bwd_dx", "qlinear_bwd_ds", "qlinear_decode"]
    n_stages = len(stage_names)
    launches_per_step = n_stages + (1 if ws is not None else 0)

    def step(i, evs=None):
        r = i % N_SETS
        qw = qws[r]
        if evs: evs[0].record()
        binding.quantize_rtn(Ws[r], bits, g, out=qw)
        if evs: evs[1].record()
        binding.qlinear_fwd(qw, Xs[r], Y)
        if evs: evs[2].record()
        binding.qlinear_bwd(qw, None, dYs[r], dX=dX, need_ds=False)
        if evs: evs[3].record()
        binding.qlinear_bwd_ds_adamw(qw, Xs[r], dYs[r], m, v, lr, 0.9, 0.999, 1e-8, 0.0, i + 1,
                                     dS=dS, workspace=ws)
        if evs: evs[4].record()
        binding.qlinear_decode(qw, Xs[r][:1], Yd)
        if evs: evs[5].record()

    for i in range(max(args.warmup, 3)):
        step(i)
    binding.check_status()
    torch.cuda.synchronize()

    sampler = ClockSampler(physical_gpu_index(torch.cuda.current_device()))
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(n_stages + 1)] for _ in range(args.steps)]
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(args.steps):
        step(i, evs[i])
    t_end.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    clocks = sampler.stop()
    binding.check_status()
    ms_total = aggregate_max(t_start.elapsed_time(t_end), dist, dev)
    ms_step = ms_total / args.steps
    stage_ms = [float(np.mean([evs[i][k].elapsed_time(evs[i][k + 1]) for i in range(args.steps)]))
                for k in range(n_stages)]

    flop_step = 6.0 * T * N * K
    value = world * flop_step / (ms_step * 1e-3) / 1e12

    # ---- end to end through the host-buffer entry point (pinned host memory both ways)
    e2e = None
    if not args.only_step:
        e2e = bench_e2e(args, binding, torch, qws, Xs, dYs, Y, dX, dS, m, v, ws, lr, dist, dev,
                        world, flop_step, T, N, K, G)

    # ---- roofline of the dominant kernel (the slowest of the three contractions)
    gemm = {k: stage_ms[k] for k in (1, 2, 3)}
    dom = max(gemm, key=gemm.get)
    ach = 2.0 * T * N * K / (gemm[dom] * 1e-3) / 1e12
    long_region = ms_total > 1000.0
    peak = peaks["bf16_tflops_sustained"] if long_region else peaks["bf16_tflops"]
    roofline = {"bound": "tensor", "kernel": stage_names[dom], "achieved": ach, "peak": peak,
                "unit": "TFLOP/s", "frac": ach / peak, "traffic": measured_traffic(stage_names[dom]),
                "traffic_unit": "DRAM bytes per launch (ncu)",
                "peak_source": f"{peak_src} bf16 {'sustained' if long_region else 'burst'}",
                "frac_of_nominal_2250": ach / 2250.0,
                "per_kernel_tflops": {stage_names[k]: 2.0 * T * N * K / (gemm[k] * 1e-3) / 1e12
                                      for k in (1, 2, 3)}}

    # ---- secondary metric: M=1 decode of the LLaMA-65B 3-bit per-channel shapes, cold in L2
    decode = None
    if rank == 0 and not args.only_step:
        decode = bench_decode(binding, dev, peaks)

    # ---- next-row item: per-channel dS from the stored output (HBM bound, 4*T*N bytes)
    ds_from_y = None
    if rank == 0 and not args.only_step:
        ds_from_y = bench_ds_from_y(binding, dev, peaks)

    out = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{WORKLOAD}: LLaMA-7B attention projection N=K=4096, 3-bit, group 128, "
                               f"T=2048 tokens; step = quantize+pack, fwd, dX, dS+AdamW (one launch), decode(M=1)",
                   "l2": f"{N_SETS} rotating input sets (~{N_SETS * 135} MB) exceed the 126 MB L2; no flush kernel",
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "flop_per_step": flop_step},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
        "stage_ms": dict(zip(stage_names, stage_ms)),
        "roofline": roofline, "decode": decode, "ds_from_y": ds_from_y,
    }
    if rank == 0 and world == 1 and not args.only_step:
        dt, fl, what = oracle_sample(spec, sets[0])
        import oracle
        out["cpu_baseline"] = {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(),
                               "kind": "oracle", "sample": what, "seconds": dt}
    if rank == 0:
        print(json.dumps(out), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def bench_e2e(args, binding, torch, qws, Xs, dYs, Y, dX, dS, m, v, ws, lr, dist, dev, world,
              flop_step, T, N, K, G):
    """Same metric through peqa_train_step_host: pinned host buffers in and out every step."""
    hX = torch.empty((T, K), dtype=torch.bfloat16).pin_memory()
    hdY = torch.empty((T, N), dtype=torch.bfloat16).pin_memory()
    hX.copy_(Xs[0].cpu())
    hdY.copy_(dYs[0].cpu())
    hY = torch.empty((T, N), dtype=torch.bfloat16).pin_memory()
    hdX = torch.empty((T, K), dtype=torch.bfloat16).pin_memory()
    hdS = torch.empty((N, G), dtype=torch.float32).pin_memory()
    dXin = torch.empty_like(Xs[0])
    ddYin = torch.empty_like(dYs[0])
    e2e_steps = max(3, min(args.steps, 50))
    for k in range(2):
        binding.train_step_host(qws[0], hX, hdY, hY, hdX, hdS, dXin, ddYin, Y, dX, dS, m, v, lr,
                                step=k + 1, workspace=ws)
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for k in range(e2e_steps):
        binding.train_step_host(qws[k % N_SETS], hX, hdY, hY, hdX, hdS, dXin, ddYin, Y, dX, dS, m, v,
                                lr, step=k + 3, workspace=ws)
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = aggregate_max(e0.elapsed_time(e1) / e2e_steps, dist, dev)
    return {"value": world * flop_step / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
            "h2d_bytes_per_step": int(hX.numel() * 2 + hdY.numel() * 2),
            "d2h_bytes_per_step": int(hY.numel() * 2 + hdX.numel() * 2 + hdS.numel() * 4),
            "ms_per_step": e2e_ms,
            "what": "peqa_train_step_host: H2D X,dY; fwd, dX, dS, AdamW; D2H Y,dX,dS"}


def bench_decode(binding, dev, peaks, reps=30):
    """GB/s of peqa_qlinear_decode at M=1 on the three LLaMA-65B shapes; weights rotate through
    enough distinct copies to exceed L2, so every launch streams from HBM."""
    import torch
    res = {}
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    for name, N, K in (("attn_8192x8192", 8192, 8192), ("gate_up_22016x8192", 22016, 8192),
                       ("down_8192x22016", 8192, 22016)):
        words = K * 3 // 32
        wbytes = N * words * 4
        copies = max(2, int(np.ceil(4 * 126e6 / wbytes)))
        qs = [torch.randint(-2 ** 31, 2 ** 31 - 1, (N, words), dtype=torch.int32, device=dev, generator=gen)
              for _ in range(copies)]
        z = torch.full((N, 1), 3, dtype=torch.uint8, device=dev)
        s = torch.full((N, 1), 0.01, dtype=torch.float32, device=dev)
        X = torch.randn((1, K), device=dev, generator=gen).to(torch.bfloat16)
        Y = torch.empty((1, N), dtype=torch.bfloat16, device=dev)
        qws = [binding.QWeight(3, N, K, 0, q, z, s) for q in qs]
        for i in range(copies):
            binding.qlinear_decode(qws[i], X, Y)
        torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(reps):
            binding.qlinear_decode(qws[i % copies], X, Y)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / reps * 1e3
        nbytes = wbytes + N * 5 + K * 2 + N * 2
        gbs = nbytes / (us * 1e-6) / 1e9
        res[name] = {"us": us, "GB/s": gbs, "frac_measured_hbm": gbs / peaks["hbm_gbs"],
                     "frac_nominal_8000": gbs / 8000.0, "bytes": nbytes, "copies": copies}
        del qs, qws
    return res


def bench_ds_from_y(binding, dev, peaks, reps=20):
    """GB/s of peqa_qlinear_bwd_ds_from_y on the LLaMA-7B MLP gate shape (N=11008, T=4096, 4-bit
    per-channel): two rotating (dY, Y) pairs of 180 MB each, so every launch streams from HBM."""
    import torch
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
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(reps):
        binding.qlinear_bwd_ds_from_y(qw, pairs[i % 2][0], pairs[i % 2][1], dS, ws)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) / reps * 1e3
    nbytes = 4 * T * N + 8 * N
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"workload": "N=11008, T=4096 (c3 gate), bf16 dY and Y", "us": us, "GB/s": gbs,
            "frac_measured_hbm": gbs / peaks["hbm_gbs"], "bytes": nbytes,
            "replaces": "the dS contraction of the same layer (2*T*N*K flop)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--only-decode", action="store_true",
                    help="run only the M=1 decode section on the three LLaMA-65B shapes")
    ap.add_argument("--only-step", action="store_true",
                    help="time the step only: skip the e2e, decode and CPU-baseline sections "
                         "(lean runs under a profiler)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
