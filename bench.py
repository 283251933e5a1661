#!/usr/bin/env python
"""Benchmark of the DEER-GRU hot path on B200.

One "step" = one whole `deer_gru_eval` (input projection + all Newton bodies:
cell + Jacobian + rhs, scan, convergence) over the headline workload, the
largest single-GPU configuration of the benchmark definition that is a forward
evaluation: config 3 (GRU n=32, m=32, B=16, T=100,000, fp32, x ~ N(0,1), zero
initial state and zero initial guess).  `value` = B*T positions evaluated per
second with the inputs resident in HBM; `e2e` = the same through the
host-buffer call (`deer_gru_eval_host`) with the H2D copy of x and the D2H copy
of y inside the timed region.  The same JSON line carries, as extra keys, the
other workloads of the definition (config 2, the config-4 training step) and
the stand-alone scans on HBM-sized inputs (n = 4 ... 64) with their rooflines.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

N > 1 (under torchrun): every rank evaluates its own batch of the same shape
(sequences are independent: no data-path collective), weak scaling; the timed
region is bracketed by barriers and the maximum over ranks is reported.
`--impl reference` times the CPU oracle's sequential fp32 loop instead.
Other modes (`--mode scan|eval|sweep|classifier`) print one JSON line each for
a single measurement; every input is drawn from the documented seeded streams
of `paper_2309_12252_b200.synth` (on the device through `synth_device`).
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

METRIC = "DEER GRU B*T steps/s"
UNIT = "steps/s"
WORKLOADS = {
    2: dict(workload="config2: GRU n=8 m=4 B=16 T=10000 fp32, x=sin(wt+phi)+0.1N(0,1), y0=0, zero guess",
            n=8, m=4, B=16, T=10000, tol=1e-4, max_iter=100),
    3: dict(workload="config3: GRU n=32 m=32 B=16 T=100000 fp32, x~N(0,1), y0=0, zero guess",
            n=32, m=32, B=16, T=100000, tol=1e-4, max_iter=100),
}
HEADLINE = 3
# stand-alone scans sized well beyond L2 (J of 1 ... 9.4 GB): where the HBM roofline claims are taken
SCANS_HBM = [dict(n=4, B=16, T=1_000_000), dict(n=8, B=16, T=1_000_000), dict(n=16, B=16, T=200_000),
             dict(n=32, B=16, T=100_000), dict(n=64, B=32, T=17_984)]


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


def tf32_peak_tflops(pk) -> float:
    """Dense TF32 tensor peak: the measured bf16 burst figure times the nominal TF32/bf16 ratio (1.1 / 2.25 PFLOP/s)."""
    return pk["bf16_tflops"] * (1.1 / 2.25)


# DRAM bytes (read + write) per position from the ncu captures summarised under profiles/ (inputs larger
# than L2; traffic grows in proportion to the positions processed, so a launch's traffic is this times B*T).
NCU_SCAN_TRAFFIC_PER_POSITION = {1: 12.8, 2: 32.7, 4: 95.3, 8: 606.6, 16: 2213.0, 32: 8622.0, 64: 34116.0}
# the two launches of the scan inside deer_gru_eval (n = 16, 32, 64): reduce, apply
NCU_FUSED_TRAFFIC_PER_POSITION = {"scan_fused_reduce_kernel": {32: 684.0}, "scan_fused_apply_kernel": {32: 916.0}}
NCU_CONFIG2_SCAN_TRAFFIC = 51.43e6                      # scan_warp8_kernel inside the config-2 step, per launch


def scan_bytes_per_position(n: int) -> int:
    """Algorithmic bytes of one stand-alone scan per position: read J and b once, write y."""
    return 4 * (n * n + n) + 4 * n


def fused_scan_bytes_per_position(n: int) -> int:
    """The scan inside deer_gru_eval for n = 16, 32, 64 (J generated from four coefficient vectors per position):
    read the coefficient rows (16n), the residual (4n) and the previous iterate (4n) once, write y (4n)."""
    return 28 * n


def fused_kernel_bytes(name: str, n: int) -> int:
    """Algorithmic bytes per position of one launch of the two-launch scan: the reduce kernels read the coefficient
    rows and the residual (20 n), the apply kernel those, y_old, and writes y (32 n)."""
    return (20 if "reduce" in name else 32) * n


def scan_flops_per_position(n: int) -> int:
    """Chunk reduce of Eq. 9: one n x n by n x (n+1) product per position (apply adds 2n^2, counted with it)."""
    return 2 * n * n * (n + 1)


def roofline_of_scan(n, positions, ms, pk, bytes_per_position, traffic_per_position, kernel, extra=None, bf16=False):
    """The slower of the byte bound (measured HBM copy rate) and the flop bound (tensor peak of the kernel's MMA
    type: TF32, or bf16 when `bf16`) is the scan's roofline; `frac` = that bound's time / measured time,
    `achieved` in the unit of the binding resource."""
    t_bytes = bytes_per_position * positions / (pk["hbm_gbs"] * 1e9) * 1e3
    tf32 = pk["bf16_tflops"] if bf16 else tf32_peak_tflops(pk)
    t_flops = scan_flops_per_position(n) * positions / (tf32 * 1e12) * 1e3
    hbm_bound = t_bytes >= t_flops
    gbs = bytes_per_position * positions / (ms * 1e-3) / 1e9
    tfs = scan_flops_per_position(n) * positions / (ms * 1e-3) / 1e12
    out = dict(bound="hbm" if hbm_bound else "tensor", kernel=kernel,
               achieved=gbs if hbm_bound else tfs, peak=pk["hbm_gbs"] if hbm_bound else tf32,
               unit="GB/s" if hbm_bound else "TFLOP/s", frac=(t_bytes if hbm_bound else t_flops) / ms,
               peak_source=pk["source"] + ("" if hbm_bound else " bf16 burst" if bf16 else " bf16 burst x 1.1/2.25 (nominal TF32/bf16 ratio)"),
               tensor_peak_tflops=tf32, tensor_dtype="bf16" if bf16 else "tf32",
               ms_per_launch=ms, positions_per_launch=positions, bytes_per_position=bytes_per_position,
               flops_per_position=scan_flops_per_position(n),
               hbm_frac=t_bytes / ms, tensor_frac=t_flops / ms, achieved_gbs=gbs, achieved_tflops=tfs,
               traffic=None if traffic_per_position is None else traffic_per_position * positions)
    if extra:
        out.update(extra)
    return out


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while GPU work runs (read-only).  Samples taken
    between mark_begin() and mark_end() are also kept apart: those are the timed region's."""

    def __init__(self, index: int, period: float = 0.005):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self.timed, self.timed_reasons, self.in_timed = [], set(), False
        self._stop_ev = threading.Event()
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
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8)),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40)),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20)),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4)),
        }
        get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self._stop_ev.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = int(get(self.h))
                hit = {k for k, bit in names.items() if mask & bit}
                self.samples.append(mhz)
                self.reasons |= hit
                if self.in_timed:
                    self.timed.append(mhz)
                    self.timed_reasons |= hit
            except Exception:
                pass
            time.sleep(self.period)

    def mark_begin(self):
        self.in_timed = True

    def mark_end(self):
        self.in_timed = False

    def stop(self):
        self._stop_ev.set()
        self.join(timeout=2)
        timed = self.timed or self.samples
        reasons = self.timed_reasons if self.timed else self.reasons
        med = int(np.median(timed)) if timed else None
        return dict(sm_mhz=med, sm_max_mhz=self.max_mhz, reasons=sorted(reasons), samples=len(timed),
                    whole_run=dict(sm_mhz=int(np.median(self.samples)) if self.samples else None,
                                   reasons=sorted(self.reasons), samples=len(self.samples)))


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def aggregate_over_ranks(local_ms: float, local_units: float, dist, device):
    """Max of the per-rank times and sum of the per-rank units (whole-job throughput)."""
    import torch
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_ms, local_units
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([local_units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def cpu_oracle_rate(w, min_seconds: float):
    """Sequential fp32 GRU loop of the oracle, repeated on the full workload until min_seconds."""
    import oracle
    oracle.gru_seq(w.params, w.x, w.y0, np.float32)          # warm-up (page-in, thread pool)
    reps, t0 = 0, time.perf_counter()
    while True:
        oracle.gru_seq(w.params, w.x, w.y0, np.float32)
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= min_seconds:
            break
    return reps * w.B * w.T / dt, reps, dt, min(oracle.num_threads(), w.B)


def run_reference(args):
    """Reference arm: the CPU oracle as it stands, on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2309_12252_b200 import synth
    import oracle
    w = synth.config(args.workload)
    for _ in range(max(args.warmup, 1)):
        oracle.gru_seq(w.params, w.x, w.y0, np.float32)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.gru_seq(w.params, w.x, w.y0, np.float32)
    dt = time.perf_counter() - t0
    value = args.steps * w.B * w.T / dt
    cores = min(oracle.num_threads(), w.B)
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=1e3 * dt / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f32", data="synthetic", impl="reference", config=dict(WORKLOADS[args.workload]),
                cpu_baseline=dict(value=value, unit=UNIT, cores=cores, kind="oracle",
                                  sample=f"{args.steps} full passes of the sequential fp32 GRU loop over the whole workload"),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


def parse_profile(text):
    out = {}
    for ln in text.strip().splitlines():
        name, cnt, ms = ln.split()
        out[name] = dict(launches=int(cnt), total_ms=float(ms))
    return out


def read_profile(bd):
    import ctypes
    L = bd.lib()
    L.deer_profile_read.restype = ctypes.c_size_t
    L.deer_profile_read.argtypes = [ctypes.c_char_p, ctypes.c_size_t]
    buf = ctypes.create_string_buffer(1 << 16)
    L.deer_profile_read(buf, len(buf))
    return parse_profile(buf.value.decode())


def is_scan_kernel(name: str) -> bool:
    return (name.startswith("scan_") and "prep" not in name) or name.startswith("gen_")


def scan_inputs(n, B, T, device, seed=0):
    """Stand-alone scan inputs from the documented streams: contractive J (entries U(+-0.9/n)), b ~ N(0,1)."""
    from paper_2309_12252_b200 import synth_device
    J = synth_device.contractive_J(B, T, n, seed=seed, tag=f"bench/scan{n}/J", scale=0.9, device=device)
    b = synth_device.normal(seed, f"bench/scan{n}/b", (B, T, n), device=device)
    return J, b


def time_scan(bd, torch, device, n, B, T, reverse, flags, steps, warmup):
    J, bb = scan_inputs(n, B, T, device)
    yy = torch.empty_like(bb)
    ws = bd.alloc_workspace(bd.DEER_OP_SCAN, B, T, n, 1, flags, device)
    stream = torch.cuda.current_stream()
    for _ in range(max(warmup, 1)):
        bd.deer_linrec_scan(J, bb, None, bool(reverse), yy, ws, flags, stream)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    torch.cuda.synchronize()
    for a, b in ev:
        a.record(stream)
        bd.deer_linrec_scan(J, bb, None, bool(reverse), yy, ws, flags, stream)
        b.record(stream)
    torch.cuda.synchronize()
    status = bd.deer_workspace_status(ws, stream)
    assert status == bd.DEER_OK, bd.deer_status_string(status)
    return float(np.median([a.elapsed_time(b) for a, b in ev]))


def scan_kernel_name(n: int, flags: int = 0) -> str:
    return {1: "scan_onepass_kernel", 2: "scan_onepass_kernel", 4: "scan_hold4_kernel", 8: "scan_warp8_kernel",
            16: "scan_warpn_kernel", 32: "scan_warpn_kernel", 64: "scan_umma64_kernel" if flags & 8 else "scan_cta64_kernel"}.get(n, "gen_*")


def run_scan_only(args):
    """Stand-alone linear-recurrence scan at the given size: prints one JSON line."""
    import torch
    from paper_2309_12252_b200 import binding as bd
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    n, B, T = args.n, args.B, args.T
    ms = time_scan(bd, torch, device, n, B, T, args.reverse, args.flags, args.steps, args.warmup)
    pk = peaks()
    r = roofline_of_scan(n, B * T, ms, pk, scan_bytes_per_position(n), NCU_SCAN_TRAFFIC_PER_POSITION.get(n),
                         scan_kernel_name(n, args.flags))
    print(json.dumps(dict(mode="scan", n=n, B=B, T=T, reverse=int(args.reverse), flags=args.flags, ms=ms,
                          positions_per_s=B * T / (ms * 1e-3), achieved_gbs=r["achieved_gbs"], peak_gbs=pk["hbm_gbs"],
                          frac=r["hbm_frac"], tensor_frac=r["tensor_frac"], bound=r["bound"], peak_source=pk["source"],
                          input_mb=(n * n + n) * 4 * B * T / 1e6, geometry=bd.deer_scan_geometry(B, T, n, args.flags))))


def eval_point(bd, synth, device, n, m, B, T, flags, steps, warmup, vjp=False, breakdown=True):
    """deer_gru_eval (optionally deer_gru_vjp) at one point of the speed grid (weights and x ~ N(0,1) from the
    streams of synth.sweep_point, y0 = 0): a dict of timings."""
    import torch
    from paper_2309_12252_b200 import synth_device
    p = bd.GruParamsDev.from_numpy(synth.gru_params(n, m, 0, tag=f"sweep{n}/gru"))
    x = synth_device.normal(0, f"sweep{n}/x", (B, T, m), device=device)
    y0 = torch.zeros((B, n), device=device)
    y = torch.empty((B, T, n), device=device)
    ws = bd.alloc_workspace(bd.DEER_OP_EVAL, B, T, n, m, flags, device)
    stream = torch.cuda.current_stream()
    run = lambda: bd.deer_gru_eval(p, x, y0, 1e-4, 100, y, ws, flags, stream)
    for _ in range(max(warmup, 1)):
        r = run()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    torch.cuda.synchronize()
    for a, b in ev:
        a.record(stream); r = run(); b.record(stream)
    torch.cuda.synchronize()
    ms = float(np.median([a.elapsed_time(b) for a, b in ev]))
    out = dict(n=n, m=m, B=B, T=T, flags=flags, ms=ms, steps_per_s=B * T / (ms * 1e-3),
               iters=r.iters, err=r.err, status=r.status)
    if breakdown:
        bd.lib().deer_profile_enable(1)
        run()
        torch.cuda.synchronize()
        bd.lib().deer_profile_enable(0)
        prof = read_profile(bd)
        out["kernels"] = {k: dict(launches=v["launches"], ms=round(v["total_ms"], 4)) for k, v in prof.items()}
        scan_ms = sum(v["total_ms"] for k, v in prof.items() if is_scan_kernel(k))
        if scan_ms > 0 and r.iters > 0:
            pk = peaks()
            per = scan_ms / r.iters
            fused = any(k.startswith("scan_fused") or k.startswith("scan_warpnf") for k in prof)
            bpp = fused_scan_bytes_per_position(n) if fused else scan_bytes_per_position(n)
            rl = roofline_of_scan(n, B * T, per, pk, bpp, None, "+".join(k for k in prof if is_scan_kernel(k)), bf16=fused)
            out["scan_ms_per_iter"] = per
            out["scan_bound"] = rl["bound"]
            out["scan_frac"] = rl["frac"]
            out["scan_bytes_per_position"] = bpp
    if vjp:
        gy = synth_device.normal(0, f"sweep{n}/gy", (B, T, n), device=device)
        del ws
        wsv = bd.alloc_workspace(bd.DEER_OP_VJP, B, T, n, m, flags, device)
        for _ in range(2):
            bd.deer_gru_vjp(p, x, y0, y, gy, True, True, wsv, flags, stream)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream); bd.deer_gru_vjp(p, x, y0, y, gy, True, True, wsv, flags, stream); b.record(stream)
        torch.cuda.synchronize()
        out["vjp_ms"] = a.elapsed_time(b)
        bd.lib().deer_profile_enable(1)
        bd.deer_gru_vjp(p, x, y0, y, gy, True, True, wsv, flags, stream)
        torch.cuda.synchronize()
        bd.lib().deer_profile_enable(0)
        out["vjp_kernels"] = {k: round(v["total_ms"], 4) for k, v in read_profile(bd).items()}
    return out


def run_eval_only(args):
    """One grid point chosen on the command line: prints one JSON line."""
    import torch
    from paper_2309_12252_b200 import binding as bd
    from paper_2309_12252_b200 import synth
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    out = eval_point(bd, synth, device, args.n, args.m or args.n, args.B, args.T, args.flags,
                     args.steps, args.warmup, vjp=bool(args.vjp))
    out["mode"] = "eval"
    print(json.dumps(out))


def time_classifier(bd, synth, torch, device, B, T, flags, steps, warmup, profile=True):
    """Config 4: full training steps (loss + all gradients) of the 2-layer GRU classifier."""
    w = synth.config4(seed=0, B=B, T=T)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device)
    l1 = bd.GruParamsDev.from_numpy(w.layers[0]); l2 = bd.GruParamsDev.from_numpy(w.layers[1])
    W_o, b_o, x, labels = dev(w.W_o), dev(w.b_o), dev(w.x), dev(w.labels)
    n, m = w.layers[0].n, w.layers[0].m
    ws = bd.alloc_workspace(bd.DEER_OP_CLASSIFIER, B, T, n, m, flags, device)
    stream = torch.cuda.current_stream()
    run = lambda: bd.deer_gru_classifier_step(l1, l2, W_o, b_o, x, labels, ws=ws, flags=flags, stream=stream)
    for _ in range(max(warmup, 1)):
        r = run()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    torch.cuda.synchronize()
    for a, b in ev:
        a.record(stream); r = run(); b.record(stream)
    torch.cuda.synchronize()
    ms = float(np.median([a.elapsed_time(b) for a, b in ev]))
    out = dict(B=B, T=T, n=n, m=m, ms=ms, steps_per_s=B * T / (ms * 1e-3), loss=r["loss"], iters=list(r["iters"]),
               status=r["status"])
    if profile:
        bd.lib().deer_profile_enable(1)
        run()
        torch.cuda.synchronize()
        bd.lib().deer_profile_enable(0)
        prof = read_profile(bd)
        out["kernels"] = {k: dict(launches=v["launches"], ms=round(v["total_ms"], 4)) for k, v in prof.items()}
    return out


def time_multihead(bd, synth, torch, device, B, T, H, n, m, steps, warmup, cpu_seconds=0.0):
    """The multi-head GRU unit of the paper's sequential-image model (Sec. 4.4, App. B.4: 32 heads of 8 channels
    on 256 input channels, strides 2^0 .. 2^7, T = 1024): forward evaluation and gradient."""
    heads = synth.multihead_params(H, n, m, 0, tag="bench/mh")
    strides = synth.multihead_strides(H)
    x_np = synth.x_gaussian(B, T, m, 0, tag="bench/mhx")
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device)
    hd = [bd.GruParamsDev.from_numpy(h) for h in heads]
    x = dev(x_np); y0 = torch.zeros((B, H, n), device=device)
    ws = bd.alloc_multihead_workspace(hd, strides, B, T, device)
    y = torch.empty((B, T, H, n), device=device)
    stream = torch.cuda.current_stream()
    run = lambda: bd.deer_gru_multihead_eval(hd, strides, x, y0, y=y, ws=ws, stream=stream)
    for _ in range(max(warmup, 1)):
        _, iters, status = run()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    torch.cuda.synchronize()
    for a, b in ev:
        a.record(stream); run(); b.record(stream)
    torch.cuda.synchronize()
    ms = float(np.median([a.elapsed_time(b) for a, b in ev]))
    gy = torch.ones_like(y)
    bd.deer_gru_multihead_vjp(hd, strides, x, y0, y, gy, ws=ws, stream=stream)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record(stream); bd.deer_gru_multihead_vjp(hd, strides, x, y0, y, gy, ws=ws, stream=stream); b.record(stream)
    torch.cuda.synchronize()
    out = dict(workload=f"multi-head GRU unit: H={H} heads x n={n}, m={m}, strides 2^(h mod 8), B={B} T={T}, x~N(0,1), y0=0",
               ms_per_step=ms, value=B * T / (ms * 1e-3), unit=UNIT, newton_iters=iters, status=status,
               vjp_ms=a.elapsed_time(b))
    if cpu_seconds > 0:
        import oracle
        y0_np = np.zeros((B, H, n), np.float32)
        oracle.multihead_seq(heads, strides, x_np, y0_np, np.float32)
        reps, t0 = 0, time.perf_counter()
        while time.perf_counter() - t0 < cpu_seconds:
            oracle.multihead_seq(heads, strides, x_np, y0_np, np.float32)
            reps += 1
        dt = time.perf_counter() - t0
        out["cpu_baseline"] = dict(value=reps * B * T / dt, unit=UNIT, cores=min(oracle.num_threads(), B), kind="oracle",
                                   sample=f"{reps} passes of the oracle's sequential multi-head loop ({dt:.1f} s)")
    return out


def run_multihead(args):
    import torch
    from paper_2309_12252_b200 import binding as bd
    from paper_2309_12252_b200 import synth
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    out = time_multihead(bd, synth, torch, device, args.B, args.T, 32, 8, 256, args.steps, args.warmup, args.cpu_seconds)
    out["mode"] = "multihead"
    print(json.dumps(out))


def run_classifier(args):
    import torch
    from paper_2309_12252_b200 import binding as bd
    from paper_2309_12252_b200 import synth
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    out = time_classifier(bd, synth, torch, device, args.B, args.T, args.flags, args.steps, args.warmup)
    out["mode"] = "classifier"
    print(json.dumps(out))


def run_sweep(args):
    """The paper's speed grid (Table of forward speed-ups), thinned: n = m in {1..64} x T in {1e3..1e6},
    B = 16, x ~ N(0,1); one JSON line with one entry per point (n = 64, T = 1e6 is left out)."""
    import torch
    from paper_2309_12252_b200 import binding as bd
    from paper_2309_12252_b200 import synth
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    points = []
    for n in (1, 2, 4, 8, 16, 32, 64):
        for T in (1000, 10000, 100000, 1000000):
            if n == 64 and T == 1000000:
                continue
            steps = 5 if n * n * T <= 10 ** 8 else 2
            pt = eval_point(bd, synth, device, n, n, 16, T, args.flags, steps, 1, breakdown=True)
            pt.pop("kernels", None)
            points.append(pt)
            torch.cuda.empty_cache()
    print(json.dumps(dict(mode="sweep", B=16, points=points)))


def measure_workload(bd, torch, synth, idx, rank, device, dist, steps, warmup, flush, sampler=None, prof_steps=10):
    """Whole deer_gru_eval calls on configuration `idx` (each rank its own batch, same weights): device-resident
    timing, the host-buffer call, and a separate profiled pass for the per-kernel breakdown."""
    cfg = WORKLOADS[idx]
    w = synth.config(idx, seed=rank)
    B, T, n, m = w.B, w.T, w.n, w.m
    p = bd.GruParamsDev.from_numpy(synth.config(idx, seed=0, B=1, T=1).params)
    x_host = torch.from_numpy(w.x).pin_memory()
    y_host = torch.empty((B, T, n), dtype=torch.float32).pin_memory()
    x = x_host.to(device)
    y0 = torch.zeros((B, n), device=device)
    y = torch.empty((B, T, n), device=device)
    ws = bd.alloc_workspace(bd.DEER_OP_EVAL, B, T, n, m, 0, device)
    stream = torch.cuda.current_stream()

    def step():
        return bd.deer_gru_eval(p, x, y0, cfg["tol"], cfg["max_iter"], y, ws, 0, stream)

    def step_host():
        return bd.deer_gru_eval_host(p, x_host, y0, y_host, x, y, ws, cfg["tol"], cfg["max_iter"], 0, stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        r = step()
    iters = r.iters
    assert r.status == 0, bd.deer_status_string(r.status)

    # ---- timed region: K steps, L2 flushed before each, per-step CUDA events on the launching stream
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    barrier()
    if sampler is not None:
        sampler.mark_begin()
    launches0 = bd.deer_launch_count()
    for a, b in ev:
        flush.fill_(1)
        a.record(stream)
        r = step()
        b.record(stream)
    barrier()
    launches = bd.deer_launch_count() - launches0
    if sampler is not None:
        sampler.mark_end()
    local_ms = sum(a.elapsed_time(b) for a, b in ev)
    total_ms, total_units = aggregate_over_ranks(local_ms, float(steps) * B * T, dist, device)

    # ---- end to end: host buffers, H2D of x and D2H of y inside the timed region
    for _ in range(3):
        step_host()
    ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    barrier()
    for a, b in ev2:
        flush.fill_(1)
        a.record(stream)
        step_host()
        b.record(stream)
    barrier()
    e2e_ms, e2e_units = aggregate_over_ranks(sum(a.elapsed_time(b) for a, b in ev2), float(steps) * B * T, dist, device)

    # ---- per-kernel breakdown of the same steps (separate pass: event pairs around every launch)
    prof_steps = min(steps, prof_steps)
    bd.lib().deer_profile_enable(1)
    for _ in range(prof_steps):
        flush.fill_(1)
        step()
    torch.cuda.synchronize()
    bd.lib().deer_profile_enable(0)
    prof = read_profile(bd)
    tot = sum(v["total_ms"] for v in prof.values()) or 1.0
    kernels = {k: dict(launches_per_step=v["launches"] / prof_steps, us_per_launch=1e3 * v["total_ms"] / v["launches"],
                       share=v["total_ms"] / tot) for k, v in prof.items()}
    return dict(cfg=cfg, B=B, T=T, n=n, m=m, iters=iters, err=r.err, value=total_units / (total_ms * 1e-3),
                ms_per_step=total_ms / steps, launches=int(launches),
                e2e=dict(value=e2e_units / (e2e_ms * 1e-3), unit=UNIT, h2d_bytes_per_step=int(x_host.numel() * 4),
                         d2h_bytes_per_step=int(y_host.numel() * 4), ms_per_step=e2e_ms / steps),
                kernels=kernels, prof=prof, prof_steps=prof_steps)


def step_scan_roofline(m, pk):
    """Roofline of the scan inside the measured step (the dominant kernel), from the profiled pass."""
    prof = m["prof"]
    names = [k for k in prof if is_scan_kernel(k)]
    scan_ms = sum(prof[k]["total_ms"] for k in names)
    launches = sum(prof[k]["launches"] for k in names if k.startswith("scan_")) or (m["prof_steps"] * m["iters"])
    if scan_ms <= 0:
        return None
    n, positions = m["n"], m["B"] * m["T"]
    per = scan_ms / launches
    fused = [k for k in names if k.startswith("scan_fused")]
    if fused:
        # two launches per scan: the roofline object is the dominant kernel's (its own bytes and flops); the pair
        # is reported against the scan's algorithmic bytes (everything read once) beside it
        per_kernel = {k: prof[k]["total_ms"] / prof[k]["launches"] for k in fused}
        dom = max(per_kernel, key=per_kernel.get)
        reduce_k = dom.startswith("scan_fused_reduce")
        out = roofline_of_scan(n, positions, per_kernel[dom], pk, fused_kernel_bytes(dom, n),
                               NCU_FUSED_TRAFFIC_PER_POSITION.get(dom, {}).get(n), dom, bf16=reduce_k,
                               extra=dict(note="dominant kernel of the step: the chunk reduce of the two-launch scan (J generated from "
                                               "coefficient rows; bf16 m16n8k16 chain products).  bytes = coefficient rows + residual "
                                               "read once (20 n per position); flops = 2 n^2 (n+1) per position",
                                          traffic_note="ncu capture of this kernel at T = 20,000 scaled by positions (profiles/)"))
        pair_ms = sum(per_kernel.values())
        out["scan_pair"] = dict(kernels=per_kernel, ms_per_scan=pair_ms, bytes_per_position=fused_scan_bytes_per_position(n),
                                hbm_frac=fused_scan_bytes_per_position(n) * positions / (pk["hbm_gbs"] * 1e9) * 1e3 / pair_ms,
                                note="reduce + apply of one Newton body against the scan's algorithmic bytes (28 n per position)")
        return out
    extra = None
    traffic = NCU_SCAN_TRAFFIC_PER_POSITION.get(n)
    if m["cfg"] is WORKLOADS[2]:
        extra = dict(traffic=NCU_CONFIG2_SCAN_TRAFFIC,
                     note="this workload (46 MB of J, b per body) is L2-resident: an effective rate, not an HBM claim")
        traffic = None
    return roofline_of_scan(n, positions, per, pk, scan_bytes_per_position(n) + 4 * n, traffic, "+".join(names), extra)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--mode", default="step", choices=["step", "scan", "eval", "sweep", "classifier", "multihead"])
    ap.add_argument("--m", type=int, default=0)
    ap.add_argument("--vjp", type=int, default=0)
    ap.add_argument("--n", type=int, default=8)
    ap.add_argument("--B", type=int, default=None, help="default 16 (classifier mode: 32, config 4)")
    ap.add_argument("--T", type=int, default=None, help="default 1,000,000 (classifier mode: 17,984, config 4)")
    ap.add_argument("--reverse", type=int, default=0)
    ap.add_argument("--flags", type=int, default=0)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="deer", choices=["deer", "reference"])
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--workload", type=int, default=HEADLINE, choices=sorted(WORKLOADS),
                    help="configuration measured as the step (default: the headline, config 3)")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the other workloads and the HBM-sized stand-alone scans (headline workload only)")
    args = ap.parse_args()
    if args.B is None:
        args.B = 32 if args.mode in ("classifier", "multihead") else 16
    if args.T is None:
        args.T = 17_984 if args.mode == "classifier" else 1024 if args.mode == "multihead" else 1_000_000
    if args.impl == "reference":
        run_reference(args)
        return
    if args.mode == "scan":
        run_scan_only(args)
        return
    if args.mode == "eval":
        run_eval_only(args)
        return
    if args.mode == "sweep":
        run_sweep(args)
        return
    if args.mode == "classifier":
        run_classifier(args)
        return
    if args.mode == "multihead":
        run_multihead(args)
        return

    import torch
    from paper_2309_12252_b200 import binding as bd
    from paper_2309_12252_b200 import synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback exists for the product path)")
    bd.lib()
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    args.warmup = max(args.warmup, 3)
    pk = peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)     # > 126 MB L2

    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    head = measure_workload(bd, torch, synth, args.workload, rank, device, dist, args.steps, args.warmup, flush, sampler)
    roofline = step_scan_roofline(head, pk)

    extras = {}
    scans = None
    if rank == 0 and not args.no_extras:
        torch.cuda.empty_cache()
        # ---- the other forward workload of the definition (L2-resident)
        other = 2 if args.workload != 2 else 3
        c2 = measure_workload(bd, torch, synth, other, 0, device, None, max(args.steps, 20), args.warmup, flush)
        extras[f"config{other}"] = dict(workload=c2["cfg"]["workload"], value=c2["value"], unit=UNIT, ms_per_step=c2["ms_per_step"],
                                 newton_iters=c2["iters"], e2e=c2["e2e"], kernels=c2["kernels"],
                                 roofline=step_scan_roofline(c2, pk))
        torch.cuda.empty_cache()
        # ---- config 4: full training step of the 2-layer n = 64 classifier
        c4 = time_classifier(bd, synth, torch, device, 32, 17_984, 0, 3, 2)
        k4 = c4["kernels"]
        per4 = lambda name: k4[name]["ms"] / k4[name]["launches"] if name in k4 else None
        fwd_ms = (per4("scan_fused_reduce64_kernel") or 0.0) + (per4("scan_fused_apply_kernel") or 0.0)
        extras["config4_training_step"] = dict(
            workload="config4: 2-layer GRU n=64 m=6 B=32 T=17984, mean-pool, 5-class head; loss + all gradients",
            ms_per_step=c4["ms"], value=c4["steps_per_s"], unit=UNIT, newton_iters=c4["iters"], loss=c4["loss"],
            kernels=k4,
            forward_scan=dict(ms_per_scan=fwd_ms, kernels="scan_fused_reduce64_kernel + scan_fused_apply_kernel",
                              bytes_per_position=fused_scan_bytes_per_position(64),
                              hbm_frac=fused_scan_bytes_per_position(64) * 32 * 17_984 / (pk["hbm_gbs"] * 1e9) * 1e3 / max(fwd_ms, 1e-9),
                              tensor_frac_bf16=scan_flops_per_position(64) * 32 * 17_984 / (pk["bf16_tflops"] * 1e12) * 1e3 / max(fwd_ms, 1e-9)),
            reverse_scan_roofline=roofline_of_scan(64, 32 * 17_984, per4("scan_cta64_kernel") or 1.0, pk, scan_bytes_per_position(64),
                                                   NCU_SCAN_TRAFFIC_PER_POSITION[64], "scan_cta64_kernel (reverse, 3 x TF32)"))
        torch.cuda.empty_cache()
        # ---- the multi-head GRU unit of the paper's sequential-image model
        extras["multihead_unit"] = time_multihead(bd, synth, torch, device, 32, 1024, 32, 8, 256, 5, 2, cpu_seconds=2.0)
        torch.cuda.empty_cache()
        # ---- stand-alone scans on HBM-sized problems: the roofline of each scan kernel
        scans = []
        for s in SCANS_HBM:
            for reverse in (0, 1):
                ms = time_scan(bd, torch, device, s["n"], s["B"], s["T"], reverse, 0, 10, 3)
                rl = roofline_of_scan(s["n"], s["B"] * s["T"], ms, pk, scan_bytes_per_position(s["n"]),
                                      NCU_SCAN_TRAFFIC_PER_POSITION[s["n"]], scan_kernel_name(s["n"]),
                                      dict(workload=f"n={s['n']} B={s['B']} T={s['T']} reverse={reverse} "
                                                    f"(J {4 * s['n'] ** 2 * s['B'] * s['T'] / 1e9:.2f} GB, inputs > L2)",
                                           reverse=reverse, n=s["n"],
                                           traffic_note="ncu capture of the forward kernel at smaller T scaled by positions (profiles/)"))
                scans.append(rl)
                torch.cuda.empty_cache()
    clocks = sampler.stop()

    cpu = None
    if rank == 0 and world == 1:
        v, reps, dt, cores = cpu_oracle_rate(synth.config(args.workload), args.cpu_seconds)
        cpu = dict(value=v, unit=UNIT, cores=cores, kind="oracle",
                   sample=f"{reps} full passes of the oracle's sequential fp32 GRU loop over the whole workload ({dt:.1f} s)")

    if rank == 0:
        hbm8 = next((s for s in (scans or []) if s["n"] == 8 and s["reverse"] == 0), None)
        line = dict(metric=METRIC, value=head["value"], unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                    ms_per_step=head["ms_per_step"], higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="f32", data="synthetic",
                    config=dict(head["cfg"], global_batch=head["B"] * world,
                                parallelism=f"batch-sharded x{world}, no collective",
                                l2="flushed (256 MiB write) before every timed step; the step's working set (> 1 GB) exceeds L2"),
                    newton_iters=head["iters"], err=head["err"], gpu_launches=head["launches"], clocks=clocks,
                    e2e={k: v for k, v in head["e2e"].items() if k != "ms_per_step"},
                    roofline=roofline, roofline_scan_hbm=hbm8, roofline_scans_hbm=scans, kernels=head["kernels"],
                    workloads=extras, cpu_baseline=cpu)
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
