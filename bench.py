#!/usr/bin/env python
"""Benchmark of the DEER-GRU hot path on B200.

One "step" = one whole `deer_gru_eval` (input projection + all Newton bodies:
cell + Jacobian + rhs, scan, convergence) over the benchmark workload
(GRU n=8, m=4, B=16, T=10,000, fp32, sinusoid+noise inputs, zero initial
state and zero initial guess).  `value` = B*T positions evaluated per second,
inputs resident in HBM; `e2e` = the same through the host-buffer call with
the H2D copy of x and the D2H copy of y inside the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

N > 1 (under torchrun): every rank evaluates its own batch of the same shape
(sequences are independent: no data-path collective), weak scaling; the timed
region is bracketed by barriers and the maximum over ranks is reported.
`--impl reference` times the CPU oracle's sequential fp32 loop instead.
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
WORKLOAD = dict(workload="config2: GRU n=8 m=4 B=16 T=10000 fp32, x=sin(wt+phi)+0.1N(0,1), y0=0, zero guess",
                n=8, m=4, B=16, T=10000, tol=1e-4, max_iter=100)
SCAN_HBM = dict(n=8, B=16, T=1_000_000)     # stand-alone scan sized well beyond L2 (J = 4.1 GB)


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


# DRAM bytes (read + write) per position of the stand-alone scan, from the ncu captures summarised in
# profiles/scan_kernels_standalone_B16.md (inputs larger than L2; traffic grows in proportion to positions).
NCU_STEP_SCAN_TRAFFIC = 51.43e6      # config-2 step, scan_warp8_kernel: dram read + write per launch
NCU_SCAN_TRAFFIC_PER_POSITION = {1: 12.8, 2: 32.7, 4: 95.3, 8: 606.6, 16: 2213.0, 32: 8622.0, 64: 34116.0}


def scan_bytes_per_position(n: int) -> int:
    """Algorithmic bytes of one scan per position: read J and b once, write y."""
    return 4 * (n * n + n) + 4 * n


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period: float = 0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
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
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(get(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_ev.set()
        self.join(timeout=2)
        med = int(np.median(self.samples)) if self.samples else None
        return dict(sm_mhz=med, sm_max_mhz=self.max_mhz, reasons=sorted(self.reasons), samples=len(self.samples))


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
    w = synth.config(2)
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
                dtype="f32", data="synthetic", impl="reference", config=dict(WORKLOAD),
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


def run_scan_only(args):
    """Stand-alone linear-recurrence scan at the given size: prints one JSON line."""
    import torch
    from paper_2309_12252_b200 import binding as bd
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    n, B, T = args.n, args.B, args.T
    g = torch.Generator(device=device); g.manual_seed(0)
    J = (torch.rand((B, T, n, n), device=device, generator=g) * 2 - 1) * (0.9 / n)
    bb = torch.randn((B, T, n), device=device, generator=g)
    yy = torch.empty_like(bb)
    ws = bd.alloc_workspace(bd.DEER_OP_SCAN, B, T, n, 1, args.flags, device)
    stream = torch.cuda.current_stream()
    for _ in range(max(args.warmup, 1)):
        bd.deer_linrec_scan(J, bb, None, bool(args.reverse), yy, ws, args.flags, stream)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    torch.cuda.synchronize()
    for a, b in ev:
        a.record(stream)
        bd.deer_linrec_scan(J, bb, None, bool(args.reverse), yy, ws, args.flags, stream)
        b.record(stream)
    torch.cuda.synchronize()
    ms = float(np.median([a.elapsed_time(b) for a, b in ev]))
    pk = peaks()
    ach = scan_bytes_per_position(n) * B * T / (ms * 1e-3) / 1e9
    print(json.dumps(dict(mode="scan", n=n, B=B, T=T, reverse=int(args.reverse), flags=args.flags, ms=ms,
                          positions_per_s=B * T / (ms * 1e-3), achieved_gbs=ach, peak_gbs=pk["hbm_gbs"],
                          frac=ach / pk["hbm_gbs"], peak_source=pk["source"],
                          input_mb=(n * n + n) * 4 * B * T / 1e6)))


def eval_point(bd, synth, device, n, m, B, T, flags, steps, warmup, vjp=False, breakdown=True):
    """deer_gru_eval (optionally deer_gru_vjp) at one sweep point (x ~ N(0,1), y0 = 0): a dict of timings."""
    import torch
    p = bd.GruParamsDev.from_numpy(synth.gru_params(n, m, 0, tag=f"sweep{n}/gru"))
    g = torch.Generator(device=device); g.manual_seed(0)
    x = torch.randn((B, T, m), device=device, generator=g)
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
        scan_ms = sum(v["total_ms"] for k, v in prof.items() if k.startswith("scan_") and "prep" not in k or k.startswith("gen_"))
        if scan_ms > 0 and r.iters > 0:
            pk = peaks()
            per = scan_ms / r.iters
            out["scan_ms_per_iter"] = per
            out["scan_frac_hbm"] = scan_bytes_per_position(n) * B * T / (per * 1e-3) / 1e9 / pk["hbm_gbs"]
    if vjp:
        gy = torch.randn((B, T, n), device=device, generator=g)
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
    """One sweep point chosen on the command line: prints one JSON line."""
    import torch
    from paper_2309_12252_b200 import binding as bd
    from paper_2309_12252_b200 import synth
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    out = eval_point(bd, synth, device, args.n, args.m or args.n, args.B, args.T, args.flags,
                     args.steps, args.warmup, vjp=bool(args.vjp))
    out["mode"] = "eval"
    print(json.dumps(out))


def run_classifier(args):
    """Config 4: one full training step (loss + all gradients) of the 2-layer GRU classifier: one JSON line."""
    import torch
    from paper_2309_12252_b200 import binding as bd
    from paper_2309_12252_b200 import synth
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    w = synth.config4(seed=0, B=args.B, T=args.T)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device)
    l1 = bd.GruParamsDev.from_numpy(w.layers[0]); l2 = bd.GruParamsDev.from_numpy(w.layers[1])
    W_o, b_o, x, labels = dev(w.W_o), dev(w.b_o), dev(w.x), dev(w.labels)
    n, m = w.layers[0].n, w.layers[0].m
    ws = bd.alloc_workspace(bd.DEER_OP_CLASSIFIER, args.B, args.T, n, m, args.flags, device)
    stream = torch.cuda.current_stream()
    run = lambda: bd.deer_gru_classifier_step(l1, l2, W_o, b_o, x, labels, ws=ws, flags=args.flags, stream=stream)
    for _ in range(max(args.warmup, 1)):
        r = run()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    torch.cuda.synchronize()
    for a, b in ev:
        a.record(stream); r = run(); b.record(stream)
    torch.cuda.synchronize()
    ms = float(np.median([a.elapsed_time(b) for a, b in ev]))
    bd.lib().deer_profile_enable(1)
    run()
    torch.cuda.synchronize()
    bd.lib().deer_profile_enable(0)
    prof = read_profile(bd)
    print(json.dumps(dict(mode="classifier", B=args.B, T=args.T, n=n, m=m, ms=ms, steps_per_s=args.B * args.T / (ms * 1e-3),
                          loss=r["loss"], iters=list(r["iters"]), status=r["status"],
                          kernels={k: dict(launches=v["launches"], ms=round(v["total_ms"], 4)) for k, v in prof.items()})))


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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--mode", default="step", choices=["step", "scan", "eval", "sweep", "classifier"])
    ap.add_argument("--m", type=int, default=0)
    ap.add_argument("--vjp", type=int, default=0)
    ap.add_argument("--n", type=int, default=8)
    ap.add_argument("--B", type=int, default=None, help="default 16 (classifier mode: 32, config 4)")
    ap.add_argument("--T", type=int, default=None, help="default 1,000,000 (classifier mode: 17,984, config 4)")
    ap.add_argument("--reverse", type=int, default=0)
    ap.add_argument("--flags", type=int, default=0)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="deer", choices=["deer", "reference"])
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--no-scan-hbm", action="store_true", help="skip the HBM-sized stand-alone scan measurement")
    args = ap.parse_args()
    if args.B is None:
        args.B = 32 if args.mode == "classifier" else 16
    if args.T is None:
        args.T = 17_984 if args.mode == "classifier" else 1_000_000
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

    w = synth.config(2, seed=rank)              # each rank: its own batch of the same shape
    B, T, n, m = w.B, w.T, w.n, w.m
    p = bd.GruParamsDev.from_numpy(synth.config(2, seed=0, B=1, T=1).params)   # same weights on every rank
    x_host = torch.from_numpy(w.x).pin_memory()
    y_host = torch.empty((B, T, n), dtype=torch.float32).pin_memory()
    x = x_host.to(device)
    y0 = torch.zeros((B, n), device=device)
    y = torch.empty((B, T, n), device=device)
    ws = bd.alloc_workspace(bd.DEER_OP_EVAL, B, T, n, m, 0, device)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)     # > 126 MB L2
    stream = torch.cuda.current_stream()

    def step():
        return bd.deer_gru_eval(p, x, y0, WORKLOAD["tol"], WORKLOAD["max_iter"], y, ws, 0, stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        r = step()
    iters = r.iters
    assert r.status == 0, bd.deer_status_string(r.status)

    # ---- timed region: K steps, L2 flushed before each, per-step CUDA events on the launching stream
    sampler = ClockSampler(physical_gpu_index(local_rank))
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    sampler.start()
    launches0 = bd.deer_launch_count()
    for a, b in ev:
        flush.fill_(1)
        a.record(stream)
        r = step()
        b.record(stream)
    barrier()
    launches = bd.deer_launch_count() - launches0
    clocks = sampler.stop()
    local_ms = sum(a.elapsed_time(b) for a, b in ev)
    total_ms, total_units = aggregate_over_ranks(local_ms, float(args.steps) * B * T, dist, device)
    value = total_units / (total_ms * 1e-3)

    # ---- end to end: host buffers, H2D of x and D2H of y inside the timed region
    for _ in range(3):
        bd.deer_gru_eval_host(p, x_host, y0, y_host, x, y, ws, WORKLOAD["tol"], WORKLOAD["max_iter"], 0, stream)
    ev2 = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    for a, b in ev2:
        flush.fill_(1)
        a.record(stream)
        bd.deer_gru_eval_host(p, x_host, y0, y_host, x, y, ws, WORKLOAD["tol"], WORKLOAD["max_iter"], 0, stream)
        b.record(stream)
    barrier()
    e2e_ms, e2e_units = aggregate_over_ranks(sum(a.elapsed_time(b) for a, b in ev2), float(args.steps) * B * T, dist, device)
    e2e = dict(value=e2e_units / (e2e_ms * 1e-3), unit=UNIT, h2d_bytes_per_step=int(x_host.numel() * 4),
               d2h_bytes_per_step=int(y_host.numel() * 4))

    # ---- per-kernel breakdown of the same steps (separate pass: event pairs around every launch)
    prof_steps = min(args.steps, 20)
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
    pk = peaks()
    scan_names = [k for k in prof if ("scan" in k or "reduce" in k or "carry" in k or "apply" in k)]
    scan_ms = sum(prof[k]["total_ms"] for k in scan_names)
    scans = prof_steps * iters
    roofline = None
    if scan_ms > 0:
        ach = scan_bytes_per_position(n) * B * T / (scan_ms / scans * 1e-3) / 1e9
        roofline = dict(bound="hbm", kernel="+".join(scan_names), achieved=ach, peak=pk["hbm_gbs"], unit="GB/s",
                        frac=ach / pk["hbm_gbs"], peak_source=pk["source"], traffic=NCU_STEP_SCAN_TRAFFIC,
                        traffic_note="DRAM bytes per scan launch of this workload under ncu (caches flushed before each "
                                     "kernel): one read of J, b, y_old; the second visit of every tile is served by L2 "
                                     "(profiles/bench_step_config2_launch_list.md)",
                        note="scan inside the step; this workload (46 MB of J,b per body) is L2-resident, "
                             "so this is an effective rate; see roofline_scan_hbm for the HBM-sized scan")

    # ---- stand-alone scan on an HBM-sized problem (rank 0 only): the roofline of the dominant kernel
    roofline_hbm = None
    if rank == 0 and not args.no_scan_hbm:
        sn, sB, sT = SCAN_HBM["n"], SCAN_HBM["B"], SCAN_HBM["T"]
        g = torch.Generator(device=device); g.manual_seed(0)
        J = (torch.rand((sB, sT, sn, sn), device=device, generator=g) * 2 - 1) * (0.9 / sn)
        bb = torch.randn((sB, sT, sn), device=device, generator=g)
        yy = torch.empty_like(bb)
        sws = bd.alloc_workspace(bd.DEER_OP_SCAN, sB, sT, sn, 1, 0, device)
        for _ in range(3):
            bd.deer_linrec_scan(J, bb, None, False, yy, sws, 0, stream)
        reps = 10
        se = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        torch.cuda.synchronize()
        for a, b in se:
            a.record(stream)
            bd.deer_linrec_scan(J, bb, None, False, yy, sws, 0, stream)
            b.record(stream)
        torch.cuda.synchronize()
        ms = float(np.median([a.elapsed_time(b) for a, b in se]))
        ach = scan_bytes_per_position(sn) * sB * sT / (ms * 1e-3) / 1e9
        roofline_hbm = dict(bound="hbm", kernel="deer_linrec_scan", workload=f"n={sn} B={sB} T={sT} (J 4.1 GB, inputs > L2)",
                            achieved=ach, peak=pk["hbm_gbs"], unit="GB/s", frac=ach / pk["hbm_gbs"],
                            peak_source=pk["source"], ms=ms,
                            traffic=NCU_SCAN_TRAFFIC_PER_POSITION[sn] * sB * sT,
                            traffic_note="bytes per launch: ncu capture at T=200000 scaled by positions "
                                         "(profiles/scan_kernels_standalone_B16.md)",
                            frac_two_reads=(scan_bytes_per_position(sn) + 4 * (sn * sn + sn)) * sB * sT
                                           / (ms * 1e-3) / 1e9 / pk["hbm_gbs"])
        del J, bb, yy, sws

    cpu = None
    if rank == 0 and world == 1:
        v, reps, dt, cores = cpu_oracle_rate(synth.config(2), args.cpu_seconds)
        cpu = dict(value=v, unit=UNIT, cores=cores, kind="oracle",
                   sample=f"{reps} full passes of the oracle's sequential fp32 GRU loop over the whole workload ({dt:.1f} s)")

    if rank == 0:
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                    ms_per_step=total_ms / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="f32", data="synthetic",
                    config=dict(WORKLOAD, global_batch=B * world, parallelism=f"batch-sharded x{world}, no collective",
                                l2="flushed (256 MiB write) before every timed step"),
                    newton_iters=iters, err=r.err, gpu_launches=int(launches), clocks=clocks, e2e=e2e,
                    roofline=roofline, roofline_scan_hbm=roofline_hbm, kernels=kernels, cpu_baseline=cpu)
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
