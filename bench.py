#!/usr/bin/env python
"""Benchmark of the FFT-convolution hot path: one step = fprop + bprop + accGrad
of one layer (all four kernels of each pass) on seeded synthetic tensors.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1] [--math auto]
    python bench.py --impl reference ...     # the float64 CPU oracle on the host cores

Prints ONE JSON line.  `value` is the paper's throughput metric (equivalent
time-domain multiply-adds per second, Section 4.2, times two flops) summed over
the three passes, with the inputs resident in HBM; `e2e` is the same metric with
the host<->device copies inside the timed region; `roofline` describes the
kernel with the largest share of the step; `cpu_baseline` is the oracle timed
on a bounded sample of the same workload.  Under torchrun every rank runs the
same layer on its own minibatch (data parallel over S: fprop and bprop need no
exchange, the weight gradient is summed with one NCCL all-reduce).
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

METRIC = "conv_gflops_equivalent_3pass"
UNIT = "GFLOP/s-equivalent"
FP32_FFMA_TFLOPS_NOMINAL = 148 * 128 * 2 * 1.965e9 / 1e12   # SMs x lanes x 2 flops x max clock
# DRAM bytes (read + write) of one launch from the ncu captures summarised under profiles/,
# keyed by (workload, kernel, pass); None where no capture exists.
NCU_TRAFFIC = {
    # (workload, kernel, pass): read + write, profiles/dram_traffic_per_launch_three_layer_configs.md
    ("mid_S128_f96_fp256_31x31_k5", "r2c_fft_both_operands", "fprop"): 156.5e6,
    ("mid_S128_f96_fp256_31x31_k5", "bin_contraction", "fprop"): 242.4e6,
    ("mid_S128_f96_fp256_31x31_k5", "c2r_ifft", "fprop"): 193.9e6,
    ("mid_S128_f96_fp256_31x31_k5", "r2c_fft_both_operands", "bprop"): 291.0e6,
    ("mid_S128_f96_fp256_31x31_k5", "bin_contraction", "bprop"): 277.1e6,
    ("mid_S128_f96_fp256_31x31_k5", "c2r_ifft", "bprop"): 54.4e6,
    ("mid_S128_f96_fp256_31x31_k5", "r2c_fft_both_operands", "accgrad"): 286.9e6,
    ("mid_S128_f96_fp256_31x31_k5", "bin_contraction", "accgrad"): 257.7e6,
    ("mid_S128_f96_fp256_31x31_k5", "c2r_ifft", "accgrad"): 107.6e6,
    ("largek_S128_f64_fp64_64x64_k11", "r2c_fft_both_operands", "fprop"): 293.1e6,
    ("largek_S128_f64_fp64_64x64_k11", "bin_contraction", "fprop"): 290.4e6,
    ("largek_S128_f64_fp64_64x64_k11", "c2r_ifft", "fprop"): 192.0e6,
    ("largek_S128_f64_fp64_64x64_k11", "r2c_fft_both_operands", "bprop"): 251.9e6,
    ("largek_S128_f64_fp64_64x64_k11", "bin_contraction", "bprop"): 290.1e6,
    ("largek_S128_f64_fp64_64x64_k11", "c2r_ifft", "bprop"): 222.4e6,
    ("largek_S128_f64_fp64_64x64_k11", "r2c_fft_both_operands", "accgrad"): 454.2e6,
    ("largek_S128_f64_fp64_64x64_k11", "bin_contraction", "accgrad"): 324.1e6,
    ("largek_S128_f64_fp64_64x64_k11", "c2r_ifft", "accgrad"): 69.3e6,
    ("deep_S128_f384_fp384_13x13_k3", "r2c_fft_both_operands", "fprop"): 210.8e6,
    ("deep_S128_f384_fp384_13x13_k3", "bin_contraction", "fprop"): 251.7e6,
    ("deep_S128_f384_fp384_13x13_k3", "c2r_ifft", "fprop"): 56.8e6,
    ("deep_S128_f384_fp384_13x13_k3", "r2c_fft_both_operands", "bprop"): 198.2e6,
    ("deep_S128_f384_fp384_13x13_k3", "bin_contraction", "bprop"): 251.8e6,
    ("deep_S128_f384_fp384_13x13_k3", "c2r_ifft", "bprop"): 57.1e6,
    ("deep_S128_f384_fp384_13x13_k3", "r2c_fft_both_operands", "accgrad"): 114.6e6,
    ("deep_S128_f384_fp384_13x13_k3", "bin_contraction", "accgrad"): 222.3e6,
    ("deep_S128_f384_fp384_13x13_k3", "c2r_ifft", "accgrad"): 172.6e6,
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            d = json.load(fh)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


# ---------------------------------------------------------------------------
# Algorithmic bytes / flops of one pass (each real tensor and each spectrum
# crosses HBM once in the FFT stages; the contraction reads two spectra and
# writes one).
# ---------------------------------------------------------------------------
def pass_model(s, which, tile=0):
    n = tile or s.n
    B = n * (n // 2 + 1)
    x_el, w_el, y_el = s.S * s.f * s.h * s.w, s.fp * s.f * s.kh * s.kw, s.S * s.fp * s.oh * s.ow
    # windows per plane with spatial tiling (fprop and accGrad tile the output plane, bprop the input)
    T = 1
    if tile:
        dh, dw = n - s.kh + 1, n - s.kw + 1
        cd = lambda a, b: (a + b - 1) // b
        T = cd(s.h, dh) * cd(s.w, dw) if which == "bprop" else cd(s.oh, dh) * cd(s.ow, dw)
    x_pl, w_pl, y_pl = s.S * s.f * T, s.fp * s.f, s.S * s.fp * T
    if which == "fprop":
        a, b, c = (x_el, x_pl), (w_el, w_pl), (y_el, y_pl)
    elif which == "bprop":
        a, b, c = (y_el, y_pl), (w_el, w_pl), (x_el, x_pl)
    else:
        a, b, c = (y_el, y_pl), (x_el, x_pl), (w_el, w_pl)
    spec = lambda planes: planes * B * 8
    stage_bytes = [a[0] * 4 + spec(a[1]), b[0] * 4 + spec(b[1]),
                   spec(a[1]) + spec(b[1]) + spec(c[1]), spec(c[1]) + c[0] * 4]
    return {
        "stage_bytes": stage_bytes,                         # fft A, fft B, contraction, ifft
        "b_fft": stage_bytes[0] + stage_bytes[1] + stage_bytes[3],
        "b_gemm": stage_bytes[2],
        "gemm_flops": 8.0 * s.S * T * s.f * s.fp * B,
        "equiv_flops": 2.0 * s.macs,
    }


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid, self.proc, self.lines = uuid, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.uuid, "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = [l for (t, l) in self.lines if t0 <= t <= t1 + 0.12] or [l for (_, l) in self.lines]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in rows:
            parts = [p.strip() for p in l.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------
def oracle_sample_run(s, x, w, dy, budget_s):
    """Times the oracle (as it stands) on a bounded sample of output elements of
    each pass; returns (equivalent flops done, seconds, description)."""
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    per = {"fprop": s.f * s.kh * s.kw, "bprop": s.fp * s.kh * s.kw, "accgrad": s.S * s.oh * s.ow}
    dims = {"fprop": (s.S, s.fp, s.oh, s.ow), "bprop": (s.S, s.f, s.h, s.w),
            "accgrad": (s.fp, s.f, s.kh, s.kw)}
    fns = {"fprop": lambda c: oracle.fprop_at(x, w, c),
           "bprop": lambda c: oracle.bprop_at(dy, w, s.h, s.w, c),
           "accgrad": lambda c: oracle.accgrad_at(dy, x, s.kh, s.kw, c)}
    total_macs, total_t, desc = 0.0, 0.0, []
    for name in ("fprop", "bprop", "accgrad"):
        # calibrate on a small sample, then size the timed sample to the budget
        c0 = wl.sample_coords(dims[name], 2048, seed=1)
        t = time.perf_counter(); fns[name](c0); dt = max(time.perf_counter() - t, 1e-6)
        rate = len(c0) / dt
        nel = int(min(max(rate * budget_s / 3.0, 2048), 50_000_000))
        c = wl.sample_coords(dims[name], nel, seed=2)
        t = time.perf_counter(); fns[name](c); dt = time.perf_counter() - t
        # bprop border elements have fewer valid taps; count the formula's nominal taps
        total_macs += float(len(c)) * per[name]
        total_t += dt
        desc.append("%s:%d elems" % (name, len(c)))
    return 2.0 * total_macs, total_t, ", ".join(desc)


def run_reference(args, s):
    """--impl reference: the float64 oracle on the host cores, bounded sample per step."""
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    cores = oracle.num_threads()
    per_step = 3.0
    for _ in range(args.warmup):
        oracle_sample_run(s, x, w, dy, 0.3)
    vals, times, desc = [], [], ""
    for _ in range(args.steps):
        fl, t, desc = oracle_sample_run(s, x, w, dy, per_step)
        vals.append(fl / t / 1e9); times.append(t)
    vals.sort()
    v = vals[len(vals) // 2]
    line = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * sum(times) / max(len(times), 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": s.name, "sample": "per step: " + desc},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "per step: " + desc},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------
def run_ours(args, s):
    import numpy as np
    import torch
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    peaks = load_peaks()
    math = {"auto": fc.MATH_AUTO, "fp32": fc.MATH_FP32, "tf32": fc.MATH_TF32}[args.math]
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    plan = fc.conv_plan(*s.args())
    fc.conv_plan_set_math(plan, math)
    if args.tile:
        fc.conv_plan_set_tiling(plan, args.tile)      # -1: the plan chooses
    tile = fc.conv_plan_tile_basis(plan)
    ws = fc.conv_plan_alloc_workspace(plan)
    eff = fc.conv_plan_effective_math(plan)
    hx, hw_, hdy = (torch.from_numpy(a).pin_memory() for a in (x, w, dy))
    xd, wd, dyd = hx.cuda(), hw_.cuda(), hdy.cuda()
    y = torch.empty((s.S, s.fp, s.oh, s.ow), device="cuda")
    dx = torch.empty((s.S, s.f, s.h, s.w), device="cuda")
    dw = torch.empty((s.fp, s.f, s.kh, s.kw), device="cuda")
    hy, hdx, hdw = (torch.empty(t.shape, dtype=torch.float32).pin_memory() for t in (y, dx, dw))

    def step():
        fc.conv_fprop(plan, xd, wd, y)
        fc.conv_bprop(plan, dyd, wd, dx)
        fc.conv_accgrad(plan, dyd, xd, dw)
        if dist is not None:
            dist.all_reduce(dw)        # data parallel over S: sum of the per-rank weight gradients

    # End to end: every step copies x, w, dy from pinned host memory and y, dx, dw back.  The
    # copies run on their own streams so that the two PCIe directions and the kernels overlap;
    # each pass waits only for the tensors it reads, each read-back for the pass that wrote it.
    main_stream = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev = {k: torch.cuda.Event() for k in ("xw", "dy", "y", "dx", "dw")}

    small = 4 * (x.size + w.size + dy.size) < (8 << 20)     # a few MB: stream hand-offs cost more than they hide

    def step_e2e():
        if small:
            xd.copy_(hx, non_blocking=True); wd.copy_(hw_, non_blocking=True)
            dyd.copy_(hdy, non_blocking=True)
            step()
            hy.copy_(y, non_blocking=True); hdx.copy_(dx, non_blocking=True)
            hdw.copy_(dw, non_blocking=True)
            return
        s_in.wait_stream(main_stream)          # the previous step has read its inputs
        with torch.cuda.stream(s_in):
            xd.copy_(hx, non_blocking=True); wd.copy_(hw_, non_blocking=True)
            ev["xw"].record(s_in)
            dyd.copy_(hdy, non_blocking=True)
            ev["dy"].record(s_in)
        main_stream.wait_stream(s_out)         # the previous step's results have left the device
        main_stream.wait_event(ev["xw"])
        fc.conv_fprop(plan, xd, wd, y)
        ev["y"].record(main_stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev["y"]); hy.copy_(y, non_blocking=True)
        main_stream.wait_event(ev["dy"])
        fc.conv_bprop(plan, dyd, wd, dx)
        ev["dx"].record(main_stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev["dx"]); hdx.copy_(dx, non_blocking=True)
        fc.conv_accgrad(plan, dyd, xd, dw)
        if dist is not None:
            dist.all_reduce(dw)
        ev["dw"].record(main_stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev["dw"]); hdw.copy_(dw, non_blocking=True)

    def e2e_drain():
        main_stream.wait_stream(s_out)         # the timed region ends when the last result is on the host

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, drain=None):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(steps):
            fn()
        if drain is not None:
            drain()
        e1.record()
        barrier()
        ms = e0.elapsed_time(e1)
        if dist is not None:
            t = torch.tensor([ms], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms

    for _ in range(max(args.warmup, 3)):
        step()
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(local).uuid).replace("GPU-", ""))
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    launches0 = fc.fftconv_launch_count()
    t0 = time.time()
    ms_total = timed(step, args.steps)
    # keep the GPU under the same load a little longer so the clock sampler sees it
    reps = 0
    while time.time() - t0 < 1.0 and reps < 200:
        step(); reps += 1
    torch.cuda.synchronize()
    t1 = time.time()
    # counted by the library.  Per pass: the forward FFTs (one launch for both operands with the
    # one-pass kernels, one per operand with the two-pass kernels), the contraction, the inverse FFT
    counted = fc.fftconv_launch_count() - launches0
    assert counted % (args.steps + reps) == 0 and counted // (args.steps + reps) in (9, 12)
    launches = counted // (args.steps + reps) * args.steps
    clocks = sampler.stop(t0, t1) if rank == 0 else None
    ms_step = ms_total / args.steps

    for _ in range(2):
        step_e2e()
    ms_e2e = timed(step_e2e, args.steps, e2e_drain) / args.steps
    assert fc.conv_plan_status(plan) == 0

    flops_step = 3 * 2.0 * s.macs
    value = world * flops_step / (ms_step * 1e-3) / 1e9
    e2e_value = world * flops_step / (ms_e2e * 1e-3) / 1e9

    names = ["fprop", "bprop", "accgrad"]
    calls = [lambda: fc.conv_fprop(plan, xd, wd, y), lambda: fc.conv_bprop(plan, dyd, wd, dx),
             lambda: fc.conv_accgrad(plan, dyd, xd, dw)]
    reps = max(args.steps, 10)

    # per-pass durations, normal launch sequence, CUDA events on the launching stream
    pass_ms = {n: [] for n in names}
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
           for _ in range(3 * reps)]
    torch.cuda.synchronize()
    k = 0
    for _ in range(reps):
        for c in calls:
            evs[k][0].record(); c(); evs[k][1].record(); k += 1
    torch.cuda.synchronize()
    k = 0
    for _ in range(reps):
        for n in names:
            pass_ms[n].append(evs[k][0].elapsed_time(evs[k][1])); k += 1

    # per-kernel durations from CUDA events recorded by the library on its stream:
    # mode 1 = the normal launch sequence (fused forward FFT, contraction, inverse FFT),
    # mode 2 = the two forward FFTs launched apart (detail only)
    def stage_times(mode):
        fc.conv_plan_enable_stage_timing(plan, mode)
        acc = {n: np.zeros(4) for n in names}
        for _ in range(reps):
            for n, c in zip(names, calls):
                c()
                acc[n] += np.array(fc.conv_plan_stage_times_ms(plan))
        fc.conv_plan_enable_stage_timing(plan, 0)
        return {n: acc[n] / reps for n in names}
    st1, st2 = stage_times(1), stage_times(2)

    tf32_peak = peaks["bf16_tflops_sustained"] / 2.0
    p_tflops = tf32_peak if eff == fc.MATH_TF32 else FP32_FFMA_TFLOPS_NOMINAL
    bw = peaks["hbm_gbs"] * 1e9
    passes, best = {}, None
    kernel_names = ["r2c_fft_both_operands", None, "bin_contraction", "c2r_ifft"]
    for n in names:
        m = pass_model(s, n, tile)
        t_ms = float(np.median(pass_ms[n]))
        t_roof = max(m["b_fft"] / bw, m["gemm_flops"] / (p_tflops * 1e12))
        t_stage = max((m["b_fft"] + m["b_gemm"]) / bw, m["gemm_flops"] / (p_tflops * 1e12))
        kbytes = [m["stage_bytes"][0] + m["stage_bytes"][1], 0, m["stage_bytes"][2], m["stage_bytes"][3]]
        passes[n] = {
            "ms": t_ms, "ms_min": float(np.min(pass_ms[n])),
            "gflops_equiv": m["equiv_flops"] / (t_ms * 1e-3) / 1e9,
            "roofline_us": t_roof * 1e6, "roofline_frac": t_roof / (t_ms * 1e-3),
            "unfused_roofline_us": t_stage * 1e6, "unfused_roofline_frac": t_stage / (t_ms * 1e-3),
            "kernel_ms": {kernel_names[k]: float(st1[n][k]) for k in (0, 2, 3)},
            "forward_fft_apart_ms": {"A": float(st2[n][0]), "B": float(st2[n][1])},
        }
        for k in (0, 2, 3):
            cand = (float(st1[n][k]), n, k, m, kbytes[k])
            if best is None or cand[0] > best[0]:
                best = cand
    dur_ms, bn, bk, bm, bbytes = best
    if bk == 2 and bm["gemm_flops"] / (p_tflops * 1e12) > bbytes / bw:
        ach = bm["gemm_flops"] / (dur_ms * 1e-3) / 1e12
        roof = {"bound": "tensor" if eff == fc.MATH_TF32 else "alu", "achieved": ach,
                "peak": p_tflops, "unit": "TFLOP/s", "frac": ach / p_tflops}
    else:
        ach = bbytes / (dur_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"]}
    roof.update({"traffic": None if tile else NCU_TRAFFIC.get((s.name, kernel_names[bk], bn)),
                 "kernel": "%s/%s" % (bn, kernel_names[bk]),
                 "kernel_ms": dur_ms, "algorithmic_bytes": bbytes,
                 "peak_source": peaks["source"] + (" sustained bf16 / 2" if roof["bound"] == "tensor" else "")})

    # extra (not the headline, which re-transforms every operand in every pass): the same
    # step with the forward spectra shared between the passes of the step
    reuse = None
    if not args.no_reuse_line and not tile:
        plan_r = fc.conv_plan(*s.args())
        fc.conv_plan_set_math(plan_r, math)
        fc.conv_plan_set_spectrum_reuse(plan_r, True)
        ws_r = fc.conv_plan_alloc_workspace(plan_r)

        def step_r():
            fc.conv_fprop(plan_r, xd, wd, y)
            fc.conv_bprop(plan_r, dyd, wd, dx)
            fc.conv_accgrad(plan_r, dyd, xd, dw)
        for _ in range(3):
            step_r()
        lr0 = fc.fftconv_launch_count()
        ms_r = timed(step_r, args.steps) / args.steps
        launches_r = (fc.fftconv_launch_count() - lr0) // args.steps
        reuse = {"ms_per_step": ms_r, "value": world * flops_step / (ms_r * 1e-3) / 1e9, "unit": UNIT,
                 "gpu_launches_per_step": launches_r, "workspace_bytes": int(ws_r.numel()),
                 "note": "x, w, dy spectra computed once per step and shared by the three passes"}
        fc.conv_plan_destroy(plan_r)
        del ws_r

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        fl, t, desc = oracle_sample_run(s, x, w, dy, args.cpu_budget)
        cpu = {"value": fl / t / 1e9, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
               "sample": desc + " (sampled output elements of each pass, plain definition, float64)"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "tf32" if eff == fc.MATH_TF32 else "f32", "data": "synthetic",
            "config": {"workload": s.name, "S": s.S, "f": s.f, "fprime": s.fp, "h": s.h, "w": s.w,
                       "kh": s.kh, "kw": s.kw, "n": s.n, "tile_basis": tile,
                       "passes": "fprop+bprop+accgrad",
                       "parallelism": "dp%d over S" % world,
                       "l2": "working set %.0f MB > 126 MB L2, no flush" % (
                           (ws.numel() + 4 * (x.size + w.size + dy.size) * 2) / 1e6)},
            "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": ms_e2e,
                    "h2d_bytes_per_step": int(4 * (x.size + w.size + dy.size)),
                    "d2h_bytes_per_step": int(4 * (y.numel() + dx.numel() + dw.numel()))},
            "gpu_launches": launches, "clocks": clocks, "roofline": roof, "cpu_baseline": cpu,
            "passes": passes, "step_with_spectrum_reuse": reuse,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1, help="0 tiny, 1 mid (default), 2 large-kernel, 3 deep")
    ap.add_argument("--shape", default=None,
                    help="S,f,fp,h,w,kh,kw,n : a layer shape of your own instead of --config "
                         "(seeded inputs as in the sweep; used for profiling single shapes)")
    ap.add_argument("--math", default="auto", choices=["auto", "fp32", "tf32"])
    ap.add_argument("--tile", type=int, default=0,
                    help="spatial tiling with this basis (8, 16, 32 or 64; 0 = off); bytes, flops and the "
                         "roofline in the output are then those of the tiled method")
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of oracle work for cpu_baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-reuse-line", action="store_true",
                    help="skip the extra measurement of a step with spectrum reuse between passes")
    args = ap.parse_args()
    from paper_1412_7580_b200 import workloads as wl
    s = wl.CONFIGS[args.config]
    if args.shape:
        dims = [int(v) for v in args.shape.split(",")]
        assert len(dims) == 8, "--shape wants S,f,fp,h,w,kh,kw,n"
        s = wl.ConvShape("custom_S%d_f%d_fp%d_%dx%d_k%dx%d_n%d" % tuple(dims), *dims, cfg=6,
                         point=sum(dims), w_dist="fan_in", dy_dist="normal")
    if args.impl == "reference":
        run_reference(args, s)
    else:
        run_ours(args, s)


if __name__ == "__main__":
    main()
