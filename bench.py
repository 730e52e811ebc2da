#!/usr/bin/env python
"""Benchmark of the FFT-convolution hot path: one step = fprop + bprop + accGrad
of one layer (all kernels of each pass) on seeded synthetic tensors.

    python bench.py [--gpus N] [--steps K] [--warmup W]      # the whole contract, one JSON line
    python bench.py --config 1 ...                           # one layer config only (0 tiny, 1 mid, 2 large-kernel, 3 deep)
    python bench.py --shape S,f,fp,h,w,kh,kw,n [--tile t]    # a layer shape of your own
    python bench.py --sweep-only --sweep-points 1000 --sweep-budget 900 --sweep-out sweep.jsonl
    python bench.py --fft2d | --fft1d                        # throughput of the bare transforms
    python bench.py --impl reference ...                     # the float64 CPU oracle on the host cores

Prints ONE JSON line.  `value` is the paper's throughput metric (equivalent
time-domain multiply-adds per second, Section 4.2, times two flops) summed over
the three passes, with the inputs resident in HBM, on the headline workload: the
large-kernel layer, the largest of the single-GPU layer configs.  The timed
region is `--steps` steps long and is repeated until at least a second of GPU
time has been measured; `ms_per_step` is the median over those blocks.  `e2e` is
the same metric with the host<->device copies inside the timed region;
`roofline` describes the kernel with the largest share of the step;
`cpu_baseline` is the oracle timed on a bounded sample of the same workload.
Without `--config` / `--shape` the line also carries `configs` (the same
measurements for all four layer configs) and `sweep` (a time-boxed, stratified
run of the parameter sweep: per-pass roofline fractions per basis).  Under
torchrun every rank runs the same layer on its own minibatch (data parallel over
S: fprop and bprop need no exchange, the weight gradient is summed with one NCCL
all-reduce).
"""
from __future__ import annotations

import argparse
import hashlib
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
HEADLINE_CONFIG = 2                                         # the large-kernel layer
FP32_FFMA_TFLOPS_NOMINAL = 148 * 128 * 2 * 1.965e9 / 1e12   # SMs x lanes x 2 flops x max clock
MIN_TIMED_MS = 1000.0                                       # GPU time measured per number
MAX_BLOCKS = 400

# DRAM bytes (read + write) of one launch from the ncu capture summarised in the profile named
# below, keyed by (workload, kernel, pass).  The capture belongs to one state of the kernel
# sources; `kernel_sources_sha256` is the digest of paper_1412_7580_b200/csrc at that state, and
# the bench reports the figure only while the sources still have that digest.
NCU_TRAFFIC_SOURCE = {
    "profile": "profiles/dram_traffic_per_launch_three_layer_configs.md",
    "ncu": "dram__bytes_read.sum + dram__bytes_write.sum, default cache control (caches flushed before each launch)",
    "kernel_sources_sha256": "8093a5cb9b8182a7ddaf386527d8b43b04cee811388ada43c98902d481bfc6b8",
}
NCU_TRAFFIC = {
    "mid_S128_f96_fp256_31x31_k5/r2c_fft_first_operand/fprop": 55.0e6,
    "mid_S128_f96_fp256_31x31_k5/r2c_fft_small_planes/fprop": 40.5e6,
    "mid_S128_f96_fp256_31x31_k5/bin_contraction/fprop": 226.1e6,
    "mid_S128_f96_fp256_31x31_k5/c2r_ifft/fprop": 194.6e6,
    "mid_S128_f96_fp256_31x31_k5/r2c_fft_first_operand/bprop": 186.8e6,
    "mid_S128_f96_fp256_31x31_k5/r2c_fft_small_planes/bprop": 41.0e6,
    "mid_S128_f96_fp256_31x31_k5/bin_contraction/bprop": 261.7e6,
    "mid_S128_f96_fp256_31x31_k5/c2r_ifft/bprop": 54.4e6,
    "mid_S128_f96_fp256_31x31_k5/r2c_fft_both_operands/accgrad": 286.6e6,
    "mid_S128_f96_fp256_31x31_k5/bin_contraction/accgrad": 240.9e6,
    "mid_S128_f96_fp256_31x31_k5/c2r_ifft/accgrad": 101.2e6,
    "largek_S128_f64_fp64_64x64_k11/r2c_fft_first_operand/fprop": 227.2e6,
    "largek_S128_f64_fp64_64x64_k11/r2c_fft_small_planes/fprop": 7.9e6,
    "largek_S128_f64_fp64_64x64_k11/bin_contraction/fprop": 280.0e6,
    "largek_S128_f64_fp64_64x64_k11/c2r_ifft/fprop": 187.9e6,
    "largek_S128_f64_fp64_64x64_k11/r2c_fft_first_operand/bprop": 183.1e6,
    "largek_S128_f64_fp64_64x64_k11/r2c_fft_small_planes/bprop": 7.8e6,
    "largek_S128_f64_fp64_64x64_k11/bin_contraction/bprop": 280.5e6,
    "largek_S128_f64_fp64_64x64_k11/c2r_ifft/bprop": 217.3e6,
    "largek_S128_f64_fp64_64x64_k11/r2c_fft_both_operands/accgrad": 457.9e6,
    "largek_S128_f64_fp64_64x64_k11/bin_contraction/accgrad": 313.7e6,
    "largek_S128_f64_fp64_64x64_k11/c2r_ifft/accgrad": 67.2e6,
    "deep_S128_f384_fp384_13x13_k3/r2c_fft_first_operand/fprop": 38.4e6,
    "deep_S128_f384_fp384_13x13_k3/r2c_fft_small_planes/fprop": 100.3e6,
    "deep_S128_f384_fp384_13x13_k3/bin_contraction/fprop": 224.6e6,
    "deep_S128_f384_fp384_13x13_k3/c2r_ifft/fprop": 56.7e6,
    "deep_S128_f384_fp384_13x13_k3/r2c_fft_first_operand/bprop": 25.3e6,
    "deep_S128_f384_fp384_13x13_k3/r2c_fft_small_planes/bprop": 99.6e6,
    "deep_S128_f384_fp384_13x13_k3/bin_contraction/bprop": 224.9e6,
    "deep_S128_f384_fp384_13x13_k3/c2r_ifft/bprop": 56.8e6,
    "deep_S128_f384_fp384_13x13_k3/r2c_fft_both_operands/accgrad": 114.7e6,
    "deep_S128_f384_fp384_13x13_k3/bin_contraction/accgrad": 196.1e6,
    "deep_S128_f384_fp384_13x13_k3/c2r_ifft/accgrad": 172.3e6,
}


def kernel_sources_digest():
    """sha256 over the CUDA sources of the library, in name order."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_1412_7580_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        if name.endswith((".cu", ".cuh")):
            with open(os.path.join(csrc, name), "rb") as fh:
                h.update(name.encode() + b"\0" + fh.read())
    return h.hexdigest()


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
    # the contraction of a pass with one-pass inverse transforms (n <= 64) leaves out the n - 2
    # bins that are conjugates of other bins: the bytes its launch really has to move
    kept = (B - (n - 2)) / B if n <= 64 else 1.0
    return {
        "stage_bytes": stage_bytes,                         # fft A, fft B, contraction, ifft
        "contraction_launch_bytes": stage_bytes[2] * kept,
        "b_fft": stage_bytes[0] + stage_bytes[1] + stage_bytes[3],
        "b_gemm": stage_bytes[2],
        "gemm_flops": 8.0 * s.S * T * s.f * s.fp * B,
        "equiv_flops": 2.0 * s.macs,
    }


def config_dict(s, tile, world, workspace_bytes):
    """The `config` object of the JSON line; both arms print the same one for the same workload."""
    working_mb = (workspace_bytes + 8 * (s.S * s.f * s.h * s.w + s.fp * s.f * s.kh * s.kw +
                                         s.S * s.fp * s.oh * s.ow)) / 1e6
    return {"workload": s.name, "S": s.S, "f": s.f, "fprime": s.fp, "h": s.h, "w": s.w,
            "kh": s.kh, "kw": s.kw, "n": s.n, "tile_basis": tile, "passes": "fprop+bprop+accgrad",
            "parallelism": "dp%d over S" % world,
            "l2": ("working set %.0f MB > 126 MB L2, no flush" % working_mb) if working_mb > 126
                  else ("working set %.1f MB is L2-resident: the figure is launch latency" % working_mb)}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi (query only) while a region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid, self.proc, self.lines = uuid, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.uuid, "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "50"],
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
        rows = [l for (t, l) in self.lines if t0 <= t <= t1 + 0.05] or [l for (_, l) in self.lines]
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
        # bprop border elements have fewer valid taps; the count is the formula's nominal taps
        total_macs += float(len(c)) * per[name]
        total_t += dt
        desc.append("%s:%d elems" % (name, len(c)))
    return 2.0 * total_macs, total_t, ", ".join(desc) + " (nominal taps per element)"


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
    import paper_1412_7580_b200 as fc
    plan = fc.conv_plan(*s.args())              # host-only: sizes the workspace the GPU arm would use
    cfg = config_dict(s, 0, args.gpus, fc.conv_plan_workspace_bytes(plan))
    fc.conv_plan_destroy(plan)
    line = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * sum(times) / max(len(times), 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": cfg,
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "per step: " + desc},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------
class Bench:
    def __init__(self, args):
        import torch
        self.torch = torch
        self.args = args
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
        torch.cuda.set_device(self.local)
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local))
            self.dist = dist
        self.peaks = load_peaks()

    def barrier(self):
        self.torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def timed_block(self, fn, steps, drain=None):
        """One timed region of exactly `steps` calls: barrier + synchronize on both sides,
        CUDA events on the launching stream, maximum over the ranks."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        e0.record()
        for _ in range(steps):
            fn()
        if drain is not None:
            drain()
        e1.record()
        self.barrier()
        ms = e0.elapsed_time(e1)
        if self.dist is not None:
            t = torch.tensor([ms], device="cuda")
            self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms

    def timed(self, fn, steps, drain=None, min_ms=MIN_TIMED_MS):
        """Repeats the timed block until `min_ms` of GPU time has been measured (the number of
        blocks is fixed from the first block, identical on every rank); returns the per-block
        times in ms."""
        first = self.timed_block(fn, steps, drain)
        blocks = int(min(max(min_ms / max(first, 1e-3), 1), MAX_BLOCKS))
        return [first] + [self.timed_block(fn, steps, drain) for _ in range(blocks - 1)]

    # -- one layer config, all measurements ---------------------------------------------
    def measure(self, s, math, tile_req=0, sample_clocks=False, reuse_line=True, cpu_budget=0.0):
        import numpy as np
        import paper_1412_7580_b200 as fc
        from paper_1412_7580_b200 import workloads as wl
        torch, args, world, dist = self.torch, self.args, self.world, self.dist
        peaks = self.peaks
        x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
        plan = fc.conv_plan(*s.args())
        fc.conv_plan_set_math(plan, math)
        if args.filter_chunks > 1:
            fc.conv_plan_set_filter_chunks(plan, args.filter_chunks)
        if args.small_planes != 1:
            fc.conv_plan_set_small_plane_kernel(plan, args.small_planes)
        if tile_req:
            fc.conv_plan_set_tiling(plan, tile_req)      # -1: the plan chooses
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

        warmup = max(args.warmup, 3)
        for _ in range(warmup):
            step()
        sampler = None
        if sample_clocks and self.rank == 0:
            sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(self.local).uuid).replace("GPU-", ""))
            sampler.start()
            time.sleep(0.25)
        launches0 = fc.fftconv_launch_count()
        t0 = time.time()
        blocks = self.timed(step, args.steps)
        t1 = time.time()
        # counted by the library.  Per pass: the forward FFTs (one launch for both operands with the
        # one-pass kernels, one per operand with the two-pass kernels), the contraction, the inverse FFT
        counted = fc.fftconv_launch_count() - launches0
        total_steps = args.steps * len(blocks)
        assert counted % total_steps == 0, (counted, total_steps)
        launches = counted // len(blocks)
        clocks = sampler.stop(t0, t1) if sampler is not None else None
        ms_step = float(np.median(blocks)) / args.steps

        for _ in range(2):
            step_e2e()
        e2e_blocks = self.timed(step_e2e, args.steps, e2e_drain, min_ms=MIN_TIMED_MS / 2)
        ms_e2e = float(np.median(e2e_blocks)) / args.steps
        assert fc.conv_plan_status(plan) == 0

        flops_step = 3 * 2.0 * s.macs
        value = world * flops_step / (ms_step * 1e-3) / 1e9
        e2e_value = world * flops_step / (ms_e2e * 1e-3) / 1e9

        names = ["fprop", "bprop", "accgrad"]
        calls = [lambda: fc.conv_fprop(plan, xd, wd, y), lambda: fc.conv_bprop(plan, dyd, wd, dx),
                 lambda: fc.conv_accgrad(plan, dyd, xd, dw)]
        reps = max(args.steps, 20)

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
        for n in names:
            m = pass_model(s, n, tile)
            t_ms = float(np.median(pass_ms[n]))
            t_roof = max(m["b_fft"] / bw, m["gemm_flops"] / (p_tflops * 1e12))
            t_stage = max((m["b_fft"] + m["b_gemm"]) / bw, m["gemm_flops"] / (p_tflops * 1e12))
            # both forward transforms share one launch unless the second operand has small planes
            # (filters), which take the small-plane kernel in a launch of their own
            apart = float(st1[n][1]) > 0.0       # the library reports 0 where that stage launched nothing
            kernel_names = ["r2c_fft_first_operand" if apart else "r2c_fft_both_operands",
                            "r2c_fft_small_planes", "bin_contraction", "c2r_ifft"]
            kbytes = [m["stage_bytes"][0] + (0 if apart else m["stage_bytes"][1]),
                      m["stage_bytes"][1] if apart else 0, m["contraction_launch_bytes"], m["stage_bytes"][3]]
            used = (0, 1, 2, 3) if apart else (0, 2, 3)
            passes[n] = {
                "ms": t_ms, "ms_min": float(np.min(pass_ms[n])),
                "gflops_equiv": m["equiv_flops"] / (t_ms * 1e-3) / 1e9,
                "roofline_us": t_roof * 1e6, "roofline_frac": t_roof / (t_ms * 1e-3),
                "unfused_roofline_us": t_stage * 1e6, "unfused_roofline_frac": t_stage / (t_ms * 1e-3),
                "kernel_ms": {kernel_names[k]: float(st1[n][k]) for k in used},
                "forward_fft_apart_ms": {"A": float(st2[n][0]), "B": float(st2[n][1])},
            }
            for k in used:
                cand = (float(st1[n][k]), n, k, m, kbytes[k], kernel_names[k])
                if best is None or cand[0] > best[0]:
                    best = cand
        dur_ms, bn, bk, bm, bbytes, bname = best
        if bk == 2 and bm["gemm_flops"] / (p_tflops * 1e12) > bbytes / bw:
            ach = bm["gemm_flops"] / (dur_ms * 1e-3) / 1e12
            roof = {"bound": "tensor" if eff == fc.MATH_TF32 else "alu", "achieved": ach,
                    "peak": p_tflops, "unit": "TFLOP/s", "frac": ach / p_tflops}
        else:
            ach = bbytes / (dur_ms * 1e-3) / 1e9
            roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": ach / peaks["hbm_gbs"]}
        digest = kernel_sources_digest()
        fresh = digest == NCU_TRAFFIC_SOURCE["kernel_sources_sha256"]
        traffic = NCU_TRAFFIC.get("%s/%s/%s" % (s.name, bname, bn)) if (fresh and not tile) else None
        roof.update({"traffic": traffic,
                     "traffic_source": dict(NCU_TRAFFIC_SOURCE, current_kernel_sources_sha256=digest,
                                            note=None if fresh else "kernel sources changed since the capture: no figure reported"),
                     "kernel": "%s/%s" % (bn, bname),
                     "kernel_ms": dur_ms, "algorithmic_bytes": bbytes,
                     "peak_source": peaks["source"] + (" sustained bf16 / 2" if roof["bound"] == "tensor" else "")})

        # extra (not the headline, which re-transforms every operand in every pass): the same
        # step with the forward spectra shared between the passes of the step
        reuse = None
        if reuse_line and not tile:
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
            ms_r = self.timed_block(step_r, args.steps) / args.steps
            launches_r = (fc.fftconv_launch_count() - lr0) // args.steps
            reuse = {"ms_per_step": ms_r, "value": world * flops_step / (ms_r * 1e-3) / 1e9, "unit": UNIT,
                     "gpu_launches_per_step": launches_r, "workspace_bytes": int(ws_r.numel()),
                     "note": "x, w, dy spectra computed once per step and shared by the three passes"}
            fc.conv_plan_destroy(plan_r)
            del ws_r

        cpu = None
        if cpu_budget > 0 and self.rank == 0 and world == 1:
            import oracle
            fl, t, desc = oracle_sample_run(s, x, w, dy, cpu_budget)
            cpu = {"value": fl / t / 1e9, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                   "sample": desc + " (sampled output elements of each pass, plain definition, float64)"}

        cfg = config_dict(s, tile, world, int(ws.numel()))
        out = {
            "value": value, "ms_per_step": ms_step, "blocks": len(blocks),
            "ms_per_step_min_max": [min(blocks) / args.steps, max(blocks) / args.steps],
            "dtype": "tf32" if eff == fc.MATH_TF32 else "f32", "config": cfg,
            "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": ms_e2e,
                    "h2d_bytes_per_step": int(4 * (x.size + w.size + dy.size)),
                    "d2h_bytes_per_step": int(4 * (y.numel() + dx.numel() + dw.numel()))},
            "gpu_launches": launches, "clocks": clocks, "roofline": roof, "cpu_baseline": cpu,
            "passes": passes, "step_with_spectrum_reuse": reuse,
        }
        fc.conv_plan_destroy(plan)
        del ws, xd, wd, dyd, y, dx, dw, hx, hw_, hdy, hy, hdx, hdw
        torch.cuda.empty_cache()
        return out

    # -- workload 5: the parameter sweep, timing only ------------------------------------
    def sweep(self, points, budget_s, out_path=None, tile="off", reps=5, max_gb=40.0):
        """Per-pass times and roofline fractions of sweep points (no oracle here: parity of the
        sweep is the job of the GPU tests; this run only checks that every result is finite).
        `points` is a list of ConvShapes; stops when the time budget is used up."""
        import numpy as np
        import paper_1412_7580_b200 as fc
        from paper_1412_7580_b200 import workloads as wl
        torch = self.torch
        bw = self.peaks["hbm_gbs"] * 1e9
        t_start = time.time()
        recs, skipped = [], 0
        fh = open(out_path, "w") if out_path else None
        for s in points:
            if time.time() - t_start > budget_s:
                break
            B = s.n * (s.n // 2 + 1)
            planes = s.S * s.f + s.fp * s.f + s.S * s.fp
            real_b = 4 * (s.S * s.f * s.h * s.w + s.fp * s.f * s.kh * s.kw + s.S * s.fp * s.oh * s.ow)
            if 8 * B * planes + 2 * real_b > max_gb * 1e9:
                skipped += 1
                continue
            x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
            p = fc.conv_plan(*s.args())
            if tile == "auto":
                fc.conv_plan_set_tiling(p, fc.TILE_AUTO)
            xd, wd, dyd = (torch.from_numpy(a).cuda() for a in (x, w, dy))
            y = torch.full((s.S, s.fp, s.oh, s.ow), float("nan"), device="cuda")
            dx = torch.full((s.S, s.f, s.h, s.w), float("nan"), device="cuda")
            dw = torch.full((s.fp, s.f, s.kh, s.kw), float("nan"), device="cuda")
            tuned = None
            if tile == "tuned":
                # measured choice: the library times a step for every admissible basis
                # (candidates that need more than 16 GB of workspace are left out by the library)
                nbytes = max(fc.conv_plan_workspace_bytes(p), min(fc.conv_plan_tune_workspace_bytes(p), 16 << 30))
                ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
                _, tuned = fc.conv_plan_tune_tiling(p, xd, wd, dyd, y, dx, dw, ws, reps=2)
            else:
                ws = fc.conv_plan_alloc_workspace(p)
            calls = [lambda: fc.conv_fprop(p, xd, wd, y), lambda: fc.conv_bprop(p, dyd, wd, dx),
                     lambda: fc.conv_accgrad(p, dyd, xd, dw)]
            ms = []
            for c in calls:
                c()                                    # warm-up
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * reps)]
                for r in range(reps):
                    ev[2 * r].record(); c(); ev[2 * r + 1].record()
                torch.cuda.synchronize()
                ms.append(float(np.median([ev[2 * r].elapsed_time(ev[2 * r + 1]) for r in range(reps)])))
            ok = fc.conv_plan_status(p) == 0 and all(bool(torch.isfinite(t).all().item()) for t in (y, dx, dw))
            t_roof_ms = (real_b + 8 * B * planes) / bw * 1e3   # byte term of the roofline; flops never bind here
            fr = [t_roof_ms / m for m in ms]
            rec = {"point": s.point, "S": s.S, "f": s.f, "fp": s.fp, "h": s.h, "k": s.kh, "n": s.n,
                   "tile_basis": fc.conv_plan_tile_basis(p),
                   "math": ["tf32" if fc.conv_plan_pass_math(p, k) == fc.MATH_TF32 else "f32" for k in range(3)],
                   "finite_and_status_ok": ok, "ms": ms, "roofline_frac": fr,
                   "gflops_equiv": [2.0 * s.macs / (m * 1e-3) / 1e9 for m in ms]}
            if tuned is not None:
                rec["tuner_step_ms"] = {str(k): v for k, v in tuned.items()}
            recs.append(rec)
            if fh:
                fh.write(json.dumps(rec) + "\n"); fh.flush()
            fc.conv_plan_destroy(p)
            del xd, wd, dyd, y, dx, dw, ws
        if fh:
            fh.close()
        per_n = {}
        for n in (16, 32, 64, 128):
            for label, sel in (("all", lambda r: True),
                               ("S_f_fp_ge_64", lambda r: min(r["S"], r["f"], r["fp"]) >= 64)):
                v = np.array([min(r["roofline_frac"]) for r in recs if r["n"] == n and sel(r)])
                if v.size:
                    per_n["n%d_%s" % (n, label)] = {
                        "points": int(v.size), "min": float(v.min()), "p10": float(np.percentile(v, 10)),
                        "median": float(np.median(v))}
        return {"points_done": len(recs), "points_requested": len(points),
                "points_not_finite_or_status": sum(not r["finite_and_status_ok"] for r in recs),
                "points_skipped_memory": skipped, "seconds": time.time() - t_start, "tile": tile,
                "roofline_frac_min_over_passes": per_n,
                "note": "roofline = FFT-stage bytes of the untiled method / measured HBM rate; parity of "
                        "these points is checked by tests/test_gpu_conv.py::test_sweep_stratified_slice"}

    # -- the bare transforms ----------------------------------------------------------------
    def bare(self, which, mb):
        """Throughput of fft2d_r2c / fft2d_c2r (n = 8..128) or fft1d_r2c / fft1d_c2r (n = 8..256)
        on `mb` megabytes of samples per launch (larger than the L2)."""
        import paper_1412_7580_b200 as fc
        torch = self.torch
        peak = self.peaks["hbm_gbs"]

        def t_us(fn, reps=20):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / reps * 1e3
        rows = []
        sizes = (8, 16, 32, 64, 128) if which == "fft2d" else (8, 16, 32, 64, 128, 256)
        for n in sizes:
            if which == "fft2d":
                batch = (mb << 20) // (n * n * 4)
                x = torch.rand((batch, n, n), device="cuda")
                X = torch.empty((batch, n, n // 2 + 1, 2), device="cuda")
                y = torch.empty_like(x)
                tf = t_us(lambda: fc.fft2d_r2c(x, X, n))
                ti = t_us(lambda: fc.fft2d_c2r(X, y, n, 1.0 / (n * n)))
            else:
                batch = (mb << 20) // (n * 4)
                x = torch.rand((batch, n), device="cuda")
                X = torch.empty((batch, n // 2 + 1, 2), device="cuda")
                y = torch.empty_like(x)
                tf = t_us(lambda: fc.fft1d_r2c(x, X, n))
                ti = t_us(lambda: fc.fft1d_c2r(X, y, n, 1.0 / n))
            nbytes = (x.numel() + X.numel()) * 4
            rows.append({"n": n, "batch": batch, "algorithmic_bytes": nbytes,
                         "forward_us": tf, "forward_gbs": nbytes / tf / 1e3, "forward_frac": nbytes / tf / 1e3 / peak,
                         "inverse_us": ti, "inverse_gbs": nbytes / ti / 1e3, "inverse_frac": nbytes / ti / 1e3 / peak})
            del x, X, y
        return {"transform": which, "mb_per_launch": mb, "peak_gbs": peak, "peak_source": self.peaks["source"],
                "rows": rows}


def run_ours(args):
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    b = Bench(args)
    math = {"auto": fc.MATH_AUTO, "fp32": fc.MATH_FP32, "tf32": fc.MATH_TF32}[args.math]
    single = (args.config is not None or args.shape is not None or args.filter_chunks > 1
              or args.small_planes != 1)
    extras = not single and not args.no_extras and b.world == 1

    if args.fft2d or args.fft1d:
        print(json.dumps({"metric": "bare_transform_throughput", "unit": "GB/s", "n_gpus": 1,
                          "data": "synthetic",
                          "tables": [b.bare(w, args.mb) for w, on in (("fft2d", args.fft2d), ("fft1d", args.fft1d)) if on]}),
              flush=True)
        return
    if args.sweep_only:
        pts = wl.sweep_points(args.sweep_points)
        import numpy as np
        order = np.random.default_rng([wl.SEED_ROOT, 55]).permutation(len(pts))   # seeded order: a time-boxed run is an unbiased sample
        res = b.sweep([pts[int(i)] for i in order], args.sweep_budget, args.sweep_out, args.sweep_tile)
        print(json.dumps({"metric": "sweep_roofline_fraction", "n_gpus": 1, "data": "synthetic", "sweep": res}),
              flush=True)
        return

    if args.shape:
        dims = [int(v) for v in args.shape.split(",")]
        assert len(dims) == 8, "--shape wants S,f,fp,h,w,kh,kw,n"
        s = wl.ConvShape("custom_S%d_f%d_fp%d_%dx%d_k%dx%d_n%d" % tuple(dims), *dims, cfg=6,
                         point=sum(dims), w_dist="fan_in", dy_dist="normal")
    else:
        s = wl.CONFIGS[HEADLINE_CONFIG if args.config is None else args.config]
    head = b.measure(s, math, args.tile, sample_clocks=True, reuse_line=not args.no_reuse_line,
                     cpu_budget=0.0 if args.no_cpu_baseline else args.cpu_budget)
    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": b.world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": head["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": head["dtype"], "data": "synthetic",
        "config": head["config"], "e2e": head["e2e"], "gpu_launches": head["gpu_launches"],
        "clocks": head["clocks"], "roofline": head["roofline"], "cpu_baseline": head["cpu_baseline"],
        "timed_blocks": head["blocks"], "ms_per_step_min_max": head["ms_per_step_min_max"],
        "passes": head["passes"], "step_with_spectrum_reuse": head["step_with_spectrum_reuse"],
    }
    if extras:
        cfgs = {}
        for idx in (0, 1, 2, 3):
            if idx == HEADLINE_CONFIG and not args.tile and math == fc.MATH_AUTO:
                r = head
            else:
                r = b.measure(wl.CONFIGS[idx], fc.MATH_AUTO, 0, sample_clocks=True, reuse_line=False)
            cfgs[wl.CONFIGS[idx].name] = {
                "ms_per_step": r["ms_per_step"], "value": r["value"], "dtype": r["dtype"],
                "gpu_launches": r["gpu_launches"], "clocks": r["clocks"], "timed_blocks": r["blocks"],
                "e2e": r["e2e"], "roofline": r["roofline"],
                "passes": {n: {k: p[k] for k in ("ms", "roofline_us", "roofline_frac", "unfused_roofline_frac",
                                                 "gflops_equiv", "kernel_ms")}
                           for n, p in r["passes"].items()}}
        line["configs"] = cfgs
        line["sweep"] = b.sweep(wl.sweep_stratified(), args.sweep_budget)
    if b.rank == 0:
        print(json.dumps(line), flush=True)
    if b.dist is not None:
        b.dist.barrier()
        b.dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20, help="steps per timed block")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=None,
                    help="0 tiny, 1 mid, 2 large-kernel (the headline), 3 deep; given: that layer only")
    ap.add_argument("--shape", default=None,
                    help="S,f,fp,h,w,kh,kw,n : a layer shape of your own instead of --config "
                         "(seeded inputs as in the sweep; used for profiling single shapes)")
    ap.add_argument("--math", default="auto", choices=["auto", "fp32", "tf32"])
    ap.add_argument("--tile", type=int, default=0,
                    help="spatial tiling with this basis (8, 16, 32 or 64; 0 = off); bytes, flops and the "
                         "roofline in the output are then those of the tiled method")
    ap.add_argument("--filter-chunks", type=int, default=1,
                    help="fprop / bprop: transform and contract the filters in this many ranges of frequency rows")
    ap.add_argument("--small-planes", type=int, default=1, choices=[0, 1, 2],
                    help="pruned-DFT kernels for small planes: 0 never, 1 where measured to pay (default), 2 wherever they apply")
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of oracle work for cpu_baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-reuse-line", action="store_true",
                    help="skip the extra measurement of a step with spectrum reuse between passes")
    ap.add_argument("--no-extras", action="store_true", help="skip the `configs` and `sweep` keys")
    ap.add_argument("--sweep-budget", type=float, default=75.0, help="seconds for the sweep")
    ap.add_argument("--sweep-only", action="store_true", help="run the seeded sweep points only (timing)")
    ap.add_argument("--sweep-points", type=int, default=1000)
    ap.add_argument("--sweep-out", default=None, help="JSON lines, one per sweep point")
    ap.add_argument("--sweep-tile", default="off", choices=["off", "auto", "tuned"],
                    help="tile basis of the sweep points: untiled, the plan's byte model, or measured")
    ap.add_argument("--fft2d", action="store_true", help="throughput table of the bare 2-D transforms")
    ap.add_argument("--fft1d", action="store_true", help="throughput table of the bare 1-D transforms")
    ap.add_argument("--mb", type=int, default=256, help="megabytes of samples per launch for --fft2d / --fft1d")
    args = ap.parse_args()
    if args.impl == "reference":
        from paper_1412_7580_b200 import workloads as wl
        s = wl.CONFIGS[HEADLINE_CONFIG if args.config is None else args.config]
        run_reference(args, s)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
