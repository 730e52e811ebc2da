#!/usr/bin/env python
"""Throughput of the bare batched 1-D transforms (fft1d_r2c / fft1d_c2r) on one GPU.

    python tests/run_fft1d_bench.py [--mb 256]

For every size n in 8..256 it transforms `--mb` megabytes of fp32 samples (inputs larger than the
L2, so every launch streams from HBM), times 20 launches with CUDA events after 3 warm-up launches
and prints a table: microseconds per launch and algorithmic GB/s (samples read + spectrum
written, or the reverse), next to the measured copy bandwidth of the GPU if MEASURED_PEAKS.json
is present.  Measurement helper; not part of the product path.
"""
import argparse
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main():
    import torch
    import paper_1412_7580_b200 as fc
    ap = argparse.ArgumentParser()
    ap.add_argument("--mb", type=int, default=256)
    args = ap.parse_args()
    peak = None
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        peak = float(json.load(open(path))["hbm_gbs"])

    def timed(fn, reps=20):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps * 1e-3

    print("| n | batch | forward us | GB/s | of peak | inverse us | GB/s | of peak |")
    print("|---|---|---|---|---|---|---|---|")
    for n in (8, 16, 32, 64, 128, 256):
        batch = (args.mb << 20) // (n * 4)
        x = torch.rand((batch, n), device="cuda")
        X = torch.empty((batch, n // 2 + 1, 2), device="cuda")
        y = torch.empty_like(x)
        tf = timed(lambda: fc.fft1d_r2c(x, X, n))
        ti = timed(lambda: fc.fft1d_c2r(X, y, n, 1.0 / n))
        nbytes = (x.numel() + X.numel()) * 4
        gf, gi = nbytes / tf / 1e9, nbytes / ti / 1e9
        frac = (lambda g: "%.2f" % (g / peak)) if peak else (lambda g: "-")
        print("| %d | %d | %.0f | %.0f | %s | %.0f | %.0f | %s |" % (n, batch, tf * 1e6, gf, frac(gf),
                                                                    ti * 1e6, gi, frac(gi)))


if __name__ == "__main__":
    main()
