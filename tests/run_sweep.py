#!/usr/bin/env python
"""Parameter sweep (the fifth workload): seeded points of the grid
S in {1,16,64,128} x f,f' in {1,16,64,128,256,384} x h in {13..128} x k in {3..13},
all three passes per point on the GPU, checked against the float64 oracle at a
seeded sample of output coordinates (the plain definition evaluated element by
element), with per-pass times and roofline fractions.

    python tests/run_sweep.py --points 1000 --budget-s 1200 --out sweep.jsonl

Writes one JSON line per finished point and a summary line at the end; points
are visited in a seeded random order so that a time-boxed run is an unbiased
sample.  This is test infrastructure (it imports the oracle); it is not part of
the product path.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

TOL = {1: 1e-4, 2: 5e-3}


def relerr(got, ref):
    m = np.max(np.abs(ref))
    return float(np.max(np.abs(got - ref)) / m) if m > 0 else float(np.max(np.abs(got)))


def main():
    import torch
    import oracle
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl

    ap = argparse.ArgumentParser()
    ap.add_argument("--points", type=int, default=1000)
    ap.add_argument("--budget-s", type=float, default=1200.0)
    ap.add_argument("--max-gb", type=float, default=40.0, help="skip points needing more device memory")
    ap.add_argument("--out", default=os.path.join(ROOT, "sweep.jsonl"))
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--tile", default="off", choices=["off", "auto"],
                    help="auto: let every plan choose a tile basis (spatial tiling, Section 6 of the paper)")
    args = ap.parse_args()

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    bw = (json.load(open(peaks_path))["hbm_gbs"] if os.path.exists(peaks_path) else 6650.0) * 1e9
    pts = wl.sweep_points(args.points)
    order = np.random.default_rng([wl.SEED_ROOT, 55]).permutation(len(pts))
    os.makedirs(os.path.dirname(os.path.abspath(args.out)), exist_ok=True)
    t_start = time.time()
    done = failed = skipped = 0
    fracs, worst = [], 0.0
    with open(args.out, "w") as fh:
        for oi in order:
            if time.time() - t_start > args.budget_s:
                break
            s = pts[int(oi)]
            B = s.n * (s.n // 2 + 1)
            planes = s.S * s.f + s.fp * s.f + s.S * s.fp
            real_b = 4 * (s.S * s.f * s.h * s.w + s.fp * s.f * s.kh * s.kw + s.S * s.fp * s.oh * s.ow)
            need = 8 * B * planes + 2 * real_b
            if need > args.max_gb * 1e9:
                skipped += 1
                continue
            x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
            p = fc.conv_plan(*s.args())
            if args.tile == "auto":
                fc.conv_plan_set_tiling(p, fc.TILE_AUTO)
            ws = fc.conv_plan_alloc_workspace(p)
            eff = fc.conv_plan_effective_math(p)
            xd, wd, dyd = (torch.from_numpy(a).cuda() for a in (x, w, dy))
            y = torch.full((s.S, s.fp, s.oh, s.ow), float("nan"), device="cuda")
            dx = torch.full((s.S, s.f, s.h, s.w), float("nan"), device="cuda")
            dw = torch.full((s.fp, s.f, s.kh, s.kw), float("nan"), device="cuda")
            calls = [lambda: fc.conv_fprop(p, xd, wd, y), lambda: fc.conv_bprop(p, dyd, wd, dx),
                     lambda: fc.conv_accgrad(p, dyd, xd, dw)]
            ms = []
            for c in calls:
                c()                                    # warm-up and the result that is checked
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * args.reps)]
                for r in range(args.reps):
                    ev[2 * r].record(); c(); ev[2 * r + 1].record()
                torch.cuda.synchronize()
                ms.append(float(np.median([ev[2 * r].elapsed_time(ev[2 * r + 1]) for r in range(args.reps)])))
            assert fc.conv_plan_status(p) == 0
            tols = [TOL[fc.conv_plan_pass_math(p, k)] for k in range(3)]
            errs = []
            for out, fn, ncoord, sd in (
                    (y, lambda c: oracle.fprop_at(x, w, c), 200, 0),
                    (dx, lambda c: oracle.bprop_at(dy, w, s.h, s.w, c), 200, 1),
                    (dw, lambda c: oracle.accgrad_at(dy, x, s.kh, s.kw, c), 48, 2)):
                c = wl.sample_coords(out.shape, ncoord, seed=s.point + sd)
                idx = torch.from_numpy(c.astype(np.int64)).cuda()
                got = out[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]].cpu().numpy().astype(np.float64)
                finite = bool(torch.isfinite(out).all().item())
                errs.append(relerr(got, fn(c)) if finite else float("inf"))
            ok = all(e <= t for e, t in zip(errs, tols))
            b_fft = real_b + 8 * B * planes
            t_roof_ms = b_fft / bw * 1e3        # byte term of the roofline; flops never bind here
            fr = [t_roof_ms / m for m in ms]
            rec = {"point": s.point, "S": s.S, "f": s.f, "fp": s.fp, "h": s.h, "k": s.kh, "n": s.n,
                   "tile_basis": fc.conv_plan_tile_basis(p),
                   "math": ["tf32" if t == TOL[2] else "f32" for t in tols], "ok": ok,
                   "max_rel_err": errs, "tol": tols,
                   "ms": ms, "roofline_frac": fr,
                   "gflops_equiv": [2.0 * s.macs / (m * 1e-3) / 1e9 for m in ms]}
            fh.write(json.dumps(rec) + "\n"); fh.flush()
            done += 1
            failed += (not ok)
            worst = max(worst, max(e / t for e, t in zip(errs, tols)))
            fracs.extend(fr)
            fc.conv_plan_destroy(p)
            del xd, wd, dyd, y, dx, dw, ws
        fr = np.array(fracs) if fracs else np.zeros(1)
        summary = {"summary": True, "points_done": done, "points_failed": failed, "points_skipped_memory": skipped,
                   "points_requested": len(pts), "seconds": time.time() - t_start,
                   "worst_err_over_tol": worst,
                   "roofline_frac_median": float(np.median(fr)), "roofline_frac_p10": float(np.percentile(fr, 10)),
                   "roofline_frac_min": float(fr.min()), "roofline_frac_max": float(fr.max())}
        fh.write(json.dumps(summary) + "\n")
    print(json.dumps(summary))
    return 1 if failed else 0


if __name__ == "__main__":
    sys.exit(main())
