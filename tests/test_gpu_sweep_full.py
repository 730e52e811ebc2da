"""The whole parameter sweep (workload 5) against the oracle -- an opt-in, long run.

    python -m pytest tests/test_gpu_sweep_full.py -m gpu -q --sweep-points 1000 \
        --sweep-budget 1500 --sweep-out sweep_parity.jsonl [--sweep-tile auto]

Every seeded point of the sweep, all three passes, default math mode: small
points are compared element by element, the others at seeded sampled
coordinates (corners, uniform, three elements of every output plane), plus a
finiteness scan of the full tensors.  Skipped unless --sweep-points is given:
the routine GPU run covers the sweep with the stratified slice in
test_gpu_conv.py; this file is how the 1,000-point evidence is produced.
"""
import json
import time

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_sweep_full(request):
    npts = request.config.getoption("--sweep-points")
    if not npts:
        pytest.skip("opt-in: pass --sweep-points N")
    import torch
    import oracle
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    from test_gpu_conv import TOL, check_sampled, relerr
    budget = request.config.getoption("--sweep-budget")
    out = request.config.getoption("--sweep-out")
    tile = request.config.getoption("--sweep-tile")
    pts = wl.sweep_points(npts)
    order = np.random.default_rng([wl.SEED_ROOT, 55]).permutation(len(pts))
    fh = open(out, "w") if out else None
    t0, done, failed, worst = time.time(), 0, [], 0.0
    for oi in order:
        if time.time() - t0 > budget:
            break
        s = pts[int(oi)]
        x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
        p = fc.conv_plan(*s.args())
        if tile == "auto":
            fc.conv_plan_set_tiling(p, fc.TILE_AUTO)
        fc.conv_plan_alloc_workspace(p)
        xd, wd, dyd = (torch.from_numpy(a).cuda() for a in (x, w, dy))
        y = torch.full((s.S, s.fp, s.oh, s.ow), float("nan"), device="cuda")
        dx = torch.full((s.S, s.f, s.h, s.w), float("nan"), device="cuda")
        dw = torch.full((s.fp, s.f, s.kh, s.kw), float("nan"), device="cuda")
        fc.conv_fprop(p, xd, wd, y)
        fc.conv_bprop(p, dyd, wd, dx)
        fc.conv_accgrad(p, dyd, xd, dw)
        torch.cuda.synchronize()
        ok = fc.conv_plan_status(p) == 0
        eff = [fc.conv_plan_pass_math(p, k) for k in range(3)]
        res = [t.cpu().numpy().astype(np.float64) for t in (y, dx, dw)]
        ok = ok and all(np.all(np.isfinite(r)) for r in res)
        ratio = float("inf")
        if ok:
            try:
                if s.macs <= 2e9:
                    refs = (oracle.fprop(x, w), oracle.bprop(dy, w, s.h, s.w), oracle.accgrad(dy, x, s.kh, s.kw))
                    ratio = max(relerr(g, r) / TOL[e] for g, r, e in zip(res, refs, eff))
                    ok = ratio <= 1.0
                else:
                    ratio = check_sampled(s, x, w, dy, res[0], res[1], res[2], eff, (200, 200, 48), seed=s.point)
            except AssertionError:
                ok = False
        rec = {"point": s.point, "name": s.name, "n": s.n, "tile_basis": fc.conv_plan_tile_basis(p),
               "math": eff, "ok": bool(ok), "worst_err_over_tol": ratio}
        if fh:
            fh.write(json.dumps(rec) + "\n"); fh.flush()
        done += 1
        worst = max(worst, ratio)
        if not ok:
            failed.append(s.name)
        fc.conv_plan_destroy(p)
        del xd, wd, dyd, y, dx, dw
    summary = {"summary": True, "points_done": done, "points_requested": len(pts), "points_failed": len(failed),
               "worst_err_over_tol": worst, "seconds": time.time() - t0, "tile": tile}
    if fh:
        fh.write(json.dumps(summary) + "\n")
        fh.close()
    print(json.dumps(summary))
    assert not failed, failed[:10]
    assert done > 0
