"""The three convolution passes on the GPU against the float64 oracle.

Tolerances (max |gpu - oracle| / max |oracle|): 1e-4 for the FP32 path, 5e-3
for the TF32 tensor-core contraction.  Small shapes are compared element by
element on full tensors; the benchmark-size layers are compared on a seeded
sample of output coordinates (the oracle evaluates the plain definition at
those coordinates) plus the adjoint identity on the full GPU tensors; in the
benchmark's own math mode they are also compared element by element.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = {1: 1e-4, 2: 5e-3}   # MATH_FP32, MATH_TF32


def relerr(got, ref):
    m = np.max(np.abs(ref))
    if m == 0:
        return float(np.max(np.abs(got)))
    return float(np.max(np.abs(got - ref)) / m)


def run_gpu(shape, x, w, dy, math, accumulate_init=None):
    import torch
    import paper_1412_7580_b200 as fc
    p = fc.conv_plan(*shape.args())
    fc.conv_plan_set_math(p, math)
    ws = fc.conv_plan_alloc_workspace(p)
    ws.view(torch.float32)[64:].fill_(float("nan"))     # stale workspace must never leak
    xd, wd, dyd = (torch.from_numpy(a).cuda() for a in (x, w, dy))
    y = torch.full((shape.S, shape.fp, shape.oh, shape.ow), float("nan"), device="cuda")
    dx = torch.full((shape.S, shape.f, shape.h, shape.w), float("nan"), device="cuda")
    dw = torch.full((shape.fp, shape.f, shape.kh, shape.kw), float("nan"), device="cuda")
    fc.conv_fprop(p, xd, wd, y)
    fc.conv_bprop(p, dyd, wd, dx)
    fc.conv_accgrad(p, dyd, xd, dw)
    torch.cuda.synchronize()
    assert fc.conv_plan_status(p) == 0
    eff = [fc.conv_plan_pass_math(p, k) for k in range(3)]     # AUTO resolves per pass
    res = (y.cpu().numpy().astype(np.float64), dx.cpu().numpy().astype(np.float64),
           dw.cpu().numpy().astype(np.float64), eff)
    fc.conv_plan_destroy(p)
    return res


SMALL = [
    # S, f, fp, h, w, kh, kw, n
    (8, 4, 8, 16, 16, 3, 3, 16),       # the tiny benchmark config
    (2, 3, 4, 8, 8, 3, 3, 8),
    (1, 1, 1, 8, 8, 8, 8, 8),
    (3, 5, 2, 7, 6, 3, 2, 8),
    (5, 33, 17, 13, 13, 3, 3, 16),
    (4, 7, 9, 16, 11, 5, 4, 16),
    (3, 18, 20, 31, 31, 5, 5, 32),
    (2, 5, 3, 27, 32, 7, 9, 32),
    (9, 1, 16, 32, 32, 13, 13, 32),
    (2, 9, 10, 64, 64, 11, 11, 64),
    (3, 4, 1, 57, 57, 3, 3, 64),
    (1, 2, 3, 128, 128, 13, 13, 128),
    (2, 3, 2, 120, 120, 5, 5, 128),
    (3, 9, 10, 128, 128, 7, 7, 128),    # two-pass transforms: a full tile of 8 planes and a ragged one
    (2, 5, 3, 97, 101, 5, 9, 128),      # plane sizes that break the 16-byte alignment of the plane copies
    (1, 17, 12, 120, 121, 13, 3, 128),
    (16, 16, 16, 13, 13, 3, 3, 16),
    (1, 64, 1, 16, 16, 5, 5, 16),
]


@pytest.mark.parametrize("dims", SMALL)
@pytest.mark.parametrize("math", [1, 2])
def test_small_shapes_full_tensors(dims, math):
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    s = wl.ConvShape("case", *dims, cfg=7, point=sum(dims))
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    y, dx, dw, eff = run_gpu(s, x, w, dy, math)
    for got in (y, dx, dw):
        assert np.all(np.isfinite(got))
    assert relerr(y, oracle.fprop(x, w)) <= TOL[eff[0]]
    assert relerr(dx, oracle.bprop(dy, w, s.h, s.w)) <= TOL[eff[1]]
    assert relerr(dw, oracle.accgrad(dy, x, s.kh, s.kw)) <= TOL[eff[2]]


def test_accgrad_accumulates():
    import torch
    import oracle
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    s = wl.ConvShape("acc", 4, 6, 5, 13, 13, 3, 3, 16, cfg=7, point=1)
    x, dy = wl.make_x(s), wl.make_dy(s)
    init = wl.make_w(s)
    p = fc.conv_plan(*s.args())
    fc.conv_plan_set_math(p, fc.MATH_FP32)
    fc.conv_plan_alloc_workspace(p)
    dw = torch.from_numpy(init.copy()).cuda()
    fc.conv_accgrad(p, torch.from_numpy(dy).cuda(), torch.from_numpy(x).cuda(), dw, accumulate=True)
    torch.cuda.synchronize()
    ref = init.astype(np.float64) + oracle.accgrad(dy, x, s.kh, s.kw)
    assert relerr(dw.cpu().numpy().astype(np.float64), ref) <= 1e-4


def test_accgrad_accumulates_two_pass_transforms():
    """accumulate = 1 through the n = 128 inverse transform."""
    import torch
    import oracle
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    s = wl.ConvShape("acc128", 2, 9, 3, 120, 120, 7, 7, 128, cfg=7, point=2)
    x, dy = wl.make_x(s), wl.make_dy(s)
    init = wl.make_w(s)
    p = fc.conv_plan(*s.args())
    fc.conv_plan_set_math(p, fc.MATH_FP32)
    fc.conv_plan_alloc_workspace(p)
    dw = torch.from_numpy(init.copy()).cuda()
    fc.conv_accgrad(p, torch.from_numpy(dy).cuda(), torch.from_numpy(x).cuda(), dw, accumulate=True)
    torch.cuda.synchronize()
    ref = init.astype(np.float64) + oracle.accgrad(dy, x, s.kh, s.kw)
    assert relerr(dw.cpu().numpy().astype(np.float64), ref) <= 1e-4


def check_sampled(s, x, w, dy, y, dx, dw, eff, counts, seed):
    """Sampled parity on full-size tensors: the oracle evaluates the plain definition at the
    16 corners and uniform random coordinates of every result, and at three elements of EVERY
    output plane (one random, one in the last row, one in the last column), so that a wrong
    tile, plane group or clipped edge anywhere shows up."""
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    fns = (lambda c: oracle.fprop_at(x, w, c), lambda c: oracle.bprop_at(dy, w, s.h, s.w, c),
           lambda c: oracle.accgrad_at(dy, x, s.kh, s.kw, c))
    worst = []
    for k, (got, fn) in enumerate(zip((y, dx, dw), fns)):
        c = np.concatenate([wl.sample_coords(got.shape, counts[k], seed=seed + 10 * k),
                            wl.plane_coords(got.shape, seed=seed + 10 * k + 1)], axis=0)
        err = relerr(got[c[:, 0], c[:, 1], c[:, 2], c[:, 3]], fn(c))
        assert err <= TOL[eff[k]], (s.name, ("fprop", "bprop", "accgrad")[k], err)
        worst.append(err / TOL[eff[k]])
    return max(worst)


@pytest.mark.parametrize("cfg", [1, 2, 3])
def test_benchmark_layers_full_tensors(cfg):
    """The three benchmark layers at full size, in the launch configuration and math mode the
    benchmark times (AUTO = TF32 tensor cores), every element of y, dx and dw against the
    float64 oracle."""
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    s = wl.CONFIGS[cfg]
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    y, dx, dw, eff = run_gpu(s, x, w, dy, 0)
    assert eff == [2, 2, 2]
    assert relerr(y, oracle.fprop(x, w)) <= TOL[eff[0]]
    assert relerr(dx, oracle.bprop(dy, w, s.h, s.w)) <= TOL[eff[1]]
    assert relerr(dw, oracle.accgrad(dy, x, s.kh, s.kw)) <= TOL[eff[2]]


@pytest.mark.parametrize("cfg", [1, 2, 3])
def test_benchmark_layers_fp32_sampled(cfg):
    """The same layers with the FP32 contraction: sampled coordinates (corners, uniform,
    three per output plane) plus the adjoint identity on the full GPU tensors."""
    from paper_1412_7580_b200 import workloads as wl
    s = wl.CONFIGS[cfg]
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    y, dx, dw, eff = run_gpu(s, x, w, dy, 1)
    assert eff == [1, 1, 1]
    for got in (y, dx, dw):
        assert np.all(np.isfinite(got))
    check_sampled(s, x, w, dy, y, dx, dw, eff, (4000, 4000, 600), seed=cfg)
    # adjoint identity on the full GPU tensors: <y,dy> = <x,dx> = <w,dw>
    a = float(np.sum(y * dy)); b = float(np.sum(dx * x)); c = float(np.sum(dw * w))
    scale = np.sqrt(float(np.sum(y * y)) * float(np.sum(dy.astype(np.float64) ** 2)))
    assert abs(a - b) <= 10 * 1e-4 * scale and abs(a - c) <= 10 * 1e-4 * scale


def test_sweep_stratified_slice():
    """A stratified, seeded slice of the 1,000-point parameter sweep, all three passes, default
    math mode: every basis n in {16, 32, 64, 128}, eight points per basis with S, f, f' >= 64
    (many contraction tiles per bin) and six smaller ones (which include shapes the plan gives
    to the FP32 contraction).  Time-boxed; the points come round robin over the bases."""
    import time
    from paper_1412_7580_b200 import workloads as wl
    pts = wl.sweep_stratified()
    assert len(pts) >= 48
    t0, done, maths, per_n = time.time(), 0, set(), {}
    for s in pts:
        if time.time() - t0 > 240.0:
            break
        x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
        y, dx, dw, eff = run_gpu(s, x, w, dy, 0)
        for got in (y, dx, dw):
            assert np.all(np.isfinite(got)), s
        small = s.macs <= 2e9
        if small:
            import oracle
            assert relerr(y, oracle.fprop(x, w)) <= TOL[eff[0]], s
            assert relerr(dx, oracle.bprop(dy, w, s.h, s.w)) <= TOL[eff[1]], s
            assert relerr(dw, oracle.accgrad(dy, x, s.kh, s.kw)) <= TOL[eff[2]], s
        else:
            check_sampled(s, x, w, dy, y, dx, dw, eff, (300, 300, 60), seed=s.point)
        done += 1
        maths.update(eff)
        per_n[s.n] = per_n.get(s.n, 0) + 1
        if min(s.S, s.f, s.fp) >= 64:
            per_n[(s.n, "large")] = per_n.get((s.n, "large"), 0) + 1
    assert done >= 40, (done, per_n)
    assert maths == {1, 2}                      # both contraction kernels were exercised
    for n in (16, 32, 64, 128):
        assert per_n.get(n, 0) >= 8 and per_n.get((n, "large"), 0) >= 5, per_n


@pytest.mark.parametrize("dims", [(6, 20, 24, 16, 16, 3, 3, 16), (4, 24, 40, 31, 31, 5, 5, 32),
                                  (2, 40, 36, 64, 64, 7, 7, 64)])
def test_steps_back_to_back_without_synchronisation(dims):
    """Kernels of consecutive passes overlap their ramp-up with the predecessor's drain.  Every
    pass reuses the same workspace, so a kernel that started reading or writing too early would
    corrupt a neighbour's spectra: several steps on changing inputs with no host synchronisation
    in between, every step's outputs checked afterwards."""
    import torch
    import oracle
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    s = wl.ConvShape("b2b", *dims, cfg=8, point=sum(dims))
    p = fc.conv_plan(*s.args())
    fc.conv_plan_set_math(p, fc.MATH_TF32)
    fc.conv_plan_alloc_workspace(p)
    steps = 4
    ins, outs = [], []
    for i in range(steps):
        si = wl.ConvShape("b2b", *dims, cfg=8, point=sum(dims) + 100 * i)
        x, w, dy = wl.make_x(si), wl.make_w(si), wl.make_dy(si)
        ins.append((x, w, dy))
        outs.append((torch.empty((s.S, s.fp, s.oh, s.ow), device="cuda"),
                     torch.empty((s.S, s.f, s.h, s.w), device="cuda"),
                     torch.empty((s.fp, s.f, s.kh, s.kw), device="cuda")))
    dev = [tuple(torch.from_numpy(a).cuda() for a in t) for t in ins]
    torch.cuda.synchronize()
    for (xd, wd, dyd), (y, dx, dw) in zip(dev, outs):
        fc.conv_fprop(p, xd, wd, y)
        fc.conv_bprop(p, dyd, wd, dx)
        fc.conv_accgrad(p, dyd, xd, dw)
    torch.cuda.synchronize()
    assert fc.conv_plan_status(p) == 0
    eff = [fc.conv_plan_pass_math(p, k) for k in range(3)]
    for (x, w, dy), (y, dx, dw) in zip(ins, outs):
        assert relerr(y.cpu().numpy().astype(np.float64), oracle.fprop(x, w)) <= TOL[eff[0]]
        assert relerr(dx.cpu().numpy().astype(np.float64), oracle.bprop(dy, w, s.h, s.w)) <= TOL[eff[1]]
        assert relerr(dw.cpu().numpy().astype(np.float64), oracle.accgrad(dy, x, s.kh, s.kw)) <= TOL[eff[2]]
    fc.conv_plan_destroy(p)
