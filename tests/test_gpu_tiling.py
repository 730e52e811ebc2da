"""Spatial tiling (Section 6 of the paper) on the GPU against the float64 oracle.

With a tile basis smaller than the plane, every pass works on windows of the
planes; the result is the same convolution, so the oracle is the plain direct
sum of the untiled pass.  Tolerances as for the untiled passes: 1e-4 (FP32
contraction), 5e-3 (TF32 tensor cores), normalised by the oracle's max-abs.
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


def run_tiled(shape, n_tile, x, w, dy, math, accumulate_init=None):
    import torch
    import paper_1412_7580_b200 as fc
    p = fc.conv_plan(*shape.args())
    fc.conv_plan_set_math(p, math)
    fc.conv_plan_set_tiling(p, n_tile)
    assert fc.conv_plan_tile_basis(p) == (n_tile if n_tile != shape.n else 0)
    ws = fc.conv_plan_alloc_workspace(p)
    ws.view(torch.float32)[64:].fill_(float("nan"))     # stale workspace must never leak
    xd, wd, dyd = (torch.from_numpy(a).cuda() for a in (x, w, dy))
    y = torch.full((shape.S, shape.fp, shape.oh, shape.ow), float("nan"), device="cuda")
    dx = torch.full((shape.S, shape.f, shape.h, shape.w), float("nan"), device="cuda")
    if accumulate_init is None:
        dw = torch.full((shape.fp, shape.f, shape.kh, shape.kw), float("nan"), device="cuda")
    else:
        dw = torch.from_numpy(accumulate_init.copy()).cuda()
    fc.conv_fprop(p, xd, wd, y)
    fc.conv_bprop(p, dyd, wd, dx)
    fc.conv_accgrad(p, dyd, xd, dw, accumulate=accumulate_init is not None)
    torch.cuda.synchronize()
    assert fc.conv_plan_status(p) == 0
    eff = [fc.conv_plan_pass_math(p, k) for k in range(3)]
    res = (y.cpu().numpy().astype(np.float64), dx.cpu().numpy().astype(np.float64),
           dw.cpu().numpy().astype(np.float64), eff)
    fc.conv_plan_destroy(p)
    return res


CASES = [
    # (S, f, fp, h, w, kh, kw, n), n_tile
    ((2, 3, 4, 16, 16, 3, 3, 16), 8),          # 14 x 14 output in 6 x 6 tiles: ragged last tile
    ((3, 5, 2, 31, 31, 5, 5, 32), 16),         # 27 = 2 * 12 + 3
    ((2, 9, 10, 64, 64, 3, 3, 64), 16),        # even split of the output, ragged split of the input
    ((1, 4, 3, 57, 61, 3, 5, 64), 16),         # rectangular plane and kernel
    ((2, 8, 8, 64, 64, 11, 11, 64), 32),       # large kernel: step 22
    ((1, 6, 5, 120, 128, 5, 5, 128), 32),      # planes that would take the two-pass transforms
    ((2, 3, 2, 128, 128, 7, 3, 128), 64),      # 64 x 64 tiles
    ((5, 33, 17, 27, 27, 8, 8, 32), 8),        # one output sample per tile and axis
    ((4, 16, 24, 32, 32, 3, 3, 32), 32),       # n_tile == n: tiling off
]


@pytest.mark.parametrize("dims,n_tile", CASES)
@pytest.mark.parametrize("math", [1, 2])
def test_tiled_passes_full_tensors(dims, n_tile, math):
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    s = wl.ConvShape("tiled", *dims, cfg=8, point=sum(dims) + n_tile)
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    y, dx, dw, eff = run_tiled(s, n_tile, x, w, dy, math)
    for got in (y, dx, dw):
        assert np.all(np.isfinite(got))            # every output element written, no stale data read
    assert relerr(y, oracle.fprop(x, w)) <= TOL[eff[0]]
    assert relerr(dx, oracle.bprop(dy, w, s.h, s.w)) <= TOL[eff[1]]
    assert relerr(dw, oracle.accgrad(dy, x, s.kh, s.kw)) <= TOL[eff[2]]


def test_tiled_accgrad_accumulates():
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    s = wl.ConvShape("tiled_acc", 3, 6, 5, 31, 31, 3, 3, 32, cfg=8, point=77)
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    init = wl.make_w(s)
    _, _, dw, _ = run_tiled(s, 16, x, w, dy, 1, accumulate_init=init)
    ref = init.astype(np.float64) + oracle.accgrad(dy, x, s.kh, s.kw)
    assert relerr(dw, ref) <= 1e-4


def test_tiled_matches_untiled_bit_for_bit_when_one_tile_covers_the_plane():
    """A tile basis that still holds the whole plane is the untiled computation on windows."""
    import torch
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    s = wl.ConvShape("one_tile", 2, 8, 8, 13, 13, 3, 3, 32, cfg=8, point=5)
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    y16, dx16, dw16, _ = run_tiled(s, 16, x, w, dy, 1)       # 16 >= 13: one window per plane
    s16 = wl.ConvShape("plain16", 2, 8, 8, 13, 13, 3, 3, 16, cfg=8, point=5)
    p = fc.conv_plan(*s16.args())
    fc.conv_plan_set_math(p, fc.MATH_FP32)
    fc.conv_plan_alloc_workspace(p)
    xd, wd, dyd = (torch.from_numpy(a).cuda() for a in (x, w, dy))
    y = torch.empty((2, 8, 11, 11), device="cuda")
    fc.conv_fprop(p, xd, wd, y)
    torch.cuda.synchronize()
    assert np.array_equal(y.cpu().numpy().astype(np.float64), y16)


@pytest.mark.parametrize("dims", [
    (2, 3, 5, 224, 224, 11, 11, 256),      # an ImageNet-size first layer
    (1, 6, 4, 200, 180, 3, 5, 256),        # rectangular
    (1, 2, 3, 300, 290, 7, 7, 512),
])
def test_planes_larger_than_the_largest_basis_run_tiled(dims):
    """n = 256 / 512 / 1024 is only the frame of a tiled plan: the plan picks a tile basis itself."""
    import torch
    import oracle
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    s = wl.ConvShape("frame", *dims, cfg=8, point=sum(dims))
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    p = fc.conv_plan(*s.args())
    assert fc.conv_plan_tile_basis(p) in (8, 16, 32, 64)
    fc.conv_plan_set_math(p, fc.MATH_FP32)
    ws = fc.conv_plan_alloc_workspace(p)
    ws.view(torch.float32)[64:].fill_(float("nan"))
    xd, wd, dyd = (torch.from_numpy(a).cuda() for a in (x, w, dy))
    y = torch.full((s.S, s.fp, s.oh, s.ow), float("nan"), device="cuda")
    dx = torch.full((s.S, s.f, s.h, s.w), float("nan"), device="cuda")
    dw = torch.full((s.fp, s.f, s.kh, s.kw), float("nan"), device="cuda")
    fc.conv_fprop(p, xd, wd, y)
    fc.conv_bprop(p, dyd, wd, dx)
    fc.conv_accgrad(p, dyd, xd, dw)
    torch.cuda.synchronize()
    assert fc.conv_plan_status(p) == 0
    assert relerr(y.cpu().numpy().astype(np.float64), oracle.fprop(x, w)) <= 1e-4
    assert relerr(dx.cpu().numpy().astype(np.float64), oracle.bprop(dy, w, s.h, s.w)) <= 1e-4
    assert relerr(dw.cpu().numpy().astype(np.float64), oracle.accgrad(dy, x, s.kh, s.kw)) <= 1e-4
    fc.conv_plan_destroy(p)


@pytest.mark.parametrize("dims,n_tile", [((16, 64, 64, 128, 128, 3, 3, 128), 32),
                                         ((32, 96, 64, 64, 64, 5, 5, 64), 16)])
def test_tiled_layers_at_benchmark_scale_sampled(dims, n_tile):
    """Hundreds of thousands of windows in the launch configuration `bench.py --tile` times:
    sampled output coordinates against the plain definition, plus the adjoint identity on the
    full GPU tensors."""
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    s = wl.ConvShape("tiled_big", *dims, cfg=8, point=sum(dims))
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    y, dx, dw, eff = run_tiled(s, n_tile, x, w, dy, 0)
    for got in (y, dx, dw):
        assert np.all(np.isfinite(got))
    cy = wl.sample_coords(y.shape, 3000, seed=11)
    assert relerr(y[cy[:, 0], cy[:, 1], cy[:, 2], cy[:, 3]], oracle.fprop_at(x, w, cy)) <= TOL[eff[0]]
    cx = wl.sample_coords(dx.shape, 3000, seed=12)
    assert relerr(dx[cx[:, 0], cx[:, 1], cx[:, 2], cx[:, 3]], oracle.bprop_at(dy, w, s.h, s.w, cx)) <= TOL[eff[1]]
    cw = wl.sample_coords(dw.shape, 200, seed=13)
    assert relerr(dw[cw[:, 0], cw[:, 1], cw[:, 2], cw[:, 3]], oracle.accgrad_at(dy, x, s.kh, s.kw, cw)) <= TOL[eff[2]]
    tol = max(TOL[e] for e in eff)
    a = float(np.sum(y * dy)); b = float(np.sum(dx * x)); c = float(np.sum(dw * w))
    scale = np.sqrt(float(np.sum(y * y)) * float(np.sum(dy.astype(np.float64) ** 2)))
    assert abs(a - b) <= 10 * tol * scale and abs(a - c) <= 10 * tol * scale


@pytest.mark.parametrize("dims", [(2, 24, 40, 64, 64, 3, 3, 64), (3, 5, 7, 31, 31, 5, 5, 32),
                                  (1, 6, 4, 150, 140, 5, 3, 256)])
def test_measured_choice_of_the_tile_basis(dims):
    """conv_plan_tune_tiling (Section 3.4: the autotuner times the candidate bases): every
    admissible basis is timed, the plan ends on the fastest with the lent workspace, and the
    results of the tuning run and of a pass after it match the oracle."""
    import torch
    import oracle
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    s = wl.ConvShape("tune", *dims, cfg=13, point=sum(dims))
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    xd, wd, dyd = (torch.from_numpy(a).cuda() for a in (x, w, dy))
    p = fc.conv_plan(*s.args())
    need = fc.conv_plan_tune_workspace_bytes(p)
    assert need >= fc.conv_plan_workspace_bytes(p)
    ws = torch.empty(need + 512, dtype=torch.uint8, device="cuda")
    ws.view(torch.float32)[64:].fill_(float("nan"))
    y = torch.full((s.S, s.fp, s.oh, s.ow), float("nan"), device="cuda")
    dx = torch.full((s.S, s.f, s.h, s.w), float("nan"), device="cuda")
    dw = torch.full((s.fp, s.f, s.kh, s.kw), float("nan"), device="cuda")
    # a workspace that is too small is refused and the plan keeps its basis
    before = fc.conv_plan_tile_basis(p)
    with pytest.raises(fc.FftConvError):
        fc.conv_plan_tune_tiling(p, xd, wd, dyd, y, dx, dw, ws[:1024], reps=1)
    assert fc.conv_plan_tile_basis(p) == before
    chosen, times = fc.conv_plan_tune_tiling(p, xd, wd, dyd, y, dx, dw, ws[:need], reps=2)
    torch.cuda.synchronize()
    admissible = [b for b in (8, 16, 32, 64) if b < s.n and b >= max(s.kh, s.kw)]
    if s.n <= 128:
        admissible = [0] + admissible
    assert sorted(times) == sorted(admissible)
    assert chosen in times and times[chosen] == min(times.values())
    assert fc.conv_plan_tile_basis(p) == chosen
    assert fc.conv_plan_status(p) == 0
    eff = [fc.conv_plan_pass_math(p, k) for k in range(3)]
    ref = (oracle.fprop(x, w), oracle.bprop(dy, w, s.h, s.w), oracle.accgrad(dy, x, s.kh, s.kw))
    for k, (got, r) in enumerate(zip((y, dx, dw), ref)):           # results of the last candidate
        assert relerr(got.cpu().numpy().astype(np.float64), r) <= TOL[eff[k]], k
    y.fill_(float("nan"))
    fc.conv_fprop(p, xd, wd, y)                                     # the plan is ready to use
    torch.cuda.synchronize()
    assert relerr(y.cpu().numpy().astype(np.float64), ref[0]) <= TOL[fc.conv_plan_pass_math(p, 0)]
    fc.conv_plan_destroy(p)
