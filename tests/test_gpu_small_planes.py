"""The small-plane kernels (pruned DFTs of the filters and of the filter gradient) and the
filter chunking.

fprop and bprop transform their filters with a kernel of their own when the filter planes
are small (at most 13 x 13 and at most a quarter of the basis); accGrad's inverse transform
has a counterpart for small square crops.  These tests run shapes on
both sides of every condition -- kernel widths with and without an instantiation, rectangular
kernels, ragged plane counts, every basis -- with the kernel switched on and off, and the
chunked form (filter spectrum produced and contracted in ranges of frequency rows), all
against the float64 oracle.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = {1: 1e-4, 2: 5e-3}

SHAPES = [
    # S, f, fp, h, w, kh, kw, n
    (3, 5, 7, 8, 8, 3, 3, 8),            # n = 8: kernels up to 4 wide qualify
    (2, 33, 35, 8, 8, 4, 2, 8),          # even width with an instantiation, ragged planes
    (4, 40, 33, 16, 16, 5, 5, 16),
    (2, 17, 40, 16, 15, 8, 7, 16),       # as wide as the kernel takes at n = 16
    (2, 9, 12, 16, 16, 9, 9, 16),        # too large for n = 16: butterfly kernels
    (3, 36, 64, 31, 31, 5, 5, 32),
    (2, 20, 70, 32, 30, 13, 11, 32),
    (2, 20, 24, 32, 32, 3, 6, 32),       # width 6 has no instantiation: butterfly kernels
    (2, 12, 10, 64, 64, 11, 11, 64),
    (1, 40, 36, 57, 64, 7, 13, 64),
    (1, 9, 10, 120, 121, 5, 9, 128),     # two-pass transforms for x, small-plane kernel for w
    (2, 96, 1, 27, 27, 3, 3, 32),        # one output plane
    (1, 1, 65, 13, 13, 1, 1, 16),        # 1 x 1 kernels
    (37, 33, 35, 16, 16, 7, 7, 16),
    (5, 70, 40, 32, 32, 11, 11, 32),     # small square crop as large as the pruned inverse kernel takes
    (9, 160, 150, 32, 32, 3, 3, 32),     # blocks enough for a warp to own one (the other work split)
]


def relerr(got, ref):
    m = np.max(np.abs(ref))
    return float(np.max(np.abs(got - ref)) / m) if m > 0 else float(np.max(np.abs(got)))


def run(s, x, w, dy, math, small, chunks):
    import torch
    import paper_1412_7580_b200 as fc
    p = fc.conv_plan(*s.args())
    fc.conv_plan_set_math(p, math)
    fc.conv_plan_set_small_plane_kernel(p, small)
    fc.conv_plan_set_filter_chunks(p, chunks)
    ws = fc.conv_plan_alloc_workspace(p)
    ws.view(torch.float32)[64:].fill_(float("nan"))
    xd, wd, dyd = (torch.from_numpy(a).cuda() for a in (x, w, dy))
    y = torch.full((s.S, s.fp, s.oh, s.ow), float("nan"), device="cuda")
    dx = torch.full((s.S, s.f, s.h, s.w), float("nan"), device="cuda")
    dw = torch.full((s.fp, s.f, s.kh, s.kw), float("nan"), device="cuda")
    dw2 = torch.full((s.fp, s.f, s.kh, s.kw), 0.5, device="cuda")
    fc.conv_fprop(p, xd, wd, y)
    fc.conv_bprop(p, dyd, wd, dx)
    fc.conv_accgrad(p, dyd, xd, dw)
    fc.conv_accgrad(p, dyd, xd, dw2, accumulate=True)
    torch.cuda.synchronize()
    assert fc.conv_plan_status(p) == 0
    eff = [fc.conv_plan_pass_math(p, k) for k in range(3)]
    fc.conv_plan_destroy(p)
    return (y.cpu().numpy().astype(np.float64), dx.cpu().numpy().astype(np.float64),
            dw.cpu().numpy().astype(np.float64), dw2.cpu().numpy().astype(np.float64), eff)


@pytest.mark.parametrize("dims", SHAPES)
@pytest.mark.parametrize("math", [1, 2])
def test_small_plane_kernel_on_off_and_chunked(dims, math):
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    s = wl.ConvShape("small", *dims, cfg=12, point=sum(dims))
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    ref_y, ref_dx = oracle.fprop(x, w), oracle.bprop(dy, w, s.h, s.w)
    ref_dw = oracle.accgrad(dy, x, s.kh, s.kw)
    for small, chunks in ((2, 1), (1, 1), (0, 1), (1, 3), (2, 100)):
        y, dx, dw, dw2, eff = run(s, x, w, dy, math, small, chunks)
        assert np.all(np.isfinite(y)) and np.all(np.isfinite(dx)) and np.all(np.isfinite(dw)), (small, chunks)
        assert relerr(y, ref_y) <= TOL[eff[0]], (small, chunks)
        assert relerr(dx, ref_dx) <= TOL[eff[1]], (small, chunks)
        assert relerr(dw, ref_dw) <= TOL[eff[2]], (small, chunks)
        assert relerr(dw2, ref_dw + 0.5) <= TOL[eff[2]], (small, chunks)      # accumulate
