"""Spectrum reuse across the passes of a training step (Section 6 of the paper lists it
as an optimisation it passed on): the reusing plan must give the same tensors as the
plain passes and the oracle, with fewer forward transforms launched."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = {1: 1e-4, 2: 5e-3}


def relerr(got, ref):
    return float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))


@pytest.mark.parametrize("small", [1, 2])
@pytest.mark.parametrize("dims", [(16, 24, 40, 13, 13, 3, 3, 16), (3, 5, 7, 27, 30, 5, 4, 32)])
def test_reuse_matches_plain_passes_and_oracle(dims, small):
    import torch
    import oracle
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    s = wl.ConvShape("reuse", *dims, cfg=10, point=sum(dims))
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    xd, wd, dyd = (torch.from_numpy(a).cuda() for a in (x, w, dy))

    def outputs():
        return (torch.full((s.S, s.fp, s.oh, s.ow), float("nan"), device="cuda"),
                torch.full((s.S, s.f, s.h, s.w), float("nan"), device="cuda"),
                torch.full((s.fp, s.f, s.kh, s.kw), float("nan"), device="cuda"))

    plain = fc.conv_plan(*s.args())
    fc.conv_plan_set_small_plane_kernel(plain, small)
    fc.conv_plan_alloc_workspace(plain)
    y0, dx0, dw0 = outputs()
    fc.conv_fprop(plain, xd, wd, y0); fc.conv_bprop(plain, dyd, wd, dx0); fc.conv_accgrad(plain, dyd, xd, dw0)

    p = fc.conv_plan(*s.args())
    fc.conv_plan_set_small_plane_kernel(p, small)
    plain_bytes = fc.conv_plan_workspace_bytes(p)
    fc.conv_plan_set_spectrum_reuse(p, True)
    assert fc.conv_plan_workspace_bytes(p) >= plain_bytes
    ws = fc.conv_plan_alloc_workspace(p)
    ws.view(torch.float32)[64:].fill_(float("nan"))
    y1, dx1, dw1 = outputs()
    before = fc.fftconv_launch_count()
    fc.conv_fprop(p, xd, wd, y1); fc.conv_bprop(p, dyd, wd, dx1); fc.conv_accgrad(p, dyd, xd, dw1)
    # fprop: x and w (one launch at these bases; with the small-plane kernel forced, w has a
    # launch of its own), contraction, inverse; bprop: dy only; accGrad: no forward transform
    # at all -- three forward transforms saved
    assert fc.fftconv_launch_count() - before == (4 if small == 2 else 3) + 3 + 2
    torch.cuda.synchronize()
    for a, b in ((y0, y1), (dx0, dx1), (dw0, dw1)):
        assert torch.equal(a, b)                                  # same kernels, same spectra
    eff = [fc.conv_plan_pass_math(p, k) for k in range(3)]
    assert relerr(y1.cpu().numpy().astype(np.float64), oracle.fprop(x, w)) <= TOL[eff[0]]
    assert relerr(dx1.cpu().numpy().astype(np.float64), oracle.bprop(dy, w, s.h, s.w)) <= TOL[eff[1]]
    assert relerr(dw1.cpu().numpy().astype(np.float64), oracle.accgrad(dy, x, s.kh, s.kw)) <= TOL[eff[2]]

    # next step: weights updated in place; fprop refreshes their spectrum, bprop picks it up
    w2 = (w * np.float32(0.5) + np.float32(0.125)).astype(np.float32)
    wd.copy_(torch.from_numpy(w2))
    fc.conv_fprop(p, xd, wd, y1); fc.conv_bprop(p, dyd, wd, dx1)
    torch.cuda.synchronize()
    assert relerr(y1.cpu().numpy().astype(np.float64), oracle.fprop(x, w2)) <= TOL[eff[0]]
    assert relerr(dx1.cpu().numpy().astype(np.float64), oracle.bprop(dy, w2, s.h, s.w)) <= TOL[eff[1]]

    # a different tensor under another pointer is transformed afresh; so is everything after
    # an explicit invalidation
    x3 = wl.make_planes(s.S * s.f, s.h, s.w, seed=77).reshape(s.S, s.f, s.h, s.w)
    x3d = torch.from_numpy(x3).cuda()
    fc.conv_accgrad(p, dyd, x3d, dw1)
    torch.cuda.synchronize()
    assert relerr(dw1.cpu().numpy().astype(np.float64), oracle.accgrad(dy, x3, s.kh, s.kw)) <= TOL[eff[2]]
    dy2 = (dy * np.float32(-2.0)).astype(np.float32)
    dyd.copy_(torch.from_numpy(dy2))                             # changed in place, same pointer
    fc.conv_plan_invalidate_spectra(p)
    before = fc.fftconv_launch_count()
    fc.conv_accgrad(p, dyd, x3d, dw1)
    # both operands afresh, in one fused launch
    assert fc.fftconv_launch_count() - before == 3
    torch.cuda.synchronize()
    assert relerr(dw1.cpu().numpy().astype(np.float64), oracle.accgrad(dy2, x3, s.kh, s.kw)) <= TOL[eff[2]]
    fc.conv_plan_destroy(p)
    fc.conv_plan_destroy(plain)
