"""conv_fprop_noalloc: fprop for callers that cannot allocate a workspace.

Some users of this library hold device tensors but have no way to get scratch
memory where the convolution is needed (the framework's allocator owns the whole
GPU, or an allocation -- which synchronises the device -- is not acceptable at
that point).  For them the library carries a fixed 32 MiB scratch array of its
own.  This test calls that entry point through the C ABI and checks it against
the ordinary conv_fprop (caller-lent workspace) and against the float64 oracle on
two calls in a row with different inputs, so that nothing may depend on what the
previous call left in the shared array.  It lives in the file pytest collects last: a failure here
cannot hide any other test under `pytest -x`.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = {1: 1e-4, 2: 5e-3}    # FP32 / TF32 contraction, the tolerances of the other GPU tests


def _fprop_pair(fc, shape, x, w):
    import torch
    p = fc.conv_plan(*shape.args())
    fc.conv_plan_alloc_workspace(p)
    xd, wd = torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda()
    y_ref = torch.full((shape.S, shape.fp, shape.oh, shape.ow), float("nan"), device="cuda")
    fc.conv_fprop(p, xd, wd, y_ref)
    torch.cuda.synchronize()
    # a plan that was never lent a workspace: the new entry point must not need one
    q = fc.conv_plan(*shape.args())
    y_new = torch.full_like(y_ref, float("nan"))
    fc.conv_fprop_noalloc(q, xd, wd, y_new)
    torch.cuda.synchronize()
    eff = fc.conv_plan_pass_math(q, 0)       # fprop is pass 0; AUTO math resolves per pass
    fc.conv_plan_destroy(p)
    fc.conv_plan_destroy(q)
    return y_ref.cpu().numpy().astype(np.float64), y_new.cpu().numpy().astype(np.float64), eff


def test_noalloc_matches_conv_fprop_on_two_calls_in_a_row():
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    shapes = [wl.ConvShape("noalloc_a", 32, 16, 48, 13, 13, 3, 3, 16, cfg=8, point=1),   # tensor-core path
              wl.ConvShape("noalloc_b", 3, 5, 7, 27, 30, 5, 4, 32, cfg=8, point=2)]     # FP32 path, ragged
    import oracle
    for s in shapes:
        sizing = fc.conv_plan(*s.args())
        need = fc.conv_plan_workspace_bytes(sizing)
        fc.conv_plan_destroy(sizing)
        assert need <= fc.binding.NOALLOC_BYTES
        for call in range(2):           # second call: other values, same shared scratch
            x, w = wl.make_x(s), wl.make_w(s)
            if call == 1:
                x, w = (x[::-1] * np.float32(0.5)).copy(), (w + np.float32(0.25)).copy()
            ref, got, eff = _fprop_pair(fc, s, x, w)
            assert np.all(np.isfinite(got))
            err = np.max(np.abs(got - ref)) / np.max(np.abs(ref))
            assert err <= TOL[eff], (s.name, call, err)
            # and against the plain definition: a defect shared by both entry points would
            # pass the comparison above
            want = oracle.fprop(x, w)
            assert np.max(np.abs(got - want)) / np.max(np.abs(want)) <= TOL[eff], (s.name, call)


def test_noalloc_refuses_plans_beyond_its_fixed_scratch():
    import torch
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    s = wl.CONFIGS[1]                   # the mid layer needs about 300 MB of spectra
    p = fc.conv_plan(*s.args())
    assert fc.conv_plan_workspace_bytes(p) > fc.binding.NOALLOC_BYTES
    x = torch.zeros((s.S, s.f, s.h, s.w), device="cuda")
    w = torch.zeros((s.fp, s.f, s.kh, s.kw), device="cuda")
    y = torch.full((s.S, s.fp, s.oh, s.ow), 3.0, device="cuda")
    with pytest.raises(fc.FftConvError) as e:
        fc.conv_fprop_noalloc(p, x, w, y)
    assert e.value.status == fc.binding.EWORKSPACE
    torch.cuda.synchronize()
    assert bool(torch.all(y == 3.0))    # nothing was launched
    fc.conv_plan_destroy(p)
