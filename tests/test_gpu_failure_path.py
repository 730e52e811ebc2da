"""The give-up paths of the kernels: a bounded device-side wait that runs out.

Every wait on an asynchronous copy or on the tensor cores has a limit; when it
runs out the kernel raises the plan's status word, waits (bounded) for what it
has in flight, frees its tensor memory and returns.  Nothing here hangs or
faults the GPU: the test only shortens the limit (a plan setting) below the
normal latency of a copy, so the waits run out by themselves, then reads the
status back, restores the limit and checks that the same plan and context still
compute correct results.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = {1: 1e-4, 2: 5e-3}


def _run(fc, torch, plan, s, xd, wd, dyd):
    y = torch.zeros((s.S, s.fp, s.oh, s.ow), device="cuda")
    dx = torch.zeros((s.S, s.f, s.h, s.w), device="cuda")
    dw = torch.zeros((s.fp, s.f, s.kh, s.kw), device="cuda")
    fc.conv_fprop(plan, xd, wd, y)
    fc.conv_bprop(plan, dyd, wd, dx)
    fc.conv_accgrad(plan, dyd, xd, dw)
    torch.cuda.synchronize()
    return y, dx, dw


@pytest.mark.parametrize("dims", [(8, 24, 40, 13, 13, 3, 3, 16),      # double-buffered inverse transform
                                  (4, 24, 40, 31, 31, 5, 5, 32),
                                  (2, 12, 10, 64, 64, 7, 7, 64),
                                  (1, 9, 10, 120, 120, 5, 5, 128)])   # two-pass transforms
@pytest.mark.parametrize("math", [1, 2])
def test_wait_limit_runs_out_and_the_plan_recovers(dims, math):
    import torch
    import oracle
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    s = wl.ConvShape("timeout", *dims, cfg=9, point=sum(dims))
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    xd, wd, dyd = (torch.from_numpy(a).cuda() for a in (x, w, dy))
    p = fc.conv_plan(*s.args())
    fc.conv_plan_set_math(p, math)
    fc.conv_plan_alloc_workspace(p)
    assert fc.conv_plan_status(p) == 0

    fc.conv_plan_set_wait_limit(p, 1)           # one SM cycle: no copy lands that fast
    _run(fc, torch, p, s, xd, wd, dyd)          # every kernel returns by itself
    assert fc.conv_plan_status(p) == fc.binding.EDEVICE_TIMEOUT
    assert fc.conv_plan_status(p) == 0          # reading the word clears it

    fc.conv_plan_set_wait_limit(p, 0)           # default limit again: same plan, same context
    y, dx, dw = _run(fc, torch, p, s, xd, wd, dyd)
    assert fc.conv_plan_status(p) == 0
    eff = [fc.conv_plan_pass_math(p, k) for k in range(3)]
    for got, ref, e in ((y, oracle.fprop(x, w), eff[0]), (dx, oracle.bprop(dy, w, s.h, s.w), eff[1]),
                        (dw, oracle.accgrad(dy, x, s.kh, s.kw), eff[2])):
        g = got.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(g - ref)) / np.max(np.abs(ref)) <= TOL[e]
    fc.conv_plan_destroy(p)


def test_wait_limit_rejects_bad_arguments():
    import paper_1412_7580_b200 as fc
    p = fc.conv_plan(2, 2, 2, 8, 8, 3, 3, 8)
    with pytest.raises(fc.FftConvError):
        fc.conv_plan_set_wait_limit(p, -5)
    fc.conv_plan_destroy(p)
