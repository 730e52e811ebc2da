"""Bare batched 1-D transforms on the GPU against the oracle's naive DFT.

Tolerance: max |gpu - oracle| / max |oracle| <= 1e-5 (the bare-transform bar).
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = 1e-5
SIZES = [2, 4, 8, 16, 32, 64, 128, 256]


def relerr(got, ref):
    m = np.max(np.abs(ref))
    return float(np.max(np.abs(got - ref)) / m) if m > 0 else float(np.max(np.abs(got)))


def gpu_r2c(x, n):
    import torch
    import paper_1412_7580_b200 as fc
    xd = torch.from_numpy(x).cuda()
    out = torch.full((x.shape[0], n // 2 + 1, 2), float("nan"), device="cuda")
    fc.fft1d_r2c(xd, out, n)
    torch.cuda.synchronize()
    o = out.cpu().numpy().astype(np.float64)
    return o[..., 0] + 1j * o[..., 1]


def gpu_c2r(X, n, olen, scale, init=None):
    import torch
    import paper_1412_7580_b200 as fc
    Xd = torch.from_numpy(np.stack([X.real, X.imag], axis=-1).astype(np.float32)).cuda()
    if init is None:
        out = torch.full((X.shape[0], olen), float("nan"), device="cuda")
    else:
        out = torch.from_numpy(init.copy()).cuda()
    fc.fft1d_c2r(Xd, out, n, scale, accumulate=init is not None)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("batch", [1, 33, 1000])
def test_forward_full_length(n, batch):
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    x = wl.make_planes(batch, 1, n, seed=n + batch)[:, 0, :].copy()
    assert relerr(gpu_r2c(x, n), oracle.dft1d_r2c(x, n)) <= TOL


@pytest.mark.parametrize("n,ln", [(2, 1), (8, 5), (16, 15), (32, 17), (64, 1), (64, 63), (128, 65), (128, 127),
                                  (256, 3), (256, 129), (256, 255)])
def test_forward_zero_padded(n, ln):
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    x = wl.make_planes(77, 1, ln, seed=n * 1000 + ln)[:, 0, :].copy()
    got = gpu_r2c(x, n)
    assert np.all(np.isfinite(got))
    assert relerr(got, oracle.dft1d_r2c(x, n)) <= TOL


@pytest.mark.parametrize("n", SIZES)
@pytest.mark.parametrize("crop", ["full", "ragged"])
def test_inverse_with_crop_and_scale(n, crop):
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    batch = 131
    x = wl.make_planes(batch, 1, n, seed=5 * n)[:, 0, :].copy()
    X = oracle.dft1d_r2c(x, n)
    X32 = (X.real.astype(np.float32) + 1j * X.imag.astype(np.float32)).astype(np.complex128)
    olen = n if crop == "full" else max(1, (2 * n) // 3)
    ref = oracle.idft1d_c2r(X32, n, olen, 1.0 / n)
    got = gpu_c2r(X32, n, olen, 1.0 / n)
    assert np.all(np.isfinite(got))
    assert relerr(got, ref) <= TOL


def test_inverse_accumulates():
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    n, batch, olen = 128, 40, 100
    x = wl.make_planes(batch, 1, n, seed=9)[:, 0, :].copy()
    X = oracle.dft1d_r2c(x, n)
    X32 = (X.real.astype(np.float32) + 1j * X.imag.astype(np.float32)).astype(np.complex128)
    init = wl.make_planes(batch, 1, olen, seed=10)[:, 0, :].copy()
    ref = init.astype(np.float64) + oracle.idft1d_c2r(X32, n, olen, 0.5 / n)
    assert relerr(gpu_c2r(X32, n, olen, 0.5 / n, init=init), ref) <= TOL


def test_round_trip_large_batch():
    import torch
    import paper_1412_7580_b200 as fc
    n, batch = 64, 200003                     # several thousand CTAs and a ragged last tile
    x = torch.rand((batch, n), device="cuda") * 2 - 1
    X = torch.empty((batch, n // 2 + 1, 2), device="cuda")
    back = torch.empty_like(x)
    fc.fft1d_r2c(x, X, n)
    fc.fft1d_c2r(X, back, n, 1.0 / n)
    torch.cuda.synchronize()
    assert float((back - x).abs().max()) <= 1e-5


def test_argument_checks():
    import ctypes
    from paper_1412_7580_b200 import binding as b
    L = b.lib()
    one, z = ctypes.c_void_p(256), ctypes.c_void_p(0)
    assert L.fft1d_r2c(one, one, 1, 9, 8, z) == b.EINVAL          # len > n
    assert L.fft1d_r2c(one, one, 1, 8, 12, z) == b.EUNSUPPORTED   # not a power of two
    assert L.fft1d_r2c(one, one, 1, 8, 512, z) == b.EUNSUPPORTED
    assert L.fft1d_r2c(z, one, 1, 8, 8, z) == b.EINVAL
    assert L.fft1d_c2r(one, one, 1, 8, 9, 1.0, 0, z) == b.EINVAL
    assert L.fft1d_c2r(one, one, 0, 8, 8, 1.0, 0, z) == b.EINVAL
