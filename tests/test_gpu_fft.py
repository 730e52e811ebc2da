"""Bare transforms on the GPU against the oracle's naive DFT (tolerance 1e-5
of the output's max-abs, the bound the task states for the bare FFTs)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL_FFT = 1e-5


def relerr(got, ref):
    m = np.max(np.abs(ref))
    if m == 0:
        return float(np.max(np.abs(got)))
    return float(np.max(np.abs(got - ref)) / m)


def gpu_r2c(x, n):
    import torch
    import paper_1412_7580_b200 as fc
    xd = torch.from_numpy(x).cuda()
    out = torch.full((x.shape[0], n, n // 2 + 1, 2), float("nan"), device="cuda")
    fc.fft2d_r2c(xd, out, n)
    torch.cuda.synchronize()
    o = out.cpu().numpy().astype(np.float64)
    return o[..., 0] + 1j * o[..., 1]


def gpu_c2r(X, n, oh, ow, scale, init=None):
    import torch
    import paper_1412_7580_b200 as fc
    Xi = np.stack([X.real, X.imag], axis=-1).astype(np.float32)
    Xd = torch.from_numpy(Xi).cuda()
    if init is None:
        out = torch.full((X.shape[0], oh, ow), float("nan"), device="cuda")
        fc.fft2d_c2r(Xd, out, n, scale)
    else:
        out = torch.from_numpy(init).cuda()
        fc.fft2d_c2r(Xd, out, n, scale, accumulate=True)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.float64)


CASES = [
    # n, batch, h, w
    (8, 1, 8, 8), (8, 37, 5, 3), (8, 64, 1, 8), (8, 33, 7, 7),
    (16, 1, 16, 16), (16, 70, 13, 13), (16, 32, 3, 3), (16, 5, 16, 1), (16, 33, 9, 14),
    (32, 1, 32, 32), (32, 35, 31, 31), (32, 16, 5, 5), (32, 19, 27, 20), (32, 17, 17, 32),
    (64, 1, 64, 64), (64, 11, 57, 57), (64, 8, 11, 11), (64, 9, 54, 33), (64, 3, 64, 1),
    (128, 1, 128, 128), (128, 3, 120, 120), (128, 2, 13, 13), (128, 3, 65, 100),
]


@pytest.mark.parametrize("n,batch,h,w", CASES)
def test_r2c_matches_naive_dft(n, batch, h, w):
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    x = wl.make_planes(batch, h, w, seed=n * 1000 + h)
    got = gpu_r2c(x, n)
    assert np.all(np.isfinite(got.real)) and np.all(np.isfinite(got.imag))
    ref = oracle.dft2d_r2c(x, n)
    assert relerr(got, ref) <= TOL_FFT


@pytest.mark.parametrize("n,batch,h,w", CASES)
def test_c2r_matches_naive_idft(n, batch, h, w):
    """Spectra of real planes (always Hermitian-consistent) back to a cropped
    window of oh x ow = h x w, through the oracle's inverse."""
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    x = wl.make_planes(batch, n, n, seed=n * 1000 + w + 7)
    X = oracle.dft2d_r2c(x, n)
    X32 = (X.real.astype(np.float32) + 1j * X.imag.astype(np.float32)).astype(np.complex128)
    scale = 1.0 / (n * n)
    got = gpu_c2r(X32, n, h, w, scale)
    assert np.all(np.isfinite(got))
    ref = oracle.idft2d_c2r(X32, n, h, w, scale)
    assert relerr(got, ref) <= TOL_FFT


def test_c2r_accumulate_and_scale():
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    n, batch, oh, ow = 16, 21, 11, 12
    x = wl.make_planes(batch, n, n, seed=5)
    X = oracle.dft2d_r2c(x, n)
    X32 = (X.real.astype(np.float32) + 1j * X.imag.astype(np.float32)).astype(np.complex128)
    init = wl.make_planes(batch, oh, ow, seed=6)
    got = gpu_c2r(X32, n, oh, ow, 0.5, init=init.copy())
    ref = init.astype(np.float64) + oracle.idft2d_c2r(X32, n, oh, ow, 0.5)
    assert relerr(got, ref) <= TOL_FFT


def test_round_trip_on_gpu():
    from paper_1412_7580_b200 import workloads as wl
    n, batch, h, w = 32, 50, 31, 29
    x = wl.make_planes(batch, h, w, seed=11)
    X = gpu_r2c(x, n)
    back = gpu_c2r(X, n, h, w, 1.0 / (n * n))
    assert relerr(back, x.astype(np.float64)) <= TOL_FFT


def test_outputs_outside_the_result_are_untouched():
    """Canary bands before and after the output stay intact (no stray writes)."""
    import torch
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    n, batch, h, w = 16, 33, 13, 13
    x = torch.from_numpy(wl.make_planes(batch, h, w, seed=3)).cuda()
    nout = batch * n * (n // 2 + 1) * 2
    guard = 4096
    buf = torch.full((nout + 2 * guard,), -7.25, device="cuda")
    out = buf[guard:guard + nout].view(batch, n, n // 2 + 1, 2)
    fc.fft2d_r2c(x, out, n)
    torch.cuda.synchronize()
    assert torch.all(buf[:guard] == -7.25) and torch.all(buf[guard + nout:] == -7.25)
    assert not torch.any(out == -7.25)


@pytest.mark.parametrize("n,batch,h,w", [(8, 37, 5, 3), (16, 70, 13, 13), (32, 35, 31, 31), (64, 9, 54, 33)])
def test_bare_transforms_with_a_spectrum_that_is_only_8_byte_aligned(n, batch, h, w):
    """A 16-byte-aligned spectrum travels by bulk copies through shared memory; one that is
    only 8-byte aligned is accessed by the threads directly.  Both must give the same numbers."""
    import torch
    import oracle
    import paper_1412_7580_b200 as fc
    from paper_1412_7580_b200 import workloads as wl
    x = wl.make_planes(batch, h, w, seed=n * 77 + w)
    xd = torch.from_numpy(x).cuda()
    nc = n // 2 + 1
    buf = torch.full((batch * n * nc * 2 + 2,), float("nan"), device="cuda")
    out = buf[2:].view(batch, n, nc, 2)                      # 8 bytes past a 16-byte boundary
    assert out.data_ptr() % 16 == 8
    fc.fft2d_r2c(xd, out, n)
    aligned = torch.full((batch, n, nc, 2), float("nan"), device="cuda")
    fc.fft2d_r2c(xd, aligned, n)
    torch.cuda.synchronize()
    assert torch.equal(out, aligned)
    assert bool(torch.isnan(buf[:2]).all())                  # nothing written in front of the view
    o = out.cpu().numpy().astype(np.float64)
    assert relerr(o[..., 0] + 1j * o[..., 1], oracle.dft2d_r2c(x, n)) <= TOL_FFT
    back_a = torch.full((batch, h, w), float("nan"), device="cuda")
    back_u = torch.full((batch, h, w), float("nan"), device="cuda")
    fc.fft2d_c2r(aligned, back_a, n, 1.0 / (n * n))
    fc.fft2d_c2r(out, back_u, n, 1.0 / (n * n))
    torch.cuda.synchronize()
    assert torch.equal(back_a, back_u)
    assert relerr(back_a.cpu().numpy().astype(np.float64), x.astype(np.float64)) <= TOL_FFT
