"""Pins for the naive-DFT part of the oracle and for the convolution theorem
that ties it to the direct sums (CPU only).

Closed forms follow from the definition in Supplement 8.2 (forward sign
minus, no normalisation); numpy.fft.rfft2 serves as a library special case.
"""
import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(7580)


def rand(*dims):
    return (RNG.random(dims, dtype=np.float32) * 2 - 1).astype(np.float32)


@pytest.mark.parametrize("n", [8, 16])
def test_dft_of_constant(n):
    c = 0.75
    X = oracle.dft2d_r2c(np.full((1, n, n), c, np.float32), n)[0]
    ref = np.zeros((n, n // 2 + 1), np.complex128)
    ref[0, 0] = c * n * n
    np.testing.assert_allclose(X, ref, rtol=0, atol=1e-11)


@pytest.mark.parametrize("n,r0,c0", [(8, 3, 5), (16, 0, 1), (16, 15, 15)])
def test_dft_of_delta_is_pure_phase(n, r0, c0):
    x = np.zeros((1, n, n), np.float32)
    x[0, r0, c0] = 1.0
    X = oracle.dft2d_r2c(x, n)[0]
    ky, kx = np.meshgrid(np.arange(n), np.arange(n // 2 + 1), indexing="ij")
    ref = np.exp(-2j * np.pi * (ky * r0 + kx * c0) / n)
    np.testing.assert_allclose(X, ref, rtol=0, atol=1e-13)


def full_spectrum_direct(x, n):
    """All n x n bins straight from the definition with numpy broadcasting."""
    h, w = x.shape
    ky = np.arange(n)[:, None, None, None]
    kx = np.arange(n)[None, :, None, None]
    r = np.arange(h)[None, None, :, None]
    c = np.arange(w)[None, None, None, :]
    return np.sum(x.astype(np.float64) * np.exp(-2j * np.pi * ((ky * r + kx * c) % n) / n),
                  axis=(2, 3))


@pytest.mark.parametrize("n,h,w", [(8, 8, 8), (8, 5, 3), (16, 13, 16), (16, 1, 9)])
def test_half_spectrum_hermitian_and_library(n, h, w):
    x = rand(1, h, w)
    X = oracle.dft2d_r2c(x, n)[0]
    F = full_spectrum_direct(x[0], n)
    # stored half equals the left half of the full transform
    np.testing.assert_allclose(X, F[:, :n // 2 + 1], rtol=0, atol=1e-12)
    # Hermitian symmetry of the full transform of a real signal
    idx = (-np.arange(n)) % n
    np.testing.assert_allclose(F, np.conj(F[np.ix_(idx, idx)]), rtol=0, atol=1e-12)
    # library routine on the zero-padded plane (special case: same definition)
    np.testing.assert_allclose(X, np.fft.rfft2(x[0].astype(np.float64), s=(n, n)), rtol=0, atol=1e-12)


@pytest.mark.parametrize("n,h,w", [(8, 8, 8), (16, 11, 7)])
def test_parseval_on_half_spectrum(n, h, w):
    x = rand(1, h, w)
    X = oracle.dft2d_r2c(x, n)[0]
    m = np.full(n // 2 + 1, 2.0)
    m[0] = m[n // 2] = 1.0
    lhs = np.sum(x.astype(np.float64) ** 2)
    rhs = np.sum(m[None, :] * np.abs(X) ** 2) / (n * n)
    assert abs(lhs - rhs) < 1e-12 * max(1.0, lhs)


def test_separability_rows_then_columns():
    n, h, w = 16, 12, 9
    x = rand(1, h, w)
    X = oracle.dft2d_r2c(x, n)[0]
    xp = np.zeros((n, n))
    xp[:h, :w] = x[0]
    k = np.arange(n)
    Wn = np.exp(-2j * np.pi * np.outer(k, k) / n)      # 1-D DFT matrix
    rows = xp @ Wn.T                                     # transform along columns index c
    both = Wn @ rows                                     # then along r
    np.testing.assert_allclose(X, both[:, :n // 2 + 1], rtol=0, atol=1e-12)


@pytest.mark.parametrize("n,h,w", [(8, 8, 8), (16, 13, 10), (16, 16, 16)])
def test_round_trip(n, h, w):
    x = rand(3, h, w)
    X = oracle.dft2d_r2c(x, n)
    back = oracle.idft2d_c2r(X, n, n, n, 1.0 / (n * n))
    ref = np.zeros((3, n, n))
    ref[:, :h, :w] = x
    np.testing.assert_allclose(back, ref, rtol=0, atol=1e-13)
    # crop window is anchored at the origin
    crop = oracle.idft2d_c2r(X, n, h, w, 1.0 / (n * n))
    np.testing.assert_allclose(crop, x.astype(np.float64), rtol=0, atol=1e-13)


def test_idft_matches_library_irfft2():
    n = 16
    x = rand(2, n, n)
    X = np.fft.rfft2(x.astype(np.float64))
    out = oracle.idft2d_c2r(X, n, n, n, 1.0 / (n * n))
    np.testing.assert_allclose(out, np.fft.irfft2(X, s=(n, n)), rtol=0, atol=1e-13)


def test_idft_scale_is_applied_linearly():
    n = 8
    X = oracle.dft2d_r2c(rand(1, n, n), n)
    a = oracle.idft2d_c2r(X, n, 5, 6, 1.0)
    b = oracle.idft2d_c2r(X, n, 5, 6, 0.25)
    np.testing.assert_allclose(b, 0.25 * a, rtol=0, atol=1e-12)


def test_bin_contract_against_einsum():
    bins, M, N, K = 5, 3, 4, 6
    A = RNG.standard_normal((bins, M, K)) + 1j * RNG.standard_normal((bins, M, K))
    B = RNG.standard_normal((bins, N, K)) + 1j * RNG.standard_normal((bins, N, K))
    for ca in (False, True):
        for cb in (False, True):
            ref = np.einsum("bmk,bnk->bmn", np.conj(A) if ca else A, np.conj(B) if cb else B)
            np.testing.assert_allclose(oracle.bin_contract(A, B, ca, cb), ref, rtol=0, atol=1e-12)


@pytest.mark.parametrize("S,f,fp,h,w,kh,kw,n", [
    (2, 3, 2, 8, 8, 3, 3, 8),
    (1, 2, 3, 13, 11, 5, 4, 16),
    (2, 1, 1, 6, 7, 6, 7, 8),
])
def test_convolution_theorem_all_three_passes(S, f, fp, h, w, kh, kw, n):
    """Direct sums == inverse DFT of per-bin products (Section 2, the
    convolution theorem with the conjugate for cross-correlation; Table 1)."""
    oh, ow = h - kh + 1, w - kw + 1
    x, wt, dy = rand(S, f, h, w), rand(fp, f, kh, kw), rand(S, fp, oh, ow)
    B = n * (n // 2 + 1)
    Xf = oracle.dft2d_r2c(x.reshape(-1, h, w), n).reshape(S, f, B)
    Wf = oracle.dft2d_r2c(wt.reshape(-1, kh, kw), n).reshape(fp, f, B)
    Gf = oracle.dft2d_r2c(dy.reshape(-1, oh, ow), n).reshape(S, fp, B)
    sc = 1.0 / (n * n)
    # fprop: conj on the weights, reduce over f
    Yf = oracle.bin_contract(Xf.transpose(2, 0, 1), Wf.transpose(2, 0, 1), False, True)  # [B,S,fp]
    y = oracle.idft2d_c2r(Yf.transpose(1, 2, 0).reshape(S * fp, n, n // 2 + 1), n, oh, ow, sc)
    np.testing.assert_allclose(y.reshape(S, fp, oh, ow), oracle.fprop(x, wt), rtol=0, atol=1e-12)
    # bprop: no conjugate, reduce over f'
    DXf = oracle.bin_contract(Gf.transpose(2, 0, 1), Wf.transpose(2, 1, 0), False, False)  # [B,S,f]
    dx = oracle.idft2d_c2r(DXf.transpose(1, 2, 0).reshape(S * f, n, n // 2 + 1), n, h, w, sc)
    np.testing.assert_allclose(dx.reshape(S, f, h, w), oracle.bprop(dy, wt, h, w), rtol=0, atol=1e-12)
    # accGrad: conj on the output gradient, reduce over S
    DWf = oracle.bin_contract(Gf.transpose(2, 1, 0), Xf.transpose(2, 1, 0), True, False)  # [B,fp,f]
    dw = oracle.idft2d_c2r(DWf.transpose(1, 2, 0).reshape(fp * f, n, n // 2 + 1), n, kh, kw, sc)
    np.testing.assert_allclose(dw.reshape(fp, f, kh, kw), oracle.accgrad(dy, x, kh, kw), rtol=0, atol=1e-12)
