"""Pins for the one-dimensional naive DFT of the oracle (CPU only).

Closed forms follow from the definition in Supplement 8.2 (forward sign minus,
no normalisation, zero-padding from len to n); numpy.fft.rfft / irfft serve as
library special cases; the 2-D transform of a one-row plane must reduce to it.
"""
import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(75801)
SIZES = [2, 4, 8, 16, 32, 64, 128, 256]


def rand(*dims):
    return (RNG.random(dims, dtype=np.float32) * 2 - 1).astype(np.float32)


@pytest.mark.parametrize("n", SIZES)
def test_constant_and_alternating(n):
    X = oracle.dft1d_r2c(np.full((1, n), 0.5, np.float32), n)[0]
    ref = np.zeros(n // 2 + 1, np.complex128)
    ref[0] = 0.5 * n
    np.testing.assert_allclose(X, ref, rtol=0, atol=1e-10)
    alt = ((-1.0) ** np.arange(n)).astype(np.float32)[None]
    X = oracle.dft1d_r2c(alt, n)[0]
    ref = np.zeros(n // 2 + 1, np.complex128)
    ref[n // 2] = n                                  # all the energy in the Nyquist bin
    np.testing.assert_allclose(X, ref, rtol=0, atol=1e-10)


@pytest.mark.parametrize("n,j0", [(8, 3), (32, 31), (256, 100)])
def test_delta_is_pure_phase_with_minus_sign(n, j0):
    x = np.zeros((1, n), np.float32)
    x[0, j0] = 1.0
    X = oracle.dft1d_r2c(x, n)[0]
    k = np.arange(n // 2 + 1)
    np.testing.assert_allclose(X, np.exp(-2j * np.pi * k * j0 / n), rtol=0, atol=1e-13)


@pytest.mark.parametrize("n,ln", [(8, 8), (16, 11), (64, 1), (128, 100), (256, 255)])
def test_against_numpy_rfft_with_zero_padding(n, ln):
    x = rand(5, ln)
    X = oracle.dft1d_r2c(x, n)
    np.testing.assert_allclose(X, np.fft.rfft(x.astype(np.float64), n=n, axis=1), rtol=0, atol=1e-11)


@pytest.mark.parametrize("n", [4, 32, 256])
def test_parseval_on_the_half_spectrum(n):
    x = rand(3, n)
    X = oracle.dft1d_r2c(x, n)
    m = np.full(n // 2 + 1, 2.0)
    m[0] = m[-1] = 1.0
    lhs = np.sum(x.astype(np.float64) ** 2, axis=1)
    rhs = np.sum(m * np.abs(X) ** 2, axis=1) / n
    np.testing.assert_allclose(lhs, rhs, rtol=1e-12)


@pytest.mark.parametrize("n,olen", [(8, 8), (16, 5), (128, 128), (256, 17)])
def test_round_trip_and_crop(n, olen):
    x = rand(4, n)
    X = oracle.dft1d_r2c(x, n)
    back = oracle.idft1d_c2r(X, n, olen, 1.0 / n)
    np.testing.assert_allclose(back, x[:, :olen].astype(np.float64), rtol=0, atol=1e-12)
    np.testing.assert_allclose(oracle.idft1d_c2r(X, n, olen, 1.0),
                               np.fft.irfft(X, n=n, axis=1)[:, :olen] * n, rtol=0, atol=1e-10)


def test_linearity_and_shift_theorem():
    n = 32
    a, b = rand(1, n), rand(1, n)
    lhs = oracle.dft1d_r2c((2.0 * a - 0.5 * b).astype(np.float32), n)
    rhs = 2.0 * oracle.dft1d_r2c(a, n) - 0.5 * oracle.dft1d_r2c(b, n)
    np.testing.assert_allclose(lhs, rhs, rtol=0, atol=1e-5)      # fp32 rounding of the combined input
    # a cyclic shift by s multiplies bin k by exp(-2 pi i k s / n)
    s = 5
    shifted = np.roll(a, s, axis=1)
    k = np.arange(n // 2 + 1)
    np.testing.assert_allclose(oracle.dft1d_r2c(shifted, n),
                               oracle.dft1d_r2c(a, n) * np.exp(-2j * np.pi * k * s / n), rtol=0, atol=1e-12)


def test_two_dimensional_transform_of_a_single_row_reduces_to_it():
    n, ln = 16, 13
    x = rand(3, ln)
    X1 = oracle.dft1d_r2c(x, n)
    X2 = oracle.dft2d_r2c(x[:, None, :], n)          # planes of one row: no dependence on ky
    for ky in range(n):
        np.testing.assert_allclose(X2[:, ky, :], X1, rtol=0, atol=1e-12)
