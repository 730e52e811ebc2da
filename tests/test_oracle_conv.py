"""Pins for the convolution oracle (CPU only).

The oracle's gather-form sums are checked against things that are not the
oracle: an independently written scatter-form brute force in pure Python,
closed forms, special cases that reduce to a matrix product, the adjoint
identity that makes bprop / accGrad the gradients of fprop (Section 2), and
linearity (Section 2, "linearity of the DFT" applies to the passes as well).
"""
import itertools

import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(20141224)


def rand(*dims):
    return (RNG.random(dims, dtype=np.float32) * 2 - 1).astype(np.float32)


def scatter_brute_force(x, w, dy):
    """One 7-deep loop nest; every product x*w / dy*w / dy*x is pushed to the
    element it belongs to (scatter form), the opposite of the oracle's
    per-output gather sums."""
    S, f, h, wd = x.shape
    fp, _, kh, kw = w.shape
    oh, ow = h - kh + 1, wd - kw + 1
    y = np.zeros((S, fp, oh, ow))
    dx = np.zeros((S, f, h, wd))
    dw = np.zeros((fp, f, kh, kw))
    x64, w64, g64 = x.astype(np.float64), w.astype(np.float64), dy.astype(np.float64)
    for s, j, i, a, b, u, v in itertools.product(range(S), range(fp), range(f), range(oh),
                                                 range(ow), range(kh), range(kw)):
        y[s, j, a, b] += x64[s, i, a + u, b + v] * w64[j, i, u, v]
        dx[s, i, a + u, b + v] += g64[s, j, a, b] * w64[j, i, u, v]
        dw[j, i, u, v] += g64[s, j, a, b] * x64[s, i, a + u, b + v]
    return y, dx, dw


@pytest.mark.parametrize("S,f,fp,h,w,kh,kw", [
    (2, 3, 4, 7, 6, 3, 2),
    (1, 1, 1, 5, 5, 5, 5),
    (3, 2, 1, 4, 9, 1, 4),
    (1, 2, 3, 6, 5, 2, 5),
])
def test_gather_forms_equal_scatter_brute_force(S, f, fp, h, w, kh, kw):
    x, wt = rand(S, f, h, w), rand(fp, f, kh, kw)
    dy = rand(S, fp, h - kh + 1, w - kw + 1)
    y, dx, dw = scatter_brute_force(x, wt, dy)
    np.testing.assert_allclose(oracle.fprop(x, wt), y, rtol=0, atol=1e-13)
    np.testing.assert_allclose(oracle.bprop(dy, wt, h, w), dx, rtol=0, atol=1e-13)
    np.testing.assert_allclose(oracle.accgrad(dy, x, kh, kw), dw, rtol=0, atol=1e-13)


def test_adjoint_identity():
    # <y, dy> = <x, dx> = <w, dw> when y = fprop(x, w), dx = bprop(dy, w),
    # dw = accGrad(dy, x): the three passes are one bilinear form.
    S, f, fp, h, w, kh, kw = 3, 4, 5, 9, 8, 3, 4
    x, wt = rand(S, f, h, w), rand(fp, f, kh, kw)
    dy = rand(S, fp, h - kh + 1, w - kw + 1)
    a = np.sum(oracle.fprop(x, wt) * dy.astype(np.float64))
    b = np.sum(oracle.bprop(dy, wt, h, w) * x.astype(np.float64))
    c = np.sum(oracle.accgrad(dy, x, kh, kw) * wt.astype(np.float64))
    assert abs(a - b) < 1e-11 * max(1.0, abs(a))
    assert abs(a - c) < 1e-11 * max(1.0, abs(a))


def test_fprop_delta_kernel_is_shifted_crop():
    S, f, h, w, kh, kw, u0, v0 = 2, 3, 8, 7, 3, 4, 2, 1
    x = rand(S, f, h, w)
    wt = np.zeros((f, f, kh, kw), np.float32)
    for j in range(f):
        wt[j, j, u0, v0] = 1.0
    y = oracle.fprop(x, wt)
    oh, ow = h - kh + 1, w - kw + 1
    np.testing.assert_array_equal(y, x[:, :, u0:u0 + oh, v0:v0 + ow].astype(np.float64))


def test_fprop_1x1_kernel_is_matrix_product():
    S, f, fp, h, w = 2, 5, 3, 4, 6
    x, wt = rand(S, f, h, w), rand(fp, f, 1, 1)
    y = oracle.fprop(x, wt)
    ref = np.einsum("ji,sihw->sjhw", wt[:, :, 0, 0].astype(np.float64), x.astype(np.float64))
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-13)


def test_fprop_full_size_kernel_is_dot_product():
    S, f, fp, h, w = 2, 3, 2, 5, 4
    x, wt = rand(S, f, h, w), rand(fp, f, h, w)
    y = oracle.fprop(x, wt)
    assert y.shape == (S, fp, 1, 1)
    ref = np.einsum("sihw,jihw->sj", x.astype(np.float64), wt.astype(np.float64))
    np.testing.assert_allclose(y[:, :, 0, 0], ref, rtol=0, atol=1e-13)


def test_all_ones_closed_forms():
    S, f, fp, h, w, kh, kw = 3, 2, 4, 7, 9, 3, 5
    oh, ow = h - kh + 1, w - kw + 1
    x = np.ones((S, f, h, w), np.float32)
    wt = np.ones((fp, f, kh, kw), np.float32)
    dy = np.ones((S, fp, oh, ow), np.float32)
    np.testing.assert_array_equal(oracle.fprop(x, wt), np.full((S, fp, oh, ow), f * kh * kw))
    np.testing.assert_array_equal(oracle.accgrad(dy, x, kh, kw),
                                  np.full((fp, f, kh, kw), S * oh * ow))
    # full convolution of two boxes: the count of overlapping taps
    ch = np.array([min(p + 1, kh, oh, h - p) for p in range(h)], np.float64)
    cw = np.array([min(q + 1, kw, ow, w - q) for q in range(w)], np.float64)
    ref = fp * ch[:, None] * cw[None, :]
    dx = oracle.bprop(dy, wt, h, w)
    for s in range(S):
        for i in range(f):
            np.testing.assert_array_equal(dx[s, i], ref)


def test_bprop_delta_kernel_is_shifted_zero_filled():
    S, f, h, w, kh, kw, u0, v0 = 2, 3, 8, 7, 3, 4, 1, 3
    oh, ow = h - kh + 1, w - kw + 1
    dy = rand(S, f, oh, ow)
    wt = np.zeros((f, f, kh, kw), np.float32)
    for j in range(f):
        wt[j, j, u0, v0] = 1.0
    dx = oracle.bprop(dy, wt, h, w)
    ref = np.zeros((S, f, h, w))
    ref[:, :, u0:u0 + oh, v0:v0 + ow] = dy
    np.testing.assert_array_equal(dx, ref)


def test_accgrad_delta_gradient_picks_window_of_x():
    h, w, kh, kw, a0, b0 = 9, 8, 4, 3, 2, 5
    oh, ow = h - kh + 1, w - kw + 1
    x = rand(1, 1, h, w)
    dy = np.zeros((1, 1, oh, ow), np.float32)
    dy[0, 0, a0, b0] = 1.0
    dw = oracle.accgrad(dy, x, kh, kw)
    np.testing.assert_array_equal(dw[0, 0], x[0, 0, a0:a0 + kh, b0:b0 + kw].astype(np.float64))


def test_bprop_matches_numpy_full_convolution_1d_rows():
    # one plane, kernel of one row: dx rows are np.convolve (full) of dy rows
    h, w, kw = 1, 12, 5
    dy, wt = rand(1, 1, 1, w - kw + 1), rand(1, 1, 1, kw)
    dx = oracle.bprop(dy, wt, h, w)
    ref = np.convolve(dy[0, 0, 0].astype(np.float64), wt[0, 0, 0].astype(np.float64), mode="full")
    np.testing.assert_allclose(dx[0, 0, 0], ref, rtol=0, atol=1e-14)
    # and fprop rows are np.correlate (valid)
    x = rand(1, 1, 1, w)
    y = oracle.fprop(x, wt)
    ref = np.correlate(x[0, 0, 0].astype(np.float64), wt[0, 0, 0].astype(np.float64), mode="valid")
    np.testing.assert_allclose(y[0, 0, 0], ref, rtol=0, atol=1e-14)


def test_linearity_in_each_operand():
    S, f, fp, h, w, kh, kw = 2, 3, 2, 6, 6, 3, 3
    # values with short mantissas so that alpha*A + beta*A' is exact in fp32
    def q(*d):
        return (RNG.integers(-64, 65, size=d) / 64.0).astype(np.float32)
    x1, x2, wt = q(S, f, h, w), q(S, f, h, w), q(fp, f, kh, kw)
    w2 = q(fp, f, kh, kw)
    dy, dy2 = q(S, fp, h - kh + 1, w - kw + 1), q(S, fp, h - kh + 1, w - kw + 1)
    al, be = 2.0, -0.5
    np.testing.assert_allclose(oracle.fprop(al * x1 + be * x2, wt),
                               al * oracle.fprop(x1, wt) + be * oracle.fprop(x2, wt), atol=1e-12)
    np.testing.assert_allclose(oracle.fprop(x1, al * wt + be * w2),
                               al * oracle.fprop(x1, wt) + be * oracle.fprop(x1, w2), atol=1e-12)
    np.testing.assert_allclose(oracle.bprop(al * dy + be * dy2, wt, h, w),
                               al * oracle.bprop(dy, wt, h, w) + be * oracle.bprop(dy2, wt, h, w),
                               atol=1e-12)
    np.testing.assert_allclose(oracle.accgrad(dy, al * x1 + be * x2, kh, kw),
                               al * oracle.accgrad(dy, x1, kh, kw) + be * oracle.accgrad(dy, x2, kh, kw),
                               atol=1e-12)


def test_sampled_variants_equal_full_tensors():
    from paper_1412_7580_b200 import workloads as wl
    S, f, fp, h, w, kh, kw = 3, 4, 5, 9, 8, 3, 4
    x, wt = rand(S, f, h, w), rand(fp, f, kh, kw)
    dy = rand(S, fp, h - kh + 1, w - kw + 1)
    y, dx, dw = oracle.fprop(x, wt), oracle.bprop(dy, wt, h, w), oracle.accgrad(dy, x, kh, kw)
    for full, fn in ((y, lambda c: oracle.fprop_at(x, wt, c)),
                     (dx, lambda c: oracle.bprop_at(dy, wt, h, w, c)),
                     (dw, lambda c: oracle.accgrad_at(dy, x, kh, kw, c))):
        c = wl.sample_coords(full.shape, 64, seed=3)
        got = fn(c)
        np.testing.assert_array_equal(got, full[c[:, 0], c[:, 1], c[:, 2], c[:, 3]])


def test_tiling_identity_section6():
    # y[i, i+d) = x[i, i+d+k-1) (star) c : a tile of the output only needs the
    # matching window of the input (Section 6).
    h, w, k, d, i0 = 1, 20, 4, 5, 7
    x, c = rand(1, 1, h, w), rand(1, 1, 1, k)
    y = oracle.fprop(x, c)
    tile = oracle.fprop(x[:, :, :, i0:i0 + d + k - 1], c)
    np.testing.assert_array_equal(tile[0, 0, 0], y[0, 0, 0, i0:i0 + d])
