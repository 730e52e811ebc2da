/*
 * CPU oracle for FFT-domain convolution of CNN layers (fprop / bprop / accGrad)
 * and for the bare batched 2-D R2C / C2R transforms.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the yardstick the CUDA library is
 * compared against; it is never part of the product path.  It shares no code,
 * header, table or constant with the CUDA sources.  Everything is the plain
 * definition, written out as nested sums in float64: no FFT, no blocking, no
 * reordering.  Inputs are fp32 arrays (converted per element), outputs are
 * float64.
 *
 * Notation follows the paper (Section 2): S minibatch, f input planes,
 * fp (= f') output planes, h x w input plane, kh x kw kernel,
 * oh x ow = (h-kh+1) x (w-kw+1) output plane ("valid" only), n = size of the
 * square Fourier basis.
 *
 * Layouts (Section 3.1, row-major "BDHW"):
 *   x [S ][f ][h ][w ]      w [fp][f][kh][kw]      y, dy [S][fp][oh][ow]
 *   dx like x, dw like w.
 *
 * Pins (tests/test_oracle_*.py): scatter-form brute force written
 * independently in Python, adjoint identity between the three passes,
 * delta-kernel / all-ones / 1x1-kernel closed forms, linearity, the
 * convolution theorem through the naive DFT below, and for the DFT: constant,
 * delta, Hermitian symmetry, Parseval, separability, round trip, and
 * numpy.fft.rfft2 as a library special case.
 *
 * OpenMP only parallelises the outermost independent output loop; each output
 * element is still one sequential sum in the order the formula states.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define API __attribute__((visibility("default")))

API int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- single output elements: the definitions, one sum each ------------- */

/* Section 2, first equation: y(s,j) = sum_i x(s,i) (star) w(j,i), valid
 * cross-correlation: y[s,j,a,b] = sum_{i,u,v} x[s,i,a+u,b+v] * w[j,i,u,v]. */
static double fprop_elem(const float *x, const float *wt, int f, int h, int w,
                         int kh, int kw, int s, int j, int a, int b) {
    double acc = 0.0;
    for (int i = 0; i < f; ++i)
        for (int u = 0; u < kh; ++u)
            for (int v = 0; v < kw; ++v) {
                double xv = x[(((size_t)s * f + i) * h + (a + u)) * w + (b + v)];
                double wv = wt[(((size_t)j * f + i) * kh + u) * kw + v];
                acc += xv * wv;
            }
    return acc;
}

/* Section 2, second equation: dL/dx(s,i) = sum_j dL/dy(s,j) * w(j,i), true
 * (full) convolution: dx[s,i,p,q] = sum_{j,u,v} dy[s,j,p-u,q-v] * w[j,i,u,v],
 * terms whose dy index falls outside [0,oh) x [0,ow) are zero. */
static double bprop_elem(const float *dy, const float *wt, int f, int fp, int h,
                         int w, int kh, int kw, int s, int i, int p, int q) {
    const int oh = h - kh + 1, ow = w - kw + 1;
    double acc = 0.0;
    for (int j = 0; j < fp; ++j)
        for (int u = 0; u < kh; ++u)
            for (int v = 0; v < kw; ++v) {
                int a = p - u, b = q - v;
                if (a < 0 || a >= oh || b < 0 || b >= ow) continue;
                double gv = dy[(((size_t)s * fp + j) * oh + a) * ow + b];
                double wv = wt[(((size_t)j * f + i) * kh + u) * kw + v];
                acc += gv * wv;
            }
    return acc;
}

/* Section 2, third equation: dL/dw(j,i) = sum_s dL/dy(s,j) (star) x(s,i); the
 * index form is the 1-D formula of Section 6, (dL/dc)_j = sum_i x_{j+i} z_i:
 * dw[j,i,u,v] = sum_{s,a,b} dy[s,j,a,b] * x[s,i,a+u,b+v]. */
static double accgrad_elem(const float *dy, const float *x, int S, int f, int fp,
                           int h, int w, int kh, int kw, int j, int i, int u, int v) {
    const int oh = h - kh + 1, ow = w - kw + 1;
    double acc = 0.0;
    for (int s = 0; s < S; ++s)
        for (int a = 0; a < oh; ++a)
            for (int b = 0; b < ow; ++b) {
                double gv = dy[(((size_t)s * fp + j) * oh + a) * ow + b];
                double xv = x[(((size_t)s * f + i) * h + (a + u)) * w + (b + v)];
                acc += gv * xv;
            }
    return acc;
}

/* ---- full tensors -------------------------------------------------------- */

API void oracle_fprop(const float *x, const float *wt, double *y, int S, int f,
                      int fp, int h, int w, int kh, int kw) {
    const int oh = h - kh + 1, ow = w - kw + 1;
    const long planes = (long)S * fp;
#pragma omp parallel for schedule(dynamic, 1)
    for (long sj = 0; sj < planes; ++sj) {
        int s = (int)(sj / fp), j = (int)(sj % fp);
        for (int a = 0; a < oh; ++a)
            for (int b = 0; b < ow; ++b)
                y[((size_t)sj * oh + a) * ow + b] =
                    fprop_elem(x, wt, f, h, w, kh, kw, s, j, a, b);
    }
}

API void oracle_bprop(const float *dy, const float *wt, double *dx, int S, int f,
                      int fp, int h, int w, int kh, int kw) {
    const long planes = (long)S * f;
#pragma omp parallel for schedule(dynamic, 1)
    for (long si = 0; si < planes; ++si) {
        int s = (int)(si / f), i = (int)(si % f);
        for (int p = 0; p < h; ++p)
            for (int q = 0; q < w; ++q)
                dx[((size_t)si * h + p) * w + q] =
                    bprop_elem(dy, wt, f, fp, h, w, kh, kw, s, i, p, q);
    }
}

API void oracle_accgrad(const float *dy, const float *x, double *dw, int S, int f,
                        int fp, int h, int w, int kh, int kw) {
    const long planes = (long)fp * f;
#pragma omp parallel for schedule(dynamic, 1)
    for (long ji = 0; ji < planes; ++ji) {
        int j = (int)(ji / f), i = (int)(ji % f);
        for (int u = 0; u < kh; ++u)
            for (int v = 0; v < kw; ++v)
                dw[((size_t)ji * kh + u) * kw + v] =
                    accgrad_elem(dy, x, S, f, fp, h, w, kh, kw, j, i, u, v);
    }
}

/* ---- the same definitions at a list of output coordinates ---------------
 * coords holds 4 ints per sample; out[k] is the value of that one element.
 * Used where a full tensor would take the CPU too long. */

API void oracle_fprop_at(const float *x, const float *wt, const int32_t *coords,
                         long ncoords, double *out, int S, int f, int fp, int h,
                         int w, int kh, int kw) {
    (void)S; (void)fp;
#pragma omp parallel for schedule(dynamic, 16)
    for (long k = 0; k < ncoords; ++k) {
        const int32_t *c = coords + 4 * k; /* s, j, a, b */
        out[k] = fprop_elem(x, wt, f, h, w, kh, kw, c[0], c[1], c[2], c[3]);
    }
}

API void oracle_bprop_at(const float *dy, const float *wt, const int32_t *coords,
                         long ncoords, double *out, int S, int f, int fp, int h,
                         int w, int kh, int kw) {
    (void)S;
#pragma omp parallel for schedule(dynamic, 16)
    for (long k = 0; k < ncoords; ++k) {
        const int32_t *c = coords + 4 * k; /* s, i, p, q */
        out[k] = bprop_elem(dy, wt, f, fp, h, w, kh, kw, c[0], c[1], c[2], c[3]);
    }
}

API void oracle_accgrad_at(const float *dy, const float *x, const int32_t *coords,
                           long ncoords, double *out, int S, int f, int fp, int h,
                           int w, int kh, int kw) {
#pragma omp parallel for schedule(dynamic, 1)
    for (long k = 0; k < ncoords; ++k) {
        const int32_t *c = coords + 4 * k; /* j, i, u, v */
        out[k] = accgrad_elem(dy, x, S, f, fp, h, w, kh, kw, c[0], c[1], c[2], c[3]);
    }
}

/* ---- naive discrete Fourier transforms -----------------------------------
 * Supplement 8.2: X_k = sum_j x_j w_n^{kj}, w_n^j = exp(-2 pi i j / n): the
 * forward transform has the minus sign and no normalisation.  In two
 * dimensions on an n x n basis, with the h x w plane zero-padded (Section
 * 3.1), and only the n/2+1 leftmost columns stored (Hermitian symmetry of a
 * real signal's spectrum):
 *   X[ky,kx] = sum_{r<h, c<w} x[r,c] exp(-2 pi i (ky r + kx c)/n),
 *   ky in [0,n), kx in [0,n/2].
 * The angle is reduced with integer arithmetic before cos/sin.
 * out: [batch][n][n/2+1][2] doubles (re, im). O(n^2 h w) per plane. */
API void oracle_dft2d_r2c(const float *in, double *out, long batch, int h, int w, int n) {
    const int nc = n / 2 + 1;
    const double two_pi = 6.283185307179586476925286766559;
#pragma omp parallel for schedule(dynamic, 1)
    for (long p = 0; p < batch; ++p) {
        const float *xp = in + (size_t)p * h * w;
        double *op = out + (size_t)p * n * nc * 2;
        for (int ky = 0; ky < n; ++ky)
            for (int kx = 0; kx < nc; ++kx) {
                double re = 0.0, im = 0.0;
                for (int r = 0; r < h; ++r)
                    for (int c = 0; c < w; ++c) {
                        int m = (int)(((long)ky * r + (long)kx * c) % n);
                        double ang = -two_pi * (double)m / (double)n;
                        double v = xp[(size_t)r * w + c];
                        re += v * cos(ang);
                        im += v * sin(ang);
                    }
                op[((size_t)ky * nc + kx) * 2 + 0] = re;
                op[((size_t)ky * nc + kx) * 2 + 1] = im;
            }
    }
}

/* Inverse: the conjugate basis (plus sign), scaled by the caller's `scale`
 * (1/n^2 undoes oracle_dft2d_r2c), evaluated only inside the crop window
 * [0,oh) x [0,ow) anchored at the origin (Section 3.1, clipping of the IFFT
 * output).  The stored half spectrum is extended to all n columns by
 * X~[ky,kx] = conj(X[(n-ky) mod n, n-kx]) for kx > n/2; the real part of the
 * sum is returned.
 * in: [batch][n][n/2+1][2] doubles; out: [batch][oh][ow] doubles. */
API void oracle_idft2d_c2r(const double *in, double *out, long batch, int n, int oh,
                           int ow, double scale) {
    const int nc = n / 2 + 1;
    const double two_pi = 6.283185307179586476925286766559;
#pragma omp parallel for schedule(dynamic, 1)
    for (long p = 0; p < batch; ++p) {
        const double *sp = in + (size_t)p * n * nc * 2;
        double *op = out + (size_t)p * oh * ow;
        for (int r = 0; r < oh; ++r)
            for (int c = 0; c < ow; ++c) {
                double acc = 0.0;
                for (int ky = 0; ky < n; ++ky)
                    for (int kx = 0; kx < n; ++kx) {
                        double re, im;
                        if (kx < nc) {
                            re = sp[((size_t)ky * nc + kx) * 2 + 0];
                            im = sp[((size_t)ky * nc + kx) * 2 + 1];
                        } else {
                            int my = (n - ky) % n, mx = n - kx;
                            re = sp[((size_t)my * nc + mx) * 2 + 0];
                            im = -sp[((size_t)my * nc + mx) * 2 + 1];
                        }
                        int m = (int)(((long)ky * r + (long)kx * c) % n);
                        double ang = two_pi * (double)m / (double)n;
                        /* Re[(re + i im)(cos + i sin)] */
                        acc += re * cos(ang) - im * sin(ang);
                    }
                op[(size_t)r * ow + c] = scale * acc;
            }
    }
}

/* One-dimensional transforms (Supplement 8.2, the definition itself; Section 5
 * evaluates batched 1-D transforms of sizes 2..256):
 *   X_k = sum_{j<len} x_j exp(-2 pi i k j / n),  k in [0, n/2],
 * the signal zero-padded from len to n samples, only the Hermitian half stored.
 * in: [batch][len] floats; out: [batch][n/2+1][2] doubles. O(n len) per signal. */
API void oracle_dft1d_r2c(const float *in, double *out, long batch, int len, int n) {
    const int nc = n / 2 + 1;
    const double two_pi = 6.283185307179586476925286766559;
#pragma omp parallel for schedule(static)
    for (long p = 0; p < batch; ++p) {
        const float *xp = in + (size_t)p * len;
        double *op = out + (size_t)p * nc * 2;
        for (int k = 0; k < nc; ++k) {
            double re = 0.0, im = 0.0;
            for (int j = 0; j < len; ++j) {
                int m = (int)(((long)k * j) % n);
                double ang = -two_pi * (double)m / (double)n;
                re += (double)xp[j] * cos(ang);
                im += (double)xp[j] * sin(ang);
            }
            op[2 * k + 0] = re;
            op[2 * k + 1] = im;
        }
    }
}

/* Inverse of the above: x_j = scale * Re sum_{k<n} X~_k exp(+2 pi i k j / n) for j < olen,
 * X~_k = X_k for k <= n/2, conj(X_{n-k}) above (Hermitian extension).
 * in: [batch][n/2+1][2] doubles; out: [batch][olen] doubles. */
API void oracle_idft1d_c2r(const double *in, double *out, long batch, int n, int olen,
                           double scale) {
    const int nc = n / 2 + 1;
    const double two_pi = 6.283185307179586476925286766559;
#pragma omp parallel for schedule(static)
    for (long p = 0; p < batch; ++p) {
        const double *sp = in + (size_t)p * nc * 2;
        double *op = out + (size_t)p * olen;
        for (int j = 0; j < olen; ++j) {
            double acc = 0.0;
            for (int k = 0; k < n; ++k) {
                double re, im;
                if (k < nc) { re = sp[2 * k]; im = sp[2 * k + 1]; }
                else        { re = sp[2 * (n - k)]; im = -sp[2 * (n - k) + 1]; }
                int m = (int)(((long)k * j) % n);
                double ang = two_pi * (double)m / (double)n;
                acc += re * cos(ang) - im * sin(ang);
            }
            op[j] = scale * acc;
        }
    }
}

/* Per-bin complex contraction of Table 1's Cgemm row, written as the plain
 * sum: C[b][m][n] = sum_k opA(A[b][m][k]) * opB(B[b][n][k]), conjA / conjB
 * select complex conjugation of that operand (Section 2: the conjugate makes
 * the product a cross-correlation).  All arrays interleaved (re, im) doubles. */
API void oracle_bin_contract(const double *A, const double *B, double *C, long bins,
                             int M, int N, int K, int conjA, int conjB) {
    const double sa = conjA ? -1.0 : 1.0, sb = conjB ? -1.0 : 1.0;
#pragma omp parallel for schedule(dynamic, 1)
    for (long b = 0; b < bins; ++b)
        for (int m = 0; m < M; ++m)
            for (int nn = 0; nn < N; ++nn) {
                double re = 0.0, im = 0.0;
                for (int k = 0; k < K; ++k) {
                    double ar = A[(((size_t)b * M + m) * K + k) * 2 + 0];
                    double ai = sa * A[(((size_t)b * M + m) * K + k) * 2 + 1];
                    double br = B[(((size_t)b * N + nn) * K + k) * 2 + 0];
                    double bi = sb * B[(((size_t)b * N + nn) * K + k) * 2 + 1];
                    re += ar * br - ai * bi;
                    im += ar * bi + ai * br;
                }
                C[(((size_t)b * M + m) * N + nn) * 2 + 0] = re;
                C[(((size_t)b * M + m) * N + nn) * 2 + 1] = im;
            }
}
