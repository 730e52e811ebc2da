// Register-resident FFT building blocks (power-of-two sizes 2..64).
//
// Everything here works on small per-thread arrays whose indices are all
// compile-time constants, so the arrays live in registers, the bit-reversal
// permutation is free (register renaming) and every twiddle factor is an
// immediate taken from a table that the compiler evaluates in double precision
// at build time and rounds once to fp32.
//
// Transform convention (Supplement 8.2 of the paper): forward
// X_k = sum_j x_j exp(-2 pi i jk/N), unnormalised; the inverse uses the
// conjugate roots and is unnormalised as well (the caller applies 1/n^2).
//
// The functions are __host__ __device__ so the arithmetic can also be exercised
// by a host-side unit harness; the product only ever runs them on the GPU.
#pragma once

#include <utility>

#if defined(__CUDACC__)
#define FC_HD __host__ __device__ __forceinline__
#else
#define FC_HD inline
#endif

namespace fc {

// ---------------------------------------------------------------------------
// Compile-time twiddle table: cos / sin of 2 pi k / N evaluated in double.
// ---------------------------------------------------------------------------
constexpr double kPi = 3.141592653589793238462643383279502884;

// Taylor series on |x| <= pi/4 (terms to x^25: error far below 1e-17).
constexpr double cx_sin_small(double x) {
    double x2 = x * x, term = x, sum = x;
    for (int i = 1; i <= 12; ++i) {
        term *= -x2 / static_cast<double>((2 * i) * (2 * i + 1));
        sum += term;
    }
    return sum;
}
constexpr double cx_cos_small(double x) {
    double x2 = x * x, term = 1.0, sum = 1.0;
    for (int i = 1; i <= 12; ++i) {
        term *= -x2 / static_cast<double>((2 * i - 1) * (2 * i));
        sum += term;
    }
    return sum;
}
// cos(2 pi k / N), N a power of two >= 1; exact octant reduction on integers.
constexpr double cx_cos2pi(int k, int N) {
    k %= N;
    if (k < 0) k += N;
    if (2 * k > N) k = N - k;                       // cos is even about pi
    if (4 * k > N) return -cx_cos2pi(N / 2 - k, N);  // cos(pi - t) = -cos t   (N even)
    if (8 * k > N) return cx_sin_small(2.0 * kPi * static_cast<double>(N / 4 - k) / N);
    return cx_cos_small(2.0 * kPi * static_cast<double>(k) / N);
}
constexpr double cx_sin2pi(int k, int N) {
    k %= N;
    if (k < 0) k += N;
    if (2 * k > N) return -cx_sin2pi(N - k, N);
    if (4 * k > N) return cx_sin2pi(N / 2 - k, N);   // sin(pi - t) = sin t
    if (8 * k > N) return cx_cos_small(2.0 * kPi * static_cast<double>(N / 4 - k) / N);
    return cx_sin_small(2.0 * kPi * static_cast<double>(k) / N);
}

// One table entry: w = exp(-2 pi i K / N) has re = c, im = -s.
template <int N, int K>
struct Tw {
    static constexpr float c = static_cast<float>(cx_cos2pi(K, N));
    static constexpr float s = static_cast<float>(cx_sin2pi(K, N));
};

// ---------------------------------------------------------------------------
// Compile-time loops.
// ---------------------------------------------------------------------------
template <class F, int... Is>
FC_HD void static_for_impl(F&& f, std::integer_sequence<int, Is...>) {
    (f(std::integral_constant<int, Is>{}), ...);
}
template <int N, class F>
FC_HD void static_for(F&& f) {
    static_for_impl(static_cast<F&&>(f), std::make_integer_sequence<int, N>{});
}

constexpr int ilog2(int n) { return n <= 1 ? 0 : 1 + ilog2(n / 2); }
constexpr int bitrev(int v, int bits) {
    int r = 0;
    for (int i = 0; i < bits; ++i) r |= ((v >> i) & 1) << (bits - 1 - i);
    return r;
}

FC_HD float fc_fma(float a, float b, float c) {
#if defined(__CUDA_ARCH__)
    return __fmaf_rn(a, b, c);
#else
    return __builtin_fmaf(a, b, c);
#endif
}

// ---------------------------------------------------------------------------
// In-register complex FFT, radix-2 decimation in time.
// INV = false: forward (roots exp(-2 pi i/N)); INV = true: conjugate roots.
// Input and output in natural order; unnormalised.
// A butterfly with a non-trivial twiddle costs six FMAs:
//   u' = u + w v  (two chained FMAs per component),  v' = 2u - u' (one FMA).
// ---------------------------------------------------------------------------
template <int N, bool INV>
FC_HD void cfft(float (&re)[N], float (&im)[N]) {
    static_assert(N >= 1 && (N & (N - 1)) == 0, "power of two");
    if constexpr (N == 1) {
        return;
    } else {
        constexpr int BITS = ilog2(N);
        float br[N], bi[N];
        static_for<N>([&](auto I) {
            constexpr int i = decltype(I)::value;
            br[i] = re[bitrev(i, BITS)];
            bi[i] = im[bitrev(i, BITS)];
        });
        static_for<BITS>([&](auto ST) {
            constexpr int len = 2 << decltype(ST)::value;
            constexpr int half = len / 2;
            static_for<N / 2>([&](auto B) {
                constexpr int b = decltype(B)::value;
                constexpr int j = b % half;
                constexpr int p = (b / half) * len + j;
                constexpr int q = p + half;
                const float ur = br[p], ui = bi[p], vr = br[q], vi = bi[q];
                if constexpr (j == 0) {
                    br[p] = ur + vr; bi[p] = ui + vi;
                    br[q] = ur - vr; bi[q] = ui - vi;
                } else if constexpr (4 * j == len) {
                    // forward: w = -i, w v = (vi, -vr); inverse: w = +i, w v = (-vi, vr)
                    if constexpr (!INV) {
                        br[p] = ur + vi; bi[p] = ui - vr;
                        br[q] = ur - vi; bi[q] = ui + vr;
                    } else {
                        br[p] = ur - vi; bi[p] = ui + vr;
                        br[q] = ur + vi; bi[q] = ui - vr;
                    }
                } else {
                    constexpr float c = Tw<len, j>::c;
                    constexpr float s = INV ? -Tw<len, j>::s : Tw<len, j>::s;
                    // w = (c, -s): w v = (c vr + s vi, c vi - s vr)
                    const float nr = fc_fma(s, vi, fc_fma(c, vr, ur));
                    const float ni = fc_fma(-s, vr, fc_fma(c, vi, ui));
                    br[p] = nr; bi[p] = ni;
                    br[q] = fc_fma(2.0f, ur, -nr);
                    bi[q] = fc_fma(2.0f, ui, -ni);
                }
            });
        });
        static_for<N>([&](auto I) {
            constexpr int i = decltype(I)::value;
            re[i] = br[i];
            im[i] = bi[i];
        });
    }
}

// ---------------------------------------------------------------------------
// Real-input FFT of length N through one complex FFT of length M = N/2.
// In : x[0..N) real.   Out: X[0..M] (M+1 bins, the Hermitian half).
// z_j = x_2j + i x_2j+1, Z = FFT_M(z); with E = FFT of the even samples and O =
// FFT of the odd samples, X_k = E_k + w_N^k O_k and X_{M-k} = conj(E_k - w_N^k O_k).
// ---------------------------------------------------------------------------
template <int N>
FC_HD void rfft(const float (&x)[N], float (&Xr)[N / 2 + 1], float (&Xi)[N / 2 + 1]) {
    constexpr int M = N / 2;
    float zr[M], zi[M];
    static_for<M>([&](auto J) {
        constexpr int j = decltype(J)::value;
        zr[j] = x[2 * j];
        zi[j] = x[2 * j + 1];
    });
    cfft<M, false>(zr, zi);
    Xr[0] = zr[0] + zi[0]; Xi[0] = 0.0f;
    Xr[M] = zr[0] - zi[0]; Xi[M] = 0.0f;
    if constexpr (M >= 2) {
        Xr[M / 2] = zr[M / 2];
        Xi[M / 2] = -zi[M / 2];
    }
    if constexpr (M >= 4) {
        static_for<M / 2 - 1>([&](auto K) {
            constexpr int k = decltype(K)::value + 1;
            constexpr float hc = 0.5f * Tw<N, k>::c;
            constexpr float hs = 0.5f * Tw<N, k>::s;
            const float ar = zr[k], ai = zi[k], brr = zr[M - k], bii = zi[M - k];
            const float er = ar + brr, ei = ai - bii;     // 2 E_k
            const float orr = ai + bii, oi = brr - ar;    // 2 O_k
            // T = (w_N^k / 2) * (2 O_k), w = (c, -s)
            const float tr = fc_fma(hs, oi, hc * orr);
            const float ti = fc_fma(-hs, orr, hc * oi);
            Xr[k] = fc_fma(0.5f, er, tr);
            Xi[k] = fc_fma(0.5f, ei, ti);
            Xr[M - k] = fc_fma(0.5f, er, -tr);
            Xi[M - k] = fc_fma(-0.5f, ei, ti);
        });
    }
}

// ---------------------------------------------------------------------------
// Inverse of rfft: Hermitian half X[0..M] -> N reals, unnormalised (returns
// N * x).  Imaginary parts of X_0 and X_M are ignored.
// Z'_k = (X_k + conj X_{M-k}) + i w_N^{-k} (X_k - conj X_{M-k}); the
// unnormalised inverse FFT_M of Z' is N (x_2j + i x_2j+1).
// ---------------------------------------------------------------------------
template <int N>
FC_HD void irfft(const float (&Xr)[N / 2 + 1], const float (&Xi)[N / 2 + 1], float (&x)[N]) {
    constexpr int M = N / 2;
    float zr[M], zi[M];
    zr[0] = Xr[0] + Xr[M];
    zi[0] = Xr[0] - Xr[M];
    if constexpr (M >= 2) {
        zr[M / 2] = 2.0f * Xr[M / 2];
        zi[M / 2] = -2.0f * Xi[M / 2];
    }
    if constexpr (M >= 4) {
        static_for<M / 2 - 1>([&](auto K) {
            constexpr int k = decltype(K)::value + 1;
            constexpr float c = Tw<N, k>::c;
            constexpr float s = Tw<N, k>::s;
            const float pr = Xr[k], pi = Xi[k], qr = Xr[M - k], qi = Xi[M - k];
            const float er = pr + qr, ei = pi - qi;   // E = P + conj Q
            const float dr = pr - qr, di = pi + qi;   // D = P - conj Q
            // U = w_N^{-k} D with w^{-k} = (c, +s): U = (c dr - s di, c di + s dr)
            const float ur = fc_fma(-s, di, c * dr);
            const float ui = fc_fma(s, dr, c * di);
            // Z'_k = E + iU = (er - ui, ei + ur); Z'_{M-k} = conj(E - iU) = (er + ui, -(ei - ur))
            zr[k] = er - ui;     zi[k] = ei + ur;
            zr[M - k] = er + ui; zi[M - k] = ur - ei;
        });
    }
    cfft<M, true>(zr, zi);
    static_for<M>([&](auto J) {
        constexpr int j = decltype(J)::value;
        x[2 * j] = zr[j];
        x[2 * j + 1] = zi[j];
    });
}

// ---------------------------------------------------------------------------
// One decimation-in-frequency split of an N-point transform over two
// cooperating threads: given all N inputs, thread q in {0,1} forms the N/2
// inputs of the half-size transform whose outputs are X_{2k+q}:
//   q = 0: a_j = x_j + x_{j+N/2}        q = 1: a_j = (x_j - x_{j+N/2}) w_N^{+-j}
// ---------------------------------------------------------------------------
template <int N, bool INV, int Q>
FC_HD void dif_split(const float (&xr)[N], const float (&xi)[N], float (&ar)[N / 2],
                     float (&ai)[N / 2]) {
    constexpr int M = N / 2;
    static_for<M>([&](auto J) {
        constexpr int j = decltype(J)::value;
        if constexpr (Q == 0) {
            ar[j] = xr[j] + xr[j + M];
            ai[j] = xi[j] + xi[j + M];
        } else {
            const float dr = xr[j] - xr[j + M], di = xi[j] - xi[j + M];
            if constexpr (j == 0) {
                ar[j] = dr; ai[j] = di;
            } else if constexpr (4 * j == N) {
                if constexpr (!INV) { ar[j] = di; ai[j] = -dr; }
                else                { ar[j] = -di; ai[j] = dr; }
            } else {
                constexpr float c = Tw<N, j>::c;
                constexpr float s = INV ? -Tw<N, j>::s : Tw<N, j>::s;
                ar[j] = fc_fma(s, di, c * dr);
                ai[j] = fc_fma(-s, dr, c * di);
            }
        }
    });
}

}  // namespace fc
