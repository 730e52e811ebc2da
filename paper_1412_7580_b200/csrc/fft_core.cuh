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

// ---------------------------------------------------------------------------
// Real-input FFT of length N split over two cooperating threads.  Both threads
// see all N samples; thread Q in {0,1} returns the bins k = 2i + Q of the
// Hermitian half 0..N/2 in O[i]: Q = 0 gets k = 0, 2, .., N/2 (N/4 + 1 bins),
// Q = 1 gets k = 1, 3, .., N/2 - 1 (N/4 bins, O[N/4] untouched).
// With z_j = x_2j + i x_2j+1 (M = N/2 points) the thread takes one
// decimation-in-frequency step, a_j = z_j +- z_{j+M/2} (times w_M^j for Q = 1),
// and an M/2-point FFT, which yields Z_{2m+Q}; the Hermitian post-pass of rfft
// pairs Z_k with Z_{M-k}, and k and M-k have the same parity, so it stays inside
// the thread.
// ---------------------------------------------------------------------------
template <int N, int Q, class Load>
FC_HD void rfft_half_split(Load&& x, float (&ar)[N / 4], float (&ai)[N / 4]) {
    static_assert(N >= 8, "needs an even quarter length");
    constexpr int M = N / 2, H = M / 2;
    static_for<H>([&](auto J) {
        constexpr int j = decltype(J)::value;
        const float lr = x(std::integral_constant<int, 2 * j>{});
        const float li = x(std::integral_constant<int, 2 * j + 1>{});
        const float hr = x(std::integral_constant<int, 2 * j + M>{});
        const float hi = x(std::integral_constant<int, 2 * j + M + 1>{});
        if constexpr (Q == 0) {
            ar[j] = lr + hr; ai[j] = li + hi;
        } else {
            const float dr = lr - hr, di = li - hi;
            if constexpr (j == 0) {
                ar[j] = dr; ai[j] = di;
            } else if constexpr (4 * j == M) {
                ar[j] = di; ai[j] = -dr;
            } else {
                constexpr float c = Tw<M, j>::c, s = Tw<M, j>::s;
                ar[j] = fc_fma(s, di, c * dr);
                ai[j] = fc_fma(-s, dr, c * di);
            }
        }
    });
}
// Second half of rfft_half: the N/4-point FFT and the Hermitian post-pass; every bin is
// handed to emit(i, re, im) with i a compile-time index (bin k = 2i + Q) as soon as it exists.
template <int N, int Q, class Emit>
FC_HD void rfft_half_finish(float (&ar)[N / 4], float (&ai)[N / 4], Emit&& emit) {
    constexpr int M = N / 2, H = M / 2;
    cfft<H, false>(ar, ai);                       // ar/ai[m] = Z_{2m+Q}
    auto pair = [&](auto K) {                     // bins k and M-k from Z_k and Z_{M-k}
        constexpr int k = decltype(K)::value;
        constexpr int m = (k - Q) / 2, mp = (M - k - Q) / 2;
        constexpr float hc = 0.5f * Tw<N, k>::c;
        constexpr float hs = 0.5f * Tw<N, k>::s;
        const float pr = ar[m], pi = ai[m], qr = ar[mp], qi = ai[mp];
        const float er = pr + qr, ei = pi - qi;       // 2 E_k
        const float orr = pi + qi, oi = qr - pr;      // 2 O_k
        const float tr = fc_fma(hs, oi, hc * orr);
        const float ti = fc_fma(-hs, orr, hc * oi);
        emit(std::integral_constant<int, m>{}, fc_fma(0.5f, er, tr), fc_fma(0.5f, ei, ti));
        emit(std::integral_constant<int, mp>{}, fc_fma(0.5f, er, -tr), fc_fma(-0.5f, ei, ti));
    };
    if constexpr (Q == 0) {
        emit(std::integral_constant<int, 0>{}, ar[0] + ai[0], 0.0f);          // k = 0
        emit(std::integral_constant<int, H>{}, ar[0] - ai[0], 0.0f);          // k = M
        emit(std::integral_constant<int, H / 2>{}, ar[H / 2], -ai[H / 2]);    // k = M/2
        static_for<H / 2 - 1>([&](auto I) {            // k = 2, 4, .., M/2 - 2
            pair(std::integral_constant<int, 2 * (decltype(I)::value + 1)>{});
        });
    } else {
        static_for<H / 2>([&](auto I) {                // k = 1, 3, .., M/2 - 1
            pair(std::integral_constant<int, 2 * decltype(I)::value + 1>{});
        });
    }
}
template <int N, int Q, class Load>
FC_HD void rfft_half(Load&& x, float (&Or)[N / 4 + 1], float (&Oi)[N / 4 + 1]) {
    float ar[N / 4], ai[N / 4];
    rfft_half_split<N, Q>(static_cast<Load&&>(x), ar, ai);
    rfft_half_finish<N, Q>(ar, ai, [&](auto I, float re, float im) {
        Or[decltype(I)::value] = re;
        Oi[decltype(I)::value] = im;
    });
}

// ---------------------------------------------------------------------------
// One radix-4 decimation-in-frequency step of an N-point complex transform split
// over four cooperating threads.  All threads see the N inputs through load(j)
// (a float2); thread Q in {0..3} forms the N/4 inputs of the quarter-size
// transform whose outputs are X_{4m+Q}:
//   a_j = (x_j + u^Q x_{j+L} + u^2Q x_{j+2L} + u^3Q x_{j+3L}) w_N^{+-Qj},  L = N/4,
// with u = -i forward and +i inverse.
// ---------------------------------------------------------------------------
template <int N, bool INV, int Q, int J>
FC_HD void split4_elem(const float2 x0, const float2 x1, const float2 x2, const float2 x3, float& outr,
                       float& outi) {
    float tr, ti;
    if constexpr (Q == 0) {
        tr = (x0.x + x2.x) + (x1.x + x3.x); ti = (x0.y + x2.y) + (x1.y + x3.y);
    } else if constexpr (Q == 2) {
        tr = (x0.x + x2.x) - (x1.x + x3.x); ti = (x0.y + x2.y) - (x1.y + x3.y);
    } else {
        const float dr = x0.x - x2.x, di = x0.y - x2.y;     // x_j - x_{j+2L}
        const float er = x1.x - x3.x, ei = x1.y - x3.y;     // x_{j+L} - x_{j+3L}
        // forward Q = 1 (inverse Q = 3): d - i e;   forward Q = 3 (inverse Q = 1): d + i e
        if constexpr ((Q == 1) != INV) { tr = dr + ei; ti = di - er; }
        else                           { tr = dr - ei; ti = di + er; }
    }
    if constexpr (Q == 0 || J == 0) {
        outr = tr; outi = ti;
    } else {
        constexpr float c = Tw<N, Q * J>::c;
        constexpr float s = INV ? -Tw<N, Q * J>::s : Tw<N, Q * J>::s;
        // w = (c, -s): w t = (c tr + s ti, c ti - s tr)
        outr = fc_fma(s, ti, c * tr);
        outi = fc_fma(-s, tr, c * ti);
    }
}
template <int N, bool INV, int Q, class Load>
FC_HD void load_split4(Load&& load, float (&ar)[N / 4], float (&ai)[N / 4]) {
    constexpr int L = N / 4;
    static_for<L>([&](auto J) {
        constexpr int j = decltype(J)::value;
        const float2 x0 = load(J), x1 = load(std::integral_constant<int, j + L>{});
        const float2 x2 = load(std::integral_constant<int, j + 2 * L>{});
        const float2 x3 = load(std::integral_constant<int, j + 3 * L>{});
        split4_elem<N, INV, Q, j>(x0, x1, x2, x3, ar[j], ai[j]);
    });
}

// ---------------------------------------------------------------------------
// Inverse of the real-input FFT split over two cooperating threads (decimation
// in time).  Thread Q in {0,1} reads the bins k = Q (mod 2) of the Hermitian half
// through X(k) (a float2; X(0) must return (Re X_0, Re X_{N/2}) -- both bins are
// real), forms Z'_{2m+Q} with the pre-pass of irfft (k and M-k have the same
// parity) and runs an M/2-point inverse FFT.  Result: Q = 0 returns E_j, Q = 1
// returns w_M^{-j} O_j (j < M/2); then z_j = E_j + w^{-j} O_j and
// z_{j+M/2} = E_j - w^{-j} O_j, with x_2j = Re z_j, x_2j+1 = Im z_j (times N).
// ---------------------------------------------------------------------------
template <int N, int Q, class LoadX>
FC_HD void irfft_half(LoadX&& X, float (&er)[N / 4], float (&ei)[N / 4]) {
    static_assert(N >= 8, "needs an even quarter length");
    constexpr int M = N / 2, H = M / 2;
    auto pair = [&](auto K) {
        constexpr int k = decltype(K)::value;
        constexpr int m = (k - Q) / 2, mp = (M - k - Q) / 2;
        constexpr float c = Tw<N, k>::c, s = Tw<N, k>::s;
        const float2 P = X(K), Qv = X(std::integral_constant<int, M - k>{});
        const float sr = P.x + Qv.x, si = P.y - Qv.y;   // P + conj Q
        const float dr = P.x - Qv.x, di = P.y + Qv.y;   // P - conj Q
        const float ur = fc_fma(-s, di, c * dr);        // w_N^{-k} D
        const float ui = fc_fma(s, dr, c * di);
        er[m] = sr - ui;  ei[m] = si + ur;
        er[mp] = sr + ui; ei[mp] = ur - si;
    };
    if constexpr (Q == 0) {
        const float2 dc = X(std::integral_constant<int, 0>{});
        er[0] = dc.x + dc.y; ei[0] = dc.x - dc.y;
        const float2 mid = X(std::integral_constant<int, H>{});
        er[H / 2] = 2.0f * mid.x; ei[H / 2] = -2.0f * mid.y;
        static_for<H / 2 - 1>([&](auto I) {
            pair(std::integral_constant<int, 2 * (decltype(I)::value + 1)>{});
        });
    } else {
        static_for<H / 2>([&](auto I) {
            pair(std::integral_constant<int, 2 * decltype(I)::value + 1>{});
        });
    }
    cfft<H, true>(er, ei);
    if constexpr (Q == 1) {
        static_for<H - 1>([&](auto J) {
            constexpr int j = decltype(J)::value + 1;
            constexpr float c = Tw<M, j>::c, s = Tw<M, j>::s;
            const float a = er[j], b = ei[j];
            er[j] = fc_fma(-s, b, c * a);
            ei[j] = fc_fma(s, a, c * b);
        });
    }
}

}  // namespace fc
