// Batched 2-D R2C / C2R FFT kernels with fused zero-padding, fused
// frequency-major transpose, crop, scale and accumulate.
//
// One CTA transforms a tile of G planes that are adjacent along the *minor*
// index of the frequency-major matrix they are written to (read from), so that
// every frequency bin receives G consecutive floats: the transposition
// BDHW -> HWBD of the paper's Table 1 happens in the store (load) itself and no
// separate transpose pass or padded tensor exists (Section 5.1: zero-copy
// padding by clipped loads; Section 5.1: transposed output removes a pass).
//
// Structure of the forward kernel (the inverse mirrors it):
//   1. coalesced copy of the G real planes into shared memory;
//   2. one thread per non-zero row: real FFT of length N in registers
//      (a complex FFT of length N/2 plus a Hermitian post-pass), half spectrum
//      (N/2+1 bins) written back to shared memory;
//   3. N/2 column transforms per plane -- columns 0 and N/2 are real and ride
//      together as one complex column (the paper's "n x n/2 with border case",
//      Section 5.2) -- each split over two threads by one
//      decimation-in-frequency step applied while loading, then an N/2-point
//      register FFT; results go straight from registers to global memory,
//      lanes running over the G planes.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "fft_core.cuh"

namespace fc {

enum { LAYOUT_FREQ_MAJOR = 0, LAYOUT_BARE = 1 };

struct FftParams {
    const float* real_in;   // forward: real planes in
    float* real_out;        // inverse: real planes out
    const float* spec_in;   // inverse: spectra in
    float* spec_out;        // forward: spectra out
    int h, w;               // forward: plane size; inverse: crop window (hc, wc)
    int R, C;               // frequency-major matrix: rows, cols (planes = R*C)
    int ld;                 // its leading dimension in floats
    long long in_rs, in_cs; // forward: input plane index = row*in_rs + col*in_cs
    int conj;               // forward: negate imaginary parts on store
    int tiles_per_row;      // ceil(C / G)
    int pitch;              // shared-memory plane pitch in complex elements
    float scale;            // inverse
    int accumulate;         // inverse
};

// Shared-memory pitch of one plane's half spectrum (rows x (N/2+1) complex)
// such that lanes running over g (and then over adjacent columns) hit distinct
// 8-byte banks: pitch = (16 / min(G,16)) * odd.
static inline int smem_plane_pitch(int rows, int N, int G) {
    int need = rows * (N / 2 + 1);
    int unit = 16 / (G < 16 ? G : 16);
    int m = (need + unit - 1) / unit;
    if ((m & 1) == 0) ++m;
    return m * unit;
}

static inline size_t r2c_smem_bytes(int N, int G, int h, int w) {
    size_t a = (size_t)G * h * (w | 1) * sizeof(float);
    size_t b = (size_t)G * smem_plane_pitch(h, N, G) * sizeof(float2);
    return a > b ? a : b;
}
static inline size_t c2r_smem_bytes(int N, int G, int hc, int wc) {
    return r2c_smem_bytes(N, G, hc, wc);
}

// Copy `count` planes of rows x cols floats between a contiguous global range
// (plane stride rows*cols) and shared memory with row pitch colsp.
// TO_SMEM: global -> shared; otherwise shared -> global (optionally adding).
template <int T, bool TO_SMEM>
__device__ __forceinline__ void copy_planes(float* smem, const float* gsrc, float* gdst,
                                            int count, long long plane_stride, int rows,
                                            int cols, int colsp, float scale, int accumulate) {
    const int hw = rows * cols;
    const int tid = threadIdx.x;
    if (colsp == cols && plane_stride == hw) {
        const int total = count * hw;
        const uintptr_t addr = TO_SMEM ? (uintptr_t)gsrc : (uintptr_t)gdst;
        if ((addr & 15) == 0) {
            const int total4 = total >> 2;
            if constexpr (TO_SMEM) {
                const float4* s4 = reinterpret_cast<const float4*>(gsrc);
                float4* d4 = reinterpret_cast<float4*>(smem);
                for (int i = tid; i < total4; i += T) d4[i] = __ldg(s4 + i);
                for (int i = (total4 << 2) + tid; i < total; i += T) smem[i] = __ldg(gsrc + i);
            } else {
                const float4* s4 = reinterpret_cast<const float4*>(smem);
                float4* d4 = reinterpret_cast<float4*>(gdst);
                for (int i = tid; i < total4; i += T) {
                    float4 v = s4[i];
                    v.x *= scale; v.y *= scale; v.z *= scale; v.w *= scale;
                    if (accumulate) {
                        float4 o = d4[i];
                        v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                    }
                    d4[i] = v;
                }
                for (int i = (total4 << 2) + tid; i < total; i += T) {
                    float v = smem[i] * scale;
                    if (accumulate) v += gdst[i];
                    gdst[i] = v;
                }
            }
        } else {
            for (int i = tid; i < total; i += T) {
                if constexpr (TO_SMEM) {
                    smem[i] = __ldg(gsrc + i);
                } else {
                    float v = smem[i] * scale;
                    if (accumulate) v += gdst[i];
                    gdst[i] = v;
                }
            }
        }
        return;
    }
    // general case: walk (g, r, c) incrementally, T elements per step
    int g = tid / hw;
    int rem = tid - g * hw;
    int r = rem / cols;
    int c = rem - r * cols;
    const int dg = T / hw;
    const int drem = T - dg * hw;
    const int dr = drem / cols;
    const int dc = drem - dr * cols;
    while (g < count) {
        const long long gi = (long long)g * plane_stride + r * cols + c;
        const int si = (g * rows + r) * colsp + c;
        if constexpr (TO_SMEM) {
            smem[si] = __ldg(gsrc + gi);
        } else {
            float v = smem[si] * scale;
            if (accumulate) v += gdst[gi];
            gdst[gi] = v;
        }
        c += dc; r += dr;
        if (c >= cols) { c -= cols; ++r; }
        g += dg;
        if (r >= rows) { r -= rows; ++g; }
    }
}

// ---------------------------------------------------------------------------
// Forward: real planes -> half spectra.
// ---------------------------------------------------------------------------
template <int N, int G, int LAYOUT>
__global__ void __launch_bounds__(N* G) r2c_kernel(const FftParams p) {
    constexpr int T = N * G, NC = N / 2 + 1, M = N / 2, HALF = T / 2;
    static_assert(HALF % 32 == 0, "the two halves of a column transform must be warp-uniform");
    extern __shared__ __align__(16) unsigned char fc_smem[];
    float* sIn = reinterpret_cast<float*>(fc_smem);
    float2* sMid = reinterpret_cast<float2*>(fc_smem);

    const int tid = threadIdx.x;
    const int row = blockIdx.x / p.tiles_per_row;
    const int c0 = (blockIdx.x - row * p.tiles_per_row) * G;
    const int gcount = min(G, p.C - c0);
    const int h = p.h, w = p.w, wp = w | 1, P = p.pitch;

    // 1. stage the tile's planes (only the h x w non-zero part exists anywhere)
    {
        const long long first = (long long)row * p.in_rs + (long long)c0 * p.in_cs;
        copy_planes<T, true>(sIn, p.real_in + first * h * w, nullptr, gcount,
                             p.in_cs * h * w, h, w, wp, 1.0f, 0);
    }
    __syncthreads();

    // 2. row transforms: thread = (plane g, row r), r < h
    {
        const int g = tid / h, r = tid - g * h;
        const bool act = (tid < G * h) && (g < gcount);
        float Xr[NC], Xi[NC];
        if (act) {
            float v[N];
            const float* src = sIn + (g * h + r) * wp;
            static_for<N>([&](auto Cc) {
                constexpr int c = decltype(Cc)::value;
                v[c] = (c < w) ? src[c] : 0.0f;
            });
            rfft<N>(v, Xr, Xi);
        }
        __syncthreads();   // every row is in registers: the staging area may be overwritten
        if (act) {
            float2* dst = sMid + g * P + r * NC;
            static_for<NC>([&](auto Kk) {
                constexpr int k = decltype(Kk)::value;
                dst[k] = make_float2(Xr[k], Xi[k]);
            });
        }
    }
    __syncthreads();

    // 3. column transforms: thread = (half q, column kxp, plane g)
    const int q = tid / HALF;
    const int u = tid - q * HALF;
    const int kxp = u / G;
    const int g = u - kxp * G;
    if (g >= gcount) return;

    float ar[M], ai[M];
    {
        const float2* col = sMid + g * P + kxp;
        const bool packed = (kxp == 0);
        auto load = [&](int r) -> float2 {
            if (r >= h) return make_float2(0.0f, 0.0f);
            float2 v = col[r * NC];
            if (packed) v.y = col[r * NC + M].x;   // Nyquist column rides as the imaginary part
            return v;
        };
        auto split = [&](auto Q) {
            constexpr int qq = decltype(Q)::value;
            static_for<M>([&](auto J) {
                constexpr int j = decltype(J)::value;
                const float2 lo = load(j), hi = load(j + M);
                if constexpr (qq == 0) {
                    ar[j] = lo.x + hi.x;
                    ai[j] = lo.y + hi.y;
                } else {
                    const float dr = lo.x - hi.x, di = lo.y - hi.y;
                    if constexpr (j == 0) {
                        ar[j] = dr; ai[j] = di;
                    } else if constexpr (4 * j == N) {
                        ar[j] = di; ai[j] = -dr;
                    } else {
                        constexpr float c = Tw<N, j>::c;
                        constexpr float s = Tw<N, j>::s;
                        ar[j] = fc_fma(s, di, c * dr);
                        ai[j] = fc_fma(-s, dr, c * di);
                    }
                }
            });
        };
        if (q == 0) split(std::integral_constant<int, 0>{});
        else        split(std::integral_constant<int, 1>{});
    }
    cfft<M, false>(ar, ai);   // ar/ai[k] = F[2k+q]

    const float sgn = p.conj ? -1.0f : 1.0f;
    if constexpr (LAYOUT == LAYOUT_FREQ_MAJOR) {
        const size_t plane = (size_t)p.R * p.ld;               // one re or im matrix
        float* base = p.spec_out + (size_t)row * p.ld + c0 + g;
        if (kxp != 0) {
            static_for<M>([&](auto Kk) {
                constexpr int k = decltype(Kk)::value;
                const int ky = 2 * k + q;
                float* o = base + (size_t)(ky * NC + kxp) * 2 * plane;
                o[0] = ar[k];
                o[plane] = sgn * ai[k];
            });
        } else {
            auto untangle = [&](auto Q) {
                constexpr int qq = decltype(Q)::value;
                static_for<M>([&](auto Kk) {
                    constexpr int k = decltype(Kk)::value;
                    constexpr int kp = (qq == 0) ? ((M - k) % M) : (M - 1 - k);
                    constexpr int ky = 2 * k + qq;
                    const float fr = ar[k], fi = ai[k], gr = ar[kp], gi = ai[kp];
                    float* o0 = base + (size_t)(ky * NC) * 2 * plane;
                    float* oN = base + (size_t)(ky * NC + M) * 2 * plane;
                    o0[0] = 0.5f * (fr + gr);
                    o0[plane] = sgn * 0.5f * (fi - gi);
                    oN[0] = 0.5f * (fi + gi);
                    oN[plane] = sgn * 0.5f * (gr - fr);
                });
            };
            if (q == 0) untangle(std::integral_constant<int, 0>{});
            else        untangle(std::integral_constant<int, 1>{});
        }
    } else {
        float2* base = reinterpret_cast<float2*>(p.spec_out) +
                       ((size_t)row * p.C + c0 + g) * (size_t)(N * NC);
        if (kxp != 0) {
            static_for<M>([&](auto Kk) {
                constexpr int k = decltype(Kk)::value;
                const int ky = 2 * k + q;
                base[ky * NC + kxp] = make_float2(ar[k], sgn * ai[k]);
            });
        } else {
            auto untangle = [&](auto Q) {
                constexpr int qq = decltype(Q)::value;
                static_for<M>([&](auto Kk) {
                    constexpr int k = decltype(Kk)::value;
                    constexpr int kp = (qq == 0) ? ((M - k) % M) : (M - 1 - k);
                    constexpr int ky = 2 * k + qq;
                    const float fr = ar[k], fi = ai[k], gr = ar[kp], gi = ai[kp];
                    base[ky * NC] = make_float2(0.5f * (fr + gr), sgn * 0.5f * (fi - gi));
                    base[ky * NC + M] = make_float2(0.5f * (fi + gi), sgn * 0.5f * (gr - fr));
                });
            };
            if (q == 0) untangle(std::integral_constant<int, 0>{});
            else        untangle(std::integral_constant<int, 1>{});
        }
    }
}

// ---------------------------------------------------------------------------
// Inverse: half spectra -> cropped, scaled real planes.
// ---------------------------------------------------------------------------
template <int N, int G, int LAYOUT>
__global__ void __launch_bounds__(N* G) c2r_kernel(const FftParams p) {
    constexpr int T = N * G, NC = N / 2 + 1, M = N / 2, HALF = T / 2;
    extern __shared__ __align__(16) unsigned char fc_smem[];
    float* sOut = reinterpret_cast<float*>(fc_smem);
    float2* sMid = reinterpret_cast<float2*>(fc_smem);

    const int tid = threadIdx.x;
    const int row = blockIdx.x / p.tiles_per_row;
    const int c0 = (blockIdx.x - row * p.tiles_per_row) * G;
    const int gcount = min(G, p.C - c0);
    const int hc = p.h, wc = p.w, wcp = wc | 1, P = p.pitch;

    // 1. column transforms straight from global memory
    {
        const int q = tid / HALF;
        const int u = tid - q * HALF;
        const int kxp = u / G;
        const int g = u - kxp * G;
        if (g < gcount) {
            const bool packed = (kxp == 0);
            const size_t plane = (size_t)p.R * p.ld;
            const float* fbase = p.spec_in + (size_t)row * p.ld + c0 + g;
            const float2* bbase = reinterpret_cast<const float2*>(p.spec_in) +
                                  ((size_t)row * p.C + c0 + g) * (size_t)(N * NC);
            auto load = [&](int ky) -> float2 {
                float2 v;
                if constexpr (LAYOUT == LAYOUT_FREQ_MAJOR) {
                    const float* a = fbase + (size_t)(ky * NC + kxp) * 2 * plane;
                    v = make_float2(__ldg(a), __ldg(a + plane));
                    if (packed) {
                        const float* b = fbase + (size_t)(ky * NC + M) * 2 * plane;
                        v.x -= __ldg(b + plane);
                        v.y += __ldg(b);
                    }
                } else {
                    v = __ldg(bbase + ky * NC + kxp);
                    if (packed) {
                        const float2 nq = __ldg(bbase + ky * NC + M);
                        v.x -= nq.y;
                        v.y += nq.x;
                    }
                }
                return v;
            };
            float ar[M], ai[M];
            auto split = [&](auto Q) {
                constexpr int qq = decltype(Q)::value;
                static_for<M>([&](auto J) {
                    constexpr int j = decltype(J)::value;
                    const float2 lo = load(j), hi = load(j + M);
                    if constexpr (qq == 0) {
                        ar[j] = lo.x + hi.x;
                        ai[j] = lo.y + hi.y;
                    } else {
                        const float dr = lo.x - hi.x, di = lo.y - hi.y;
                        if constexpr (j == 0) {
                            ar[j] = dr; ai[j] = di;
                        } else if constexpr (4 * j == N) {
                            ar[j] = -di; ai[j] = dr;
                        } else {
                            constexpr float c = Tw<N, j>::c;
                            constexpr float s = -Tw<N, j>::s;
                            ar[j] = fc_fma(s, di, c * dr);
                            ai[j] = fc_fma(-s, dr, c * di);
                        }
                    }
                });
            };
            if (q == 0) split(std::integral_constant<int, 0>{});
            else        split(std::integral_constant<int, 1>{});
            cfft<M, true>(ar, ai);   // ar/ai[m] = column value at row r = 2m+q
            float2* dst = sMid + g * P + kxp;
            static_for<M>([&](auto Mm) {
                constexpr int m = decltype(Mm)::value;
                const int r = 2 * m + q;
                if (r < hc) {
                    if (!packed) {
                        dst[r * NC] = make_float2(ar[m], ai[m]);
                    } else {
                        dst[r * NC] = make_float2(ar[m], 0.0f);
                        dst[r * NC + M] = make_float2(ai[m], 0.0f);
                    }
                }
            });
        }
    }
    __syncthreads();

    // 2. row transforms: thread = (plane g, row r), r < hc
    {
        const int g = tid / hc, r = tid - g * hc;
        const bool act = (tid < G * hc) && (g < gcount);
        float v[N];
        if (act) {
            float Xr[NC], Xi[NC];
            const float2* src = sMid + g * P + r * NC;
            static_for<NC>([&](auto Kk) {
                constexpr int k = decltype(Kk)::value;
                const float2 t = src[k];
                Xr[k] = t.x; Xi[k] = t.y;
            });
            irfft<N>(Xr, Xi, v);
        }
        __syncthreads();   // all spectra consumed: reuse the buffer for the real output
        if (act) {
            float* dst = sOut + (g * hc + r) * wcp;
            static_for<N>([&](auto Cc) {
                constexpr int c = decltype(Cc)::value;
                if (c < wc) dst[c] = v[c];
            });
        }
    }
    __syncthreads();

    // 3. coalesced copy-out with scale / accumulate; output planes are contiguous
    {
        const long long first = (long long)row * p.C + c0;
        copy_planes<T, false>(sOut, nullptr, p.real_out + first * hc * wc, gcount,
                              (long long)hc * wc, hc, wc, wcp, p.scale, p.accumulate);
    }
}

// ---------------------------------------------------------------------------
// Host-side launchers.
// ---------------------------------------------------------------------------
template <int N>
struct TileOf;   // planes per CTA for each transform size
template <> struct TileOf<8>   { static constexpr int G = 32; };
template <> struct TileOf<16>  { static constexpr int G = 32; };
template <> struct TileOf<32>  { static constexpr int G = 16; };
template <> struct TileOf<64>  { static constexpr int G = 8; };
template <> struct TileOf<128> { static constexpr int G = 2; };

template <int N, int LAYOUT>
static cudaError_t launch_r2c_n(FftParams p, cudaStream_t st) {
    constexpr int G = TileOf<N>::G;
    p.tiles_per_row = (p.C + G - 1) / G;
    p.pitch = smem_plane_pitch(p.h, N, G);
    const size_t smem = r2c_smem_bytes(N, G, p.h, p.w);
    auto kern = r2c_kernel<N, G, LAYOUT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const long long blocks = (long long)p.R * p.tiles_per_row;
    if (blocks <= 0 || blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    kern<<<(unsigned)blocks, N * G, smem, st>>>(p);
    return cudaGetLastError();
}

template <int N, int LAYOUT>
static cudaError_t launch_c2r_n(FftParams p, cudaStream_t st) {
    constexpr int G = TileOf<N>::G;
    p.tiles_per_row = (p.C + G - 1) / G;
    p.pitch = smem_plane_pitch(p.h, N, G);
    const size_t smem = c2r_smem_bytes(N, G, p.h, p.w);
    auto kern = c2r_kernel<N, G, LAYOUT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const long long blocks = (long long)p.R * p.tiles_per_row;
    if (blocks <= 0 || blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    kern<<<(unsigned)blocks, N * G, smem, st>>>(p);
    return cudaGetLastError();
}

template <int LAYOUT>
static cudaError_t launch_r2c(int n, const FftParams& p, cudaStream_t st) {
    switch (n) {
        case 8:   return launch_r2c_n<8, LAYOUT>(p, st);
        case 16:  return launch_r2c_n<16, LAYOUT>(p, st);
        case 32:  return launch_r2c_n<32, LAYOUT>(p, st);
        case 64:  return launch_r2c_n<64, LAYOUT>(p, st);
        case 128: return launch_r2c_n<128, LAYOUT>(p, st);
    }
    return cudaErrorInvalidValue;
}
template <int LAYOUT>
static cudaError_t launch_c2r(int n, const FftParams& p, cudaStream_t st) {
    switch (n) {
        case 8:   return launch_c2r_n<8, LAYOUT>(p, st);
        case 16:  return launch_c2r_n<16, LAYOUT>(p, st);
        case 32:  return launch_c2r_n<32, LAYOUT>(p, st);
        case 64:  return launch_c2r_n<64, LAYOUT>(p, st);
        case 128: return launch_c2r_n<128, LAYOUT>(p, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace fc
