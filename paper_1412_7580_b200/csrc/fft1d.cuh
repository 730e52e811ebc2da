// Batched one-dimensional R2C / C2R transforms, sizes 2 .. 256 (the range the
// paper's Section 5 evaluates), with the zero-padding fused into the load and
// crop, scale and accumulate fused into the store.
//
// A CTA of 128 threads takes a tile of consecutive signals.  The tile is copied
// between global and shared memory with fully coalesced accesses (consecutive
// threads, consecutive addresses); in shared memory every signal sits at an odd
// pitch, so that threads working on different signals hit different banks.
//   n <= 64 : one thread per signal, the whole real transform in registers.
//   n >= 128: four threads per signal.  The real transform of length n is a complex
//             transform of length n/2 on z_j = x_2j + i x_2j+1 (Supplement 8.2 notation)
//             plus a Hermitian post-pass; the complex transform is split over the four
//             threads by one radix-4 decimation-in-frequency step applied while loading,
//             each thread finishing with an n/8-point register transform; the post-pass
//             (which pairs bins k and n/2-k, held by different threads) runs on the
//             shared-memory copy.  The inverse mirrors this: pre-pass in shared memory,
//             then the split inverse complex transform.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "fft_core.cuh"

namespace fc {

constexpr int F1_THREADS = 128;

struct Fft1dParams {
    const float* real_in;   // forward: [batch][len]
    float2* spec_out;       // forward: [batch][n/2+1]
    const float2* spec_in;  // inverse: [batch][n/2+1]
    float* real_out;        // inverse: [batch][len]
    long long batch;
    int len;                // forward: samples per signal; inverse: samples kept (crop at the origin)
    float scale;            // inverse
    int accumulate;         // inverse
};

template <int N> struct F1Cfg {
    static constexpr int TPT = (N <= 64) ? 1 : 4;           // threads per signal
    static constexpr int TB = F1_THREADS / TPT;             // signals per CTA
    static constexpr int NC = N / 2 + 1;
    static constexpr int PITCH_C = NC | 1;                  // complex pitch (float2 units), odd
    static constexpr int PITCH_R = N | 1;                   // real pitch of a full-length signal, odd
    static constexpr int SMEM = TB * (PITCH_C * 8 > PITCH_R * 4 ? PITCH_C * 8 : PITCH_R * 4);
};

// Asynchronous copy of BYTES (4 or 8) from global to shared memory.
template <int BYTES>
__device__ __forceinline__ void f1_cp_async(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2;"
                 ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst))), "l"(gmem_src), "n"(BYTES)
                 : "memory");
}

// cos and sin of 2 pi k / n for a run-time k (post- and pre-pass of the split transforms)
__device__ __forceinline__ void f1_twiddle(int k, int n, float& c, float& s) {
    sincospif(2.0f * (float)k / (float)n, &s, &c);
}

template <int N>
__global__ void __launch_bounds__(F1_THREADS)
fft1d_r2c_kernel(const Fft1dParams p) {
    using C = F1Cfg<N>;
    constexpr int TB = C::TB, NC = C::NC, PC = C::PITCH_C, M = N / 2;
    extern __shared__ __align__(16) unsigned char f1_smem[];
    float* sR = reinterpret_cast<float*>(f1_smem);
    float2* sC = reinterpret_cast<float2*>(f1_smem);
    const int tid = threadIdx.x;
    const int len = p.len, pr = len | 1;
    const long long t0 = (long long)blockIdx.x * TB;
    const int cnt = (int)((p.batch - t0) < TB ? (p.batch - t0) : TB);

    // coalesced copy of the tile's samples
    {
        const float* src = p.real_in + t0 * len;
        int r = tid / len, j = tid - r * len;
        const int dr = F1_THREADS / len, dj = F1_THREADS - dr * len;
        for (int idx = tid; idx < cnt * len; idx += F1_THREADS) {
            f1_cp_async<4>(sR + r * pr + j, src + idx);     // asynchronous: the loop only issues
            r += dr; j += dj;
            if (j >= len) { j -= len; ++r; }
        }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncthreads();

    if constexpr (C::TPT == 1) {
        float Xr[NC], Xi[NC];
        {
            float v[N];
            const float* row = sR + tid * pr;
            static_for<N>([&](auto J) {
                constexpr int j = decltype(J)::value;
                v[j] = (tid < cnt && j < len) ? row[j] : 0.0f;
            });
            rfft<N>(v, Xr, Xi);
        }
        __syncthreads();                    // every sample read: the buffer becomes the spectrum tile
        float2* orow = sC + tid * PC;
        static_for<NC>([&](auto K) {
            constexpr int k = decltype(K)::value;
            orow[k] = make_float2(Xr[k], Xi[k]);
        });
    } else {
        // quarter Q of the complex transform of length M: warp-uniform Q, lane = signal
        constexpr int L = M / 4;
        const int Q = tid / TB, t = tid - Q * TB;
        float ar[L], ai[L];
        {
            const float* row = sR + t * pr;
            auto load = [&](auto J) -> float2 {
                constexpr int j = decltype(J)::value;
                float2 z;
                z.x = (t < cnt && 2 * j < len) ? row[2 * j] : 0.0f;
                z.y = (t < cnt && 2 * j + 1 < len) ? row[2 * j + 1] : 0.0f;
                return z;
            };
            if (Q == 0) load_split4<M, false, 0>(load, ar, ai);
            else if (Q == 1) load_split4<M, false, 1>(load, ar, ai);
            else if (Q == 2) load_split4<M, false, 2>(load, ar, ai);
            else load_split4<M, false, 3>(load, ar, ai);
        }
        cfft<L, false>(ar, ai);             // ar/ai[m] = Z_{4m+Q}
        __syncthreads();
        {
            float2* zrow = sC + t * PC + Q;
            static_for<L>([&](auto Mm) {
                constexpr int m = decltype(Mm)::value;
                zrow[4 * m] = make_float2(ar[m], ai[m]);
            });
        }
        __syncthreads();
        // Hermitian post-pass on the shared copy: X_k = E_k + w_N^k O_k, X_{M-k} = conj(E_k - w_N^k O_k)
        // with 2 E_k = Z_k + conj Z_{M-k}, 2 O_k = -i (Z_k - conj Z_{M-k}); one (signal, k) pair per step
        for (int it = tid; it < TB * (M / 2 + 1); it += F1_THREADS) {
            const int tt = it % TB, k = it / TB;
            float2* z = sC + tt * PC;
            if (k == 0) {
                const float2 a = z[0];
                z[0] = make_float2(a.x + a.y, 0.0f);
                z[M] = make_float2(a.x - a.y, 0.0f);
            } else if (2 * k == M) {
                const float2 a = z[k];
                z[k] = make_float2(a.x, -a.y);
            } else {
                float c, s;
                f1_twiddle(k, N, c, s);
                const float2 a = z[k], b = z[M - k];
                const float er = a.x + b.x, ei = a.y - b.y;
                const float orr = a.y + b.y, oi = b.x - a.x;
                const float tr = 0.5f * (s * oi + c * orr), ti = 0.5f * (c * oi - s * orr);
                z[k] = make_float2(0.5f * er + tr, 0.5f * ei + ti);
                z[M - k] = make_float2(0.5f * er - tr, ti - 0.5f * ei);
            }
        }
    }
    __syncthreads();

    // coalesced copy of the tile's spectra
    float2* dst = p.spec_out + t0 * NC;
    for (int idx = tid; idx < cnt * NC; idx += F1_THREADS) {
        const int r = idx / NC, k = idx - r * NC;
        dst[idx] = sC[r * PC + k];
    }
}

template <int N>
__global__ void __launch_bounds__(F1_THREADS)
fft1d_c2r_kernel(const Fft1dParams p) {
    using C = F1Cfg<N>;
    constexpr int TB = C::TB, NC = C::NC, PC = C::PITCH_C, PR = C::PITCH_R, M = N / 2;
    extern __shared__ __align__(16) unsigned char f1_smem[];
    float* sR = reinterpret_cast<float*>(f1_smem);
    float2* sC = reinterpret_cast<float2*>(f1_smem);
    const int tid = threadIdx.x;
    const int len = p.len;
    const long long t0 = (long long)blockIdx.x * TB;
    const int cnt = (int)((p.batch - t0) < TB ? (p.batch - t0) : TB);

    {
        const float2* src = p.spec_in + t0 * NC;
        for (int idx = tid; idx < cnt * NC; idx += F1_THREADS) {
            const int r = idx / NC, k = idx - r * NC;
            f1_cp_async<8>(sC + r * PC + k, src + idx);
        }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncthreads();

    if constexpr (C::TPT == 1) {
        float v[N];
        {
            float Xr[NC], Xi[NC];
            const float2* row = sC + tid * PC;
            static_for<NC>([&](auto K) {
                constexpr int k = decltype(K)::value;
                const float2 t = (tid < cnt) ? row[k] : make_float2(0.0f, 0.0f);
                Xr[k] = t.x; Xi[k] = t.y;
            });
            irfft<N>(Xr, Xi, v);
        }
        __syncthreads();
        float* orow = sR + tid * PR;
        static_for<N>([&](auto J) {
            constexpr int j = decltype(J)::value;
            orow[j] = v[j];
        });
    } else {
        // pre-pass on the shared copy: Z'_k = (X_k + conj X_{M-k}) + i w_N^{-k} (X_k - conj X_{M-k})
        for (int it = tid; it < TB * (M / 2 + 1); it += F1_THREADS) {
            const int tt = it % TB, k = it / TB;
            float2* z = sC + tt * PC;
            if (k == 0) {
                const float x0 = z[0].x, xm = z[M].x;
                z[0] = make_float2(x0 + xm, x0 - xm);
            } else if (2 * k == M) {
                const float2 a = z[k];
                z[k] = make_float2(2.0f * a.x, -2.0f * a.y);
            } else {
                float c, s;
                f1_twiddle(k, N, c, s);
                const float2 a = z[k], b = z[M - k];
                const float er = a.x + b.x, ei = a.y - b.y;
                const float dr = a.x - b.x, di = a.y + b.y;
                const float ur = c * dr - s * di, ui = s * dr + c * di;
                z[k] = make_float2(er - ui, ei + ur);
                z[M - k] = make_float2(er + ui, ur - ei);
            }
        }
        __syncthreads();
        constexpr int L = M / 4;
        const int Q = tid / TB, t = tid - Q * TB;
        float ar[L], ai[L];
        {
            const float2* row = sC + t * PC;
            auto load = [&](auto J) -> float2 { return row[decltype(J)::value]; };
            if (Q == 0) load_split4<M, true, 0>(load, ar, ai);
            else if (Q == 1) load_split4<M, true, 1>(load, ar, ai);
            else if (Q == 2) load_split4<M, true, 2>(load, ar, ai);
            else load_split4<M, true, 3>(load, ar, ai);
        }
        cfft<L, true>(ar, ai);              // ar/ai[m] = z_{4m+Q} = x_{2(4m+Q)} + i x_{2(4m+Q)+1}, times N
        __syncthreads();
        float* orow = sR + t * PR + 2 * Q;
        static_for<L>([&](auto Mm) {
            constexpr int m = decltype(Mm)::value;
            orow[8 * m] = ar[m];
            orow[8 * m + 1] = ai[m];
        });
    }
    __syncthreads();

    // coalesced, cropped, scaled store
    float* dst = p.real_out + t0 * len;
    const float scale = p.scale;
    const bool acc = p.accumulate != 0;
    int r = tid / len, j = tid - r * len;
    const int dr = F1_THREADS / len, dj = F1_THREADS - dr * len;
    for (int idx = tid; idx < cnt * len; idx += F1_THREADS) {
        float o = sR[r * PR + j] * scale;
        if (acc) o += dst[idx];
        dst[idx] = o;
        r += dr; j += dj;
        if (j >= len) { j -= len; ++r; }
    }
}

template <int N>
static cudaError_t launch_fft1d_n(const Fft1dParams& p, bool inverse, cudaStream_t st) {
    using C = F1Cfg<N>;
    const long long ctas = (p.batch + C::TB - 1) / C::TB;
    if (ctas < 1 || ctas > 0x7fffffffLL) return cudaErrorInvalidValue;
    if (inverse) fft1d_c2r_kernel<N><<<(unsigned)ctas, F1_THREADS, C::SMEM, st>>>(p);
    else fft1d_r2c_kernel<N><<<(unsigned)ctas, F1_THREADS, C::SMEM, st>>>(p);
    return cudaGetLastError();
}

static cudaError_t launch_fft1d(int n, const Fft1dParams& p, bool inverse, cudaStream_t st) {
    switch (n) {
        case 2:   return launch_fft1d_n<2>(p, inverse, st);
        case 4:   return launch_fft1d_n<4>(p, inverse, st);
        case 8:   return launch_fft1d_n<8>(p, inverse, st);
        case 16:  return launch_fft1d_n<16>(p, inverse, st);
        case 32:  return launch_fft1d_n<32>(p, inverse, st);
        case 64:  return launch_fft1d_n<64>(p, inverse, st);
        case 128: return launch_fft1d_n<128>(p, inverse, st);
        case 256: return launch_fft1d_n<256>(p, inverse, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace fc
