// Forward 2-D R2C transform of SMALL planes (filters: kh x kw <= 13 x 13 samples padded
// to n x n) straight into the frequency-major layout, as a pruned separable DFT.
//
// A filter plane has so few non-zero samples that its padded transform (Table 1, the
// "FFT B" row; Section 5.1: the zero padding is never materialised) is cheaper as a direct
// sum than as a butterfly network, and -- what matters on this machine -- the direct sum can
// be organised around the STORES instead of around the planes: a warp takes 32 planes that
// are adjacent along the minor index of the frequency-major matrix (lane = plane), every
// lane evaluates the same frequency bin of its own plane at the same time, and the warp's
// result for one (part, bin) is one contiguous 128-byte line, written from registers.  No
// staging tile, no TMA box of short rows: every store is a whole line, which is the only
// access size at which the memory system runs at its streaming rate.
//
// Per task (32 planes x a group of <= KY rows ky of the kept half ky <= n/2):
//   1. the 32 planes (contiguous in the BDHW tensor) are copied to shared memory with
//      coalesced loads; lane l then reads plane l at an odd pitch (no bank conflicts);
//   2. column sums   T[ky][v] = sum_u w[u][v] e^{-2 pi i ky u / n}        (registers)
//   3. row sums      X[ky][kx] = sum_v T[ky][v] e^{-2 pi i kx v / n}  for all kx, four
//      outputs kx0 + m n/4 at a time: the samples are grouped by v mod 4 into four partial
//      sums P_q (e^{-2 pi i (n/4) v / n} = (-i)^v), so that the four outputs cost one set of
//      kw complex multiply-adds plus additions (one radix-4 decimation-in-frequency step).
// Twiddles come from a 128-entry table in constant memory (evaluated in double at build
// time); their index is lane-uniform, so they travel through the uniform datapath.
// The kernel can be asked for a range of rows ky only, i.e. for a subset of the bins.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "fft_core.cuh"
#include "fft_kernels.cuh"
#include "fft_big.cuh"

namespace fc {

constexpr int SMALL_MAX_K = 13;       // largest plane side this kernel takes
// rows ky per task (upper bound): the column sums T[ky][v] of a task live in registers, so
// wide planes get fewer rows; narrow ones more (the staging of the planes is then shared by more bins)
constexpr int small_ky(int kw) { return kw <= 3 ? 6 : (kw <= 5 ? 4 : (kw <= 9 ? 3 : 2)); }
constexpr int SMALL_WARPS = 4;        // warps per CTA, each with its own tasks

struct TwTable128 { float2 v[128]; };
constexpr TwTable128 make_tw128() {
    TwTable128 t{};
    for (int k = 0; k < 128; ++k) {
        t.v[k].x = static_cast<float>(cx_cos2pi(k, 128));
        t.v[k].y = static_cast<float>(cx_sin2pi(k, 128));
    }
    return t;
}
// (cos, sin) of 2 pi k / 128
__constant__ TwTable128 c_tw128 = make_tw128();

struct SmallParams {
    const float* real_in;
    float* spec_out;
    int n, kh, kw;              // basis, plane rows, plane columns
    int R, C, ld;               // frequency-major matrix: rows, cols (plane = row*C + col), leading dim
    int ky_begin, ky_end;       // rows ky of the kept half [0, n/2] to produce
    int groups;                 // tasks per block of 32 planes: the ky range in `groups` nearly equal parts
    int cblocks;                // ceil(C / 32)
    long long tasks;            // R * cblocks * groups
    int pitch;                  // floats per plane in shared memory (odd)
    int concurrent;             // launched to run beside its predecessor: do not wait for it (see launch_r2c_small)
    int skip_conj;              // do not store the bins (kx > n/2, ky in {0, n/2}): the contraction leaves them out
};

template <int N, int KW>
__global__ void __launch_bounds__(SMALL_WARPS * 32)
r2c_small_kernel(const SmallParams p) {
    extern __shared__ __align__(16) float sm_small[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* sw = sm_small + (size_t)warp * 32 * p.pitch;
    constexpr int NC = N / 2 + 1, NQ = N / 4, TWS = 128 / N, MASK = N - 1, SMALL_KY = small_ky(KW);
    const int ksq = p.kh * KW;
    const size_t mat = (size_t)p.R * p.ld;              // floats per bin
    const size_t part = (size_t)N * NC * mat;           // real parts -> imaginary parts
    const int span = p.ky_end - p.ky_begin, base = span / p.groups, rem = span - base * p.groups;

    dep_trigger();
    // `concurrent`: the predecessor in the stream is the other operand's forward transform, which
    // this kernel neither reads from nor overwrites, so it does not wait for it before it starts.
    // It waits for it at its END instead (below): this grid then completes only after its
    // predecessor has, and the kernel launched after it as a programmatic dependent, which waits
    // for this grid alone, is ordered after both.
    if (!p.concurrent) dep_wait();  // no global access above this line

    const long long stride = (long long)gridDim.x * SMALL_WARPS;
    for (long long t = (long long)blockIdx.x * SMALL_WARPS + warp; t < p.tasks; t += stride) {
        const int g = (int)(t % p.groups);
        const long long pb = t / p.groups;
        const int cb = (int)(pb % p.cblocks), r = (int)(pb / p.cblocks);
        const int c0 = cb * 32, count = min(32, p.C - c0);
        const int ky0 = p.ky_begin + g * base + min(g, rem), kys = base + (g < rem ? 1 : 0);

        // 1. stage the planes: `count` planes of ksq floats, contiguous in memory
        __syncwarp();
        {
            const float* src = p.real_in + ((size_t)r * p.C + c0) * ksq;
            const int total = count * ksq;
            if (p.pitch == ksq) {
                // odd plane size: the shared-memory image is the memory image
                if ((reinterpret_cast<uintptr_t>(src) & 15) == 0) {
                    const int vec = total >> 2;
                    for (int e = lane; e < vec; e += 32)
                        reinterpret_cast<float4*>(sw)[e] = __ldg(reinterpret_cast<const float4*>(src) + e);
                    for (int e = 4 * vec + lane; e < total; e += 32) sw[e] = __ldg(src + e);
                } else {
                    for (int e = lane; e < total; e += 32) sw[e] = __ldg(src + e);
                }
            } else {
                for (int pl = 0; pl < count; ++pl)
                    for (int e = lane; e < ksq; e += 32) sw[pl * p.pitch + e] = __ldg(src + pl * ksq + e);
            }
        }
        __syncwarp();
        const float* mine = sw + (lane < count ? lane : 0) * p.pitch;

        // 2. column sums for the rows ky0 .. ky0 + kys - 1 (absent rows computed and dropped)
        float Tr[SMALL_KY][KW], Ti[SMALL_KY][KW];
#pragma unroll
        for (int j = 0; j < SMALL_KY; ++j)
#pragma unroll
            for (int v = 0; v < KW; ++v) Tr[j][v] = Ti[j][v] = 0.0f;
        for (int u = 0; u < p.kh; ++u) {
            float2 tw[SMALL_KY];
#pragma unroll
            for (int j = 0; j < SMALL_KY; ++j) tw[j] = c_tw128.v[(((ky0 + j) * u) & MASK) * TWS];
#pragma unroll
            for (int v = 0; v < KW; ++v) {
                const float wv = mine[u * KW + v];
#pragma unroll
                for (int j = 0; j < SMALL_KY; ++j) {
                    Tr[j][v] = fc_fma(wv, tw[j].x, Tr[j][v]);
                    Ti[j][v] = fc_fma(-wv, tw[j].y, Ti[j][v]);
                }
            }
        }

        // 3. row sums, four outputs per step, one 128-byte line per (part, bin) and warp; the
        //    twiddles are compile-time constants (immediate operands)
        const bool live = lane < count;
        // bin = kx * NC + ky; the four outputs of a step are NQ * NC bins apart
        const size_t step = (size_t)NC * mat, quarter = (size_t)NQ * step;
        float* o0 = p.spec_out + (size_t)ky0 * mat + (size_t)r * p.ld + c0 + lane;
#pragma unroll
        for (int j = 0; j < SMALL_KY; ++j) {
            if (j >= kys) break;
            float* o = o0 + (size_t)j * mat;
            // rows ky = 0 and ky = n/2: the bins kx > n/2 are conjugates of kept bins (GemmParams::herm_n)
            const bool herm_row = p.skip_conj && (ky0 + j == 0 || ky0 + j == N / 2);
            static_for<NQ>([&](auto KX0) {
                constexpr int kx0 = decltype(KX0)::value;
                float Pr[4] = {0.0f, 0.0f, 0.0f, 0.0f}, Pi[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                static_for<KW>([&](auto V) {
                    constexpr int v = decltype(V)::value;
                    // T[v] * e^{-i th}, th = 2 pi kx0 v / N:  (Tr c + Ti s, Ti c - Tr s)
                    constexpr int idx = (kx0 * v) & MASK;
                    constexpr float c = Tw<N, idx>::c, sn = Tw<N, idx>::s;
                    if constexpr (idx == 0) {
                        Pr[v & 3] += Tr[j][v]; Pi[v & 3] += Ti[j][v];
                    } else {
                        Pr[v & 3] = fc_fma(Tr[j][v], c, fc_fma(Ti[j][v], sn, Pr[v & 3]));
                        Pi[v & 3] = fc_fma(Ti[j][v], c, fc_fma(-Tr[j][v], sn, Pi[v & 3]));
                    }
                });
                // X[kx0 + m N/4] = sum_q (-i)^(q m) P_q
                const float ar = Pr[0] + Pr[2], ai = Pi[0] + Pi[2], br = Pr[0] - Pr[2], bi = Pi[0] - Pi[2];
                const float cr = Pr[1] + Pr[3], ci = Pi[1] + Pi[3], dr = Pr[1] - Pr[3], di = Pi[1] - Pi[3];
                if (live) {
                    float* q = o + (size_t)kx0 * step;
                    q[0] = ar + cr;                 q[part] = ai + ci;                       // m = 0
                    q[quarter] = br + di;           q[quarter + part] = bi - dr;             // m = 1: P0 - iP1 - P2 + iP3
                    if (kx0 == 0 || !herm_row) {
                        q[2 * quarter] = ar - cr;   q[2 * quarter + part] = ai - ci;         // m = 2
                    }
                    if (!herm_row) {
                        q[3 * quarter] = br - di;   q[3 * quarter + part] = bi + dr;         // m = 3: P0 + iP1 - P2 - iP3
                    }
                }
            });
        }
    }
    if (p.concurrent) dep_wait();   // see above: complete only after the predecessor has
}

// True if the small-plane kernel takes this operand: planes that fill at most a quarter of
// the basis (beyond that the butterfly kernels are as fast) and whose width has an instantiation.
static inline bool small_supported(int n, int kh, int kw) {
    if (n < 8 || n > 128 || kh < 1 || kw < 1 || kh > SMALL_MAX_K || kw > SMALL_MAX_K) return false;
    if (2 * kh > n || 2 * kw > n) return false;
    return kw <= 5 || kw == 7 || kw == 9 || kw == 11 || kw == 13;
}

template <int N, int KW>
static cudaError_t launch_r2c_small_nk(const SmallParams& p, cudaStream_t st, bool overlap) {
    if constexpr (2 * KW > N) {
        return cudaErrorNotSupported;
    } else {
        auto kern = r2c_small_kernel<N, KW>;
        const size_t smem = (size_t)SMALL_WARPS * 32 * p.pitch * sizeof(float);
        int grid = 0;
        const long long ctas = (p.tasks + SMALL_WARPS - 1) / SMALL_WARPS;
        cudaError_t e = persistent_grid(reinterpret_cast<const void*>(kern), SMALL_WARPS * 32, smem, ctas, &grid);
        if (e != cudaSuccess) return e;
        return dep_launch(overlap, kern, dim3(grid), dim3(SMALL_WARPS * 32), smem, st, p);
    }
}
template <int N>
static cudaError_t launch_r2c_small_n(const SmallParams& p, cudaStream_t st, bool overlap) {
    switch (p.kw) {
        case 1:  return launch_r2c_small_nk<N, 1>(p, st, overlap);
        case 2:  return launch_r2c_small_nk<N, 2>(p, st, overlap);
        case 3:  return launch_r2c_small_nk<N, 3>(p, st, overlap);
        case 4:  return launch_r2c_small_nk<N, 4>(p, st, overlap);
        case 5:  return launch_r2c_small_nk<N, 5>(p, st, overlap);
        case 7:  return launch_r2c_small_nk<N, 7>(p, st, overlap);
        case 9:  return launch_r2c_small_nk<N, 9>(p, st, overlap);
        case 11: return launch_r2c_small_nk<N, 11>(p, st, overlap);
        case 13: return launch_r2c_small_nk<N, 13>(p, st, overlap);
    }
    return cudaErrorNotSupported;
}

// Forward transform of one operand whose planes are small (see small_supported); produces the
// rows ky in [ky_begin, ky_end) of the kept half, all kx.
// overlap: launch as a programmatic dependent of the previous kernel.  concurrent (with overlap):
// additionally start without waiting for that kernel, so that the two run side by side (the wait
// moves to the end of this kernel, which keeps the chain of dependent launches ordered).
static cudaError_t launch_r2c_small(int n, const FftParams& f, int ky_begin, int ky_end, cudaStream_t st,
                                    bool overlap = false, bool concurrent = false, bool skip_conj = false) {
    if (!small_supported(n, f.h, f.w) || f.win) return cudaErrorNotSupported;
    if (ky_begin < 0 || ky_end > n / 2 + 1 || ky_begin >= ky_end) return cudaErrorInvalidValue;
    SmallParams p{};
    p.real_in = f.real_in; p.spec_out = f.spec_out;
    p.n = n; p.kh = f.h; p.kw = f.w;
    p.R = f.R; p.C = f.C; p.ld = f.ld;
    p.ky_begin = ky_begin; p.ky_end = ky_end;
    const int span = ky_end - ky_begin;
    p.cblocks = (f.C + 31) / 32;
    // rows ky per task: as many as SMALL_KY (the column sums are shared by them), fewer when
    // the operand has too few planes to fill the machine with tasks otherwise
    int ky_per = small_ky(f.w);
    const long long blocks = (long long)f.R * p.cblocks, want = (long long)fft_sm_count() * 24;
    while (ky_per > 1 && blocks * ((span + ky_per - 1) / ky_per) < want) --ky_per;
    p.groups = (span + ky_per - 1) / ky_per;
    p.tasks = blocks * p.groups;
    p.pitch = (f.h * f.w) | 1;
    p.concurrent = (overlap && concurrent) ? 1 : 0;
    p.skip_conj = skip_conj ? 1 : 0;
    switch (n) {
        case 8:   return launch_r2c_small_n<8>(p, st, overlap);
        case 16:  return launch_r2c_small_n<16>(p, st, overlap);
        case 32:  return launch_r2c_small_n<32>(p, st, overlap);
        case 64:  return launch_r2c_small_n<64>(p, st, overlap);
        case 128: return launch_r2c_small_n<128>(p, st, overlap);
    }
    return cudaErrorNotSupported;
}

// ---------------------------------------------------------------------------
// Inverse transform with a SMALL crop (the filter gradient of accGrad: K x K outputs of an
// n x n inverse transform, Table 1 "IFFT C" with the clipping of Section 3.1), as a pruned
// separable inverse DFT that is organised around the LOADS: a warp takes 32 planes adjacent
// along the minor index (lane = plane) and reads, for one frequency row ky, all n columns kx
// of both parts as whole 128-byte lines (one 4-D TMA box per row, double- or triple-buffered
// per warp), so the memory system only sees full lines.  With the stored half ky <= n/2 and
// the Hermitian extension,
//   out[u][v] = scale * sum_{ky <= n/2} m(ky) Re( e^{+2 pi i ky u / n} Z[ky][v] ),
//   Z[ky][v]  = sum_kx X[ky][kx] e^{+2 pi i kx v / n},    m = 1 for ky in {0, n/2}, else 2.
// Z is formed four columns kx0 + m n/4 at a time (the four inputs are first combined for the
// four classes v mod 4 with additions only, e^{2 pi i (n/4) v / n} = i^v; then K complex
// multiply-adds with compile-time twiddles), and each row's Z is folded into the K x K
// accumulators, which live in registers.  The four warps of a CTA take the rows ky = w, w + 4,
// ... of one block of 32 planes and add their accumulators in a fixed order at the end, so the
// result does not depend on timing.
// ---------------------------------------------------------------------------
struct SmallInvParams {
    float* real_out;
    int n, k;                   // basis, crop (k x k outputs per plane)
    int R, C;                   // matrix rows, cols (plane = row*C + col)
    int cblocks;                // ceil(C / 32)
    long long blocks;           // R * cblocks blocks of 32 planes
    int split;                  // warps that share a block: 4 (rows ky = w, w + 4, ..) or 1 (a warp owns a block)
    float scale;
    int accumulate;
    int* status;
    long long wait_cycles;
};

template <int N> struct SmallInvCfg { static constexpr int NST = (N >= 64) ? 2 : 3; };
constexpr int SMALLINV_WARPS = 4;

template <int N, int K>
__global__ void __launch_bounds__(SMALLINV_WARPS * 32)
c2r_small_kernel(const __grid_constant__ CUtensorMap tmS, const __grid_constant__ CUtensorMap tmH,
                 const SmallInvParams p) {
    constexpr int NC = N / 2 + 1, NQ = N / 4, TWS = 128 / N, MASK = N - 1, NST = SmallInvCfg<N>::NST;
    constexpr int ROW_FLOATS = 2 * N * 32;              // one frequency row: [part*N + kx][32 planes]
    constexpr int KSQ = K * K;
    extern __shared__ __align__(128) unsigned char fc_smem[];
    __shared__ __align__(8) unsigned long long bar_storage[SMALLINV_WARPS * NST];
    __shared__ int failed;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* ring = reinterpret_cast<float*>(fc_smem) + (size_t)warp * NST * ROW_FLOATS;
    // behind the rings: one [KSQ][33] block of accumulators per warp (summed over the warps of a
    // block when they share it, and the way to coalesced stores in either case)
    float* red = reinterpret_cast<float*>(fc_smem) + (size_t)SMALLINV_WARPS * NST * ROW_FLOATS;
    const uint32_t bars = fk_smem_u32(&bar_storage[warp * NST]);

    dep_trigger();
    if (threadIdx.x == 0) failed = 0;
    if (lane == 0) {
        for (int s = 0; s < NST; ++s) fk_mbar_init(bars + 8u * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    dep_wait();                     // no global access above this line

    // Work of this warp: the rows ky = member, member + split, ... of the blocks first, first +
    // stride, ...; the (block, row) items form one stream, so that the rows of the next block
    // are already on their way while a block is finished.
    const bool shared = p.split == SMALLINV_WARPS;
    const int split = shared ? SMALLINV_WARPS : 1, member = shared ? warp : 0;
    const long long first = shared ? (long long)blockIdx.x : (long long)blockIdx.x * SMALLINV_WARPS + warp;
    const long long stride = shared ? (long long)gridDim.x : (long long)gridDim.x * SMALLINV_WARPS;
    const int my_rows = (NC - member + split - 1) / split;
    const long long my_blocks = first < p.blocks ? (p.blocks - first + stride - 1) / stride : 0;
    const long long items = my_blocks * my_rows;
    // the issuing side runs NST items ahead of the consuming side; both walk (block, row) with
    // counters of their own (no divisions in the loop)
    long long iss_blk = first;
    int iss_row = 0, iss_stage = 0;
    auto issue = [&]() {
        if (lane == 0) {
            const int cb = (int)(iss_blk % p.cblocks), r = (int)(iss_blk / p.cblocks);
            const int ky = member + split * iss_row;
            const uint32_t dst = fk_smem_u32(ring + (size_t)iss_stage * ROW_FLOATS);
            if (ky == 0 || ky == N / 2) {
                // Hermitian rows: only the lines kx <= N/2 of either part are fetched
                fk_mbar_expect_tx(bars + 8u * iss_stage, (uint32_t)(2 * (N / 2 + 1) * 32 * 4));
                fk_tma_load_4d(dst, &tmH, cb * 32, r, ky, 0, bars + 8u * iss_stage);
                fk_tma_load_4d(dst + (uint32_t)(N * 32 * 4), &tmH, cb * 32, r, ky, N, bars + 8u * iss_stage);
            } else {
                fk_mbar_expect_tx(bars + 8u * iss_stage, (uint32_t)(ROW_FLOATS * 4));
                fk_tma_load_4d(dst, &tmS, cb * 32, r, ky, 0, bars + 8u * iss_stage);
            }
        }
        if (++iss_row == my_rows) { iss_row = 0; iss_blk += stride; }
        if (++iss_stage == NST) iss_stage = 0;
    };
    for (long long j = 0; j < NST && j < items; ++j) issue();

    uint32_t phase = 0;             // bit s: phase of this warp's stage s
    bool ok = true;
    float acc[K][K];
    long long blk = first;
    int i = 0, s = 0;
    for (long long j = 0; j < items; ++j) {
        const int ky = member + split * i;
        if (i == 0) {
#pragma unroll
            for (int u = 0; u < K; ++u)
#pragma unroll
                for (int v = 0; v < K; ++v) acc[u][v] = 0.0f;
        }
        if (ok && !fk_wait_or_report(bars + 8u * s, (phase >> s) & 1u, p.wait_cycles, p.status)) ok = false;
        phase ^= (1u << s);
        if (ok) {
            if (ky == 0 || ky == N / 2) {
                // These two rows are Hermitian in kx and their bins kx > N/2 are never read (the
                // contraction leaves them out, see GemmParams::herm_n): every lane rebuilds them
                // in its own column of the row.
                float* wr = ring + (size_t)s * ROW_FLOATS + lane;
                float* wi = wr + N * 32;
#pragma unroll
                for (int kx = N / 2 + 1; kx < N; ++kx) {
                    wr[kx * 32] = wr[(N - kx) * 32];
                    wi[kx * 32] = -wi[(N - kx) * 32];
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // before the next TMA fill of this stage
            }
            const float* xr = ring + (size_t)s * ROW_FLOATS + lane;     // [kx][32]
            const float* xi = xr + N * 32;
            float Zr[K], Zi[K];
#pragma unroll
            for (int v = 0; v < K; ++v) Zr[v] = Zi[v] = 0.0f;
            static_for<NQ>([&](auto KX0) {
                constexpr int kx0 = decltype(KX0)::value;
                const float ar = xr[kx0 * 32], ai = xi[kx0 * 32];
                const float br = xr[(kx0 + NQ) * 32], bi = xi[(kx0 + NQ) * 32];
                const float cr = xr[(kx0 + 2 * NQ) * 32], ci = xi[(kx0 + 2 * NQ) * 32];
                const float dr = xr[(kx0 + 3 * NQ) * 32], di = xi[(kx0 + 3 * NQ) * 32];
                // Y_q = sum_m i^(m q) x_m for the classes q = v mod 4
                const float pr = ar + cr, pi = ai + ci, mr = ar - cr, mi = ai - ci;
                const float sr = br + dr, si = bi + di, tr = br - dr, ti = bi - di;
                const float Yr[4] = {pr + sr, mr - ti, pr - sr, mr + ti};
                const float Yi[4] = {pi + si, mi + tr, pi - si, mi - tr};
                static_for<K>([&](auto V) {
                    constexpr int v = decltype(V)::value;
                    constexpr int idx = (kx0 * v) & MASK;
                    constexpr float c = Tw<N, idx>::c, sn = Tw<N, idx>::s;     // e^{+i th} = (c, +s)
                    if constexpr (idx == 0) {
                        Zr[v] += Yr[v & 3]; Zi[v] += Yi[v & 3];
                    } else {
                        Zr[v] = fc_fma(Yr[v & 3], c, fc_fma(-Yi[v & 3], sn, Zr[v]));
                        Zi[v] = fc_fma(Yr[v & 3], sn, fc_fma(Yi[v & 3], c, Zi[v]));
                    }
                });
            });
            const float wgt = (ky == 0 || ky == N / 2) ? 1.0f : 2.0f;
#pragma unroll
            for (int u = 0; u < K; ++u) {
                const float2 tw = c_tw128.v[((ky * u) & MASK) * TWS];   // e^{+i th} = (cos, +sin)
                const float cu = wgt * tw.x, su = wgt * tw.y;
#pragma unroll
                for (int v = 0; v < K; ++v) acc[u][v] = fc_fma(Zr[v], cu, fc_fma(-Zi[v], su, acc[u][v]));
            }
        }
        __syncwarp();                                   // the row is consumed by every lane
        if (j + NST < items) issue();
        if (++s == NST) s = 0;
        if (++i != my_rows) continue;

        // the block is complete for this warp
        i = 0;
        const int cb = (int)(blk % p.cblocks), r = (int)(blk / p.cblocks);
        blk += stride;
        const int c0 = cb * 32, count = min(32, p.C - c0);
        float* out = p.real_out + ((size_t)r * p.C + c0) * KSQ;    // the block's planes are contiguous
        {
            float* mine = red + (size_t)warp * KSQ * 33 + lane;
#pragma unroll
            for (int u = 0; u < K; ++u)
#pragma unroll
                for (int v = 0; v < K; ++v) mine[(u * K + v) * 33] = acc[u][v];
        }
        if (shared) {
            // the four warps' accumulators are added in a fixed order
            if (!ok) failed = 1;
            __syncthreads();
            if (failed) return;                         // a load never came: status raised, leave
            for (int e = threadIdx.x; e < count * KSQ; e += SMALLINV_WARPS * 32) {
                const int pl = e / KSQ, idx = e - pl * KSQ;
                float sum = 0.0f;
#pragma unroll
                for (int w = 0; w < SMALLINV_WARPS; ++w) sum += red[(size_t)w * KSQ * 33 + idx * 33 + pl];
                sum *= p.scale;
                if (p.accumulate) sum += out[e];
                out[e] = sum;
            }
            __syncthreads();                            // before the accumulators are written again
        } else {
            if (!ok) return;
            __syncwarp();
            const float* mine = red + (size_t)warp * KSQ * 33;
            for (int e = lane; e < count * KSQ; e += 32) {
                const int pl = e / KSQ, idx = e - pl * KSQ;
                float sum = mine[idx * 33 + pl] * p.scale;
                if (p.accumulate) sum += out[e];
                out[e] = sum;
            }
            __syncwarp();
        }
    }
}

// Taken at n = 32 and 64 (measured: filter gradient of the mid layer 31.7 -> 25.1 us, of the
// large-kernel layer 34.6 -> 24.3 us); at n = 16 the butterfly kernel with its 64-byte rows is
// as fast or faster (deep layer 41.4 against 45.2 us) and keeps the job.
static inline bool small_inv_supported(int n, int hc, int wc) {
    if (n < 32 || n > 64 || hc != wc || 2 * hc > n) return false;
    return hc <= 5 || hc == 7 || hc == 9 || hc == 11;
}

// box_kx: lines of one box (2 N: a whole row, both parts; N/2 + 1: the kept half of one part)
template <int N>
static bool small_inv_map(CUtensorMap* map, const float* spec, const FftParams& p, int box_kx) {
    tc_encode_fn enc = tc_get_encode();
    if (!enc) return false;
    constexpr int NC = N / 2 + 1;
    const cuuint64_t mat = (cuuint64_t)p.R * p.ld * 4;
    cuuint64_t dims[4] = {(cuuint64_t)p.C, (cuuint64_t)p.R, (cuuint64_t)NC, (cuuint64_t)2 * N};
    cuuint64_t strides[3] = {(cuuint64_t)p.ld * 4, mat, mat * NC};
    cuuint32_t box[4] = {32u, 1u, 1u, (cuuint32_t)box_kx};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(spec), dims, strides, box,
               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int N, int K>
static cudaError_t launch_c2r_small_nk(const FftParams& f, cudaStream_t st) {
    if constexpr (2 * K > N) {
        return cudaErrorNotSupported;
    } else {
        CUtensorMap tm, tmh;
        memset(&tm, 0, sizeof(tm));
        memset(&tmh, 0, sizeof(tmh));
        if (!small_inv_map<N>(&tm, f.spec_in, f, 2 * N) || !small_inv_map<N>(&tmh, f.spec_in, f, N / 2 + 1))
            return cudaErrorInvalidValue;
        SmallInvParams p{};
        p.real_out = f.real_out; p.n = N; p.k = K; p.R = f.R; p.C = f.C;
        p.cblocks = (f.C + 31) / 32;
        p.blocks = (long long)f.R * p.cblocks;
        p.scale = f.scale; p.accumulate = f.accumulate; p.status = f.status; p.wait_cycles = f.wait_cycles;
        auto kern = c2r_small_kernel<N, K>;
        const size_t smem = (size_t)SMALLINV_WARPS * SmallInvCfg<N>::NST * 2 * N * 32 * sizeof(float) +
                            (size_t)SMALLINV_WARPS * K * K * 33 * sizeof(float);
        // a warp owns a block of 32 planes where there are blocks enough to fill the machine
        // that way; otherwise the four warps of a CTA share a block
        p.split = (p.blocks >= (long long)fft_sm_count() * 4 * SMALLINV_WARPS) ? 1 : SMALLINV_WARPS;
        const long long ctas = p.split == 1 ? (p.blocks + SMALLINV_WARPS - 1) / SMALLINV_WARPS : p.blocks;
        int grid = 0;
        cudaError_t e = persistent_grid(reinterpret_cast<const void*>(kern), SMALLINV_WARPS * 32, smem, ctas, &grid);
        if (e != cudaSuccess) return e;
        return dep_launch(f.overlap != 0, kern, dim3(grid), dim3(SMALLINV_WARPS * 32), smem, st, tm, tmh, p);
    }
}
template <int N>
static cudaError_t launch_c2r_small_n(const FftParams& f, cudaStream_t st) {
    switch (f.h) {
        case 1:  return launch_c2r_small_nk<N, 1>(f, st);
        case 2:  return launch_c2r_small_nk<N, 2>(f, st);
        case 3:  return launch_c2r_small_nk<N, 3>(f, st);
        case 4:  return launch_c2r_small_nk<N, 4>(f, st);
        case 5:  return launch_c2r_small_nk<N, 5>(f, st);
        case 7:  return launch_c2r_small_nk<N, 7>(f, st);
        case 9:  return launch_c2r_small_nk<N, 9>(f, st);
        case 11: return launch_c2r_small_nk<N, 11>(f, st);
    }
    return cudaErrorNotSupported;
}
// Inverse transform of a spectrum whose crop is small and square (see small_inv_supported).
static cudaError_t launch_c2r_small(int n, const FftParams& f, cudaStream_t st) {
    if (!small_inv_supported(n, f.h, f.w) || f.win) return cudaErrorNotSupported;
    switch (n) {
        case 32: return launch_c2r_small_n<32>(f, st);
        case 64: return launch_c2r_small_n<64>(f, st);
    }
    return cudaErrorNotSupported;
}

}  // namespace fc
