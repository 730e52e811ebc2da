// Per-frequency-bin complex contraction with FP32 FFMA (Table 1, the Cgemm row).
//
// For every bin b:  C[b][m][n] = sum_k op(A)[b][m][k] * op(B)[b][n][k]  (complex;
// op = identity or complex conjugate).
// Operands are planar: all real matrices of the bins first, then all imaginary
// ones.  A is [2][bins][M][lda] (k contiguous) or, with transA, [2][bins][K][lda]
// (m contiguous); B likewise [2][bins][N][ldb] or, with transB, [2][bins][K][ldb];
// C is [2][bins][M][ldc].
//
// CTA tile 64 x 64 of one bin, 256 threads, each thread a 4 x 4 block of complex
// outputs (64 FFMAs per k against four 16-byte shared loads); k-blocks of 16 arrive by
// asynchronous copies, double-buffered.  This is the exact
// fp32 path and the fallback for shapes too small for the tensor-core kernel.
#pragma once

#include <cuda_runtime.h>

#include "dep_launch.cuh"

namespace fc {

struct GemmParams {
    const float* A;
    const float* B;
    float* C;
    int bins, M, N, K;
    int lda, ldb, ldc;
    int transA, transB;   // operand stored [K][rows] instead of [rows][K]
    int conjA, conjB;     // use the complex conjugate of the operand
    int overlap;          // host only: launch as a programmatic dependent of the previous kernel
    long long wait_cycles; // host only: limit of a bounded wait in the tensor-core kernel (<= 0: default)
    // Tensor-core kernel only: contract a subset of the bins.  Bins are numbered kx * nc + ky;
    // with ky_count > 0 only the rows ky in [ky_begin, ky_begin + ky_count) of every kx are
    // contracted (bins / nc values of kx).  ky_count == 0: all bins.
    int nc, ky_begin, ky_count;
    // Tensor-core kernel only, host only: the next launch in the stream is a transform that is to
    // run beside this contraction; the kernel then keeps 64 KB of shared memory free (two pipeline
    // stages instead of three) and releases its dependent only after its own wait.
    int shared_sms;
    // Both kernels: herm_n = n > 0 leaves out the bins (kx > n/2, ky in {0, n/2}) of an n x (n/2+1)
    // half spectrum.  They are the complex conjugates of the bins (n - kx, ky) (Section 5.2: the
    // rows ky = 0 and ky = n/2 of a real signal's spectrum are Hermitian in kx), the inverse
    // transforms rebuild them from those, and the contraction neither reads nor writes them:
    // n - 2 bins of n (n/2 + 1), 9.7 % at n = 16, 5.5 % at n = 32, 2.9 % at n = 64.
    int herm_n;
};

// Bins kept by herm_n = n, and the bin of the spectra behind the b-th kept bin (kept bins in
// increasing order: all of kx <= n/2, then ky = 1 .. n/2 - 1 of every kx > n/2).
__host__ __device__ inline int herm_kept_bins(int n) { return n * (n / 2 + 1) - (n - 2); }
__host__ __device__ inline int herm_bin(int b, int n) {
    const int nc = n / 2 + 1, head = nc * nc;
    if (b < head) return b;
    b -= head;
    const int kx = nc + b / (nc - 2);
    return kx * nc + 1 + (b - (kx - nc) * (nc - 2));
}

constexpr int FG_BM = 64, FG_BN = 64, FG_BK = 16, FG_PAD = 4, FG_T = 256;

// 4-byte asynchronous copy global -> shared; `ok` false writes a zero (zero-fill of the
// ragged edges of M, N and K).
__device__ __forceinline__ void fg_cp4(float* dst, const float* src, bool ok) {
    const unsigned d = static_cast<unsigned>(__cvta_generic_to_shared(dst));
    const int nbytes = ok ? 4 : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(d), "l"(src), "r"(nbytes) : "memory");
}

// TA / TB: operand stored [K][rows] instead of [rows][K]; CA / CB: use its complex conjugate.
// The k-blocks are double-buffered in shared memory: the asynchronous copies of block kb + 1
// are in flight while block kb is multiplied.
// BN: columns of a tile, 64 (4 per thread) or 96 (6 per thread; chosen where it leaves fewer
// padded columns, e.g. N = 96: one tile of 96 instead of 64 + 32 of 64).
template <bool TA, bool TB, bool CA, bool CB, int BN>
__global__ void __launch_bounds__(FG_T) cgemm_ffma_kernel(const GemmParams p) {
    static_assert(BN == 64 || BN == 96, "16 thread columns of 4 or 6 outputs");
    constexpr int TN = BN / 16;
    __shared__ __align__(16) float sA[2][2][FG_BK][FG_BM + FG_PAD];
    __shared__ __align__(16) float sB[2][2][FG_BK][BN + FG_PAD];

    dep_trigger();
    dep_wait();                     // no global access above this line
    const int tid = threadIdx.x;
    // grid: x = (row block, column block) linearised (tiled plans can have millions of row
    // blocks, more than grid.y takes), y = bin
    const int bin = p.herm_n ? herm_bin((int)blockIdx.y, p.herm_n) : (int)blockIdx.y;
    const int n_blocks = (p.N + BN - 1) / BN;
    const int m_blk = (int)(blockIdx.x / n_blocks) * FG_BM, n_blk = (int)(blockIdx.x % n_blocks) * BN;
    const size_t planeA = (size_t)(TA ? p.K : p.M) * p.lda,
                 planeB = (size_t)(TB ? p.K : p.N) * p.ldb, planeC = (size_t)p.M * p.ldc;
    const float* Ab = p.A + (size_t)bin * planeA;
    const float* Bb = p.B + (size_t)bin * planeB;
    float* Cb = p.C + (size_t)bin * planeC;
    const size_t imA = (size_t)p.bins * planeA, imB = (size_t)p.bins * planeB,
                 imC = (size_t)p.bins * planeC;

    const int tx = tid & 15, ty = tid >> 4;      // 16 x 16 threads
    const int lk = tid & 15, lr = tid >> 4;      // loader, k-contiguous operand: k within block, row group
    const int tr = tid & 63, tk = tid >> 6;      // loader, row-contiguous operand: row, k group

    // global -> shared as [k][row]; lanes run along the contiguous index of each operand
    auto issue = [&](int k0, int st) {
        if constexpr (!TA) {
            const int k = k0 + lk;
#pragma unroll
            for (int it = 0; it < FG_BM / 16; ++it) {
                const int r = lr + 16 * it, m = m_blk + r;
                const bool ok = (k < p.K) && (m < p.M);
                const float* src = ok ? Ab + (size_t)m * p.lda + k : Ab;
                fg_cp4(&sA[st][0][lk][r], src, ok);
                fg_cp4(&sA[st][1][lk][r], src + imA, ok);
            }
        } else {
            const int m = m_blk + tr;
#pragma unroll
            for (int it = 0; it < FG_BK / 4; ++it) {
                const int kk = tk + 4 * it, k = k0 + kk;
                const bool ok = (k < p.K) && (m < p.M);
                const float* src = ok ? Ab + (size_t)k * p.lda + m : Ab;
                fg_cp4(&sA[st][0][kk][tr], src, ok);
                fg_cp4(&sA[st][1][kk][tr], src + imA, ok);
            }
        }
        if constexpr (!TB) {
            const int k = k0 + lk;
#pragma unroll
            for (int it = 0; it < BN / 16; ++it) {
                const int r = lr + 16 * it, n = n_blk + r;
                const bool ok = (k < p.K) && (n < p.N);
                const float* src = ok ? Bb + (size_t)n * p.ldb + k : Bb;
                fg_cp4(&sB[st][0][lk][r], src, ok);
                fg_cp4(&sB[st][1][lk][r], src + imB, ok);
            }
        } else {
#pragma unroll
            for (int rr = tr; rr < BN; rr += 64) {
                const int n = n_blk + rr;
#pragma unroll
                for (int it = 0; it < FG_BK / 4; ++it) {
                    const int kk = tk + 4 * it, k = k0 + kk;
                    const bool ok = (k < p.K) && (n < p.N);
                    const float* src = ok ? Bb + (size_t)k * p.ldb + n : Bb;
                    fg_cp4(&sB[st][0][kk][rr], src, ok);
                    fg_cp4(&sB[st][1][kk][rr], src + imB, ok);
                }
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    float cr[4][TN], ci[4][TN];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) cr[i][j] = ci[i][j] = 0.0f;

    const int k_blocks = (p.K + FG_BK - 1) / FG_BK;
    issue(0, 0);
    for (int kb = 0; kb < k_blocks; ++kb) {
        const int st = kb & 1;
        if (kb + 1 < k_blocks) {
            issue((kb + 1) * FG_BK, st ^ 1);
            asm volatile("cp.async.wait_group 1;" ::: "memory");    // block kb has landed (for this thread)
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();                                            // ... and for everyone
#pragma unroll
        for (int kk = 0; kk < FG_BK; ++kk) {
            const float4 a_r = *reinterpret_cast<const float4*>(&sA[st][0][kk][ty * 4]);
            const float4 a_i = *reinterpret_cast<const float4*>(&sA[st][1][kk][ty * 4]);
            const float ar[4] = {a_r.x, a_r.y, a_r.z, a_r.w};
            const float ai[4] = {a_i.x, a_i.y, a_i.z, a_i.w};
            float br[TN], bi[TN];
            if constexpr (TN == 4) {
                const float4 b_r = *reinterpret_cast<const float4*>(&sB[st][0][kk][tx * 4]);
                const float4 b_i = *reinterpret_cast<const float4*>(&sB[st][1][kk][tx * 4]);
                br[0] = b_r.x; br[1] = b_r.y; br[2] = b_r.z; br[3] = b_r.w;
                bi[0] = b_i.x; bi[1] = b_i.y; bi[2] = b_i.z; bi[3] = b_i.w;
            } else {
#pragma unroll
                for (int j = 0; j < TN; j += 2) {       // 8-byte loads, 6 words apart across the lanes
                    const float2 v_r = *reinterpret_cast<const float2*>(&sB[st][0][kk][tx * TN + j]);
                    const float2 v_i = *reinterpret_cast<const float2*>(&sB[st][1][kk][tx * TN + j]);
                    br[j] = v_r.x; br[j + 1] = v_r.y;
                    bi[j] = v_i.x; bi[j + 1] = v_i.y;
                }
            }
            // (ar + i sa ai)(br + i sb bi), sa / sb = -1 for a conjugated operand:
            // re = ar br - sa sb ai bi,  im = sb ar bi + sa ai br
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) {
                    cr[i][j] = fmaf(ar[i], br[j], cr[i][j]);
                    cr[i][j] = fmaf((CA != CB) ? ai[i] : -ai[i], bi[j], cr[i][j]);
                    ci[i][j] = fmaf(CB ? -ar[i] : ar[i], bi[j], ci[i][j]);
                    ci[i][j] = fmaf(CA ? -ai[i] : ai[i], br[j], ci[i][j]);
                }
        }
        __syncthreads();                                            // stage st may be refilled
    }

    const int n0 = n_blk + tx * TN;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m_blk + ty * 4 + i;
        if (m >= p.M) continue;
        float* o_r = Cb + (size_t)m * p.ldc + n0;
        float* o_i = o_r + imC;
        bool vec = false;
        if constexpr (TN == 4) {
            if (n0 + 3 < p.N) {
                *reinterpret_cast<float4*>(o_r) = make_float4(cr[i][0], cr[i][1], cr[i][2], cr[i][3]);
                *reinterpret_cast<float4*>(o_i) = make_float4(ci[i][0], ci[i][1], ci[i][2], ci[i][3]);
                vec = true;
            }
        }
        if (!vec) {
#pragma unroll
            for (int j = 0; j < TN; ++j)
                if (n0 + j < p.N) { o_r[j] = cr[i][j]; o_i[j] = ci[i][j]; }
        }
    }
}

template <bool TA, bool TB, int BN>
static cudaError_t launch_cgemm_ffma_t(const GemmParams& p, dim3 grid, cudaStream_t st) {
    const bool ov = p.overlap != 0;
    if (p.conjA) return p.conjB ? dep_launch(ov, cgemm_ffma_kernel<TA, TB, true, true, BN>, grid, dim3(FG_T), 0, st, p)
                                : dep_launch(ov, cgemm_ffma_kernel<TA, TB, true, false, BN>, grid, dim3(FG_T), 0, st, p);
    return p.conjB ? dep_launch(ov, cgemm_ffma_kernel<TA, TB, false, true, BN>, grid, dim3(FG_T), 0, st, p)
                   : dep_launch(ov, cgemm_ffma_kernel<TA, TB, false, false, BN>, grid, dim3(FG_T), 0, st, p);
}
template <int BN>
static cudaError_t launch_cgemm_ffma_bn(const GemmParams& p, cudaStream_t st) {
    const long long blocks = (long long)((p.N + BN - 1) / BN) * ((p.M + FG_BM - 1) / FG_BM);
    if (blocks > 0x7fffffffLL || p.bins > 65535) return cudaErrorInvalidValue;
    if (p.herm_n && (p.herm_n < 8 || p.bins != p.herm_n * (p.herm_n / 2 + 1))) return cudaErrorInvalidValue;
    dim3 grid((unsigned)blocks, (unsigned)(p.herm_n ? herm_kept_bins(p.herm_n) : p.bins), 1);
    if (p.transA) return p.transB ? launch_cgemm_ffma_t<true, true, BN>(p, grid, st) : launch_cgemm_ffma_t<true, false, BN>(p, grid, st);
    return p.transB ? launch_cgemm_ffma_t<false, true, BN>(p, grid, st) : launch_cgemm_ffma_t<false, false, BN>(p, grid, st);
}

static cudaError_t launch_cgemm_ffma(const GemmParams& p, cudaStream_t st) {
    // the tile width that pads N the least (on a tie the 64-wide tile: 10 % faster per multiply-add, measured)
    const int pad64 = (p.N + 63) / 64 * 64, pad96 = (p.N + 95) / 96 * 96;
    return pad96 < pad64 ? launch_cgemm_ffma_bn<96>(p, st) : launch_cgemm_ffma_bn<FG_BN>(p, st);
}

}  // namespace fc
