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
// outputs (64 FFMAs per k against four 16-byte shared loads).  This is the exact
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
};

constexpr int FG_BM = 64, FG_BN = 64, FG_BK = 16, FG_PAD = 4, FG_T = 256;

__global__ void __launch_bounds__(FG_T) cgemm_ffma_kernel(const GemmParams p) {
    __shared__ __align__(16) float sA[2][FG_BK][FG_BM + FG_PAD];
    __shared__ __align__(16) float sB[2][FG_BK][FG_BN + FG_PAD];

    dep_trigger();
    dep_wait();                     // no global access above this line
    const int tid = threadIdx.x;
    // grid: x = (row block, column block) linearised (tiled plans can have millions of row
    // blocks, more than grid.y takes), y = bin
    const int bin = blockIdx.y;
    const int n_blocks = (p.N + FG_BN - 1) / FG_BN;
    const int m_blk = (int)(blockIdx.x / n_blocks) * FG_BM, n_blk = (int)(blockIdx.x % n_blocks) * FG_BN;
    const size_t planeA = (size_t)(p.transA ? p.K : p.M) * p.lda,
                 planeB = (size_t)(p.transB ? p.K : p.N) * p.ldb, planeC = (size_t)p.M * p.ldc;
    const float sa = p.conjA ? -1.0f : 1.0f, sb = p.conjB ? -1.0f : 1.0f;
    const float* Ab = p.A + (size_t)bin * planeA;
    const float* Bb = p.B + (size_t)bin * planeB;
    float* Cb = p.C + (size_t)bin * planeC;
    const size_t imA = (size_t)p.bins * planeA, imB = (size_t)p.bins * planeB,
                 imC = (size_t)p.bins * planeC;

    const int tx = tid & 15, ty = tid >> 4;      // 16 x 16 threads
    const int lk = tid & 15, lr = tid >> 4;      // loader: k within chunk, row group

    float cr[4][4], ci[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) cr[i][j] = ci[i][j] = 0.0f;

    for (int k0 = 0; k0 < p.K; k0 += FG_BK) {
        // global -> shared as [k][row]; zero-fill outside M/N/K; lanes run along the
        // contiguous index of each operand
        if (!p.transA) {
            const int k = k0 + lk;
#pragma unroll
            for (int it = 0; it < FG_BM / 16; ++it) {
                const int r = lr + 16 * it, m = m_blk + r;
                float are = 0.f, aim = 0.f;
                if (k < p.K && m < p.M) {
                    are = __ldg(Ab + (size_t)m * p.lda + k);
                    aim = sa * __ldg(Ab + imA + (size_t)m * p.lda + k);
                }
                sA[0][lk][r] = are; sA[1][lk][r] = aim;
            }
        } else {
            const int r = tid & 63, m = m_blk + r;
#pragma unroll
            for (int it = 0; it < FG_BK / 4; ++it) {
                const int kk = (tid >> 6) + 4 * it, k = k0 + kk;
                float are = 0.f, aim = 0.f;
                if (k < p.K && m < p.M) {
                    are = __ldg(Ab + (size_t)k * p.lda + m);
                    aim = sa * __ldg(Ab + imA + (size_t)k * p.lda + m);
                }
                sA[0][kk][r] = are; sA[1][kk][r] = aim;
            }
        }
        if (!p.transB) {
            const int k = k0 + lk;
#pragma unroll
            for (int it = 0; it < FG_BN / 16; ++it) {
                const int r = lr + 16 * it, n = n_blk + r;
                float bre = 0.f, bim = 0.f;
                if (k < p.K && n < p.N) {
                    bre = __ldg(Bb + (size_t)n * p.ldb + k);
                    bim = sb * __ldg(Bb + imB + (size_t)n * p.ldb + k);
                }
                sB[0][lk][r] = bre; sB[1][lk][r] = bim;
            }
        } else {
            const int r = tid & 63, n = n_blk + r;
#pragma unroll
            for (int it = 0; it < FG_BK / 4; ++it) {
                const int kk = (tid >> 6) + 4 * it, k = k0 + kk;
                float bre = 0.f, bim = 0.f;
                if (k < p.K && n < p.N) {
                    bre = __ldg(Bb + (size_t)k * p.ldb + n);
                    bim = sb * __ldg(Bb + imB + (size_t)k * p.ldb + n);
                }
                sB[0][kk][r] = bre; sB[1][kk][r] = bim;
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < FG_BK; ++kk) {
            const float4 a_r = *reinterpret_cast<const float4*>(&sA[0][kk][ty * 4]);
            const float4 a_i = *reinterpret_cast<const float4*>(&sA[1][kk][ty * 4]);
            const float4 b_r = *reinterpret_cast<const float4*>(&sB[0][kk][tx * 4]);
            const float4 b_i = *reinterpret_cast<const float4*>(&sB[1][kk][tx * 4]);
            const float ar[4] = {a_r.x, a_r.y, a_r.z, a_r.w};
            const float ai[4] = {a_i.x, a_i.y, a_i.z, a_i.w};
            const float br[4] = {b_r.x, b_r.y, b_r.z, b_r.w};
            const float bi[4] = {b_i.x, b_i.y, b_i.z, b_i.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    cr[i][j] = fmaf(ar[i], br[j], cr[i][j]);
                    cr[i][j] = fmaf(-ai[i], bi[j], cr[i][j]);
                    ci[i][j] = fmaf(ar[i], bi[j], ci[i][j]);
                    ci[i][j] = fmaf(ai[i], br[j], ci[i][j]);
                }
        }
        __syncthreads();
    }

    const int n0 = n_blk + tx * 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m_blk + ty * 4 + i;
        if (m >= p.M) continue;
        float* o_r = Cb + (size_t)m * p.ldc + n0;
        float* o_i = o_r + imC;
        if (n0 + 3 < p.N) {
            *reinterpret_cast<float4*>(o_r) = make_float4(cr[i][0], cr[i][1], cr[i][2], cr[i][3]);
            *reinterpret_cast<float4*>(o_i) = make_float4(ci[i][0], ci[i][1], ci[i][2], ci[i][3]);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (n0 + j < p.N) { o_r[j] = cr[i][j]; o_i[j] = ci[i][j]; }
        }
    }
}

static cudaError_t launch_cgemm_ffma(const GemmParams& p, cudaStream_t st) {
    const long long blocks = (long long)((p.N + FG_BN - 1) / FG_BN) * ((p.M + FG_BM - 1) / FG_BM);
    if (blocks > 0x7fffffffLL || p.bins > 65535) return cudaErrorInvalidValue;
    dim3 grid((unsigned)blocks, (unsigned)p.bins, 1);
    return dep_launch(p.overlap != 0, cgemm_ffma_kernel, grid, dim3(FG_T), 0, st, p);
}

}  // namespace fc
