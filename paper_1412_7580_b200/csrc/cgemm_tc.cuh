// Per-frequency-bin complex contraction on the 5th-generation tensor cores
// (Table 1, the Cgemm row): for every bin b,
//     C[b][m][n] = sum_k op(A)[b][m][k] * op(B)[b][n][k]      (complex)
// with planar operands (see cgemm_ffma.cuh for the layouts): each operand is
// stored either k-contiguous ([rows][k]) or row-contiguous ([k][rows]); the
// second form is fed to the tensor cores as an "MN-major" shared-memory matrix,
// so no pass ever needs a transposed copy of a spectrum.  op() is an optional
// complex conjugate, folded into the negate bits below.
//
// The complex product is four real TF32 MMAs per k-step into two FP32
// accumulators in tensor memory,
//     C_re += A_re B_re ; C_re += (-A_im) B_im ; C_im += A_re B_im ; C_im += A_im B_re,
// the minus sign coming from the instruction descriptor's negate-A bit, so no
// expanded or interleaved copy of an operand is ever built.
//
// One persistent CTA per SM, warp-specialised:
//   warp 0      TMA producer: 128-byte-swizzled boxes of 32 k-values x 128 rows
//               of A_re, A_im, B_re, B_im per stage (64 KB), 3 stages in flight;
//   warp 1      issues tcgen05.mma (one lane), owns the TMEM allocation;
//   warps 2..5  epilogue: tcgen05.ld of the finished accumulators, a swizzled
//               staging tile per warp in shared memory and TMA stores (full
//               128-byte lines, clipped at the matrix edge by the tensor map),
//               overlapped with the next tile's MMAs through two accumulator
//               buffers (2 x 256 TMEM columns).
// The per-bin problems are small and the kernel streams: it is bound by HBM
// bytes (two spectra in, one out), not by tensor throughput.
//
// Every wait on an mbarrier is bounded; when one runs out the kernel raises the
// caller's status word, drains what it issued, frees its tensor memory and
// returns normally.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "cgemm_ffma.cuh"
#include "tma_util.cuh"
#include "dep_launch.cuh"
#include "fft_kernels.cuh"

namespace fc {

constexpr int TC_BM = 128, TC_BN = 128, TC_BK = 32, TC_STAGES = 3;
constexpr int TC_THREADS = 192;
constexpr uint32_t TC_TILE_BYTES = TC_BM * TC_BK * 4;            // one 128 x 32 fp32 box: 16 KB
constexpr uint32_t TC_STAGE_BYTES = 4 * TC_TILE_BYTES;           // A_re, A_im, B_re, B_im
constexpr uint32_t TC_EPI_BUF_BYTES = 32 * 128;                  // 32 rows x 32 fp32, one TMA store box
constexpr uint32_t TC_EPI_BYTES = 4 * 2 * TC_EPI_BUF_BYTES;      // 4 warps x 2 buffers
constexpr uint32_t tc_smem_bytes(int stages) { return 1024 + stages * TC_STAGE_BYTES + TC_EPI_BYTES + 256; }
constexpr uint32_t TC_SMEM_BYTES = tc_smem_bytes(TC_STAGES);
// A launch that shares the SMs with a transform kernel (the filter spectrum produced range by range
// beside the contraction) runs a ring of two stages and leaves 64 KB of shared memory to that kernel.
constexpr int TC_STAGES_SHARED = 2;
constexpr uint32_t TC_TMEM_COLS = 512;
constexpr long long TC_WAIT_CYCLES = 2000000000LL;               // about one second

struct TcParams {
    int bins, M, N, K;
    int m_tiles, n_tiles, k_blocks;
    int conjA, conjB;
    int* status;
    long long wait_cycles;      // limit of one wait in SM clock cycles (the draining waits keep TC_WAIT_CYCLES)
    int bins_run;               // bins contracted by this launch (all of them, or a ky range of every kx)
    int nc, ky_begin, ky_count; // ky_count > 0: local bin b -> kx = b / ky_count, ky = ky_begin + b % ky_count
    int late_trigger;           // let the dependent launch start after this one's wait instead of before it
    int herm_n;                 // > 0: the launch runs the kept bins of GemmParams::herm_n (local bin -> herm_bin)
};

static inline bool tc_shape_supported(int M, int N, int K) {
    return M >= 1 && N >= 1 && K >= 1;
}
// The kernel streams: rows and k-values outside the matrices are zero-filled by the
// TMA without being fetched, so even mostly-empty 128 x 128 x 32 tiles cost little;
// only really tiny problems are left to the FP32 kernel (which is exact).  Measured on B200: with
// one or three summed terms (first layers, f = 3) the streaming kernel is still 3-4 x faster than
// the FP32 one (164 against 564 us for S128 f3 f'96 at n = 128), so the summed length does not
// enter the choice.
static inline bool tc_shape_profitable(int M, int N, int K) {
    (void)K;
    return (long long)M * N >= 128;
}

// ---- PTX wrappers ----------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit ran out or another role already gave up.  The first
// probe does not block; before every further (possibly suspending) attempt the clock and
// the abort flag are checked.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          long long limit) {
    if (fk_mbar_test_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (*abort_flag) return false;
        if (clock64() - t0 > limit) return false;
        if (mbar_try_wait(bar, parity)) return true;
    }
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                            int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int c0, int c1,
                                             int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
        ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                            uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32"
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15,"
        " %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31},"
        " [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]),
          "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]),
          "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows 128 B
// apart, groups of eight rows 1024 B apart (the layout a 128B-swizzled TMA box of
// 32 fp32 x rows produces).  Tile bases are 1024-byte aligned.
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | (1ull << 16) | (64ull << 32) | (1ull << 46) |
           (2ull << 61);
}
// MN-major TF32 operand: the only shared-memory layout the tensor cores take for
// it is the 128-byte swizzle with a 32-byte base (32-byte chunks of a 128-byte
// row are permuted by the row index modulo 4), which the TMA produces with its
// "128B, 32B atom" mode.  The tile is four blocks of 32 rows-of-the-matrix
// (128 B, contiguous in memory) x 32 k; inside a block consecutive k are 128 B
// apart, groups of four k 512 B apart (stride offset); blocks are 4096 B apart
// (leading offset).  One MMA consumes eight k = 1024 bytes.
__device__ __forceinline__ uint64_t tc_smem_desc_mn(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | (256ull << 16) | (32ull << 32) | (1ull << 46) |
           (1ull << 61);
}
// Instruction descriptor: D = FP32, A = B = TF32, M x N tile; majorness per operand.
__host__ __device__ constexpr uint32_t tc_idesc(int M, int N, bool negA, bool mnA, bool mnB) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((negA ? 1u : 0u) << 13) |
           ((mnA ? 1u : 0u) << 15) | ((mnB ? 1u : 0u) << 16) |
           ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

template <bool TA, bool TB, int ST>
__global__ void __launch_bounds__(TC_THREADS, 1)
cgemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmC, const TcParams p) {
    extern __shared__ uint8_t tc_raw[];
    const uint32_t raw_addr = smem_u32(tc_raw);
    const uint32_t tiles = (raw_addr + 1023u) & ~1023u;             // stage buffers, 1024-aligned
    const uint32_t epi = tiles + ST * TC_STAGE_BYTES;        // epilogue staging, 1024-aligned
    uint8_t* ctl = tc_raw + (tiles - raw_addr) + ST * TC_STAGE_BYTES + TC_EPI_BYTES;
    const uint32_t bars = epi + TC_EPI_BYTES;
    // barrier slots (8 bytes each): full[3] empty[3] tfull[2] tempty[2] drain
    auto full = [&](int s) { return bars + 8u * s; };
    auto empty = [&](int s) { return bars + 8u * (ST + s); };
    auto tfull = [&](int b) { return bars + 8u * (2 * ST + b); };
    auto tempty = [&](int b) { return bars + 8u * (2 * ST + 2 + b); };
    const uint32_t drain = bars + 8u * (2 * ST + 4);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctl + 128);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ctl + 136);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (!p.late_trigger) dep_trigger();
    if (tid == 0) {
        for (int s = 0; s < ST; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull(b), 1); mbar_init(tempty(b), 128); }
        mbar_init(drain, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(TC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    dep_wait();                     // no global access above this line
    // late: the dependent is a transform that runs beside this contraction (not after it) and
    // must not start before the operands of this launch are complete
    if (p.late_trigger) dep_trigger();

    const int num_tiles = p.bins_run * p.m_tiles * p.n_tiles;
    // local bin of this launch -> bin of the spectra
    auto global_bin = [&](int b) {
        if (p.herm_n) return herm_bin(b, p.herm_n);
        if (p.ky_count == 0) return b;
        const int kx = b / p.ky_count;
        return kx * p.nc + p.ky_begin + (b - kx * p.ky_count);
    };
    auto give_up = [&]() {
        *abort_flag = 1;
        if (p.status) atomicExch(p.status, 1);
    };

    if (warp == 0) {
        if (lane == 0) {
            // ---- producer ------------------------------------------------------
            int it = 0;
            bool ok = true;
            for (int t = blockIdx.x; ok && t < num_tiles; t += gridDim.x) {
                const int n_t = t % p.n_tiles;
                const int m_t = (t / p.n_tiles) % p.m_tiles;
                const int bin = global_bin(t / (p.n_tiles * p.m_tiles));
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % ST;
                    const uint32_t ph = (uint32_t)(it / ST) & 1u;
                    if (!mbar_wait(empty(s), ph ^ 1u, abort_flag, p.wait_cycles)) { ok = false; break; }
                    const uint32_t dst = tiles + s * TC_STAGE_BYTES;
                    mbar_expect_tx(full(s), TC_STAGE_BYTES);
#pragma unroll
                    for (int part = 0; part < 2; ++part) {
                        if constexpr (!TA) {
                            tma_load_3d(dst + part * TC_TILE_BYTES, &tmA, kb * TC_BK, m_t * TC_BM,
                                        part * p.bins + bin, full(s));
                        } else {
#pragma unroll
                            for (int blk = 0; blk < 4; ++blk)
                                tma_load_3d(dst + part * TC_TILE_BYTES + blk * 4096, &tmA,
                                            m_t * TC_BM + blk * 32, kb * TC_BK, part * p.bins + bin, full(s));
                        }
                        if constexpr (!TB) {
                            tma_load_3d(dst + (2 + part) * TC_TILE_BYTES, &tmB, kb * TC_BK, n_t * TC_BN,
                                        part * p.bins + bin, full(s));
                        } else {
#pragma unroll
                            for (int blk = 0; blk < 4; ++blk)
                                tma_load_3d(dst + (2 + part) * TC_TILE_BYTES + blk * 4096, &tmB,
                                            n_t * TC_BN + blk * 32, kb * TC_BK, part * p.bins + bin, full(s));
                        }
                    }
                }
            }
            if (!ok) {
                give_up();
                // let the copies already issued land before the CTA's memory goes away
                const int back = it < ST ? it : ST;
                for (int j = it - back; j < it; ++j) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(full(j % ST), (uint32_t)(j / ST) & 1u) &&
                           clock64() - t0 < TC_WAIT_CYCLES) {}
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer ----------------------------------------------------
            constexpr uint32_t idesc_pos = tc_idesc(TC_BM, TC_BN, false, TA, TB);
            constexpr uint32_t idesc_neg = tc_idesc(TC_BM, TC_BN, true, TA, TB);
            // (Ar + i sA Ai)(Br + i sB Bi): re = ArBr - sA sB AiBi ; im = sB ArBi + sA AiBr
            const uint32_t id_ii = (p.conjA != p.conjB) ? idesc_pos : idesc_neg;
            const uint32_t id_ri = p.conjB ? idesc_neg : idesc_pos;
            const uint32_t id_ir = p.conjA ? idesc_neg : idesc_pos;
            int it = 0, tl = 0;
            bool ok = true;
            for (int t = blockIdx.x; ok && t < num_tiles; t += gridDim.x, ++tl) {
                const int buf = tl & 1;
                if (!mbar_wait(tempty(buf), ((uint32_t)(tl >> 1) & 1u) ^ 1u, abort_flag, p.wait_cycles)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d_re = tmem_base + (uint32_t)buf * 256u;
                const uint32_t d_im = d_re + 128u;
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % ST;
                    if (!mbar_wait(full(s), (uint32_t)(it / ST) & 1u, abort_flag, p.wait_cycles)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t src = tiles + s * TC_STAGE_BYTES;
                    const uint64_t a_re = TA ? tc_smem_desc_mn(src) : tc_smem_desc(src);
                    const uint64_t a_im = TA ? tc_smem_desc_mn(src + TC_TILE_BYTES)
                                             : tc_smem_desc(src + TC_TILE_BYTES);
                    const uint64_t b_re = TB ? tc_smem_desc_mn(src + 2 * TC_TILE_BYTES)
                                             : tc_smem_desc(src + 2 * TC_TILE_BYTES);
                    const uint64_t b_im = TB ? tc_smem_desc_mn(src + 3 * TC_TILE_BYTES)
                                             : tc_smem_desc(src + 3 * TC_TILE_BYTES);
                    // per k-step of 8: K-major advances 32 bytes inside the swizzled row,
                    // MN-major advances eight 128-byte k-rows (address field is in 16 B units)
                    constexpr uint64_t stepA = TA ? 64 : 2, stepB = TB ? 64 : 2;
#pragma unroll
                    for (int k = 0; k < TC_BK / 8; ++k) {
                        const uint64_t da = stepA * k, db = stepB * k;
                        const uint32_t acc = (kb | k) != 0 ? 1u : 0u;
                        tc_mma_tf32(d_re, a_re + da, b_re + db, idesc_pos, acc);
                        tc_mma_tf32(d_re, a_im + da, b_im + db, id_ii, 1u);
                        tc_mma_tf32(d_im, a_re + da, b_im + db, id_ri, acc);
                        tc_mma_tf32(d_im, a_im + da, b_re + db, id_ir, 1u);
                    }
                    tc_commit(empty(s));          // stage reusable once these MMAs have read it
                }
                if (ok) tc_commit(tfull(buf));    // accumulators complete
            }
            if (!ok) {
                give_up();
                tc_commit(drain);                 // wait (bounded) for the MMAs already issued
                const long long t0 = clock64();
                while (!mbar_try_wait(drain, 0u) && clock64() - t0 < TC_WAIT_CYCLES) {}
            }
        }
    } else {
        // ---- epilogue: warps 2..5, each owns the TMEM lanes of its quarter ------
        const int q = warp & 3;
        const uint32_t my_buf = epi + (uint32_t)q * 2u * TC_EPI_BUF_BYTES;
        int tl = 0;
        uint32_t nstore = 0;
        bool ok = true;
        for (int t = blockIdx.x; ok && t < num_tiles; t += gridDim.x, ++tl) {
            const int n_t = t % p.n_tiles;
            const int m_t = (t / p.n_tiles) % p.m_tiles;
            const int bin = global_bin(t / (p.n_tiles * p.m_tiles));
            const int buf = tl & 1;
            if (!mbar_wait(tfull(buf), (uint32_t)(tl >> 1) & 1u, abort_flag, p.wait_cycles)) { ok = false; break; }
            tc_fence_after_sync();
            const int row0 = m_t * TC_BM + q * 32;
            const int col0 = n_t * TC_BN;
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * 256u;
            if (row0 < p.M) {                                           // warp-uniform
#pragma unroll 1
                for (int part = 0; part < 2; ++part) {
#pragma unroll 1
                    for (int c = 0; c < TC_BN; c += 32) {
                        if (col0 + c >= p.N) break;                     // warp-uniform
                        uint32_t v[32];
                        tc_ld32(t_row + (uint32_t)(part * 128 + c), v);
                        // the staging buffer used two stores ago must have been read out
                        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                        __syncwarp();
                        tc_wait_ld();
                        // row = lane; 16-byte chunk j goes to slot j ^ (row % 8) (128-byte swizzle)
                        const uint32_t sbuf = my_buf + (nstore & 1u) * TC_EPI_BUF_BYTES;
                        const uint32_t srow = sbuf + (uint32_t)lane * 128u;
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};"
                                         ::"r"(srow + (uint32_t)((j ^ (lane & 7)) << 4)), "r"(v[4 * j]),
                                           "r"(v[4 * j + 1]), "r"(v[4 * j + 2]), "r"(v[4 * j + 3])
                                         : "memory");
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                        if (lane == 0) {
                            tma_store_3d(&tmC, sbuf, col0 + c, row0, part * p.bins + bin);
                            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        }
                        ++nstore;
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(tempty(buf));
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        __syncwarp();
        if (!ok && lane == 0) give_up();
    }

    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     ::"r"(tmem_base), "r"(TC_TMEM_COLS) : "memory");
    }
}

// ---- host side -------------------------------------------------------------
template <bool TA, bool TB, int ST>
static cudaError_t launch_cgemm_tc_t(const GemmParams& g, int* status, cudaStream_t st, int sm_count) {
    auto kern = cgemm_tc_kernel<TA, TB, ST>;
    static std::atomic<unsigned long long> attr_set_devices{0};     // one bit per device ordinal
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
    if (dev < 0 || dev >= 64 || !((attr_set_devices.load(std::memory_order_acquire) >> dev) & 1ull)) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)tc_smem_bytes(ST));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set_devices.fetch_or(1ull << dev, std::memory_order_release);
    }
    CUtensorMap tmA, tmB, tmC;
    // k-contiguous: rows = M (or N), cols = K, box 32 k x 128 rows;
    // row-contiguous: rows = K, cols = M (or N), box 32 rows-of-the-matrix x 32 k.
    const bool okA = TA ? tc_make_map(&tmA, g.A, g.bins, g.K, g.M, g.lda, 32, TC_BK,
                                      CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B)
                        : tc_make_map(&tmA, g.A, g.bins, g.M, g.K, g.lda, TC_BK, TC_BM);
    const bool okB = TB ? tc_make_map(&tmB, g.B, g.bins, g.K, g.N, g.ldb, 32, TC_BK,
                                      CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B)
                        : tc_make_map(&tmB, g.B, g.bins, g.N, g.K, g.ldb, TC_BK, TC_BN);
    const bool okC = tc_make_map(&tmC, g.C, g.bins, g.M, g.N, g.ldc, 32, 32);
    if (!okA || !okB || !okC) return cudaErrorInvalidValue;
    TcParams p{};
    p.bins = g.bins; p.M = g.M; p.N = g.N; p.K = g.K;
    p.m_tiles = (g.M + TC_BM - 1) / TC_BM;
    p.n_tiles = (g.N + TC_BN - 1) / TC_BN;
    p.k_blocks = (g.K + TC_BK - 1) / TC_BK;
    p.conjA = g.conjA; p.conjB = g.conjB;
    p.status = status;
    p.wait_cycles = g.wait_cycles > 0 ? g.wait_cycles : TC_WAIT_CYCLES;
    p.bins_run = g.bins; p.nc = g.nc; p.ky_begin = g.ky_begin; p.ky_count = 0;
    p.late_trigger = g.shared_sms ? 1 : 0;
    p.herm_n = 0;
    if (g.herm_n) {
        if (g.ky_count > 0 || g.herm_n < 8 || g.bins != g.herm_n * (g.herm_n / 2 + 1)) return cudaErrorInvalidValue;
        p.herm_n = g.herm_n;
        p.bins_run = herm_kept_bins(g.herm_n);
    }
    if (g.ky_count > 0) {
        if (g.nc < 1 || g.bins % g.nc != 0 || g.ky_begin < 0 || g.ky_begin + g.ky_count > g.nc)
            return cudaErrorInvalidValue;
        if (g.ky_count < g.nc) { p.ky_count = g.ky_count; p.bins_run = (g.bins / g.nc) * g.ky_count; }
    }
    const long long tiles = (long long)p.bins_run * p.m_tiles * p.n_tiles;
    if (tiles > 0x7fffffffLL) return cudaErrorInvalidValue;
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    return dep_launch(g.overlap != 0, kern, dim3(grid), dim3(TC_THREADS), tc_smem_bytes(ST), st, tmA, tmB, tmC, p);
}

static cudaError_t launch_cgemm_tc(const GemmParams& g, int* status, cudaStream_t st) {
    const int sm_count = fft_sm_count();        // of the current device
    if (sm_count < 1) return cudaErrorInvalidDevice;
    if (g.shared_sms) {
        constexpr int S2 = TC_STAGES_SHARED;
        if (g.transA) return g.transB ? launch_cgemm_tc_t<true, true, S2>(g, status, st, sm_count)
                                      : launch_cgemm_tc_t<true, false, S2>(g, status, st, sm_count);
        return g.transB ? launch_cgemm_tc_t<false, true, S2>(g, status, st, sm_count)
                        : launch_cgemm_tc_t<false, false, S2>(g, status, st, sm_count);
    }
    if (g.transA) return g.transB ? launch_cgemm_tc_t<true, true, TC_STAGES>(g, status, st, sm_count)
                                  : launch_cgemm_tc_t<true, false, TC_STAGES>(g, status, st, sm_count);
    return g.transB ? launch_cgemm_tc_t<false, true, TC_STAGES>(g, status, st, sm_count)
                    : launch_cgemm_tc_t<false, false, TC_STAGES>(g, status, st, sm_count);
}

}  // namespace fc
