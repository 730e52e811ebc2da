// Batched 2-D R2C / C2R FFT kernels with fused zero-padding, fused
// frequency-major transpose, crop, scale and accumulate.
//
// One CTA transforms tiles of G planes that are adjacent along the minor index
// of the frequency-major matrix they are written to (read from), so that every
// frequency bin receives G consecutive floats: the transposition BDHW -> HWBD of
// the paper's Table 1 happens in the store (load) itself and no separate
// transpose pass or padded tensor exists (Section 5.1: zero-copy padding by
// clipped loads; returning the transposed spectrum removes a pass).
//
// Frequency bins.  For a real plane only half the spectrum is kept (Section 3.1).
// Inside the convolution passes the kept half is ky in [0, n/2], kx in [0, n),
// numbered bin = kx*(n/2+1) + ky, because the first 1-D pass then runs down the
// columns of the plane with one thread per column, which reads shared memory
// without bank conflicts for every plane width and lets the planes be staged by
// one bulk asynchronous copy.  The per-bin contraction does not care which half
// is kept or how bins are numbered.  The bare transforms present the
// conventional [n][n/2+1] half instead; the kernels translate through the
// Hermitian symmetry X[ky][kx] = conj X[-ky][-kx].
//
// Spectra in global memory are planar: [2][bins][R][ld] floats, all real parts
// first.  A tile's spectrum is assembled in shared memory as [part][bin][G] and
// moved by the TMA as boxes of G columns x 1 row x D bins, so the SM never
// issues a scattered global access and every shared-memory access of a warp is
// one contiguous 128-byte line with an immediate offset.
//
// Forward kernel, per tile (the inverse mirrors it):
//   1. bulk asynchronous copy of the G real planes into shared memory; the copy
//      of the next tile is issued as soon as step 2 has read the current one;
//   2. one thread per non-zero column: real FFT of length N down the column, in
//      registers (complex FFT of length N/2 plus a Hermitian post-pass), half
//      spectrum (N/2+1 rows) written back to shared memory;
//   3. N/2 row transforms per plane -- rows ky = 0 and ky = N/2 are real and ride
//      together as one complex row (the paper's "n x n/2 with border case",
//      Section 5.2) -- each split over two threads by one decimation-in-frequency
//      step applied while loading, then an N/2-point register FFT; results go to
//      the staging tile and from there to global memory by TMA stores.
// CTAs are persistent and walk the tiles with a grid stride.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "fft_core.cuh"
#include "tma_util.cuh"
#include "dep_launch.cuh"

namespace fc {

// LAYOUT_FREQ_TMA / _DIRECT: planar frequency-major spectra, moved by the TMA or
// by plain per-thread accesses; LAYOUT_BARE: [plane][n][n/2+1] interleaved pairs, accessed
// by the threads directly; LAYOUT_BARE_STAGED: the same layout, but a tile's planes (which
// are contiguous in memory) travel between global and shared memory as one bulk
// asynchronous copy per plane and the threads only touch the shared-memory image.
enum { LAYOUT_FREQ_TMA = 0, LAYOUT_BARE = 1, LAYOUT_FREQ_DIRECT = 2, LAYOUT_BARE_STAGED = 3 };

// Pitch (in complex elements) of one plane of the bare layout in shared memory: the plane
// itself, rounded up so that every plane starts on a 16-byte boundary, plus a few elements so
// that lanes running over the planes of a tile and over adjacent rows hit distinct banks.
template <int N, int G>
struct BareGeom {
    static constexpr int PLANE = N * (N / 2 + 1);
    static constexpr int SKEW = (G >= 8) ? 2 : 16 / G;
    static constexpr int P2 = ((PLANE + 15) / 16) * 16 + SKEW;
    static constexpr size_t BYTES = (((size_t)G * P2 * 8 + 127) / 128) * 128;
};

struct FftParams {
    const float* real_in;   // forward: real planes in
    float* real_out;        // inverse: real planes out
    const float* spec_in;   // inverse: spectra in
    float* spec_out;        // forward: spectra out
    int h, w;               // forward: plane size; inverse: crop window (hc, wc)
    int R, C;               // frequency-major matrix: rows, cols (plane = row*C + col)
    int ld;                 // its leading dimension in floats
    int tiles_per_row;      // ceil(C / G)
    int num_tiles;          // R * tiles_per_row
    int in_bytes;           // shared-memory bytes reserved for the real tile (multiple of 128)
    float scale;            // inverse
    int accumulate;         // inverse
    // Spatial tiling (Section 6): win != 0 makes every matrix row (s, ty, tx) a window of plane s
    // of a larger H x W plane instead of a whole plane.  Tiles step by (step_y, step_x).
    // Forward: the window of h x w samples starts at (ty step_y + oy, tx step_x + ox), samples
    // outside the plane read as zero.  Inverse: rows [oy, oy + h) and columns [ox, ox + w) of the
    // transform's output go to the plane at (ty step_y, tx step_x), clipped at the plane's edge.
    int win;
    int H, W;
    int nty, ntx;
    int step_y, step_x;
    int oy, ox;
    int overlap;            // host only: launch as a programmatic dependent of the previous kernel
    int* status;            // device status word raised when a bounded wait runs out (may be null)
    long long wait_cycles;  // limit of one wait in SM clock cycles; <= 0 selects FK_WAIT_CYCLES
};

// Geometry of the half-spectrum scratch ("mid") of one plane in shared memory:
// (N/2+1) rows of N+1 complex, plane pitch = (16 / min(G,16)) * odd so that lanes
// running over the plane index and then over adjacent rows hit distinct 8-byte
// banks.
template <int N, int G>
struct MidGeom {
    static constexpr int PW = N + 1;
    static constexpr int NEED = (N / 2 + 1) * PW;   // the forward kernel uses N/2 rows of it
    static constexpr int UNIT = 16 / (G < 16 ? G : 16);
    static constexpr int MUL = ((NEED + UNIT - 1) / UNIT) | 1;
    static constexpr int P = MUL * UNIT;
    static constexpr int BYTES = ((G * P * 8 + 127) / 128) * 128;
};
// Bins moved per TMA box: the largest divisor of N*(N/2+1) that is <= 256.
constexpr int tma_bins_per_box(int N) {
    int B = N * (N / 2 + 1), best = 1;
    for (int d = 1; d <= 256; ++d)
        if (B % d == 0) best = d;
    return best;
}
static inline int real_tile_bytes(int G, int rows, int cols) {
    return (G * rows * cols * 4 + 127) & ~127;
}

// ---- small PTX helpers (bulk asynchronous copies) ---------------------------
__device__ __forceinline__ uint32_t fk_smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void fk_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fk_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool fk_mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool fk_mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Every wait on an mbarrier is bounded: about a second by default, or the limit the plan
// was given.  Returns false when the limit ran out.  The first probe does not block;
// try_wait may suspend the thread for a hardware-defined time, so the clock is read before
// every further attempt and a very short limit really is short.
constexpr long long FK_WAIT_CYCLES = 2000000000LL;
__device__ __forceinline__ bool fk_mbar_wait(uint32_t bar, uint32_t parity, long long limit) {
    if (fk_mbar_test_wait(bar, parity)) return true;
    if (limit <= 0) limit = FK_WAIT_CYCLES;
    const long long t0 = clock64();
    for (;;) {
        if (clock64() - t0 > limit) return false;
        if (fk_mbar_try_wait(bar, parity)) return true;
    }
}
// A wait that reports: when the plan's limit runs out the status word is raised, and the copy
// is then given the full default limit to land -- it must not arrive in shared memory that
// already belongs to another CTA.  True if the data is there (possibly late, status raised),
// false if it never came: the caller then leaves its remaining tiles undone and returns.
__device__ __forceinline__ bool fk_wait_or_report(uint32_t bar, uint32_t parity, long long limit,
                                                  int* status) {
    if (fk_mbar_wait(bar, parity, limit)) return true;
    if (status) atomicExch(status, 1);
    return fk_mbar_wait(bar, parity, FK_WAIT_CYCLES);
}
__device__ __forceinline__ void fk_bulk_g2s(uint32_t dst, const void* src, uint32_t bytes,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fk_bulk_s2g(void* dst, uint32_t src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void fk_tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                               int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void fk_tma_store_3d(const CUtensorMap* map, uint32_t src, int c0,
                                                int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
        ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void fk_bulk_commit() {
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void fk_bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

// One decimation-in-frequency step fused into the loads of an N-point complex
// transform split over two threads (q = 0: even outputs, q = 1: odd outputs).
template <int N, bool INV, int Q, class Load>
__device__ __forceinline__ void load_split(Load&& load, float (&ar)[N / 2], float (&ai)[N / 2]) {
    constexpr int M = N / 2;
    static_for<M>([&](auto J) {
        constexpr int j = decltype(J)::value;
        const float2 lo = load(J), hi = load(std::integral_constant<int, j + M>{});
        if constexpr (Q == 0) {
            ar[j] = lo.x + hi.x;
            ai[j] = lo.y + hi.y;
        } else {
            const float dr = lo.x - hi.x, di = lo.y - hi.y;
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

// The same step when only the first N/2 inputs can be non-zero (zero-padded rows of a
// narrow plane): the butterflies degenerate to a copy (q = 0) or one twiddle (q = 1).
// `live` is the number of inputs that exist; the rest read as zero.
template <int N, bool INV, int Q, class Load>
__device__ __forceinline__ void load_split_narrow(Load&& load, int live, float (&ar)[N / 2],
                                                  float (&ai)[N / 2]) {
    constexpr int M = N / 2;
    static_for<M>([&](auto J) {
        constexpr int j = decltype(J)::value;
        float2 lo = make_float2(0.0f, 0.0f);
        if (j < live) lo = load(J);
        if constexpr (Q == 0 || j == 0) {
            ar[j] = lo.x; ai[j] = lo.y;
        } else if constexpr (4 * j == N) {
            if constexpr (!INV) { ar[j] = lo.y; ai[j] = -lo.x; }
            else                { ar[j] = -lo.y; ai[j] = lo.x; }
        } else {
            constexpr float c = Tw<N, j>::c;
            constexpr float sn = INV ? -Tw<N, j>::s : Tw<N, j>::s;
            ar[j] = fc_fma(sn, lo.y, c * lo.x);
            ai[j] = fc_fma(-sn, lo.x, c * lo.y);
        }
    });
}

// ---------------------------------------------------------------------------
// Forward: real planes -> half spectra.
// ALIAS: the half-spectrum scratch overwrites the staging area of the real tile
// (no prefetch of the next tile); used where one tile nearly fills shared memory.
// ---------------------------------------------------------------------------
template <int N, int G, int LAYOUT, bool ALIAS, bool SALIAS, int MINB, bool WIN = false>
__global__ void __launch_bounds__(N* G, MINB)
r2c_kernel(const __grid_constant__ CUtensorMap tmS0, const __grid_constant__ CUtensorMap tmS1,
           const FftParams p0, const FftParams p1) {
    // Two operands can share one launch (both forward transforms of a pass): tiles
    // [0, p0.num_tiles) belong to the first, the rest to the second.
    constexpr int T = N * G, NC = N / 2 + 1, M = N / 2, HALF = T / 2, B = N * NC;
    constexpr int PW = MidGeom<N, G>::PW, P = MidGeom<N, G>::P;
    constexpr bool TMA = (LAYOUT == LAYOUT_FREQ_TMA);
    constexpr bool BSTG = (LAYOUT == LAYOUT_BARE_STAGED);
    constexpr bool BARE = (LAYOUT == LAYOUT_BARE) || BSTG;
    constexpr int P2 = BareGeom<N, G>::P2;
    constexpr int D = tma_bins_per_box(N);
    // The packed row (ky = 0 with ky = N/2) is taken apart either by the two threads that
    // transformed it or, with the TMA staging, afterwards by the whole CTA (one more barrier,
    // but no warp does more than the others).  Measured on B200: the CTA-wide form is 3-10 %
    // faster per launch for N <= 32; at N = 64 (16-byte staging rows) it is faster too, except
    // that the second large operand of accGrad then runs 40 % slower, so N = 64 keeps the
    // thread-local form.
    constexpr bool WIDE_UNTANGLE = TMA && N <= 32;
    static_assert(HALF % 32 == 0, "the two halves of a row transform must be warp-uniform");
    extern __shared__ __align__(128) unsigned char fc_smem[];
    float* sIn = reinterpret_cast<float*>(fc_smem);
    unsigned char* mid_base = fc_smem + (ALIAS ? 0 : p0.in_bytes);
    float2* sMid = reinterpret_cast<float2*>(mid_base);
    // SALIAS: the staging tile reuses the scratch (one more barrier per tile, a third less
    // shared memory, so more CTAs stay resident)
    float* sStage = reinterpret_cast<float*>(
        SALIAS ? mid_base
               : mid_base + (ALIAS ? (p0.in_bytes > MidGeom<N, G>::BYTES ? p0.in_bytes : MidGeom<N, G>::BYTES)
                                   : MidGeom<N, G>::BYTES));
    __shared__ __align__(8) unsigned long long bar_storage;
    const uint32_t bar = fk_smem_u32(&bar_storage);

    const int tid = threadIdx.x;
    const int total_tiles = p0.num_tiles + p1.num_tiles;
    // thread roles of step 3, fixed for the whole kernel: (half, row ky, plane)
    const int q = tid / HALF, u = tid - q * HALF;
    const int kyp = u / G, gB = u - kyp * G;
    const int q4 = tid / (T / 4), u4 = tid - q4 * (T / 4);      // step 2, narrow planes: quarter
    // operand-dependent state, set by select()
    int h = 1, w = 1, hw = 1, opC = 1, tpr = 1, step_rows = 0, step_cols = 0;
    bool split4 = false;                                        // narrow planes: 4 threads per column
    bool narrow = false;                                        // at most half the columns are live
    auto select = [&](bool second) {
        h = second ? p1.h : p0.h;
        w = second ? p1.w : p0.w;
        opC = second ? p1.C : p0.C;
        tpr = second ? p1.tiles_per_row : p0.tiles_per_row;
        hw = h * w;
        split4 = (4 * w <= N);
        narrow = (2 * w <= N);
        step_rows = gridDim.x / tpr; step_cols = gridDim.x - step_rows * tpr;
    };
    // step 2 roles: N lanes per plane (a warp never straddles two planes, so neither its
    // reads of the real tile nor its writes to the scratch collide on a bank); narrow planes
    // use N/4 lanes per plane and quarter
    const int gA = tid / N, cA = tid % N;
    const int g4 = u4 / (N / 4), c4 = u4 % (N / 4);
    // tile index -> (operand, row, tile in row)
    auto locate = [&](int tile, bool& second, int& row, int& tcol) {
        second = tile >= p0.num_tiles;
        const int t = second ? tile - p0.num_tiles : tile;
        const int tpr = second ? p1.tiles_per_row : p0.tiles_per_row;
        row = t / tpr;
        tcol = t - row * tpr;
    };

    dep_trigger();
    if (tid == 0) {
        fk_mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    dep_wait();                     // no global access above this line

    // Side jobs are spread over different warps so that no single thread strings them
    // together: thread T/2 issues the input copy, the last warp issues the TMA stores.
    constexpr int NB = 2 * B / D;                       // TMA boxes per tile
    static_assert(!TMA || NB <= 32, "one lane per TMA box");
    const bool is_loader = (tid == T / 2);
    const bool is_storer = (tid >= T - 32) && ((tid & 31) < NB);

    // Stage the planes of a tile.  Returns true if the copy is asynchronous (wait on the
    // barrier before reading), false if it was done with plain loads by all threads.
    bool win_pending = false;       // windowed tile on its way in through cp.async
    auto stage = [&](bool second, int row, int tcol) -> bool {
        const int sh = second ? p1.h : p0.h, sw = second ? p1.w : p0.w;
        const int sC = second ? p1.C : p0.C;
        const float* base = second ? p1.real_in : p0.real_in;
        const int c0 = tcol * G;
        const int gcount = min(G, sC - c0);
        if (WIN && (second ? p1.win : p0.win)) {
            // window of a larger plane: clipped loads (Section 5.1), one plane row per N lanes
            const FftParams& pw = second ? p1 : p0;
            const int nt = pw.nty * pw.ntx;
            const int s = row / nt, t = row - s * nt;
            const int ty = t / pw.ntx, tx = t - ty * pw.ntx;
            const int y0 = ty * pw.step_y + pw.oy, x0 = tx * pw.step_x + pw.ox;
            const int rr = tid / N, cc = tid - rr * N;
            const int xx = x0 + cc;
            const bool col_ok = (cc < sw) && xx >= 0 && xx < pw.W;
            // 4-byte asynchronous copies; a sample outside the plane is a copy of zero bytes,
            // which writes a zero.  Completion: every thread waits for its own copies, then a
            // barrier (win_pending, at the top of the tile loop).  The row test and the address
            // are formed once per row sweep; the planes of the tile only advance pointers.
            if (cc < sw) {
                const int r_lo = max(0, -y0), r_hi = min(sh, pw.H - y0);    // window rows inside the plane
                const size_t plane = (size_t)pw.H * pw.W;
                const float* pl0 = base + ((size_t)s * sC + c0) * plane;
                const long long off0 = (long long)y0 * pw.W + xx;
                const uint32_t tile_stride = 4u * (uint32_t)(sh * sw);
                const uint32_t dst0 = fk_smem_u32(sIn + cc);
                for (int r = rr; r < sh; r += G) {
                    const bool ok = col_ok && r >= r_lo && r < r_hi;
                    const float* src = ok ? pl0 + (off0 + (long long)r * pw.W) : pl0;
                    const size_t step = ok ? plane : 0;
                    const int nbytes = ok ? 4 : 0;
                    uint32_t dstp = dst0 + 4u * (uint32_t)(r * sw);
                    for (int g = 0; g < gcount; ++g) {
                        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;"
                                     ::"r"(dstp), "l"(src), "r"(nbytes) : "memory");
                        dstp += tile_stride;
                        src += step;
                    }
                }
            }
            win_pending = true;
            return false;
        }
        const float* src = base + ((size_t)row * sC + c0) * (sh * sw);
        const int total = gcount * sh * sw;
        if ((reinterpret_cast<uintptr_t>(src) & 15) == 0) {
            const int bulk = total & ~3;
            if (is_loader && bulk > 0) {
                fk_mbar_expect_tx(bar, (uint32_t)bulk * 4u);
                fk_bulk_g2s(fk_smem_u32(sIn), src, (uint32_t)bulk * 4u, bar);
            }
            if (tid < total - bulk) sIn[bulk + tid] = __ldg(src + bulk + tid);
            return bulk > 0;
        }
        for (int i = tid; i < total; i += T) sIn[i] = __ldg(src + i);
        return false;
    };

    uint32_t phase = 0;
    bool pending = false, store_pending = false;
    bool second = false, second_n = false;
    int row = 0, tcol = 0, row_n = 0, tcol_n = 0;
    if ((int)blockIdx.x < total_tiles) {
        locate(blockIdx.x, second_n, row_n, tcol_n);
        pending = stage(second_n, row_n, tcol_n);
        select(second_n);
    }
    __syncthreads();           // plain-load parts of the first tile are visible to everyone

    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        if (second_n != second) select(second_n);       // divisions only when the operand changes
        second = second_n; row = row_n; tcol = tcol_n;
        const FftParams& p = second ? p1 : p0;
        const CUtensorMap* tmS = second ? &tmS1 : &tmS0;
        const int c0 = tcol * G;
        const int gcount = min(G, opC - c0);
        const int next = tile + gridDim.x;
        if (next < total_tiles) {
            if (!second && next >= p0.num_tiles) {
                locate(next, second_n, row_n, tcol_n);  // crossing into the second operand
            } else {
                row_n = row + step_rows; tcol_n = tcol + step_cols;
                if (tcol_n >= tpr) { tcol_n -= tpr; ++row_n; }
            }
        }

        if (pending) {
            if (!fk_wait_or_report(bar, phase, p0.wait_cycles, p0.status)) {
                // the copy never landed: let the stores already issued finish and leave
                if ((TMA || BSTG) && store_pending && (TMA ? is_storer : tid >= T - 32))
                    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
                return;
            }
            phase ^= 1u;
        }
        if (WIN && win_pending) {
            asm volatile("cp.async.wait_all;" ::: "memory");
            __syncthreads();
            win_pending = false;
        }

        // 2. column transforms.  Wide planes: thread = (plane gA, column cA), cA < w, one real
        //    FFT of length N each.  Narrow planes (filters): four threads per column, thread
        //    q4 computing the outputs ky = 4k + q4 through one radix-4 decimation-in-frequency
        //    step and a complex FFT of length N/4, so that the few columns still occupy the CTA.
        {
            constexpr int L = N / 4;
            float Xr[NC], Xi[NC];
            float br[L], bi[L];
            bool act;
            if (!split4) {
                act = (gA < gcount) && (cA < w);
                if (act) {
                    float v[N];
                    const float* src = sIn + gA * hw + cA;
                    // Zero-padding below the plane.  Rows r < N/2 exist whenever h > N/2 (the
                    // usual case: N is the next power of two), so they are plain loads; the
                    // others are loaded unconditionally (clamped) and zeroed by a select --
                    // a branch per element would serialise the shared-memory loads.
                    if (h > M) {
                        static_for<N>([&](auto Rr) {
                            constexpr int r = decltype(Rr)::value;
                            if constexpr (r < M + 1) {
                                v[r] = src[r * w];
                            } else {
                                const float t = src[min(r, h - 1) * w];
                                v[r] = (r < h) ? t : 0.0f;
                            }
                        });
                    } else {
                        static_for<N>([&](auto Rr) {
                            constexpr int r = decltype(Rr)::value;
                            if constexpr (r < M) v[r] = (r < h) ? src[r * w] : 0.0f;
                            else v[r] = 0.0f;
                        });
                    }
                    rfft<N>(v, Xr, Xi);
                }
            } else {
                act = (c4 < w) && (g4 < gcount);
                if (act) {
                    const float* src = sIn + g4 * hw + c4;
                    auto quarter = [&](auto Q) {
                        constexpr int qq = decltype(Q)::value;
                        static_for<L>([&](auto J) {
                            constexpr int j = decltype(J)::value;
                            const float x0 = (j < h) ? src[j * w] : 0.0f;
                            const float x1 = (j + L < h) ? src[(j + L) * w] : 0.0f;
                            const float x2 = (j + 2 * L < h) ? src[(j + 2 * L) * w] : 0.0f;
                            const float x3 = (j + 3 * L < h) ? src[(j + 3 * L) * w] : 0.0f;
                            if constexpr (qq == 0) {
                                br[j] = (x0 + x2) + (x1 + x3); bi[j] = 0.0f;
                            } else if constexpr (qq == 2) {
                                const float t = (x0 + x2) - (x1 + x3);
                                br[j] = t * Tw<N, 2 * j>::c; bi[j] = -t * Tw<N, 2 * j>::s;
                            } else {
                                // d = (x0 - x2) -+ i (x1 - x3), times w_N^(qq j) = (c, -s)
                                const float dr = x0 - x2, di = (qq == 1) ? (x3 - x1) : (x1 - x3);
                                constexpr float c = Tw<N, qq * j>::c, sn = Tw<N, qq * j>::s;
                                br[j] = fc_fma(sn, di, c * dr);
                                bi[j] = fc_fma(-sn, dr, c * di);
                            }
                        });
                    };
                    if (q4 == 0) quarter(std::integral_constant<int, 0>{});
                    else if (q4 == 1) quarter(std::integral_constant<int, 1>{});
                    else if (q4 == 2) quarter(std::integral_constant<int, 2>{});
                    else quarter(std::integral_constant<int, 3>{});
                    cfft<L, false>(br, bi);             // br/bi[k] = X[ky = 4k + q4]
                }
            }
            if ((TMA || BSTG) && store_pending && (TMA ? is_storer : tid >= T - 32)) fk_bulk_wait_read();  // staging tile free again
            __syncthreads();   // tile consumed (and the previous tile's step 3 is done with sMid)
            if (!ALIAS) pending = (next < total_tiles) ? stage(second_n, row_n, tcol_n) : false;
            // Rows ky = 0 and ky = N/2 of a real column transform are real: they share the
            // scratch row 0 as (re, im) and are transformed together in step 3.
            if (!split4) {
                if (gA < gcount) {
                    float2* dst = sMid + gA * P + cA;
                    if (act) {
                        dst[0] = make_float2(Xr[0], Xr[M]);
                        static_for<M - 1>([&](auto Kk) {
                            constexpr int k = decltype(Kk)::value + 1;
                            dst[k * PW] = make_float2(Xr[k], Xi[k]);
                        });
                    } else if (!narrow) {
                        // idle lanes zero the columns past the plane, so that step 3 reads
                        // whole rows without a test per element
                        static_for<M>([&](auto Kk) {
                            constexpr int k = decltype(Kk)::value;
                            dst[k * PW] = make_float2(0.0f, 0.0f);
                        });
                    }
                }
            } else if (act) {
                float2* dst = sMid + g4 * P + c4 + q4 * PW;
                if (q4 == 0) bi[0] = br[L / 2];     // ky = N/2 sits at k = N/8 of quarter 0
                static_for<L>([&](auto Kk) {
                    constexpr int k = decltype(Kk)::value;
                    if (4 * k + q4 < M) dst[4 * k * PW] = make_float2(br[k], bi[k]);
                });
            }
        }
        __syncthreads();

        // 3. row transforms: thread = (half q, row kyp, plane gB)
        if (TMA || gB < gcount) {
            float ar[M], ai[M];
            const float2* rowp = sMid + gB * P + kyp * PW;
            const bool packed = (kyp == 0);
            auto load = [&](auto Cc) -> float2 { return rowp[decltype(Cc)::value]; };
            if (narrow) {
                // at most N/2 live columns: the other half of every butterfly is zero
                if (q == 0) load_split_narrow<N, false, 0>(load, w, ar, ai);
                else        load_split_narrow<N, false, 1>(load, w, ar, ai);
            } else {
                // every column of the scratch row is valid (zeros past the plane)
                if (q == 0) load_split<N, false, 0>(load, ar, ai);
                else        load_split<N, false, 1>(load, ar, ai);
            }
            if constexpr (TMA && SALIAS) __syncthreads();   // scratch consumed: it becomes the staging tile
            cfft<M, false>(ar, ai);                     // ar/ai[k] = F[kx = 2k+q]

            if constexpr (!BARE) {
                // element (part, bin = kx*NC + ky, plane g): staging offset (part*B + bin)*G + g,
                // global offset ((part*B + bin)*R + row)*ld + col
                float* o;
                size_t sb, sp;      // strides of one bin and of one part
                if constexpr (TMA) {
                    o = sStage + (q * NC + kyp) * G + gB;
                    sb = G; sp = (size_t)B * G;
                } else {
                    const size_t mat = (size_t)p.R * p.ld;
                    o = p.spec_out + (size_t)(q * NC + kyp) * mat + (size_t)row * p.ld + c0 + gB;
                    sb = mat; sp = (size_t)B * mat;
                }
                // With the TMA staging the packed row is written like any other row and taken
                // apart afterwards by the whole CTA (below): the lanes that hold it then do no
                // more work than the rest.
                if (WIDE_UNTANGLE || !packed) {
                    static_for<M>([&](auto Kk) {
                        constexpr int k = decltype(Kk)::value;
                        o[(size_t)(2 * k * NC) * sb] = ar[k];
                        o[(size_t)(2 * k * NC) * sb + sp] = ai[k];
                    });
                } else {
                    auto untangle = [&](auto Q) {
                        constexpr int qq = decltype(Q)::value;
                        static_for<M>([&](auto Kk) {
                            constexpr int k = decltype(Kk)::value;
                            constexpr int kp = (qq == 0) ? ((M - k) % M) : (M - 1 - k);
                            const float fr = ar[k], fi = ai[k], gr = ar[kp], gi = ai[kp];
                            float* o0 = o + (size_t)(2 * k * NC) * sb;      // row ky = 0
                            float* oN = o0 + (size_t)M * sb;                // row ky = N/2
                            o0[0] = 0.5f * (fr + gr);
                            o0[sp] = 0.5f * (fi - gi);
                            oN[0] = 0.5f * (fi + gi);
                            oN[sp] = 0.5f * (gr - fr);
                        });
                    };
                    if (q == 0) untangle(std::integral_constant<int, 0>{});
                    else        untangle(std::integral_constant<int, 1>{});
                }
            } else {
                // conventional half [ky][kx <= N/2]; the other rows come from the mirror bin
                float2* base = BSTG ? reinterpret_cast<float2*>(sStage) + gB * P2
                                    : reinterpret_cast<float2*>(p.spec_out) +
                                          ((size_t)row * p.C + c0 + gB) * (size_t)(N * NC);
                if (!packed) {
                    static_for<M>([&](auto Kk) {
                        constexpr int k = decltype(Kk)::value;
                        const int kx = 2 * k + q;
                        if (kx <= M) base[kyp * NC + kx] = make_float2(ar[k], ai[k]);
                        const int mx = (N - kx) & (N - 1);
                        if (mx <= M) base[(N - kyp) * NC + mx] = make_float2(ar[k], -ai[k]);
                    });
                } else {
                    auto untangle = [&](auto Q) {
                        constexpr int qq = decltype(Q)::value;
                        static_for<M>([&](auto Kk) {
                            constexpr int k = decltype(Kk)::value;
                            constexpr int kp = (qq == 0) ? ((M - k) % M) : (M - 1 - k);
                            constexpr int kx = 2 * k + qq;
                            if constexpr (kx <= M) {
                                const float fr = ar[k], fi = ai[k], gr = ar[kp], gi = ai[kp];
                                base[kx] = make_float2(0.5f * (fr + gr), 0.5f * (fi - gi));
                                base[M * NC + kx] = make_float2(0.5f * (fi + gi), 0.5f * (gr - fr));
                            }
                        });
                    };
                    if (q == 0) untangle(std::integral_constant<int, 0>{});
                    else        untangle(std::integral_constant<int, 1>{});
                }
            }
        }
        if constexpr (TMA) {
            // Row ky = 0 of every plane holds Z = FFT(X_0 + i X_{N/2}) of the two real rows:
            // X_0[k] = (Z_k + conj Z_{-k}) / 2,  X_{N/2}[k] = (Z_k - conj Z_{-k}) / (2i); one
            // (plane, k <= N/2) pair per thread, each touching only its own four bins.
            if constexpr (WIDE_UNTANGLE) {
            __syncthreads();
            for (int it = tid; it < G * (M + 1); it += T) {
                const int g = it % G, k = it / G, kp = (N - k) & (N - 1);
                float* a = sStage + g;
                const int ik = k * NC * G, ip = kp * NC * G;
                const float fr = a[ik], fi = a[B * G + ik], gr = a[ip], gi = a[B * G + ip];
                const float x0r = 0.5f * (fr + gr), x0i = 0.5f * (fi - gi);
                const float xnr = 0.5f * (fi + gi), xni = 0.5f * (gr - fr);
                a[ik] = x0r;          a[B * G + ik] = x0i;
                a[ip] = x0r;          a[B * G + ip] = -x0i;
                a[ik + M * G] = xnr;  a[B * G + ik + M * G] = xni;
                a[ip + M * G] = xnr;  a[B * G + ip + M * G] = -xni;
            }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncthreads();
            if (is_storer) {
                // one box per lane; columns beyond the matrix edge (ragged tile) are clipped
                // by the tensor map
                const int b0 = (tid & 31) * D;
                fk_tma_store_3d(tmS, fk_smem_u32(sStage + (size_t)b0 * G), c0, row, b0);
                fk_bulk_commit();
            }
            store_pending = true;
        }
        if constexpr (BSTG) {
            // the planes of the tile are contiguous in memory: one bulk copy per plane, issued
            // by the lanes of the last warp
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncthreads();
            if (tid >= T - 32 && (tid & 31) < gcount) {
                const int g = tid & 31;
                fk_bulk_s2g(reinterpret_cast<float2*>(p.spec_out) + ((size_t)row * p.C + c0 + g) * (size_t)(N * NC),
                            fk_smem_u32(reinterpret_cast<float2*>(sStage) + g * P2), (uint32_t)(N * NC * 8));
                fk_bulk_commit();
            }
            store_pending = true;
        }
        if (ALIAS) {
            if (!TMA) __syncthreads();   // step 3 done with the shared buffer before the next tile lands in it
            pending = (next < total_tiles) ? stage(second_n, row_n, tcol_n) : false;
            __syncthreads();
        }
    }
    if ((TMA || BSTG) && store_pending && (TMA ? is_storer : tid >= T - 32))
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// ---------------------------------------------------------------------------
// Inverse: half spectra -> cropped, scaled real planes.
// ---------------------------------------------------------------------------
// DB: two staging tiles, so that the load of the tile after the next one is issued as soon as
// a tile has been pulled into registers and the TMA never waits for the CTA (used where only
// one CTA is resident per SM and a tile's load takes longer than its arithmetic).
template <int N, int G, int LAYOUT, int MINB, bool WIN = false, bool DB = false>
__global__ void __launch_bounds__(N* G, MINB)
c2r_kernel(const __grid_constant__ CUtensorMap tmS, const FftParams p) {
    constexpr int T = N * G, NC = N / 2 + 1, M = N / 2, HALF = T / 2, B = N * NC;
    constexpr int PW = MidGeom<N, G>::PW, P = MidGeom<N, G>::P;
    constexpr bool TMA = (LAYOUT == LAYOUT_FREQ_TMA);
    constexpr bool BSTG = (LAYOUT == LAYOUT_BARE_STAGED);
    constexpr int P2 = BareGeom<N, G>::P2;
    constexpr int D = tma_bins_per_box(N);
    static_assert(!DB || TMA, "double-buffered staging needs the TMA layout");
    constexpr int STAGE_FLOATS = 2 * B * G;
    extern __shared__ __align__(128) unsigned char fc_smem[];
    float2* sMid = reinterpret_cast<float2*>(fc_smem);
    float* sStage0 = reinterpret_cast<float*>(fc_smem + MidGeom<N, G>::BYTES);
    float* sStage = sStage0;
    __shared__ __align__(8) unsigned long long bar_storage[2];
    const uint32_t bar0 = fk_smem_u32(&bar_storage[0]);
    uint32_t bar = bar0;

    const int tid = threadIdx.x;
    const int hc = p.h, wc = p.w, hw = hc * wc;
    const int gA = tid / N, cA = tid % N;                       // step 2: (plane, column), N lanes per plane
    const int q = tid / HALF, u = tid - q * HALF;               // step 1: (half, row ky, plane)
    const int kyp = u / G, gB = u - kyp * G;
    const bool packed = (kyp == 0);

    const int tpr = p.tiles_per_row;
    const int step_rows = gridDim.x / tpr, step_cols = gridDim.x - step_rows * tpr;
    auto advance = [&](int& row, int& tcol) {
        row += step_rows; tcol += step_cols;
        if (tcol >= tpr) { tcol -= tpr; ++row; }
    };
    // the last warp fetches the spectrum tiles: lane 0 arms the barrier, one TMA box per lane
    constexpr int NB = 2 * B / D;
    static_assert(!TMA || NB <= 32, "one lane per TMA box");
    const bool is_fetcher = (tid >= T - 32);
    auto fetch_into = [&](int row, int tcol, float* stage, uint32_t barrier) {   // whole last warp
        if ((tid & 31) == 0) fk_mbar_expect_tx(barrier, (uint32_t)(2 * B * G * 4));
        __syncwarp();
        if ((tid & 31) < NB) {
            const int b0 = (tid & 31) * D;
            fk_tma_load_3d(fk_smem_u32(stage + (size_t)b0 * G), &tmS, tcol * G, row, b0, barrier);
        }
    };
    auto fetch_tile = [&](int row, int tcol) { fetch_into(row, tcol, sStage, bar); };
    // bare layout, staged: the planes of a tile are contiguous in memory; one bulk copy per plane
    auto fetch_bare = [&](int row, int tcol) {                                   // whole last warp
        const int c0 = tcol * G, cnt = min(G, p.C - c0);
        if ((tid & 31) == 0) fk_mbar_expect_tx(bar0, (uint32_t)(cnt * N * NC * 8));
        __syncwarp();
        if ((tid & 31) < cnt) {
            const int g = tid & 31;
            fk_bulk_g2s(fk_smem_u32(reinterpret_cast<float2*>(sStage0) + g * P2),
                        reinterpret_cast<const float2*>(p.spec_in) + ((size_t)row * p.C + c0 + g) * (size_t)(N * NC),
                        (uint32_t)(N * NC * 8), bar0);
        }
    };
    uint32_t phase = 0;             // DB: bit b is the phase of buffer b's barrier
    int row = blockIdx.x / tpr, tcol = blockIdx.x - (blockIdx.x / tpr) * tpr;
    dep_trigger();
    if constexpr (TMA || BSTG) {
        if (tid == 0) {
            fk_mbar_init(bar0, 1);
            if (DB) fk_mbar_init(bar0 + 8u, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncthreads();
        dep_wait();                 // no global access above this line
        if constexpr (BSTG) {
            if (is_fetcher && blockIdx.x < p.num_tiles) fetch_bare(row, tcol);
        } else {
            if (is_fetcher && blockIdx.x < p.num_tiles) fetch_tile(row, tcol);
        }
        if constexpr (DB) {
            if (is_fetcher && blockIdx.x + gridDim.x < p.num_tiles) {
                int r1 = row, c1 = tcol;
                advance(r1, c1);
                fetch_into(r1, c1, sStage0 + STAGE_FLOATS, bar0 + 8u);
            }
        }
    } else {
        dep_wait();
    }
    int buf = 0;

    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x, advance(row, tcol)) {
        const int c0 = tcol * G;
        const int gcount = min(G, p.C - c0);
        int row_n = row, tcol_n = tcol;
        advance(row_n, tcol_n);

        // 1. row transforms (along kx): thread = (half q, row kyp, plane gB)
        float ar[M], ai[M];
        if constexpr (TMA) {
            if constexpr (DB) {
                sStage = sStage0 + buf * STAGE_FLOATS;
                bar = bar0 + 8u * (uint32_t)buf;
                if (!fk_wait_or_report(bar, (phase >> buf) & 1u, p.wait_cycles, p.status)) {
                    // never landed: before the CTA's shared memory is released, wait (bounded)
                    // for the load in flight into the other buffer as well
                    if (tile + (int)gridDim.x < p.num_tiles)
                        (void)fk_mbar_wait(bar0 + 8u * (uint32_t)(buf ^ 1), (phase >> (buf ^ 1)) & 1u, FK_WAIT_CYCLES);
                    return;
                }
                phase ^= (1u << buf);
            } else {
                if (!fk_wait_or_report(bar, phase, p.wait_cycles, p.status)) return;
                phase ^= 1u;
            }
            // Rows ky = 0 and ky = N/2 are real after the column pass, so they travel through
            // the row pass as one complex row Z = X_0 + i X_{N/2}.  For N <= 32 the whole CTA
            // forms Z in the staging tile first (one element per thread, one more barrier), so
            // that the two warps holding the packed rows do no more work than the others.
            constexpr bool WIDE_COMBINE = (N <= 64);
            if constexpr (WIDE_COMBINE) {
                // The two rows are Hermitian in kx, and their bins kx > N/2 are never read: the
                // thread of kx <= N/2 also forms Z[N - kx] = conj X_0[kx] + i conj X_{N/2}[kx]
                // (the contraction leaves those bins out, see GemmParams::herm_n).
                for (int it = tid; it < G * (M + 1); it += T) {
                    const int g = it % G, kx = it / G;
                    float* a = sStage + (size_t)kx * NC * G + g;
                    const float x0r = a[0], x0i = a[B * G], xnr = a[M * G], xni = a[(B + M) * G];
                    a[0] = x0r - xni;
                    a[B * G] = x0i + xnr;
                    if (kx > 0 && kx < M) {
                        float* m = sStage + (size_t)(N - kx) * NC * G + g;
                        m[0] = x0r + xni;
                        m[B * G] = xnr - x0i;
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // before the next TMA fill
                __syncthreads();
            }
            const float* sb = sStage + kyp * G + gB;
            auto load = [&](auto Kx) -> float2 {
                constexpr int kx = decltype(Kx)::value;
                float2 v = make_float2(sb[kx * NC * G], sb[(B + kx * NC) * G]);
                if (!WIDE_COMBINE && packed) {       // row ky = N/2 rides as i times itself
                    v.x -= sb[(B + kx * NC + M) * G];
                    v.y += sb[(kx * NC + M) * G];
                }
                return v;
            };
            if (q == 0) load_split<N, true, 0>(load, ar, ai);
            else        load_split<N, true, 1>(load, ar, ai);
            __syncthreads();        // staging tile consumed; previous tile's step 2 is done with sMid
            if constexpr (DB) {
                // this buffer takes the tile after the next one
                if (is_fetcher && tile + 2 * (int)gridDim.x < p.num_tiles) {
                    int r2 = row_n, c2 = tcol_n;
                    advance(r2, c2);
                    fetch_tile(r2, c2);
                }
                buf ^= 1;
            } else {
            if (is_fetcher && tile + (int)gridDim.x < p.num_tiles) fetch_tile(row_n, tcol_n);
            }
        } else if constexpr (BSTG) {
            if (!fk_wait_or_report(bar0, phase, p.wait_cycles, p.status)) return;
            phase ^= 1u;
            if (gB < gcount) {
                const float2* bbase = reinterpret_cast<const float2*>(sStage0) + gB * P2;
                auto load = [&](auto Kx) -> float2 {
                    constexpr int kx = decltype(Kx)::value;
                    // stored half: kx <= N/2; the other columns are mirror bins, conjugated
                    auto fetch = [&](int ky) -> float2 {
                        if (kx <= M) return bbase[ky * NC + kx];
                        float2 t = bbase[((N - ky) & (N - 1)) * NC + (N - kx)];
                        t.y = -t.y;
                        return t;
                    };
                    float2 v = fetch(kyp);
                    if (packed) {
                        const float2 nq = fetch(M);
                        v.x -= nq.y;
                        v.y += nq.x;
                    }
                    return v;
                };
                if (q == 0) load_split<N, true, 0>(load, ar, ai);
                else        load_split<N, true, 1>(load, ar, ai);
            }
            __syncthreads();        // planes in registers; previous tile's step 2 is done with sMid
            if (is_fetcher && tile + (int)gridDim.x < p.num_tiles) fetch_bare(row_n, tcol_n);
        } else {
            if (gB < gcount) {
                const size_t mat = (size_t)p.R * p.ld;
                const float* fbase = p.spec_in + (size_t)kyp * mat + (size_t)row * p.ld + c0 + gB;
                const float2* bbase = reinterpret_cast<const float2*>(p.spec_in) +
                                      ((size_t)row * p.C + c0 + gB) * (size_t)(N * NC);
                auto load = [&](auto Kx) -> float2 {
                    constexpr int kx = decltype(Kx)::value;
                    float2 v;
                    if constexpr (LAYOUT == LAYOUT_FREQ_DIRECT) {
                        const float* a = fbase + (size_t)(kx * NC) * mat;
                        v = make_float2(__ldg(a), __ldg(a + (size_t)B * mat));
                        if (packed) {
                            v.x -= __ldg(a + (size_t)(B + M) * mat);
                            v.y += __ldg(a + (size_t)M * mat);
                        }
                    } else {
                        auto fetch = [&](int ky) -> float2 {
                            if (kx <= M) return __ldg(bbase + ky * NC + kx);
                            float2 t = __ldg(bbase + ((N - ky) & (N - 1)) * NC + (N - kx));
                            t.y = -t.y;
                            return t;
                        };
                        v = fetch(kyp);
                        if (packed) {
                            const float2 nq = fetch(M);
                            v.x -= nq.y;
                            v.y += nq.x;
                        }
                    }
                    return v;
                };
                if (q == 0) load_split<N, true, 0>(load, ar, ai);
                else        load_split<N, true, 1>(load, ar, ai);
            }
            __syncthreads();        // previous tile's step 2 is done with sMid
        }
        if (TMA || gB < gcount) {
            cfft<M, true>(ar, ai);  // ar/ai[m] = value at column c = 2m+q
            // the packed row comes out as (row ky = 0, row ky = N/2) in (re, im): it stays
            // packed in scratch row 0 and step 2 takes it apart
            float2* dst = sMid + gB * P + kyp * PW + q;
            static_for<M>([&](auto Mm) {
                constexpr int m = decltype(Mm)::value;
                dst[2 * m] = make_float2(ar[m], ai[m]);
            });
        }
        __syncthreads();

        // 2. column transforms: thread = (plane gA, column cA), cA < wc; results go straight
        //    to global memory (lanes run along the row of the plane: contiguous segments)
        int win_hc = hc, win_wc = wc;
        size_t win_base = 0;
        if (WIN && p.win) {
            const int nt = p.nty * p.ntx;
            const int s = row / nt, t = row - s * nt;
            const int ty = t / p.ntx, tx = t - ty * p.ntx;
            win_hc = min(hc, p.H - ty * p.step_y);
            win_wc = min(wc, p.W - tx * p.step_x);
            win_base = ((size_t)s * p.C + c0 + gA) * ((size_t)p.H * p.W) +
                       (size_t)(ty * p.step_y) * p.W + tx * p.step_x;
        }
        if (gA < gcount && ((WIN && p.win) ? (cA >= p.ox && cA < p.ox + win_wc) : (cA < wc))) {
            float v[N];
            {
                float Xr[NC], Xi[NC];
                const float2* src = sMid + gA * P + cA;
                static_for<M>([&](auto Kk) {
                    constexpr int k = decltype(Kk)::value;
                    const float2 t = src[k * PW];
                    if constexpr (k == 0) {
                        Xr[0] = t.x; Xi[0] = 0.0f; Xr[M] = t.y; Xi[M] = 0.0f;
                    } else {
                        Xr[k] = t.x; Xi[k] = t.y;
                    }
                });
                irfft<N>(Xr, Xi, v);
            }
            // the crop is the first hc rows.  One running pointer and one predicated store
            // per row: written as PTX so that the row test stays a predicate (the compiler
            // otherwise builds a branch and fresh 64-bit address arithmetic per row)
            float* dst = p.real_out + ((size_t)row * p.C + c0 + gA) * hw + cA;
            const float scale = p.scale;
            if (WIN && p.win) {
                // rows [oy, oy + win_hc) of the transform go to the tile's place in the plane
                dst = p.real_out + win_base + (cA - p.ox);
                const bool acc = p.accumulate != 0;
                const int r0 = p.oy, r1 = p.oy + win_hc, pitch = p.W;
                static_for<N>([&](auto Rr) {
                    constexpr int r = decltype(Rr)::value;
                    if (r >= r0 && r < r1) {
                        float o = v[r] * scale;
                        if (acc) o += *dst;
                        *dst = o;
                        dst += pitch;
                    }
                });
            } else if (!p.accumulate && 2 * hc > N) {
                static_for<N>([&](auto Rr) {
                    constexpr int r = decltype(Rr)::value;
                    asm volatile(
                        "{\n\t.reg .pred p;\n\t"
                        "setp.lt.s32 p, %2, %3;\n\t"
                        "@p st.global.f32 [%0], %1;\n\t}"
                        ::"l"(dst), "f"(v[r] * scale), "r"(r), "r"(hc) : "memory");
                    dst += wc;
                });
            } else {
                // short crops (filter gradients) and accumulation: a uniform branch per row
                const bool acc = p.accumulate != 0;
                static_for<N>([&](auto Rr) {
                    constexpr int r = decltype(Rr)::value;
                    if (r < hc) {
                        float o = v[r] * scale;
                        if (acc) o += *dst;
                        *dst = o;
                        dst += wc;
                    }
                });
            }
        }
    }
}

// ---------------------------------------------------------------------------
// Host-side launchers.
// ---------------------------------------------------------------------------
template <int N> struct FftCfg;   // planes per CTA, buffer aliasing, min CTAs per SM, TMA staging
template <> struct FftCfg<8>   { static constexpr int G = 32; static constexpr bool ALIAS = false, SALIAS = true;  static constexpr int MINB = 4, MINB_INV = 4; static constexpr bool TMA = true; };
template <> struct FftCfg<16>  { static constexpr int G = 16; static constexpr bool ALIAS = false, SALIAS = false;  static constexpr int MINB = 4, MINB_INV = 4; static constexpr bool TMA = true; };
template <> struct FftCfg<32>  { static constexpr int G = 8;  static constexpr bool ALIAS = false, SALIAS = false;  static constexpr int MINB = 2, MINB_INV = 3; static constexpr bool TMA = true; };
template <> struct FftCfg<64>  { static constexpr int G = 4;  static constexpr bool ALIAS = false, SALIAS = false; static constexpr int MINB = 1, MINB_INV = 1; static constexpr bool TMA = true; };
template <> struct FftCfg<128> { static constexpr int G = 2;  static constexpr bool ALIAS = true,  SALIAS = false; static constexpr int MINB = 1, MINB_INV = 1; static constexpr bool TMA = false; };

// SM count of the current device (0 on failure); looked up once per device ordinal.
static inline int fft_sm_count() {
    static std::atomic<int> sms[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    const bool slot = dev >= 0 && dev < 64;
    int v = slot ? sms[dev].load(std::memory_order_relaxed) : 0;
    if (v == 0) {
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        if (slot) sms[dev].store(v, std::memory_order_relaxed);
    }
    return v;
}

// Grid of a persistent kernel: one CTA per resident slot.  The attribute call and the
// occupancy query cost microseconds of host time each, so their result is remembered per
// (kernel, shared-memory size).
static cudaError_t persistent_grid(const void* kern, int threads, size_t smem, long long tiles,
                                   int* grid) {
    struct Entry { const void* kern; size_t smem; int dev; int per_sm; };
    struct Limit { const void* kern; int dev; size_t max_smem; };
    static Entry cache[128];
    static Limit limits[64];
    static int cached = 0, nlimits = 0;
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    // the opt-in shared-memory limit of a kernel is only ever raised
    Limit* lim = nullptr;
    for (int i = 0; i < nlimits; ++i)
        if (limits[i].kern == kern && limits[i].dev == dev) lim = &limits[i];
    if (!lim || lim->max_smem < smem) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (lim) lim->max_smem = smem;
        else if (nlimits < 64) limits[nlimits++] = Limit{kern, dev, smem};
    }
    int per_sm = 0;
    for (int i = 0; i < cached; ++i)
        if (cache[i].kern == kern && cache[i].smem == smem && cache[i].dev == dev) {
            per_sm = cache[i].per_sm;
            break;
        }
    if (per_sm == 0) {
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, smem);
        if (e != cudaSuccess) return e;
        if (per_sm < 1) return cudaErrorInvalidConfiguration;
        if (cached < 128) cache[cached++] = Entry{kern, smem, dev, per_sm};
    }
    const int sms = fft_sm_count();
    if (sms < 1) return cudaErrorInvalidConfiguration;
    const long long slots = (long long)per_sm * sms;
    *grid = (int)(tiles < slots ? tiles : slots);
    return cudaSuccess;
}

// Tensor map of a planar spectrum for the staging tiles: box = G columns x 1 row x D bins.
template <int N, int G>
static bool make_spec_map(CUtensorMap* tm, const float* spec, const FftParams& p) {
    return tc_make_map(tm, spec, N * (N / 2 + 1), p.R, p.C, p.ld, G, 1, CU_TENSOR_MAP_SWIZZLE_NONE,
                       tma_bins_per_box(N));
}

template <int G>
static bool fill_tiling(FftParams& p) {
    p.tiles_per_row = (p.C + G - 1) / G;
    const long long tiles = (long long)p.R * p.tiles_per_row;
    if (tiles <= 0 || tiles > 0x3fffffffLL) return false;
    p.num_tiles = (int)tiles;
    return true;
}

// Forward transform of one operand, or of two operands in one launch (pb may be null).
template <int N, int LAYOUT>
static cudaError_t launch_r2c_layout(FftParams pa, const FftParams* pb_in, cudaStream_t st) {
    using Cfg = FftCfg<N>;
    constexpr int G = Cfg::G;
    FftParams pb{};
    if (!fill_tiling<G>(pa)) return cudaErrorInvalidValue;
    int in_bytes = real_tile_bytes(G, pa.h, pa.w);
    if (pb_in) {
        pb = *pb_in;
        if (!fill_tiling<G>(pb)) return cudaErrorInvalidValue;
        const int b = real_tile_bytes(G, pb.h, pb.w);
        if (b > in_bytes) in_bytes = b;
    }
    pa.in_bytes = pb.in_bytes = in_bytes;
    const size_t mid = MidGeom<N, G>::BYTES;
    size_t smem = Cfg::ALIAS ? (mid > (size_t)in_bytes ? mid : (size_t)in_bytes) : mid + (size_t)in_bytes;
    CUtensorMap tma, tmb;
    memset(&tma, 0, sizeof(tma));
    memset(&tmb, 0, sizeof(tmb));
    constexpr bool SALIAS = Cfg::SALIAS && LAYOUT == LAYOUT_FREQ_TMA;
    if (LAYOUT == LAYOUT_FREQ_TMA) {
        const size_t stage = (size_t)2 * N * (N / 2 + 1) * G * sizeof(float);
        if (SALIAS) smem = (size_t)in_bytes + (stage > mid ? stage : mid);
        else smem += stage;
        if (!make_spec_map<N, G>(&tma, pa.spec_out, pa)) return cudaErrorInvalidValue;
        if (pb_in && !make_spec_map<N, G>(&tmb, pb.spec_out, pb)) return cudaErrorInvalidValue;
    }
    if (LAYOUT == LAYOUT_BARE_STAGED) smem += BareGeom<N, G>::BYTES;
    // the windowed variant (spatial tiling) is a separate instantiation, so that the plain
    // kernels carry none of its code
    const bool win = pa.win || (pb_in && pb.win);
    auto kern = (win && LAYOUT == LAYOUT_FREQ_TMA) ? r2c_kernel<N, G, LAYOUT, Cfg::ALIAS, SALIAS, Cfg::MINB, LAYOUT == LAYOUT_FREQ_TMA>
                                                   : r2c_kernel<N, G, LAYOUT, Cfg::ALIAS, SALIAS, Cfg::MINB, false>;
    if (win && LAYOUT != LAYOUT_FREQ_TMA) return cudaErrorInvalidValue;
    int grid = 0;
    cudaError_t e = persistent_grid(reinterpret_cast<const void*>(kern), N * G, smem,
                                    (long long)pa.num_tiles + pb.num_tiles, &grid);
    if (e != cudaSuccess) return e;
    return dep_launch(false, kern, dim3(grid), dim3(N * G), smem, st, tma, tmb, pa, pb);
}

// Bare layout: staged through shared memory with bulk copies where a tile with its staging
// image fits (n <= 64) and the spectrum is 16-byte aligned, else accessed by the threads.
template <int N, bool FREQ>
static cudaError_t launch_r2c_n(const FftParams& pa, const FftParams* pb_in, cudaStream_t st) {
    using Cfg = FftCfg<N>;
    if constexpr (FREQ) {
        return launch_r2c_layout<N, Cfg::TMA ? LAYOUT_FREQ_TMA : LAYOUT_FREQ_DIRECT>(pa, pb_in, st);
    } else {
        if constexpr (N <= 64) {
            if ((reinterpret_cast<uintptr_t>(pa.spec_out) & 15) == 0)
                return launch_r2c_layout<N, LAYOUT_BARE_STAGED>(pa, pb_in, st);
        }
        return launch_r2c_layout<N, LAYOUT_BARE>(pa, pb_in, st);
    }
}

// Plane sizes whose inverse transform double-buffers its staging tile.
// Measured on B200: n = 64 (one resident CTA) 76-79 -> 72 us on the large-kernel layer, n = 16 44 -> 41 us
// on the deep layer's accGrad; n = 32 loses a resident CTA to the second tile and gains nothing.
template <int N> struct C2rDoubleBuffer { static constexpr bool value = (N == 64 || N == 16); };

template <int N, int LAYOUT>
static cudaError_t launch_c2r_layout(FftParams p, cudaStream_t st) {
    using Cfg = FftCfg<N>;
    constexpr int G = Cfg::G;
    constexpr bool DB = C2rDoubleBuffer<N>::value && LAYOUT == LAYOUT_FREQ_TMA;
    if (!fill_tiling<G>(p)) return cudaErrorInvalidValue;
    p.in_bytes = 0;
    size_t smem = MidGeom<N, G>::BYTES;
    CUtensorMap tm;
    memset(&tm, 0, sizeof(tm));
    if (LAYOUT == LAYOUT_FREQ_TMA) {
        smem += (size_t)(DB ? 2 : 1) * 2 * N * (N / 2 + 1) * G * sizeof(float);
        if (!make_spec_map<N, G>(&tm, p.spec_in, p)) return cudaErrorInvalidValue;
    }
    if (LAYOUT == LAYOUT_BARE_STAGED) smem += BareGeom<N, G>::BYTES;
    if (p.win && LAYOUT != LAYOUT_FREQ_TMA) return cudaErrorInvalidValue;
    auto kern = (p.win && LAYOUT == LAYOUT_FREQ_TMA) ? c2r_kernel<N, G, LAYOUT, Cfg::MINB_INV, LAYOUT == LAYOUT_FREQ_TMA, DB>
                                                     : c2r_kernel<N, G, LAYOUT, Cfg::MINB_INV, false, DB>;
    int grid = 0;
    cudaError_t e = persistent_grid(reinterpret_cast<const void*>(kern), N * G, smem, p.num_tiles, &grid);
    if (e != cudaSuccess) return e;
    return dep_launch(p.overlap != 0, kern, dim3(grid), dim3(N * G), smem, st, tm, p);
}

template <int N, bool FREQ>
static cudaError_t launch_c2r_n(const FftParams& p, cudaStream_t st) {
    using Cfg = FftCfg<N>;
    if constexpr (FREQ) {
        return launch_c2r_layout<N, Cfg::TMA ? LAYOUT_FREQ_TMA : LAYOUT_FREQ_DIRECT>(p, st);
    } else {
        if constexpr (N <= 64) {
            if ((reinterpret_cast<uintptr_t>(p.spec_in) & 15) == 0)
                return launch_c2r_layout<N, LAYOUT_BARE_STAGED>(p, st);
        }
        return launch_c2r_layout<N, LAYOUT_BARE>(p, st);
    }
}

template <bool FREQ>
static cudaError_t launch_r2c(int n, const FftParams& p, const FftParams* second, cudaStream_t st) {
    switch (n) {
        case 8:   return launch_r2c_n<8, FREQ>(p, second, st);
        case 16:  return launch_r2c_n<16, FREQ>(p, second, st);
        case 32:  return launch_r2c_n<32, FREQ>(p, second, st);
        case 64:  return launch_r2c_n<64, FREQ>(p, second, st);
        case 128: return launch_r2c_n<128, FREQ>(p, second, st);
    }
    return cudaErrorInvalidValue;
}
template <bool FREQ>
static cudaError_t launch_c2r(int n, const FftParams& p, cudaStream_t st) {
    switch (n) {
        case 8:   return launch_c2r_n<8, FREQ>(p, st);
        case 16:  return launch_c2r_n<16, FREQ>(p, st);
        case 32:  return launch_c2r_n<32, FREQ>(p, st);
        case 64:  return launch_c2r_n<64, FREQ>(p, st);
        case 128: return launch_c2r_n<128, FREQ>(p, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace fc
