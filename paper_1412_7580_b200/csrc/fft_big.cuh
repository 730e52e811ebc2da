// 2-D R2C / C2R transforms for planes too large for the one-pass kernels
// (n = 128: the half spectrum of even two planes does not fit in shared memory
// beside the real tile and the staging tile).
//
// A CTA owns tiles of 8 adjacent planes, as in the one-pass kernels, so that a
// frequency bin still receives 8 consecutive floats (32 bytes) and the
// transposition BDHW -> HWBD of the paper's Table 1 still happens inside the TMA
// store (load).  The half spectrum between the two 1-D passes goes through a
// CTA-private scratch area in global memory, 512 KB per CTA, which the CTA
// rewrites for every tile: with one CTA per SM the scratch of the whole grid is
// about 76 MB and stays resident in the 126 MB L2, so it costs L2 bandwidth, not
// HBM bandwidth.
//
// A CTA is two teams of 256 threads, each with one 65 KB buffer; inside a phase
// the teams only synchronise among themselves (named barriers), so one team's
// copies overlap the other team's arithmetic.
//
// Forward, per tile:
//   A. planes alternate between the teams.  The real plane is copied into the
//      team's buffer (16-byte asynchronous copies); two threads per column pull
//      their samples into registers (one decimation-in-frequency step on the
//      loads: rfft_half_split), the copy of the team's next plane starts, and the
//      N/4-point register FFT with the thread-local Hermitian post-pass writes
//      rows ky = 0..N/2-1 of the half spectrum to the scratch, row 0 carrying the
//      two real rows ky = 0 and ky = N/2 as (re, im) (Section 5.2's border case);
//   B. chunks of 8 rows ky (x 8 planes = 64 rows) alternate between the teams.
//      The rows come back from the scratch by asynchronous copies, four threads
//      per row run the N-point complex FFT (one radix-4 decimation-in-frequency
//      step on the loads, N/4-point register FFT), the results overwrite the
//      buffer as a staging tile [part*N + kx][ky][plane] and one TMA store writes
//      the 4-D box (8 planes, 1 matrix row, 8 ky, 2N kx-and-part); the packed row
//      of chunk 0 is taken apart in the staging tile by the whole team.
// The inverse runs the same steps backwards (TMA loads, row transforms, scratch,
// column transforms by two threads with a decimation-in-time exchange through
// the team's buffer, cropped / scaled / accumulated stores).
#pragma once

#include "fft_kernels.cuh"

namespace fc {

constexpr int BIG_G = 8;          // planes per tile
constexpr int BIG_MAX_SMS = 160;  // scratch is sized for this many SMs

// teams per CTA and CTAs per SM the kernels are built for
template <int N> struct BigCfg;
template <> struct BigCfg<128> { static constexpr int NT = 2, MINB = 1; };
template <> struct BigCfg<64>  { static constexpr int NT = 4, MINB = 2; };

template <int N>
struct BigGeom {
    static constexpr int M = N / 2, NC = M + 1, L = N / 4, H = N / 4;
    static constexpr int TEAM = 2 * N;                           // threads per team
    static constexpr int ROWS = N / 2;                           // rows per chunk (four threads per row)
    static constexpr int KC = ROWS / BIG_G;                      // rows ky per chunk
    static constexpr int PITCH = N + 2;                          // float2 per row: 16-byte multiple, odd in 16-byte units
    static constexpr size_t INBUF = (size_t)ROWS * PITCH * 8;
    static constexpr size_t STAGE = (size_t)2 * N * ROWS * 4;
    static constexpr size_t STAGE_NY = (size_t)2 * N * BIG_G * 4;
    static constexpr size_t PLANE = (size_t)N * N * 4;
    static constexpr size_t SCRATCH_PER_CTA = (size_t)BIG_G * M * N * 8;
    static constexpr int NT = BigCfg<N>::NT;                     // teams per CTA
    static constexpr int THREADS = NT * TEAM;
    static constexpr size_t SMEM = NT * INBUF + STAGE_NY;      // one buffer per team + the ky = N/2 staging
    // The scratch kept in shared memory instead (n = 64: 132 KB, one CTA per SM): rows of N + 2 and
    // planes of M rows + 2 complex, so that both the rows of one plane and the same row of
    // adjacent planes start an odd number of 16-byte units apart (conflict-free 16-byte loads).
    static constexpr int SPITCH = N + 2;
    static constexpr int SPLANE = M * SPITCH + 2;
    static constexpr size_t SSCRATCH = (size_t)BIG_G * SPLANE * 8;
    static constexpr size_t SMEM_SS = SMEM + SSCRATCH;
    static_assert(PLANE <= INBUF && STAGE <= INBUF, "a team's buffer holds a plane, a chunk or a staging tile");
    static_assert((size_t)2 * H * N * 8 <= INBUF, "the exchange buffer fits a team's buffer");
    static_assert(TEAM == 4 * ROWS && KC >= 1 && M % KC == 0, "thread roles");
};

// n = 64: the scratch fits in shared memory (one CTA per SM); n = 128 needs the global area.
constexpr bool big_smem_scratch(int n) { return n == 64; }

static inline size_t big_scratch_bytes(int n) {
    if (n == 128) return (size_t)BIG_MAX_SMS * BigCfg<128>::MINB * BigGeom<128>::SCRATCH_PER_CTA;
    return 0;
}

// Planar spectrum [2][N][NC][R][ld] seen as a 4-D tensor (col, row, ky, part*N + kx):
// bin = kx*NC + ky and the parts are N*NC bins apart, so the last stride is uniform.
template <int N>
static bool big_make_map(CUtensorMap* map, const float* spec, const FftParams& p, int box_ky) {
    tc_encode_fn enc = tc_get_encode();
    if (!enc) return false;
    constexpr int NC = N / 2 + 1;
    const cuuint64_t mat = (cuuint64_t)p.R * p.ld * 4;
    cuuint64_t dims[4] = {(cuuint64_t)p.C, (cuuint64_t)p.R, (cuuint64_t)NC, (cuuint64_t)2 * N};
    cuuint64_t strides[3] = {(cuuint64_t)p.ld * 4, mat, mat * NC};
    cuuint32_t box[4] = {(cuuint32_t)BIG_G, 1u, (cuuint32_t)box_ky, (cuuint32_t)2 * N};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<float*>(spec), dims, strides, box,
               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

__device__ __forceinline__ void fk_tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1,
                                                int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
        ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void fk_tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1,
                                               int c2, int c3, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void fk_cp16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void big_st2(float2* a, float2 v) { *a = v; }
__device__ __forceinline__ void big_st4(float4* a, float4 v) { __stcg(a, v); }
__device__ __forceinline__ float2 big_ld2(const float2* a) { return __ldcg(a); }
template <int TEAM>
__device__ __forceinline__ void big_team_sync(int team) {
    asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "n"(TEAM) : "memory");
}
__device__ __forceinline__ void fk_cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void fk_cp_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory");
}

// Radix-4 split of a row whose elements sit as consecutive float2 in shared memory
// (16-byte aligned): two elements per 16-byte load.
template <int N, bool INV, int Q>
__device__ __forceinline__ void big_split4_rows(const float2* rowp, float (&ar)[N / 4], float (&ai)[N / 4]) {
    constexpr int L = N / 4;
    static_for<L / 2>([&](auto JJ) {
        constexpr int j = 2 * decltype(JJ)::value;
        const float4 v0 = *reinterpret_cast<const float4*>(rowp + j);
        const float4 v1 = *reinterpret_cast<const float4*>(rowp + j + L);
        const float4 v2 = *reinterpret_cast<const float4*>(rowp + j + 2 * L);
        const float4 v3 = *reinterpret_cast<const float4*>(rowp + j + 3 * L);
        split4_elem<N, INV, Q, j>(make_float2(v0.x, v0.y), make_float2(v1.x, v1.y), make_float2(v2.x, v2.y),
                                  make_float2(v3.x, v3.y), ar[j], ai[j]);
        split4_elem<N, INV, Q, j + 1>(make_float2(v0.z, v0.w), make_float2(v1.z, v1.w),
                                      make_float2(v2.z, v2.w), make_float2(v3.z, v3.w), ar[j + 1], ai[j + 1]);
    });
}

// ---------------------------------------------------------------------------
// Forward.
// ---------------------------------------------------------------------------
// SS: the scratch between the two 1-D passes lives in shared memory (fits for n = 64 with one
// CTA per SM) instead of the CTA-private global area; the row pass then reads it in place.
template <int N, bool SS>
__global__ void __launch_bounds__(BigGeom<N>::THREADS, SS ? 1 : BigCfg<N>::MINB)
r2c_big_kernel(const __grid_constant__ CUtensorMap tmS, const __grid_constant__ CUtensorMap tmNy,
               const FftParams p, float2* __restrict__ scratch_all) {
    using Gm = BigGeom<N>;
    constexpr int M = Gm::M, L = Gm::L, H = Gm::H, G = BIG_G, T = Gm::TEAM, NT = Gm::NT, KC = Gm::KC, PITCH = Gm::PITCH;
    constexpr int RS = SS ? Gm::SPITCH : N;                // scratch: complex per row
    constexpr int PS = SS ? Gm::SPLANE : M * N;            // scratch: complex per plane
    extern __shared__ __align__(128) unsigned char fc_smem[];
    float2* scratch;
    if constexpr (SS) scratch = reinterpret_cast<float2*>(fc_smem + Gm::SMEM);
    else scratch = scratch_all + (size_t)blockIdx.x * (G * M * N);

    const int team = threadIdx.x / T, tid = threadIdx.x - team * T;      // tid: index inside the team
    unsigned char* buf = fc_smem + (size_t)team * Gm::INBUF;            // the team's buffer
    float* sNy = reinterpret_cast<float*>(fc_smem + NT * Gm::INBUF);
    const int q2 = tid / N, cA = tid - q2 * N;             // step A: (half, column)
    const int q4 = tid / Gm::ROWS, rB = tid - q4 * Gm::ROWS;   // step B: (quarter, row = ky_local*8 + plane)
    const int h = p.h, w = p.w, hw = h * w;
    const int tpr = p.tiles_per_row;
    dep_trigger();
    dep_wait();                     // no global access above this line

    // copy of one real plane into the team's buffer
    auto issue_plane = [&](int row, int c0, int g) {
        const float* src = p.real_in + ((size_t)row * p.C + c0 + g) * hw;
        float* dst = reinterpret_cast<float*>(buf);
        if ((reinterpret_cast<uintptr_t>(src) & 15) == 0) {
            const int vec = hw >> 2;
            for (int i = tid; i < vec; i += T) fk_cp16(fk_smem_u32(dst + 4 * i), src + 4 * i);
            for (int i = 4 * vec + tid; i < hw; i += T) dst[i] = __ldg(src + i);
        } else {
            for (int i = tid; i < hw; i += T) dst[i] = __ldg(src + i);
        }
    };
    // copy of chunk `ci` (rows ky = 8 ci .. 8 ci + 7 of all planes) from the scratch
    auto issue_chunk = [&](int ci) {
        float2* dst = reinterpret_cast<float2*>(buf);
        constexpr int PER_ROW = N / 2;                     // 16-byte pieces per row
#pragma unroll 4
        for (int i = tid; i < Gm::ROWS * PER_ROW; i += T) {
            const int rr = i / PER_ROW, pc = i - rr * PER_ROW;
            const int g = rr & (G - 1), ky = ci * KC + (rr >> 3);
            fk_cp16(fk_smem_u32(dst + rr * PITCH + 2 * pc), scratch + ((size_t)(g * M + ky) * N + 2 * pc));
        }
    };

    bool store_pending = false;
    bool team_store_pending = false;        // SS: the team's last store may still be reading its buffer
    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
        const int row = tile / tpr, tcol = tile - row * tpr;
        const int c0 = tcol * G;
        const int gcount = min(G, p.C - c0);

        // ---- A: column transforms; planes team, team + NT, .. ----------------------------
        if constexpr (SS) {
            if (team_store_pending) {
                if (tid == 0) fk_bulk_wait_read();
                big_team_sync<T>(team);                       // the buffer takes a plane again
                team_store_pending = false;
            }
        }
        if (team < gcount) issue_plane(row, c0, team);
        fk_cp_commit();
        for (int g = team; g < gcount; g += NT) {
            fk_cp_wait<0>();
            big_team_sync<T>(team);                           // plane g has landed for the team
            const float* pl = reinterpret_cast<const float*>(buf) + cA;
            float ar[H], ai[H];
            const bool live = cA < w;
            if (live) {
                auto x = [&](auto Rr) -> float {
                    constexpr int r = decltype(Rr)::value;
                    return (r < h) ? pl[r * w] : 0.0f;
                };
                if (q2 == 0) rfft_half_split<N, 0>(x, ar, ai);
                else         rfft_half_split<N, 1>(x, ar, ai);
            }
            big_team_sync<T>(team);                           // plane g is in registers: the buffer takes the next one
            if (g + NT < gcount) issue_plane(row, c0, g + NT);
            fk_cp_commit();
            float2* dst = scratch + (size_t)g * PS + cA;
            auto put = [&](float2* a, float2 v) {
                if constexpr (SS) *a = v; else big_st2(a, v);
            };
            if (live) {
                if (q2 == 0) {
                    // bins k = 2i; rows ky = 0 and ky = N/2 are real and share row 0 as (re, im)
                    float x0 = 0.0f;
                    rfft_half_finish<N, 0>(ar, ai, [&](auto I, float re, float im) {
                        constexpr int i = decltype(I)::value;
                        if constexpr (i == 0) x0 = re;
                        else if constexpr (i == H) put(dst, make_float2(x0, re));
                        else put(dst + (size_t)(2 * i) * RS, make_float2(re, im));
                    });
                } else {
                    rfft_half_finish<N, 1>(ar, ai, [&](auto I, float re, float im) {
                        constexpr int i = decltype(I)::value;
                        put(dst + (size_t)(2 * i + 1) * RS, make_float2(re, im));
                    });
                }
            } else {
                static_for<H>([&](auto I) {
                    constexpr int i = decltype(I)::value;
                    put(dst + (size_t)(2 * i + q2) * RS, make_float2(0.0f, 0.0f));
                });
            }
        }
        fk_cp_wait<0>();
        __syncthreads();                                   // the scratch is complete

        // ---- B: row transforms; chunks team, team + NT, .. --------------------------------
        constexpr int CHUNKS = M / KC;
        for (int ci = team; ci < CHUNKS; ci += NT) {
            float ar[L], ai[L];
            const float2* rowp;
            if constexpr (SS) {
                // read the row in place: row rB of the chunk is (plane rB % 8, ky = ci KC + rB / 8)
                rowp = scratch + (size_t)(rB & (G - 1)) * PS + (size_t)(ci * KC + (rB >> 3)) * RS;
            } else {
                issue_chunk(ci);
                fk_cp_commit();
                fk_cp_wait<0>();
                big_team_sync<T>(team);                       // chunk ci has landed for the team
                rowp = reinterpret_cast<const float2*>(buf) + rB * PITCH;
            }
            if (q4 == 0)      big_split4_rows<N, false, 0>(rowp, ar, ai);
            else if (q4 == 1) big_split4_rows<N, false, 1>(rowp, ar, ai);
            else if (q4 == 2) big_split4_rows<N, false, 2>(rowp, ar, ai);
            else              big_split4_rows<N, false, 3>(rowp, ar, ai);
            if constexpr (SS) {
                // the rows were read in place; the team's buffer is still the previous staging
                // tile until its store has been read out
                if (tid == 0 && team_store_pending) fk_bulk_wait_read();
            }
            big_team_sync<T>(team);                           // the chunk is in registers: the buffer becomes the staging tile
            cfft<L, false>(ar, ai);                        // ar/ai[m] = F[kx = 4m + q4]
            float* sStage = reinterpret_cast<float*>(buf);
            float* o = sStage + q4 * Gm::ROWS + rB;
            static_for<L>([&](auto Mm) {
                constexpr int m = decltype(Mm)::value;
                o[(4 * m) * Gm::ROWS] = ar[m];
                o[(N + 4 * m) * Gm::ROWS] = ai[m];
            });
            if (ci == 0) {
                // row 0 of every plane holds Z = FFT(X_0 + i X_{N/2}); take it apart:
                // X_0[k] = (Z_k + conj Z_{-k}) / 2,  X_{N/2}[k] = (Z_k - conj Z_{-k}) / (2i)
                big_team_sync<T>(team);
                for (int it = tid; it < G * (M + 1); it += T) {
                    const int g = it & (G - 1), k = it >> 3, kp = (N - k) & (N - 1);
                    float* a = sStage + g;                 // ky_local = 0: row index = plane
                    const float fr = a[k * Gm::ROWS], fi = a[(N + k) * Gm::ROWS];
                    const float gr = a[kp * Gm::ROWS], gi = a[(N + kp) * Gm::ROWS];
                    const float x0r = 0.5f * (fr + gr), x0i = 0.5f * (fi - gi);
                    const float xnr = 0.5f * (fi + gi), xni = 0.5f * (gr - fr);
                    a[k * Gm::ROWS] = x0r;  a[(N + k) * Gm::ROWS] = x0i;
                    a[kp * Gm::ROWS] = x0r; a[(N + kp) * Gm::ROWS] = -x0i;
                    float* b = sNy + g;
                    b[k * G] = xnr;  b[(N + k) * G] = xni;
                    b[kp * G] = xnr; b[(N + kp) * G] = -xni;
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            big_team_sync<T>(team);
            if (tid == 0) {
                fk_tma_store_4d(&tmS, fk_smem_u32(sStage), c0, row, ci * KC, 0);
                if (ci == 0) fk_tma_store_4d(&tmNy, fk_smem_u32(sNy), c0, row, M, 0);
                fk_bulk_commit();
                if constexpr (!SS) fk_bulk_wait_read();    // the buffer may be overwritten after this
            }
            store_pending = true;
            team_store_pending = true;
            if constexpr (!SS) big_team_sync<T>(team);
        }
        __syncthreads();                                   // both teams are done with the scratch
    }
    if (tid == 0 && store_pending) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// ---------------------------------------------------------------------------
// Inverse.
// ---------------------------------------------------------------------------
template <int N, bool SS>
__global__ void __launch_bounds__(BigGeom<N>::THREADS, SS ? 1 : BigCfg<N>::MINB)
c2r_big_kernel(const __grid_constant__ CUtensorMap tmS, const __grid_constant__ CUtensorMap tmNy,
               const FftParams p, float2* __restrict__ scratch_all) {
    using Gm = BigGeom<N>;
    constexpr int M = Gm::M, L = Gm::L, H = Gm::H, G = BIG_G, T = Gm::TEAM, NT = Gm::NT, KC = Gm::KC, PITCH = Gm::PITCH;
    constexpr int RS = SS ? Gm::SPITCH : N;
    constexpr int PS = SS ? Gm::SPLANE : M * N;
    extern __shared__ __align__(128) unsigned char fc_smem[];
    __shared__ __align__(8) unsigned long long bar_storage[NT];
    float2* scratch;
    if constexpr (SS) scratch = reinterpret_cast<float2*>(fc_smem + Gm::SMEM);
    else scratch = scratch_all + (size_t)blockIdx.x * (G * M * N);

    const int team = threadIdx.x / T, tid = threadIdx.x - team * T;
    unsigned char* buf = fc_smem + (size_t)team * Gm::INBUF;
    float* sNy = reinterpret_cast<float*>(fc_smem + NT * Gm::INBUF);
    const uint32_t bar = fk_smem_u32(&bar_storage[team]);
    const int q2 = tid / N, cA = tid - q2 * N;
    const int q4 = tid / Gm::ROWS, rB = tid - q4 * Gm::ROWS;
    const int hc = p.h, wc = p.w, hw = hc * wc;
    const int tpr = p.tiles_per_row;
    const float scale = p.scale;
    const bool acc = p.accumulate != 0;
    constexpr int CHUNKS = M / KC;

    dep_trigger();
    if (tid == 0) {
        fk_mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    dep_wait();                     // no global access above this line
    uint32_t phase = 0u;
    bool dead = false;          // a load never landed: keep walking through the barriers, stop waiting

    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
        const int row = tile / tpr, tcol = tile - row * tpr;
        const int c0 = tcol * G;
        const int gcount = min(G, p.C - c0);

        // ---- B: row transforms; chunks team, team + NT, .. --------------------------------
        for (int ci = team; ci < CHUNKS; ci += NT) {
            if (tid == 0) {
                fk_mbar_expect_tx(bar, (uint32_t)(Gm::STAGE + (ci == 0 ? Gm::STAGE_NY : 0)));
                fk_tma_load_4d(fk_smem_u32(buf), &tmS, c0, row, ci * KC, 0, bar);
                if (ci == 0) fk_tma_load_4d(fk_smem_u32(sNy), &tmNy, c0, row, M, 0, bar);
            }
            if (!dead && !fk_wait_or_report(bar, phase, p.wait_cycles, p.status)) dead = true;
            phase ^= 1u;
            float* st = reinterpret_cast<float*>(buf);
            if (ci == 0) {
                // row 0 becomes X_0 + i X_{N/2}: one complex row that carries both real rows
                for (int it = tid; it < G * N; it += T) {
                    const int g = it & (G - 1), kx = it >> 3;
                    const float a = st[kx * Gm::ROWS + g], b = st[(N + kx) * Gm::ROWS + g];
                    const float c = sNy[kx * G + g], d = sNy[(N + kx) * G + g];
                    st[kx * Gm::ROWS + g] = a - d;
                    st[(N + kx) * Gm::ROWS + g] = b + c;
                }
                big_team_sync<T>(team);
            }
            float ar[L], ai[L];
            {
                const float* sb = st + rB;
                auto load = [&](auto Kx) -> float2 {
                    constexpr int kx = decltype(Kx)::value;
                    return make_float2(sb[kx * Gm::ROWS], sb[(N + kx) * Gm::ROWS]);
                };
                if (q4 == 0)      load_split4<N, true, 0>(load, ar, ai);
                else if (q4 == 1) load_split4<N, true, 1>(load, ar, ai);
                else if (q4 == 2) load_split4<N, true, 2>(load, ar, ai);
                else              load_split4<N, true, 3>(load, ar, ai);
            }
            big_team_sync<T>(team);                           // staging tile in registers: the buffer takes the rows
            cfft<L, true>(ar, ai);                         // ar/ai[m] = value at column 4m + q4
            if constexpr (SS) {
                // straight into the shared-memory scratch: row rB is (plane rB % 8, ky = ci KC + rB / 8)
                float2* dst = scratch + (size_t)(rB & (G - 1)) * PS + (size_t)(ci * KC + (rB >> 3)) * RS + q4;
                static_for<L>([&](auto Mm) {
                    constexpr int m = decltype(Mm)::value;
                    dst[4 * m] = make_float2(ar[m], ai[m]);
                });
            } else {
            float2* sRows = reinterpret_cast<float2*>(buf);
            float2* dst = sRows + rB * PITCH + q4;
            static_for<L>([&](auto Mm) {
                constexpr int m = decltype(Mm)::value;
                dst[4 * m] = make_float2(ar[m], ai[m]);
            });
            big_team_sync<T>(team);
            constexpr int PER_ROW = N / 2;
#pragma unroll 4
            for (int i = tid; i < Gm::ROWS * PER_ROW; i += T) {
                const int rr = i / PER_ROW, pc = i - rr * PER_ROW;
                const int g = rr & (G - 1), ky = ci * KC + (rr >> 3);
                const float4 v = *reinterpret_cast<const float4*>(sRows + rr * PITCH + 2 * pc);
                big_st4(reinterpret_cast<float4*>(scratch + ((size_t)(g * M + ky) * N + 2 * pc)), v);
            }
            big_team_sync<T>(team);                           // the buffer is free for the next chunk
            }
        }
        __syncthreads();                                   // the scratch is complete for this CTA

        // ---- A: column transforms; planes team, team + NT, .. ------------------------------
        float2* sX = reinterpret_cast<float2*>(buf);
        for (int g = team; g < gcount; g += NT) {
            float er[H], ei[H];
            const float2* src = scratch + (size_t)g * PS + cA;
            auto X = [&](auto K) -> float2 {
                constexpr int k = decltype(K)::value;
                if constexpr (SS) return src[(size_t)k * RS];
                else return big_ld2(src + (size_t)k * N);
            };
            if (q2 == 0) irfft_half<N, 0>(X, er, ei);
            else         irfft_half<N, 1>(X, er, ei);
            float2* mine = sX + (size_t)q2 * (H * N) + cA;
            const float2* other = sX + (size_t)(1 - q2) * (H * N) + cA;
            static_for<H>([&](auto J) {
                constexpr int j = decltype(J)::value;
                mine[j * N] = make_float2(er[j], ei[j]);
            });
            big_team_sync<T>(team);
            if (cA < wc) {
                float* out = p.real_out + ((size_t)row * p.C + c0 + g) * hw + cA;
                // z_j = E_j + O'_j (rows 2j, 2j+1),  z_{j+H} = E_j - O'_j (rows N/2 + 2j, ...)
                static_for<H>([&](auto J) {
                    constexpr int j = decltype(J)::value;
                    const float2 t = other[j * N];
                    // q2 = 0 holds E and reads O'; q2 = 1 holds O' and reads E
                    const float zr = (q2 == 0) ? er[j] + t.x : t.x - er[j];
                    const float zi = (q2 == 0) ? ei[j] + t.y : t.y - ei[j];
                    const int r0 = q2 * M + 2 * j;
                    if (r0 < hc) {
                        float* o = out + (size_t)r0 * wc;
                        float v = zr * scale;
                        if (acc) v += *o;
                        *o = v;
                    }
                    if (r0 + 1 < hc) {
                        float* o = out + (size_t)(r0 + 1) * wc;
                        float v = zi * scale;
                        if (acc) v += *o;
                        *o = v;
                    }
                });
            }
            big_team_sync<T>(team);                           // exchange buffer free for the next plane
        }
        __syncthreads();                                   // both teams are done with the scratch
    }
}

// ---------------------------------------------------------------------------
// Launchers.
// ---------------------------------------------------------------------------
template <int N>
static cudaError_t launch_r2c_big(FftParams p, float* scratch, size_t scratch_bytes, cudaStream_t st) {
    using Gm = BigGeom<N>;
    if (!fill_tiling<BIG_G>(p)) return cudaErrorInvalidValue;
    CUtensorMap tm, tmny;
    memset(&tm, 0, sizeof(tm));
    memset(&tmny, 0, sizeof(tmny));
    if (!big_make_map<N>(&tm, p.spec_out, p, Gm::KC) || !big_make_map<N>(&tmny, p.spec_out, p, 1))
        return cudaErrorInvalidValue;
    int grid = 0;
    if constexpr (big_smem_scratch(N)) {
        (void)scratch; (void)scratch_bytes;
        auto kern = r2c_big_kernel<N, true>;
        cudaError_t e = persistent_grid(reinterpret_cast<const void*>(kern), Gm::THREADS, Gm::SMEM_SS, p.num_tiles, &grid);
        if (e != cudaSuccess) return e;
        return dep_launch(false, kern, dim3(grid), dim3(Gm::THREADS), Gm::SMEM_SS, st, tm, tmny, p, (float2*)nullptr);
    } else {
    auto kern = r2c_big_kernel<N, false>;
    cudaError_t e = persistent_grid(reinterpret_cast<const void*>(kern), Gm::THREADS, Gm::SMEM, p.num_tiles, &grid);
    if (e != cudaSuccess) return e;
    const long long fit = (long long)(scratch_bytes / Gm::SCRATCH_PER_CTA);
    if (fit < 1) return cudaErrorInvalidValue;
    if (grid > fit) grid = (int)fit;
    return dep_launch(false, kern, dim3(grid), dim3(Gm::THREADS), Gm::SMEM, st, tm, tmny, p, reinterpret_cast<float2*>(scratch));
    }
}

template <int N>
static cudaError_t launch_c2r_big(FftParams p, float* scratch, size_t scratch_bytes, cudaStream_t st) {
    using Gm = BigGeom<N>;
    if (!fill_tiling<BIG_G>(p)) return cudaErrorInvalidValue;
    CUtensorMap tm, tmny;
    memset(&tm, 0, sizeof(tm));
    memset(&tmny, 0, sizeof(tmny));
    if (!big_make_map<N>(&tm, p.spec_in, p, Gm::KC) || !big_make_map<N>(&tmny, p.spec_in, p, 1))
        return cudaErrorInvalidValue;
    int grid = 0;
    if constexpr (big_smem_scratch(N)) {
        (void)scratch; (void)scratch_bytes;
        auto kern = c2r_big_kernel<N, true>;
        cudaError_t e = persistent_grid(reinterpret_cast<const void*>(kern), Gm::THREADS, Gm::SMEM_SS, p.num_tiles, &grid);
        if (e != cudaSuccess) return e;
        return dep_launch(false, kern, dim3(grid), dim3(Gm::THREADS), Gm::SMEM_SS, st, tm, tmny, p, (float2*)nullptr);
    } else {
    auto kern = c2r_big_kernel<N, false>;
    constexpr size_t SMEM = Gm::SMEM;
    cudaError_t e = persistent_grid(reinterpret_cast<const void*>(kern), Gm::THREADS, SMEM, p.num_tiles, &grid);
    if (e != cudaSuccess) return e;
    const long long fit = (long long)(scratch_bytes / Gm::SCRATCH_PER_CTA);
    if (fit < 1) return cudaErrorInvalidValue;
    if (grid > fit) grid = (int)fit;
    return dep_launch(false, kern, dim3(grid), dim3(Gm::THREADS), SMEM, st, tm, tmny, p, reinterpret_cast<float2*>(scratch));
    }
}

// Which plane sizes take the two-pass kernels.  (They are also instantiated for n = 64, with
// the scratch in shared memory; measured slower there than the one-pass kernels, so not used.)
static inline bool big_uses_two_pass(int n) { return n == 128; }
static cudaError_t launch_r2c_two_pass(int n, const FftParams& p, float* scratch, size_t bytes, cudaStream_t st) {
    return n == 128 ? launch_r2c_big<128>(p, scratch, bytes, st) : launch_r2c_big<64>(p, scratch, bytes, st);
}
static cudaError_t launch_c2r_two_pass(int n, const FftParams& p, float* scratch, size_t bytes, cudaStream_t st) {
    return n == 128 ? launch_c2r_big<128>(p, scratch, bytes, st) : launch_c2r_big<64>(p, scratch, bytes, st);
}

}  // namespace fc
