// Sub-batched variant of the one-pass forward 2-D transform, for the plane size at which a tile
// of planes that fits shared memory is too narrow for the memory system (n = 64).
//
// The frequency-major spectrum receives, per (part, bin), one row of as many floats as the
// tile has planes.  At n = 64 the plain kernels can hold 4 planes per CTA (real tile, half-
// spectrum scratch and staging tile together), i.e. rows of 16 bytes -- half a 32-byte
// sector, and the memory system retires such requests at the same rate as 32-byte ones.
// Here a CTA still works on 4 planes at a time, but the staging tile is 8 planes wide: two
// sub-batches of 4 planes go through the two 1-D passes one after the other and fill the
// halves of the staging tile, which then leaves as rows of 32 bytes.  To make room, the
// half-spectrum scratch overwrites the real tile once the column pass has pulled it into
// registers, and the next sub-batch's planes are requested as soon as the row pass has pulled
// the scratch into registers.  (Measured on B200, large-kernel layer: forward transform of x
// 88 -> 79 us.  The inverse transform does not gain from the same arrangement: one staging
// tile of 8 planes leaves no room for a second one, and it loses more by waiting for its
// single tile than the longer rows return -- 80 against 71 us -- so it keeps the plain kernel
// with two 4-plane staging tiles.)
//
// Thread roles, the packed DC / Nyquist row, the bin numbering and the layouts are those of
// fft_kernels.cuh; only wide planes are handled (narrow ones -- filters -- take the small-
// plane kernel or the plain kernels).
#pragma once

#include "fft_kernels.cuh"

namespace fc {

template <int N, int G, int SUB>
struct SubGeom {
    static constexpr int GS = G * SUB;                          // planes per staging tile
    static constexpr int B = N * (N / 2 + 1);
    static constexpr size_t STAGE_BYTES = (size_t)2 * B * GS * sizeof(float);
    static constexpr size_t MID_BYTES = MidGeom<N, G>::BYTES;
};

// ---------------------------------------------------------------------------
// Forward.  Tiles are groups of GS adjacent planes; tiles [0, p0.num_tiles) belong to the
// first operand, the rest to the second (both forward transforms of a pass in one launch).
// ---------------------------------------------------------------------------
template <int N, int G, int SUB, int MINB>
__global__ void __launch_bounds__(N* G, MINB)
r2c_sub_kernel(const __grid_constant__ CUtensorMap tmS0, const __grid_constant__ CUtensorMap tmS1,
               const FftParams p0, const FftParams p1) {
    constexpr int T = N * G, NC = N / 2 + 1, M = N / 2, HALF = T / 2, B = N * NC, GS = G * SUB;
    constexpr int PW = MidGeom<N, G>::PW, P = MidGeom<N, G>::P;
    constexpr int D = tma_bins_per_box(N);
    constexpr int NB = 2 * B / D;
    static_assert(NB <= 32, "one lane per TMA box");
    static_assert(HALF % 32 == 0, "the two halves of a row transform must be warp-uniform");
    extern __shared__ __align__(128) unsigned char fc_smem[];
    float* sIn = reinterpret_cast<float*>(fc_smem);                 // real planes of a sub-batch, then ...
    float2* sMid = reinterpret_cast<float2*>(fc_smem);              // ... its half spectrum (same memory)
    float* sStage = reinterpret_cast<float*>(fc_smem + p0.in_bytes);   // in_bytes: max(real tile, scratch)
    __shared__ __align__(8) unsigned long long bar_storage;
    const uint32_t bar = fk_smem_u32(&bar_storage);

    const int tid = threadIdx.x;
    const int total_tiles = p0.num_tiles + p1.num_tiles;
    const int q = tid / HALF, u = tid - q * HALF;               // row pass: (half, row ky, plane)
    const int kyp = u / G, gB = u - kyp * G;
    const int gA = tid / N, cA = tid % N;                       // column pass: (plane, column)
    const bool is_loader = (tid == T / 2);
    const bool is_storer = (tid >= T - 32) && ((tid & 31) < NB);

    dep_trigger();
    if (tid == 0) {
        fk_mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    dep_wait();                     // no global access above this line

    // A work item is one sub-batch: (tile, sb).  Items are walked in order; `cur` / `nxt` hold
    // the operand, matrix row, first plane and plane count of the current and the next item.
    struct Item { int tile, sb, second, row, c0, gcount, last; };
    auto make_item = [&](int tile, int sb) {
        Item it;
        it.tile = tile; it.sb = sb;
        it.second = tile >= p0.num_tiles;
        const FftParams& p = it.second ? p1 : p0;
        const int t = it.second ? tile - p0.num_tiles : tile;
        it.row = t / p.tiles_per_row;
        const int tcol = t - it.row * p.tiles_per_row;
        it.c0 = tcol * GS + sb * G;
        const int left = p.C - it.c0;
        it.gcount = left < G ? left : G;
        it.last = (sb == SUB - 1) || (left <= G);               // last sub-batch of its tile
        return it;
    };
    auto next_item = [&](const Item& it) {
        if (!it.last) return make_item(it.tile, it.sb + 1);
        const int nt = it.tile + (int)gridDim.x;
        if (nt < total_tiles) return make_item(nt, 0);
        Item e = it;
        e.tile = -1;
        return e;
    };
    // Copy of the real planes of an item.  Sets `pending` if (part of) it is asynchronous (wait on
    // the barrier) and `plain` if threads stored (part of) it themselves (barrier before reading).
    bool pending = false, plain = false;
    auto stage = [&](const Item& it) {
        const FftParams& p = it.second ? p1 : p0;
        const int hw = p.h * p.w;
        const float* src = p.real_in + ((size_t)it.row * p.C + it.c0) * hw;
        const int total = it.gcount * hw;
        if ((reinterpret_cast<uintptr_t>(src) & 15) == 0) {
            const int bulk = total & ~3;
            if (is_loader && bulk > 0) {
                fk_mbar_expect_tx(bar, (uint32_t)bulk * 4u);
                fk_bulk_g2s(fk_smem_u32(sIn), src, (uint32_t)bulk * 4u, bar);
            }
            if (tid < total - bulk) sIn[bulk + tid] = __ldg(src + bulk + tid);
            pending = bulk > 0;
            plain = total != bulk;
            return;
        }
        for (int i = tid; i < total; i += T) sIn[i] = __ldg(src + i);
        pending = false;
        plain = true;
    };

    uint32_t phase = 0;
    bool store_pending = false;
    Item cur{};
    cur.tile = -1;
    if ((int)blockIdx.x < total_tiles) {
        cur = make_item(blockIdx.x, 0);
        stage(cur);
    }

    while (cur.tile >= 0) {
        const FftParams& p = cur.second ? p1 : p0;
        const int h = p.h, w = p.w, hw = h * w, gcount = cur.gcount;
        const Item nxt = next_item(cur);

        if (plain) __syncthreads();     // samples that threads stored themselves are visible to everyone
        if (pending) {
            if (!fk_wait_or_report(bar, phase, p0.wait_cycles, p0.status)) {
                if (store_pending && is_storer) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
                return;
            }
            phase ^= 1u;
        }

        // column transforms: thread = (plane gA, column cA), one real FFT of length N in registers
        {
            float Xr[NC], Xi[NC];
            const bool act = (gA < gcount) && (cA < w);
            if (act) {
                float v[N];
                const float* src = sIn + gA * hw + cA;
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
            // the staging tile must be free again before this tile's first row pass writes it
            if (cur.sb == 0 && store_pending && is_storer) fk_bulk_wait_read();
            __syncthreads();   // the real planes are in registers: their memory becomes the scratch
            if (gA < gcount) {
                float2* dst = sMid + gA * P + cA;
                if (act) {
                    // rows ky = 0 and ky = N/2 of a real column transform are real: they share
                    // scratch row 0 as (re, im) and are transformed together in the row pass
                    dst[0] = make_float2(Xr[0], Xr[M]);
                    static_for<M - 1>([&](auto Kk) {
                        constexpr int k = decltype(Kk)::value + 1;
                        dst[k * PW] = make_float2(Xr[k], Xi[k]);
                    });
                } else {
                    static_for<M>([&](auto Kk) {
                        constexpr int k = decltype(Kk)::value;
                        dst[k * PW] = make_float2(0.0f, 0.0f);      // columns past the plane
                    });
                }
            }
        }
        __syncthreads();

        // row transforms: thread = (half q, row kyp, plane gB); one DIF step on the loads
        {
            float ar[M], ai[M];
            const float2* rowp = sMid + gB * P + kyp * PW;
            const bool packed = (kyp == 0);
            auto load = [&](auto Cc) -> float2 { return rowp[decltype(Cc)::value]; };
            if (q == 0) load_split<N, false, 0>(load, ar, ai);
            else        load_split<N, false, 1>(load, ar, ai);
            __syncthreads();   // the scratch is in registers: its memory takes the next planes
            pending = plain = false;
            if (nxt.tile >= 0) stage(nxt);
            cfft<M, false>(ar, ai);                     // ar/ai[k] = F[kx = 2k+q]

            // element (part, bin = kx*NC + ky, plane): staging offset (part*B + bin)*GS + plane
            float* o = sStage + (q * NC + kyp) * GS + cur.sb * G + gB;
            constexpr size_t sp = (size_t)B * GS;
            if (!packed) {
                static_for<M>([&](auto Kk) {
                    constexpr int k = decltype(Kk)::value;
                    o[(size_t)(2 * k * NC) * GS] = ar[k];
                    o[(size_t)(2 * k * NC) * GS + sp] = ai[k];
                });
            } else {
                // Z = FFT(X_0 + i X_{N/2}): X_0[k] = (Z_k + conj Z_{-k}) / 2, X_{N/2}[k] = (Z_k - conj Z_{-k}) / (2i)
                auto untangle = [&](auto Q) {
                    constexpr int qq = decltype(Q)::value;
                    static_for<M>([&](auto Kk) {
                        constexpr int k = decltype(Kk)::value;
                        constexpr int kp = (qq == 0) ? ((M - k) % M) : (M - 1 - k);
                        const float fr = ar[k], fi = ai[k], gr = ar[kp], gi = ai[kp];
                        float* o0 = o + (size_t)(2 * k * NC) * GS;      // row ky = 0
                        float* oN = o0 + (size_t)M * GS;                // row ky = N/2
                        o0[0] = 0.5f * (fr + gr);
                        o0[sp] = 0.5f * (fi - gi);
                        oN[0] = 0.5f * (fi + gi);
                        oN[sp] = 0.5f * (gr - fr);
                    });
                };
                if (q == 0) untangle(std::integral_constant<int, 0>{});
                else        untangle(std::integral_constant<int, 1>{});
            }
        }
        if (cur.last) {
            // the staging tile is complete: one box of GS columns x D bins per lane of the last
            // warp; columns beyond the matrix edge are clipped by the tensor map
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncthreads();
            if (is_storer) {
                const int b0 = (tid & 31) * D;
                const int tile_c0 = cur.c0 - cur.sb * G;
                fk_tma_store_3d(cur.second ? &tmS1 : &tmS0, fk_smem_u32(sStage + (size_t)b0 * GS), tile_c0, cur.row, b0);
                fk_bulk_commit();
            }
            store_pending = true;
        }
        cur = nxt;
    }
    if (store_pending && is_storer) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// ---------------------------------------------------------------------------
// Launchers.  Return cudaErrorNotSupported where the plain kernels must be used instead.
// ---------------------------------------------------------------------------
template <int N> struct SubCfg { static constexpr bool USE = false; static constexpr int G = 1, SUB = 1, MINB = 1; };
template <> struct SubCfg<64> { static constexpr bool USE = true; static constexpr int G = 4, SUB = 2, MINB = 1; };
// (Instantiated for n = 32 with G = 8 and n = 16 with G = 16 as well, the arrangement is slower than
// the plain kernels there -- mid layer 25.8 -> 32.4 us, deep layer 24 -> 27 us for the transform of
// x: those sizes are not bound by the row length, and lose the prefetch of the next tile.)

template <int N>
static cudaError_t launch_r2c_sub(FftParams pa, const FftParams* pb_in, cudaStream_t st) {
    if constexpr (!SubCfg<N>::USE) {
        return cudaErrorNotSupported;
    } else {
        constexpr int G = SubCfg<N>::G, SUB = SubCfg<N>::SUB, GS = G * SUB;
        // wide planes only
        if (pa.win || 2 * pa.w <= N) return cudaErrorNotSupported;
        if (pb_in && (pb_in->win || 2 * pb_in->w <= N)) return cudaErrorNotSupported;
        FftParams pb{};
        if (!fill_tiling<GS>(pa)) return cudaErrorInvalidValue;
        int in_bytes = real_tile_bytes(G, pa.h, pa.w);
        if (pb_in) {
            pb = *pb_in;
            if (!fill_tiling<GS>(pb)) return cudaErrorInvalidValue;
            const int b = real_tile_bytes(G, pb.h, pb.w);
            if (b > in_bytes) in_bytes = b;
        }
        if ((size_t)in_bytes < SubGeom<N, G, SUB>::MID_BYTES) in_bytes = (int)SubGeom<N, G, SUB>::MID_BYTES;
        pa.in_bytes = pb.in_bytes = in_bytes;
        const size_t smem = (size_t)in_bytes + SubGeom<N, G, SUB>::STAGE_BYTES;
        CUtensorMap tma, tmb;
        memset(&tma, 0, sizeof(tma));
        memset(&tmb, 0, sizeof(tmb));
        if (!make_spec_map<N, GS>(&tma, pa.spec_out, pa)) return cudaErrorInvalidValue;
        if (pb_in && !make_spec_map<N, GS>(&tmb, pb.spec_out, pb)) return cudaErrorInvalidValue;
        auto kern = r2c_sub_kernel<N, G, SUB, SubCfg<N>::MINB>;
        int grid = 0;
        cudaError_t e = persistent_grid(reinterpret_cast<const void*>(kern), N * G, smem,
                                        (long long)pa.num_tiles + pb.num_tiles, &grid);
        if (e != cudaSuccess) return e;
        return dep_launch(false, kern, dim3(grid), dim3(N * G), smem, st, tma, tmb, pa, pb);
    }
}

// The sub-batched kernels exist for these plane sizes only.
static cudaError_t launch_r2c_sub_any(int n, const FftParams& pa, const FftParams* pb, cudaStream_t st) {
    return n == 64 ? launch_r2c_sub<64>(pa, pb, st) : cudaErrorNotSupported;
}

}  // namespace fc
