// Host-side helper: encode TMA tensor maps without linking against libcuda (the
// driver entry point is fetched through the runtime), so the library also loads
// on machines that have no GPU driver.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>

namespace fc {

typedef CUresult (*tc_encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                 const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                 const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The entry point is the same for every device and thread: looked up once, published
// through an atomic (concurrent first calls all store the same pointer).
static tc_encode_fn tc_get_encode() {
    static std::atomic<void*> cached{nullptr};
    static std::atomic<bool> tried{false};
    void* sym = cached.load(std::memory_order_acquire);
    if (!sym && !tried.load(std::memory_order_acquire)) {
        cudaDriverEntryPointQueryResult qres;
        void* found = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &found, cudaEnableDefault, &qres) ==
                cudaSuccess && qres == cudaDriverEntryPointSuccess)
            sym = found;
        cached.store(sym, std::memory_order_release);
        tried.store(true, std::memory_order_release);
    }
    return reinterpret_cast<tc_encode_fn>(sym);
}

// Planar matrix family [2][bins][rows][ld] (all real matrices, then all imaginary
// ones) seen as a 3-D tensor (col, row, part*bins+bin) with `cols` valid columns;
// out-of-range coordinates read as zero and are clipped on store, which is what
// makes ragged M, N, K and ragged plane tiles work.
static bool tc_make_map(CUtensorMap* map, const float* base, int bins, int rows, int cols, int ld,
                        int box_cols, int box_rows,
                        CUtensorMapSwizzle swz = CU_TENSOR_MAP_SWIZZLE_128B, int box_depth = 1) {
    tc_encode_fn enc = tc_get_encode();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)bins * 2};
    cuuint64_t strides[2] = {(cuuint64_t)ld * 4, (cuuint64_t)rows * ld * 4};
    cuuint32_t box[3] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows, (cuuint32_t)box_depth};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides,
               box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace fc
