// Programmatic dependent launch for the kernels of a pass.
//
// A pass is three kernels in one stream (forward transforms, contraction, inverse
// transform) and a training step is nine.  Launched the plain way, each kernel starts
// only after its predecessor has drained completely, so every boundary costs a launch
// latency plus the kernel's own prologue (barrier setup, tensor-memory allocation).
// With the stream-serialization attribute the next grid may be scheduled while the
// previous one drains: its CTAs run their prologue and then block in dep_wait() until
// the previous grid has completed and its writes are visible.  Every kernel calls
// dep_wait() before its first global-memory access (reads AND writes: a kernel may
// overwrite workspace that its predecessor still reads), so results are those of the
// serial order.  Without the attribute both device calls are no-ops.
#pragma once

#include <cuda_runtime.h>
#include <utility>

namespace fc {

// Allow the next kernel in the stream to be scheduled as soon as resources free up.
__device__ __forceinline__ void dep_trigger() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
// Block until every kernel this launch depends on has completed and flushed its writes.
__device__ __forceinline__ void dep_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// `overlap` = false launches the plain way.  Where overlapping pays was measured on B200
// (three layer configurations and a 1,000-point sweep of the parameter grid):
//  * contraction after one-pass forward transforms, inverse transform after the contraction:
//    1-7 % shorter passes at n <= 64 with the tensor-core contraction;
//  * the forward transforms as dependents of the previous pass's inverse transform gain
//    nothing at n <= 32, and at n = 64 a training step took 1.14 ms instead of 0.74;
//  * with the two-pass transforms (n = 128) a pass is 0.5 % longer with the contraction as a
//    dependent and 2.5 % longer with the inverse transform as one (2-6 % over the sweep);
//  * the FFMA contraction at n <= 16 with a long reduction (K > 64) loses up to 12 % (its
//    small CTAs share SMs with the waiting CTAs of the inverse transform); with K <= 64 the
//    passes are shorter (24 -> 21 us on an S8 f4 f'8 16 x 16 layer).
// The callers set the flag accordingly; everything else is launched the plain way.
template <typename... KArgs, typename... Args>
static cudaError_t dep_launch(bool overlap, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                              cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

}  // namespace fc
