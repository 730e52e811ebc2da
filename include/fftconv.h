/*
 * fftconv -- FFT-domain convolution for CNN layers on NVIDIA B200 (sm_100a).
 *
 * C ABI of libfftconv.so.  Every pass is computed as the paper's Table 1
 * pipeline: batched 2-D real-to-complex FFTs of the implicitly zero-padded
 * planes, a per-frequency-bin complex contraction over the summed index, and
 * an inverse complex-to-real FFT with crop and 1/n^2 scale.  All kernels are
 * hand-written CUDA; there is no CPU fallback and no library call on the
 * compute path.
 *
 * Notation (paper, Section 2): S minibatch, f input planes, fprime (f') output
 * planes, h x w input plane, kh x kw kernel, oh x ow = (h-kh+1) x (w-kw+1)
 * output plane ("valid" only), n = side of the square power-of-two Fourier
 * basis, n >= max(h, w).
 *
 * Conventions for all entry points
 *  - Data pointers are DEVICE pointers owned by the caller, fp32, contiguous
 *    row-major ("BDHW", Section 3.1), at least 4-byte aligned (16-byte
 *    alignment lets the loads vectorise):
 *        x, dx [S][f][h][w]     w, dw [fprime][f][kh][kw]
 *        y, dy [S][fprime][oh][ow]
 *  - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *    Calls enqueue kernels on it and return; they never synchronise.  The conv
 *    and transform calls allocate no device memory (the caller lends the plan
 *    its workspace).
 *  - Inputs are never modified.  The device used is the one current when the
 *    call is made; plan, workspace and data must live on that device.
 *  - Return value: FFTCONV_OK (0) or a negative fftconv_status.  Nothing is
 *    thrown across the boundary.  On error no kernel has been launched.
 */
#ifndef FFTCONV_H_
#define FFTCONV_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct conv_plan_s conv_plan_t; /* opaque; created and destroyed by the library */

typedef enum {
    FFTCONV_OK = 0,
    FFTCONV_EINVAL = -1,        /* null pointer, non-positive count, kh > h, n < max(h, w) ... */
    FFTCONV_EUNSUPPORTED = -2,  /* n not in {8,16,32,64,128}, unknown math mode            */
    FFTCONV_EWORKSPACE = -3,    /* workspace missing, misaligned or too small              */
    FFTCONV_ECUDA = -4,         /* a CUDA runtime / driver call failed                     */
    FFTCONV_EDEVICE_TIMEOUT = -5 /* a bounded device-side wait ran out (status word set)   */
} fftconv_status;

typedef enum {
    FFTCONV_MATH_AUTO = 0, /* tensor cores unless a bin's result has fewer than 128 elements,
                              where the FP32 kernel is as fast and exact                  */
    FFTCONV_MATH_FP32 = 1, /* per-bin contraction with FP32 FFMA                  */
    FFTCONV_MATH_TF32 = 2  /* per-bin contraction on tcgen05 tensor cores, TF32
                              inputs, FP32 accumulation in tensor memory         */
} fftconv_math;

/* Plan for one layer shape (Section 3.4: one strategy per problem size, chosen
 * once).  Host-only: validates the shape, picks kernels and sizes the
 * workspace.  Needs no GPU.  *out receives the plan; destroy it with
 * conv_plan_destroy.  EINVAL: null out, a count < 1, kh > h, kw > w,
 * n < max(h, w).  EUNSUPPORTED: n not a power of two in [8, 128] -- except that n = 256, 512 or
 * 1024 is accepted for planes of up to n x n samples as the frame of a spatially tiled plan: the
 * plan then chooses a tile basis at once (see conv_plan_set_tiling; another basis may be set, tiling
 * cannot be switched off) and no transform of that size is ever run. */
int conv_plan(conv_plan_t** out, int S, int f, int fprime, int h, int w, int kh, int kw, int n);

/* Select the arithmetic of the per-bin contraction (fftconv_math).  Changes the
 * workspace size: query it again afterwards. */
int conv_plan_set_math(conv_plan_t* plan, int math);

/* Math mode the plan actually runs once AUTO is resolved.  The three passes
 * contract over different indices (f, f', S), so AUTO resolves per pass:
 * conv_plan_pass_math returns FFTCONV_MATH_FP32 or _TF32 for pass 0 (fprop),
 * 1 (bprop) or 2 (accGrad); conv_plan_effective_math returns _TF32 only if all
 * three passes run on the tensor cores, else _FP32. */
int conv_plan_effective_math(const conv_plan_t* plan);
int conv_plan_pass_math(const conv_plan_t* plan, int pass);

/* Bytes of device scratch the three passes need: the frequency-domain copies of
 * the two operands and of the result (Section 6 lists the same buffers), in the
 * plan's private frequency-major layout; plans with n = 128 add the scratch
 * that the transforms of large planes pass their half spectra through between
 * the two 1-D passes (80 MiB = 83.9e6 bytes: 512 KiB for each of up to 160
 * resident CTAs).  0 on a null plan. */
size_t conv_plan_workspace_bytes(const conv_plan_t* plan);

/* Lend the plan `bytes` of device memory at `dev_ptr` (256-byte aligned).  The
 * caller keeps ownership and must keep it alive while the plan is used.
 * Contents need no initialisation and are overwritten by every pass.  Passes of
 * one plan must not overlap in time (one workspace).  The call clears the
 * 256-byte header in front of the spectra (the device status word lives there)
 * with a synchronous cudaMemset: it is a set-up call, not for the hot loop.
 * EWORKSPACE if too small or misaligned. */
int conv_plan_set_workspace(conv_plan_t* plan, void* dev_ptr, size_t bytes);

/* fprop (Section 2, first equation): y(s,j) = sum_i x(s,i) (star) w(j,i), valid
 * cross-correlation.  Overwrites y [S][fprime][oh][ow]. */
int conv_fprop(conv_plan_t* plan, const float* x, const float* w, float* y, void* cuda_stream);

/* fprop without any device allocation by anybody (the paper has no counterpart:
 * its buffer manager always allocates).  Same computation and same kernels as
 * conv_fprop, but the frequency-domain scratch lives in a fixed array that is
 * part of the library image (FFTCONV_NOALLOC_BYTES = 32 MiB of device memory,
 * held by every GPU that loads the library until the process exits) instead of
 * a workspace lent by the caller.  It is meant for callers that have tensors
 * but no way to obtain scratch memory at the call site: code running after a
 * framework's allocator has claimed the whole device, loops in which an
 * allocation (which synchronises the device) is not acceptable, plug-ins that
 * are handed buffers but no allocator.  The plan's own workspace, if any, is
 * ignored and left untouched; x, w, y are passed as for conv_fprop.
 *  - Returns FFTCONV_EWORKSPACE, launching nothing, when
 *    conv_plan_workspace_bytes(plan) exceeds FFTCONV_NOALLOC_BYTES.
 *  - Calls no cudaMalloc / cudaFree and no allocating library routine.  The
 *    first call on each device looks up the array's device address (one
 *    cudaGetSymbolAddress, with that device current); make that first call
 *    outside any stream capture.
 *  - All calls on a device share the one array and it keeps whatever the last
 *    call left in it; each call clears the small status header it relies on and
 *    overwrites every spectrum it reads.  Two calls that overlap on the GPU
 *    (different streams, no dependency) race on the array: serialise them.
 *  - A bounded device-side wait that runs out is recorded in the array's header,
 *    which no entry point reads back; use conv_fprop + conv_plan_status where
 *    that diagnosis matters.
 *  - The first calls on a device may come from several host threads at once:
 *    they all look up and store the same address. */
#define FFTCONV_NOALLOC_BYTES (32u << 20)
int conv_fprop_noalloc(conv_plan_t* plan, const float* x, const float* w, float* y,
                       void* cuda_stream);

/* bprop (Section 2, second equation): dx(s,i) = sum_j dy(s,j) * w(j,i), full
 * convolution.  Overwrites dx [S][f][h][w]. */
int conv_bprop(conv_plan_t* plan, const float* dy, const float* w, float* dx, void* cuda_stream);

/* accGrad (Section 2, third equation; index form in Section 6):
 * dw(j,i) = sum_s dy(s,j) (star) x(s,i).  accumulate == 0 overwrites
 * dw [fprime][f][kh][kw]; accumulate != 0 adds to it. */
int conv_accgrad(conv_plan_t* plan, const float* dy, const float* x, float* dw, int accumulate,
                 void* cuda_stream);

/* Transforms of small planes.  Operand planes of at most 13 x 13 samples that fill at most a
 * quarter of the basis (the filters of fprop and bprop) are transformed by a pruned separable
 * DFT that evaluates one frequency bin for 32 adjacent planes at a time and writes whole
 * 128-byte lines of the frequency-major spectrum (Section 5.1: the padding is never
 * materialised -- here it is never even multiplied), instead of by the butterfly kernels that
 * the large planes use; the operand then has a launch of its own, which runs beside the other
 * operand's transform (a pass is four launches).  Likewise the inverse transform of accGrad,
 * whose result is clipped to the kh x kw filter window (Section 3.1), is a pruned inverse DFT
 * that reads whole lines for 32 adjacent planes when the window is square, at most 11 x 11 and
 * at most a quarter of the basis (n = 32 and 64).  enable == 1 (the default) uses the forward
 * kernel where it was measured to pay -- bases of 64 and 128; at n <= 32 planes of at most 1/16
 * of the basis whose spectrum exceeds 96 MB; the filter operand of a chunked pass (below);
 * otherwise the filters share the other operand's launch -- and the inverse kernel wherever it
 * applies; enable >= 2 uses both wherever they apply; enable <= 0
 * sends everything through the butterfly kernels.  Same results up to rounding in every mode. */
int conv_plan_set_small_plane_kernel(conv_plan_t* plan, int enable);

/* Filter spectrum through the cache (Section 6 asks for fewer passes over memory between the
 * stages).  With chunks > 1, fprop and bprop transform the filters and contract them in
 * `chunks` ranges of frequency rows: each part of the filter spectrum is consumed by the
 * contraction right after it was produced (the transform of the next range runs beside the
 * contraction of the current one), so that it can be read back from the L2 cache where a
 * range fits it.  Needs the small-plane kernel and the tensor-core contraction; otherwise, and
 * with chunks <= 1 (the default: on B200 the unchunked pass measured faster on every layer
 * tried), the pass runs unchunked.  Results do not depend on the setting. */
int conv_plan_set_filter_chunks(conv_plan_t* plan, int chunks);

/* Spectrum reuse across the passes of one training step (the paper's Section 6
 * notes that the forward transforms could be shared between passes, saving a
 * third of them, and passes on it for memory reasons).  With enable != 0 the
 * workspace holds one region per tensor family (x, w, dy) plus one for the
 * result spectrum -- query conv_plan_workspace_bytes again and lend a workspace
 * of that size -- and the spectra survive a pass: conv_fprop always transforms x
 * and w afresh; conv_bprop transforms dy and takes w's spectrum from the
 * preceding conv_fprop if it is given the same w pointer; conv_accgrad takes
 * dy's and x's spectra from the preceding passes if given the same pointers.
 * A tensor passed under a pointer whose spectrum is cached must not have been
 * modified since that spectrum was computed, and the passes must be ordered on
 * one stream (or synchronised by the caller); otherwise call
 * conv_plan_invalidate_spectra first.  Changing the setting or the workspace
 * invalidates everything.  Results are identical to the non-reusing passes.
 * EUNSUPPORTED together with spatial tiling (the passes then use different windows). */
int conv_plan_set_spectrum_reuse(conv_plan_t* plan, int enable);
int conv_plan_invalidate_spectra(conv_plan_t* plan);

/* Spatial tiling (Section 6): with n_tile in {8, 16, 32, 64} smaller than the plan's basis n,
 * every pass decomposes its planes into tiles that fit an n_tile x n_tile basis instead of
 * padding kernels and planes to n x n.  With steps dh = n_tile - kh + 1, dw = n_tile - kw + 1:
 *   fprop  : each dh x dw tile of y is the valid cross-correlation of the n_tile x n_tile window
 *            of x at the same origin with w (the paper's y[i, i+d] = x[i, i+d+w] (star) c);
 *   bprop  : each dh x dw tile of dx is the full convolution of w with the n_tile x n_tile window
 *            of dy that starts kh-1 rows and kw-1 columns before the tile (zero outside dy);
 *   accGrad: dw is the sum over the minibatch AND over the tiles of (dh x dw tile of dy)
 *            (star) (n_tile x n_tile window of x), the paper's tiled sum for the kernel gradient.
 * The window index joins the minibatch index in the per-bin contraction (S T rows instead of S,
 * T = tiles per plane), the weight spectra shrink from n(n/2+1) to n_tile(n_tile/2+1) bins, and
 * windows are read with clipped loads and written straight into the planes: nothing is
 * gathered or padded in memory.  Results are those of the untiled passes up to rounding.
 * n_tile == 0 (or == n) switches tiling off.  Changes the workspace size: query it again and
 * lend a workspace of that size.  EUNSUPPORTED: n_tile not in {8,16,32,64}, spectrum reuse
 * enabled, or more than 2^30 windows; EINVAL: n_tile > n or n_tile < max(kh, kw).
 * n_tile == FFTCONV_TILE_AUTO lets the plan choose: it estimates a training step for every
 * admissible basis from the bytes each kernel moves (Section 3.4's one strategy per problem size,
 * decided by a static model instead of trial runs) and keeps tiling off unless a tile basis is
 * estimated at least 10 % faster. */
#define FFTCONV_TILE_AUTO (-1)
int conv_plan_set_tiling(conv_plan_t* plan, int n_tile);

/* Measured choice of the tile basis (Section 3.4: the paper's autotuner times the candidate
 * bases of a problem size and keeps the fastest; FFTCONV_TILE_AUTO above ranks them with a byte
 * model instead).  Runs one warm-up and `reps` (1..100) timed training steps -- fprop, bprop,
 * accGrad -- for the untiled basis (where the plan's n <= 128) and for every admissible tile
 * basis in {8, 16, 32, 64} below n, on the caller's tensors (device pointers, the layouts of
 * conv_fprop / conv_bprop / conv_accgrad), timed with CUDA events on `cuda_stream`, and leaves
 * the plan on the fastest basis with `workspace` lent to it.  y, dx and dw are overwritten (the
 * last candidate's results, which equal every other candidate's up to rounding).  `workspace`:
 * device memory, 256-byte aligned; conv_plan_tune_workspace_bytes(plan) is the largest workspace
 * of any candidate, and a candidate that needs more than `workspace_bytes` is left out (small
 * tile bases of large planes can need many times the untiled workspace); it stays with the
 * caller and is the plan's workspace afterwards.  *chosen_basis (host, may be null) receives the basis, 0 = untiled; step_ms (host,
 * may be null) receives FFTCONV_TUNE_CANDIDATES step times in milliseconds in the order
 * untiled, 8, 16, 32, 64, negative where a candidate is not admissible or was left out.
 * Synchronises the stream.  EUNSUPPORTED with spectrum reuse enabled or when no candidate is
 * admissible and fits the workspace; ECUDA when a run fails or a device wait gives up (the plan
 * then keeps the basis it had). */
#define FFTCONV_TUNE_CANDIDATES 5
size_t conv_plan_tune_workspace_bytes(conv_plan_t* plan);
int conv_plan_tune_tiling(conv_plan_t* plan, const float* x, const float* w, const float* dy,
                          float* y, float* dx, float* dw, void* workspace, size_t workspace_bytes,
                          int reps, void* cuda_stream, int* chosen_basis, float* step_ms);

/* The tile basis in use, 0 when tiling is off. */
int conv_plan_tile_basis(const conv_plan_t* plan);

/* Reads the plan's device status word (synchronises the device).  FFTCONV_OK,
 * or FFTCONV_EDEVICE_TIMEOUT if a bounded wait inside a kernel gave up since
 * the last call (the word is then cleared), or ECUDA.  Every kernel of a pass
 * -- the forward and inverse transforms and the tensor-core contraction --
 * bounds each wait on an asynchronous copy or on the tensor cores; when a limit
 * runs out the kernel raises this word, lets the copies and MMAs it has issued
 * finish (again bounded), frees its tensor memory and returns, so the context
 * stays usable.  The results of such a pass are unspecified. */
int conv_plan_status(conv_plan_t* plan);

/* Limit of one bounded device-side wait, in SM clock cycles; 0 restores the
 * default (2e9 cycles, about a second).  A diagnostic hook: a limit shorter
 * than a copy's normal latency makes the waits run out on purpose, which is how
 * the tests exercise the give-up paths without hanging anything (the draining
 * waits after a give-up always keep the default limit).  EINVAL: null plan or a
 * negative limit. */
int conv_plan_set_wait_limit(conv_plan_t* plan, long long sm_cycles);

/* Frees the plan (host memory and its timing events; never the workspace). */
int conv_plan_destroy(conv_plan_t* plan);

/* Per-stage device timing for benchmarks.  enable != 0 makes every following
 * pass record CUDA events on its stream around its kernels -- the columns of the
 * paper's Table 4 with the transposes fused away.  enable == 1 keeps the normal
 * launch sequence (both forward FFTs in one kernel, per-bin contraction, inverse
 * FFT); enable == 2 launches the two forward FFTs as separate kernels so that
 * they can be timed apart.  Creates the events on first use (the only state the
 * plan owns on the device side). */
int conv_plan_enable_stage_timing(conv_plan_t* plan, int enable);

/* Waits for the last pass issued with timing enabled and writes durations in
 * milliseconds to out_ms[0..3]: forward FFT of the first operand (mode 1: of both
 * operands where they share one kernel), forward FFT of the second operand
 * (exactly zero where it had no launch of its own: mode 1 unless the operand takes
 * the small-plane kernel), contraction, inverse FFT.  EINVAL if timing is off or no
 * pass has run. */
int conv_plan_stage_times_ms(conv_plan_t* plan, float* out_ms);

/* Bare batched 2-D real-to-complex transform (Supplement 8.2 definition,
 * forward sign minus, unnormalised; Section 3.1 half-spectrum storage):
 *   out[p][ky][kx] = sum_{r<h,c<w} in[p][r][c] exp(-2 pi i (ky r + kx c)/n)
 * in : device [batch][h][w] fp32, zero-padded implicitly to n x n (never
 *      materialised, Section 5.1).
 * out: device [batch][n][n/2+1] interleaved (re, im) fp32 pairs, 8-byte aligned. */
int fft2d_r2c(const float* in, void* out_c, int batch, int h, int w, int n, void* cuda_stream);

/* Bare batched 2-D complex-to-real inverse transform with crop and scale
 * (Section 3.1: the inverse transform's result is clipped):
 *   out[p][r][c] (+)= scale * Re sum_{ky,kx<n} X~[p][ky][kx] exp(+2 pi i (ky r + kx c)/n)
 * for r < oh, c < ow (window anchored at the origin), X~ the Hermitian
 * extension of the stored half.  The input must be Hermitian-consistent (the
 * spectrum of a real plane); otherwise the result is unspecified.
 * in : device [batch][n][n/2+1] interleaved fp32 pairs.
 * out: device [batch][oh][ow] fp32; accumulate != 0 adds to it. */
int fft2d_c2r(const void* in_c, float* out, int batch, int n, int oh, int ow, float scale,
              int accumulate, void* cuda_stream);

/* Bare batched 1-D real-to-complex transform, n a power of two in [2, 256] (the sizes of the
 * paper's Section 5.2 / 5.4 evaluation of batched 1-D transforms; definition in Supplement 8.2):
 *   out[p][k] = sum_{j<len} in[p][j] exp(-2 pi i k j / n),   k in [0, n/2]
 * in : device [batch][len] fp32, zero-padded implicitly to n samples (len <= n).
 * out: device [batch][n/2+1] interleaved (re, im) fp32 pairs, 8-byte aligned.
 * EUNSUPPORTED: n not a power of two in [2, 256]; EINVAL: null pointer, batch < 1, len not in [1, n]. */
int fft1d_r2c(const float* in, void* out_c, long long batch, int len, int n, void* cuda_stream);

/* Bare batched 1-D complex-to-real inverse transform with crop and scale:
 *   out[p][j] (+)= scale * Re sum_{k<n} X~[p][k] exp(+2 pi i k j / n),   j < olen,
 * X~ the Hermitian extension of the stored half (the imaginary parts of bins 0 and n/2 are
 * ignored); scale = 1/n undoes fft1d_r2c.
 * in : device [batch][n/2+1] interleaved fp32 pairs, 8-byte aligned.
 * out: device [batch][olen] fp32; accumulate != 0 adds to it. */
int fft1d_c2r(const void* in_c, float* out, long long batch, int n, int olen, float scale,
              int accumulate, void* cuda_stream);

/* Per-bin complex contraction alone (Table 1, the Cgemm row), exposed for
 * testing and profiling: for every bin b,
 *   C[b][m][nn] = sum_k op(A)[b][m][k] * op(B)[b][nn][k]
 * with op = identity, or the complex conjugate when conjA / conjB is non-zero
 * (Section 2: the conjugate turns the product into a cross-correlation).
 * Operands are planar device arrays: the real matrices of all bins first, then
 * the imaginary matrices of all bins:
 *   A: [2][bins][M][lda], k contiguous (lda >= K); with transA != 0 it is stored
 *      [2][bins][K][lda], m contiguous (lda >= M);
 *   B: [2][bins][N][ldb] (ldb >= K), or with transB != 0 [2][bins][K][ldb] (ldb >= N);
 *   C: [2][bins][M][ldc], ldc >= N; the padding columns N..ldc-1 are scratch
 *      (they may be overwritten with zeros).
 * lda, ldb, ldc must be multiples of 4 and the pointers 16-byte aligned.
 * math: FFTCONV_MATH_FP32 or FFTCONV_MATH_TF32 (AUTO resolves by shape).
 * status_word: device int the tensor-core kernel sets non-zero if a bounded wait
 * gives up; may be NULL for the FP32 path. */
int fftconv_bin_contract(const float* A, const float* B, float* C, int bins, int M, int N, int K,
                         int lda, int ldb, int ldc, int transA, int transB, int conjA, int conjB,
                         int math, int* status_word, void* cuda_stream);

/* Text for a status code; never NULL. */
const char* fftconv_status_string(int status);

/* Number of kernel launches issued by this library since load (all plans, all
 * threads); lets a benchmark state how many of this library's kernels ran. */
unsigned long long fftconv_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* FFTCONV_H_ */
