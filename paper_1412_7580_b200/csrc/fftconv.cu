// C ABI of libfftconv.so: plans, the three convolution passes, the bare
// transforms and the bare per-bin contraction.  Host code only validates,
// sizes and launches; every step of the computation runs in the kernels of
// fft_kernels.cuh, cgemm_ffma.cuh and cgemm_tc.cuh.
#include "../../include/fftconv.h"

#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <cstring>
#include <new>

#include "cgemm_ffma.cuh"
#include "cgemm_tc.cuh"
#include "fft_kernels.cuh"
#include "fft_big.cuh"
#include "fft_small.cuh"
#include "fft_sub.cuh"
#include "fft1d.cuh"

#define FFTCONV_API extern "C" __attribute__((visibility("default")))

namespace {

std::atomic<unsigned long long> g_launches{0};

constexpr size_t kAlign = 256;
constexpr size_t kHeaderBytes = 256;   // workspace header: the device status word lives here

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline int round4(int v) { return (v + 3) & ~3; }

// One frequency-major matrix family: [2][bins][R][ld] floats (real parts, then imaginary parts).
struct SpecDesc {
    int R, C, ld;
    size_t bytes(int bins) const { return (size_t)bins * 2 * R * ld * sizeof(float); }
};

// One real tensor of a pass and its spectrum: plane (row, col) of the BDHW tensor
// is matrix element (row, col) of every bin.
struct OperandDesc {
    SpecDesc spec;
    int h, w;               // plane size (forward) or crop window (inverse)
    int kind;               // which tensor family: 0 = x / dx, 1 = w / dw, 2 = y / dy
    // spatial tiling: the operand's matrix rows are windows (s, ty, tx) of H x W planes
    int win, H, W, nty, ntx, step_y, step_x, oy, ox;
};

struct PassDesc {
    OperandDesc a, b, c;    // c: result (h, w = crop window)
    int M, N, K;            // per-bin contraction C[M][N] = sum_K op(A)[M][K] op(B)[N][K]
    int transA, transB, conjA, conjB;
};

enum { PASS_FPROP = 0, PASS_BPROP = 1, PASS_ACCGRAD = 2 };

}  // namespace

struct conv_plan_s {
    int S, f, fp, h, w, kh, kw, n;
    int oh, ow, bins;
    int n_full;        // the basis given to conv_plan; n is the one in use (the tile's when tiling)
    int math;          // requested fftconv_math
    void* ws;
    size_t ws_bytes;
    int reuse;              // keep the forward spectra between the passes of a training step
    const float* cached[3]; // reuse: tensor whose spectrum sits in region 0 (x), 1 (w), 2 (dy)
    int timing;             // record events around the four kernels of a pass
    bool timed;             // a timed pass has been issued
    bool second_stage_used; // the timed pass launched something between the second and third event
    cudaEvent_t ev[5];
    bool ev_made;
    long long wait_cycles;  // limit of a bounded device-side wait in SM cycles; 0 = the kernels' default
    int small_planes;       // pruned-DFT kernels for small planes: 0 never, 1 where measured to pay, 2 wherever they apply
    int filter_chunks;      // > 1: the filter spectrum is produced and contracted in this many bin ranges
};

namespace {

// Operand roles per pass (Table 1 and Section 2; which operand carries the
// conjugate follows from the convolution theorem for cross-correlation).  Every
// spectrum keeps the plane order of its tensor ([S][f], [f'][f], [S][f']); where
// the summed index is not the minor one the contraction reads the operand
// "transposed" ([k][rows]) instead of the FFT writing a transposed copy.
//   fprop  : Y^[b][s][j]  = sum_i X^[b][s][i]        conj W^[b][j][i]
//   bprop  : dX^[b][s][i] = sum_j dY^[b][s][j]       W^[b][j][i]        (B read as [k=j][i])
//   accGrad: dW^[b][j][i] = sum_s conj dY^[b][s][j]  X^[b][s][i]        (A as [k=s][j], B as [k=s][i])
// Spatial tiling (Section 6): with a tile basis n < the plane, every pass works on windows.
// Steps dh = n - kh + 1, dw = n - kw + 1.
//   fprop  : y tile (ty, tx) of dh x dw       = x window of n x n at the same origin (star) w
//   bprop  : dx tile of dh x dw at (ty dh, ..) = rows kh-1.. of (dy window of n x n starting
//            kh-1 rows and kw-1 columns before the tile's origin, zero outside the plane) * w
//   accGrad: dw = sum over s and tiles of  dy tile of dh x dw (star) x window of n x n
// The window index joins the minibatch index: matrix rows (s, ty, tx), S T of them; accGrad
// sums over them.  fprop and accGrad tile the output plane, bprop tiles the input plane.
PassDesc describe_tiled(const conv_plan_s& p, int pass) {
    PassDesc d{};
    auto spec = [](int R, int C) { return SpecDesc{R, C, round4(C)}; };
    const int n = p.n, dh = n - p.kh + 1, dw = n - p.kw + 1;
    auto cdiv = [](int a, int b) { return (a + b - 1) / b; };
    const int oty = cdiv(p.oh, dh), otx = cdiv(p.ow, dw);       // tiles of the output plane
    const int ity = cdiv(p.h, dh), itx = cdiv(p.w, dw);         // tiles of the input plane
    auto mn = [](int a, int b) { return a < b ? a : b; };
    const OperandDesc W = {spec(p.fp, p.f), p.kh, p.kw, 1, 0, 0, 0, 0, 0, 0, 0, 0, 0};
    switch (pass) {
        case PASS_FPROP: {
            const int T = oty * otx;
            d.a = {spec(p.S * T, p.f), mn(n, p.h), mn(n, p.w), 0, 1, p.h, p.w, oty, otx, dh, dw, 0, 0};
            d.b = W;
            d.c = {spec(p.S * T, p.fp), mn(dh, p.oh), mn(dw, p.ow), 2, 1, p.oh, p.ow, oty, otx, dh, dw, 0, 0};
            d.M = p.S * T; d.N = p.fp; d.K = p.f;
            d.transA = 0; d.transB = 0; d.conjA = 0; d.conjB = 1;
            break;
        }
        case PASS_BPROP: {
            const int T = ity * itx;
            d.a = {spec(p.S * T, p.fp), n, n, 2, 1, p.oh, p.ow, ity, itx, dh, dw, -(p.kh - 1), -(p.kw - 1)};
            d.b = W;
            d.c = {spec(p.S * T, p.f), mn(dh, p.h), mn(dw, p.w), 0, 1, p.h, p.w, ity, itx, dh, dw,
                   p.kh - 1, p.kw - 1};
            d.M = p.S * T; d.N = p.f; d.K = p.fp;
            d.transA = 0; d.transB = 1; d.conjA = 0; d.conjB = 0;
            break;
        }
        default: {
            const int T = oty * otx;
            d.a = {spec(p.S * T, p.fp), mn(dh, p.oh), mn(dw, p.ow), 2, 1, p.oh, p.ow, oty, otx, dh, dw, 0, 0};
            d.b = {spec(p.S * T, p.f), mn(n, p.h), mn(n, p.w), 0, 1, p.h, p.w, oty, otx, dh, dw, 0, 0};
            d.c = W;
            d.M = p.fp; d.N = p.f; d.K = p.S * T;
            d.transA = 1; d.transB = 1; d.conjA = 1; d.conjB = 0;
            break;
        }
    }
    return d;
}

PassDesc describe(const conv_plan_s& p, int pass) {
    if (p.n != p.n_full) return describe_tiled(p, pass);
    PassDesc d{};
    auto spec = [](int R, int C) { return SpecDesc{R, C, round4(C)}; };
    const OperandDesc X = {spec(p.S, p.f), p.h, p.w, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
    const OperandDesc W = {spec(p.fp, p.f), p.kh, p.kw, 1, 0, 0, 0, 0, 0, 0, 0, 0, 0};
    const OperandDesc Y = {spec(p.S, p.fp), p.oh, p.ow, 2, 0, 0, 0, 0, 0, 0, 0, 0, 0};
    switch (pass) {
        case PASS_FPROP:
            d.a = X; d.b = W; d.c = Y;
            d.M = p.S; d.N = p.fp; d.K = p.f;
            d.transA = 0; d.transB = 0; d.conjA = 0; d.conjB = 1;
            break;
        case PASS_BPROP:
            d.a = Y; d.b = W; d.c = X;
            d.M = p.S; d.N = p.f; d.K = p.fp;
            d.transA = 0; d.transB = 1; d.conjA = 0; d.conjB = 0;
            break;
        default:
            d.a = Y; d.b = X; d.c = W;
            d.M = p.fp; d.N = p.f; d.K = p.S;
            d.transA = 1; d.transB = 1; d.conjA = 1; d.conjB = 0;
            break;
    }
    return d;
}

int resolve_math(const conv_plan_s& p, const PassDesc& d) {
    if (p.math == FFTCONV_MATH_FP32) return FFTCONV_MATH_FP32;
    const bool fits = fc::tc_shape_supported(d.M, d.N, d.K);
    if (p.math == FFTCONV_MATH_TF32) return fits ? FFTCONV_MATH_TF32 : FFTCONV_MATH_FP32;
    return (fits && fc::tc_shape_profitable(d.M, d.N, d.K)) ? FFTCONV_MATH_TF32 : FFTCONV_MATH_FP32;
}

size_t pass_bytes(const conv_plan_s& p, int pass) {
    PassDesc d = describe(p, pass);
    return align_up(d.a.spec.bytes(p.bins), kAlign) + align_up(d.b.spec.bytes(p.bins), kAlign) +
           align_up(d.c.spec.bytes(p.bins), kAlign);
}

// Bytes of the spectra regions (with the header); the scratch of the two-pass transforms
// (n = 128) follows them.
size_t spectra_bytes(const conv_plan_s* plan) {
    if (plan->reuse) {
        // one region per tensor family plus one for the result spectrum of the running pass
        const PassDesc d = describe(*plan, PASS_FPROP);      // a = x, b = w, c = y
        const size_t bx = align_up(d.a.spec.bytes(plan->bins), kAlign),
                     bw = align_up(d.b.spec.bytes(plan->bins), kAlign),
                     by = align_up(d.c.spec.bytes(plan->bins), kAlign);
        const size_t br = bx > bw ? (bx > by ? bx : by) : (bw > by ? bw : by);
        return kHeaderBytes + bx + bw + by + br;
    }
    size_t m = 0;
    for (int pass = 0; pass < 3; ++pass) {
        size_t b = pass_bytes(*plan, pass);
        if (b > m) m = b;
    }
    return kHeaderBytes + m;
}

bool valid_n(int n) { return n == 8 || n == 16 || n == 32 || n == 64 || n == 128; }

int run_pass(conv_plan_s* plan, int pass, const float* a_in, const float* b_in, float* c_out,
             int accumulate, cudaStream_t st) {
    if (!plan || !a_in || !b_in || !c_out) return FFTCONV_EINVAL;
    if (!plan->ws || plan->ws_bytes < conv_plan_workspace_bytes(plan)) return FFTCONV_EWORKSPACE;
    const PassDesc d = describe(*plan, pass);
    unsigned char* base = static_cast<unsigned char*>(plan->ws);
    int* status = reinterpret_cast<int*>(base);
    float* specA = reinterpret_cast<float*>(base + kHeaderBytes);
    float* specB = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(specA) +
                                            align_up(d.a.spec.bytes(plan->bins), kAlign));
    float* specC = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(specB) +
                                            align_up(d.b.spec.bytes(plan->bins), kAlign));
    // Which forward transforms this pass has to run.  Without reuse: both.  With reuse the
    // spectra live in fixed per-tensor regions and survive the pass: fprop always refreshes
    // x and w (new data every step), bprop refreshes dy and takes w's spectrum from fprop,
    // accGrad takes both from the earlier passes -- whenever the same device pointer is
    // passed again; otherwise the spectrum is recomputed.
    bool need_a = true, need_b = true;
    if (plan->reuse) {
        const PassDesc f = describe(*plan, PASS_FPROP);
        unsigned char* r0 = base + kHeaderBytes;
        unsigned char* r1 = r0 + align_up(f.a.spec.bytes(plan->bins), kAlign);
        unsigned char* r2 = r1 + align_up(f.b.spec.bytes(plan->bins), kAlign);
        unsigned char* r3 = r2 + align_up(f.c.spec.bytes(plan->bins), kAlign);
        unsigned char* region[3] = {r0, r1, r2};
        specA = reinterpret_cast<float*>(region[d.a.kind]);
        specB = reinterpret_cast<float*>(region[d.b.kind]);
        specC = reinterpret_cast<float*>(r3);
        const bool fresh_a = (pass != PASS_ACCGRAD), fresh_b = (pass == PASS_FPROP);
        need_a = fresh_a || plan->cached[d.a.kind] != a_in;
        need_b = fresh_b || plan->cached[d.b.kind] != b_in;
        // a spectrum counts as cached only once its transform has been launched (below)
        if (need_a) plan->cached[d.a.kind] = nullptr;
        if (need_b) plan->cached[d.b.kind] = nullptr;
    }

    auto operand = [&](const OperandDesc& o, const float* in, float* spec) {
        fc::FftParams fp{};
        fp.real_in = in; fp.spec_out = spec;
        fp.h = o.h; fp.w = o.w;
        fp.R = o.spec.R; fp.C = o.spec.C; fp.ld = o.spec.ld;
        fp.win = o.win; fp.H = o.H; fp.W = o.W; fp.nty = o.nty; fp.ntx = o.ntx;
        fp.step_y = o.step_y; fp.step_x = o.step_x; fp.oy = o.oy; fp.ox = o.ox;
        fp.status = status; fp.wait_cycles = plan->wait_cycles;
        return fp;
    };
    const bool timing = plan->timing && plan->ev_made;
    auto mark = [&](int i) { if (timing) cudaEventRecord(plan->ev[i], st); };
    // large planes run the two-pass transforms (one launch per operand, scratch behind the spectra)
    const bool tiled = plan->n != plan->n_full;
    const bool big = !tiled && fc::big_uses_two_pass(plan->n);
    float* scratch = reinterpret_cast<float*>(base + align_up(spectra_bytes(plan), kAlign));
    const size_t scratch_bytes = tiled ? 0 : fc::big_scratch_bytes(plan->n);
    // One forward launch: both operands in one kernel (one-pass transforms), or one operand.
    auto forward = [&](const fc::FftParams& pa, const fc::FftParams* pb) -> cudaError_t {
        g_launches.fetch_add((big && pb) ? 2 : 1, std::memory_order_relaxed);
        if (!big) {
            // wide planes at n = 64: the sub-batched kernels (rows twice as long); else the plain ones
            const cudaError_t es = fc::launch_r2c_sub_any(plan->n, pa, pb, st);
            return es != cudaErrorNotSupported ? es : fc::launch_r2c<true>(plan->n, pa, pb, st);
        }
        cudaError_t e = fc::launch_r2c_two_pass(plan->n, pa, scratch, scratch_bytes, st);
        if (e == cudaSuccess && pb) e = fc::launch_r2c_two_pass(plan->n, *pb, scratch, scratch_bytes, st);
        return e;
    };
    // Small planes (the filters of fprop and bprop) take the pruned-DFT kernel, whose stores are
    // whole 128-byte lines; it runs after the other operand's transform, as its programmatic
    // dependent where that transform is a one-pass kernel.
    // Mode 1 (default) takes it where it was measured to pay: at n >= 64 (passes 1.1-1.4 x
    // shorter); at n <= 32 only for planes of at most 1/16 of the basis whose spectrum is much
    // larger than the L2 (mid and deep layers: 1-2 % shorter passes), because otherwise the one
    // launch for both operands is as fast or faster (the filter spectrum is bound by the store
    // rate either way, a fourth launch costs 3-5 us on small layers, and wider filters at
    // n <= 32 are 7-25 % slower as direct sums); and for the filter operand of a chunked pass.
    // Mode 2 takes it wherever it applies.
    const bool tensor = resolve_math(*plan, d) == FFTCONV_MATH_TF32;
    const bool want_chunks = plan->filter_chunks > 1 && tensor && !timing;
    auto is_small = [&](const fc::FftParams& f, bool filter_operand) {
        if (!plan->small_planes || f.win || !fc::small_supported(plan->n, f.h, f.w)) return false;
        if (plan->small_planes == 2 || plan->n >= 64 || (filter_operand && want_chunks)) return true;
        const double spec_bytes = 8.0 * plan->bins * (double)f.R * f.ld;
        return 16 * f.h * f.w <= plan->n * plan->n && spec_bytes >= 96e6;
    };
    // dep: another forward transform of this pass was launched just before; the small-plane kernel
    // then runs beside it (neither touches the other's data) and completes only after it.
    // one-pass inverse transforms (n <= 64) rebuild the conjugate bins of the rows ky = 0 and
    // ky = n/2 themselves, so the contraction leaves them out (and the small-plane transform,
    // whose stores are single lines, does not write them)
    const int herm_n = (!big && plan->n <= 64) ? plan->n : 0;
    auto forward_small = [&](const fc::FftParams& f, bool dep) -> cudaError_t {
        g_launches.fetch_add(1, std::memory_order_relaxed);
        const bool conc = dep && !big && !timing;
        return fc::launch_r2c_small(plan->n, f, 0, plan->n / 2 + 1, st, conc, conc, herm_n != 0);
    };
    mark(0);
    const fc::FftParams fa = operand(d.a, a_in, specA), fb = operand(d.b, b_in, specB);
    const bool small_a = need_a && is_small(fa, false), small_b = need_b && is_small(fb, true);
    // the kernels of a pass overlap their ramp-up with the predecessor's drain where that
    // was measured to pay (see dep_launch.cuh)
    const bool overlap = !big && !timing && (tensor || plan->n >= 32 || d.K <= 64);

    fc::GemmParams gp{};
    gp.A = specA; gp.B = specB; gp.C = specC;
    gp.bins = plan->bins; gp.M = d.M; gp.N = d.N; gp.K = d.K;
    gp.lda = d.a.spec.ld; gp.ldb = d.b.spec.ld; gp.ldc = d.c.spec.ld;
    gp.transA = d.transA; gp.transB = d.transB; gp.conjA = d.conjA; gp.conjB = d.conjB;
    gp.wait_cycles = plan->wait_cycles;
    gp.nc = plan->n / 2 + 1;

    const int nc = plan->n / 2 + 1;
    const int chunks = (want_chunks && small_b) ? (plan->filter_chunks < nc ? plan->filter_chunks : nc) : 1;
    if (chunks > 1) {
        // Filter spectrum through the L2: the small-plane kernel can produce any range of rows
        // ky, so the filter operand is transformed and contracted range by range -- each part
        // of its spectrum is read back by the contraction right after it was written, while it
        // is still in the cache, instead of crossing HBM twice.
        bool launched = false;
        if (need_a) {
            if ((small_a ? forward_small(fa, false) : forward(fa, nullptr)) != cudaSuccess) return FFTCONV_ECUDA;
            launched = true;
        }
        // The transform of range c + 1 runs beside the contraction of range c: it is launched as
        // that contraction's programmatic dependent, starts without waiting (it touches nothing the
        // contraction touches) once the contraction has its operands, and completes only after it.
        for (int c = 0; c < chunks; ++c) {
            const int ky0 = (int)((long long)nc * c / chunks), ky1 = (int)((long long)nc * (c + 1) / chunks);
            g_launches.fetch_add(2, std::memory_order_relaxed);
            const bool dep = launched && !big;
            if (fc::launch_r2c_small(plan->n, fb, ky0, ky1, st, dep, dep) != cudaSuccess) return FFTCONV_ECUDA;
            launched = true;
            gp.ky_begin = ky0; gp.ky_count = ky1 - ky0;
            gp.overlap = big ? 0 : 1;
            gp.shared_sms = (!big && c + 1 < chunks) ? 1 : 0;
            if (fc::launch_cgemm_tc(gp, status, st) != cudaSuccess) return FFTCONV_ECUDA;
        }
        gp.shared_sms = 0;
        if (plan->reuse) {
            plan->cached[d.a.kind] = a_in;
            plan->cached[d.b.kind] = b_in;
        }
    } else {
    if (need_a && !small_a && need_b && !small_b && (!timing || plan->timing == 1)) {
        // both forward transforms in one launch: one ramp-up, one tail
        if (forward(fa, &fb) != cudaSuccess) return FFTCONV_ECUDA;
        mark(1);
        if (timing) plan->second_stage_used = false;
    } else {
        // one kernel per operand (small planes, spectrum reuse, or timing mode 2)
        bool launched = false;
        if (need_a && !small_a) { if (forward(fa, nullptr) != cudaSuccess) return FFTCONV_ECUDA; launched = true; }
        if (need_a && small_a) { if (forward_small(fa, launched) != cudaSuccess) return FFTCONV_ECUDA; launched = true; }
        mark(1);
        if (need_b && !small_b) { if (forward(fb, nullptr) != cudaSuccess) return FFTCONV_ECUDA; launched = true; }
        if (need_b && small_b) { if (forward_small(fb, launched) != cudaSuccess) return FFTCONV_ECUDA; }
        if (timing) plan->second_stage_used = need_b;
    }
    mark(2);
    if (plan->reuse) {
        plan->cached[d.a.kind] = a_in;
        plan->cached[d.b.kind] = b_in;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    gp.overlap = (overlap && (need_a || need_b)) ? 1 : 0;       // predecessor: this pass's forward transforms
    gp.herm_n = herm_n;
    cudaError_t ge;
    if (tensor) ge = fc::launch_cgemm_tc(gp, status, st);
    else ge = fc::launch_cgemm_ffma(gp, st);
    if (ge != cudaSuccess) return FFTCONV_ECUDA;
    }
    mark(3);

    fc::FftParams ip{};
    ip.spec_in = specC; ip.real_out = c_out;
    ip.h = d.c.h; ip.w = d.c.w;
    ip.R = d.c.spec.R; ip.C = d.c.spec.C; ip.ld = d.c.spec.ld;
    ip.win = d.c.win; ip.H = d.c.H; ip.W = d.c.W; ip.nty = d.c.nty; ip.ntx = d.c.ntx;
    ip.step_y = d.c.step_y; ip.step_x = d.c.step_x; ip.oy = d.c.oy; ip.ox = d.c.ox;
    ip.scale = 1.0f / ((float)plan->n * (float)plan->n);
    ip.accumulate = accumulate ? 1 : 0;
    ip.overlap = overlap ? 1 : 0;
    ip.status = status; ip.wait_cycles = plan->wait_cycles;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    // a small square crop (the filter gradient of accGrad) takes the pruned inverse kernel,
    // whose loads are whole 128-byte lines; everything else the butterfly kernels
    cudaError_t ie = plan->small_planes ? fc::launch_c2r_small(plan->n, ip, st) : cudaErrorNotSupported;
    if (ie == cudaErrorNotSupported)
        ie = big ? fc::launch_c2r_two_pass(plan->n, ip, scratch, scratch_bytes, st)
                 : fc::launch_c2r<true>(plan->n, ip, st);
    if (ie != cudaSuccess) return FFTCONV_ECUDA;
    mark(4);
    if (timing) plan->timed = true;
    return FFTCONV_OK;
}

}  // namespace

namespace {
double estimate_step_us(const conv_plan_s& p);
}

FFTCONV_API int conv_plan(conv_plan_t** out, int S, int f, int fprime, int h, int w, int kh,
                          int kw, int n) {
    if (!out) return FFTCONV_EINVAL;
    *out = nullptr;
    if (S < 1 || f < 1 || fprime < 1 || h < 1 || w < 1 || kh < 1 || kw < 1 || n < 1)
        return FFTCONV_EINVAL;
    if (kh > h || kw > w) return FFTCONV_EINVAL;
    // bases above 128 exist only as the frame of a tiled plan (planes up to 1024 x 1024)
    const bool frame_only = (n == 256 || n == 512 || n == 1024);
    if (!valid_n(n) && !frame_only) return FFTCONV_EUNSUPPORTED;
    if (n < h || n < w) return FFTCONV_EINVAL;
    // plane counts and per-tensor element counts must stay inside 31-bit grids / 63-bit offsets
    const long long planes_max = 1LL << 30;
    if ((long long)S * f > planes_max || (long long)S * fprime > planes_max ||
        (long long)f * fprime > planes_max)
        return FFTCONV_EUNSUPPORTED;
    conv_plan_s* p = new (std::nothrow) conv_plan_s();
    if (!p) return FFTCONV_EINVAL;
    p->S = S; p->f = f; p->fp = fprime; p->h = h; p->w = w; p->kh = kh; p->kw = kw; p->n = n;
    p->n_full = n;
    p->oh = h - kh + 1; p->ow = w - kw + 1;
    p->bins = n * (n / 2 + 1);
    p->math = FFTCONV_MATH_AUTO;
    p->ws = nullptr; p->ws_bytes = 0;
    p->timing = 0; p->timed = false; p->ev_made = false;
    p->reuse = 0; p->cached[0] = p->cached[1] = p->cached[2] = nullptr;
    p->wait_cycles = 0;
    p->small_planes = 1;
    p->filter_chunks = 1;
    if (frame_only) {
        // pick the tile basis now: the estimate ranks 8..64 against each other (the untiled
        // candidate does not exist), smallest admissible basis as the fallback
        int best = 0;
        double best_us = 0.0;
        const int cand[4] = {8, 16, 32, 64};
        for (int i = 0; i < 4; ++i) {
            if (conv_plan_set_tiling(p, cand[i]) != FFTCONV_OK) continue;
            const double us = estimate_step_us(*p);
            if (best == 0 || us < best_us) { best = cand[i]; best_us = us; }
        }
        if (best == 0 || conv_plan_set_tiling(p, best) != FFTCONV_OK) {
            delete p;
            return FFTCONV_EUNSUPPORTED;
        }
    }
    *out = p;
    return FFTCONV_OK;
}

FFTCONV_API int conv_plan_set_math(conv_plan_t* plan, int math) {
    if (!plan) return FFTCONV_EINVAL;
    if (math != FFTCONV_MATH_AUTO && math != FFTCONV_MATH_FP32 && math != FFTCONV_MATH_TF32)
        return FFTCONV_EUNSUPPORTED;
    plan->math = math;
    return FFTCONV_OK;
}

FFTCONV_API int conv_plan_effective_math(const conv_plan_t* plan) {
    if (!plan) return FFTCONV_EINVAL;
    // the mode all three passes share: TF32 only if every pass resolves to it
    for (int pass = 0; pass < 3; ++pass)
        if (resolve_math(*plan, describe(*plan, pass)) != FFTCONV_MATH_TF32) return FFTCONV_MATH_FP32;
    return FFTCONV_MATH_TF32;
}

FFTCONV_API int conv_plan_pass_math(const conv_plan_t* plan, int pass) {
    if (!plan || pass < 0 || pass > 2) return FFTCONV_EINVAL;
    return resolve_math(*plan, describe(*plan, pass));
}

FFTCONV_API size_t conv_plan_workspace_bytes(const conv_plan_t* plan) {
    if (!plan) return 0;
    return align_up(spectra_bytes(plan), kAlign) +
           (plan->n != plan->n_full ? 0 : fc::big_scratch_bytes(plan->n));
}

namespace {
// Plan-time estimate of one training step (three passes) in microseconds, from the bytes each
// kernel family moves and the rates measured for it on B200 (TB/s = bytes per picosecond):
// transforms 4.4 (n <= 32), 3.0 (n = 64), 2.2 (n = 128), windowed forward transforms 3.4
// (2.4 at n = 8: the fixed cost per window weighs more),
// contraction 5.5; plus a fixed cost per launch.  Only used to rank tile bases against each other.
double estimate_step_us(const conv_plan_s& p) {
    const bool tiled = p.n != p.n_full;
    const double fft_rate = p.n <= 32 ? 4.4e6 : (p.n == 64 ? 3.0e6 : 2.2e6);     // bytes per us
    const double win_rate = p.n >= 16 ? 3.4e6 : 2.4e6;
    double us = 0.0;
    for (int pass = 0; pass < 3; ++pass) {
        const PassDesc d = describe(p, pass);
        const OperandDesc* ops[3] = {&d.a, &d.b, &d.c};
        double spectra = 0.0;
        for (int i = 0; i < 3; ++i) {
            const OperandDesc& o = *ops[i];
            const double spec = (double)o.spec.bytes(p.bins);
            const double real = 4.0 * o.spec.R * o.spec.C * o.h * o.w;
            const bool windowed_load = tiled && o.win && i < 2;
            us += (spec + real) / (windowed_load ? win_rate : fft_rate);
            spectra += spec;
        }
        us += spectra / 5.5e6 + 3 * 4.0;
    }
    return us;
}
}  // namespace

FFTCONV_API int conv_plan_set_tiling(conv_plan_t* plan, int n_tile) {
    if (!plan) return FFTCONV_EINVAL;
    if (n_tile == FFTCONV_TILE_AUTO) {
        // keep the basis whose estimated step is shortest (the paper's autotuner measures; this
        // is a static ranking in the spirit of its one-strategy-per-problem-size cache)
        if (plan->reuse) return FFTCONV_EUNSUPPORTED;
        int best = 0;
        double best_us = 0.0;
        if (plan->n_full <= 128) {
            conv_plan_set_tiling(plan, 0);
            best_us = estimate_step_us(*plan);
        }
        const int cand[4] = {8, 16, 32, 64};
        for (int i = 0; i < 4; ++i) {
            if (cand[i] >= plan->n_full) break;
            if (conv_plan_set_tiling(plan, cand[i]) != FFTCONV_OK) continue;
            const double us = estimate_step_us(*plan);
            const bool first = (plan->n_full > 128 && best == 0);
            if (first || us < 0.9 * best_us) { best_us = us; best = cand[i]; }   // tiling must win clearly
        }
        return conv_plan_set_tiling(plan, best);
    }
    if (n_tile == 0 || n_tile == plan->n_full) {
        if (plan->n_full > 128) return FFTCONV_EUNSUPPORTED;   // such a basis exists only tiled
        plan->n = plan->n_full;
    } else {
        // one-pass transforms only; a tile must produce at least one output sample per axis
        if (n_tile != 8 && n_tile != 16 && n_tile != 32 && n_tile != 64) return FFTCONV_EUNSUPPORTED;
        if (n_tile > plan->n_full) return FFTCONV_EINVAL;
        if (n_tile < plan->kh || n_tile < plan->kw) return FFTCONV_EINVAL;
        if (plan->reuse) return FFTCONV_EUNSUPPORTED;
        const long long dh = n_tile - plan->kh + 1, dw = n_tile - plan->kw + 1;
        const long long T = ((plan->h + dh - 1) / dh) * ((plan->w + dw - 1) / dw);
        const long long pmax = plan->f > plan->fp ? plan->f : plan->fp;
        if ((long long)plan->S * T * pmax > (1LL << 30)) return FFTCONV_EUNSUPPORTED;
        plan->n = n_tile;
    }
    plan->bins = plan->n * (plan->n / 2 + 1);
    plan->cached[0] = plan->cached[1] = plan->cached[2] = nullptr;
    return FFTCONV_OK;
}

// ---------------------------------------------------------------------------
// Measured choice of the tile basis (the paper's autotuner, Section 3.4, times the candidate
// bases of a problem and keeps the fastest).
// ---------------------------------------------------------------------------
namespace {
const int kTuneCand[FFTCONV_TUNE_CANDIDATES] = {0, 8, 16, 32, 64};      // 0: untiled
}

FFTCONV_API size_t conv_plan_tune_workspace_bytes(conv_plan_t* plan) {
    if (!plan || plan->reuse) return 0;
    const int keep = plan->n != plan->n_full ? plan->n : 0;
    size_t m = 0;
    for (int i = 0; i < FFTCONV_TUNE_CANDIDATES; ++i) {
        if (kTuneCand[i] >= plan->n_full && kTuneCand[i] != 0) continue;
        if (conv_plan_set_tiling(plan, kTuneCand[i]) != FFTCONV_OK) continue;
        const size_t b = conv_plan_workspace_bytes(plan);
        if (b > m) m = b;
    }
    if (conv_plan_set_tiling(plan, keep) != FFTCONV_OK) return 0;
    return m;
}

FFTCONV_API int conv_plan_tune_tiling(conv_plan_t* plan, const float* x, const float* w, const float* dy,
                                      float* y, float* dx, float* dw, void* workspace,
                                      size_t workspace_bytes, int reps, void* cuda_stream,
                                      int* chosen_basis, float* step_ms) {
    if (!plan || !x || !w || !dy || !y || !dx || !dw || !workspace) return FFTCONV_EINVAL;
    if (plan->reuse) return FFTCONV_EUNSUPPORTED;
    if (reps < 1) reps = 1;
    if (reps > 100) reps = 100;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const int keep = plan->n != plan->n_full ? plan->n : 0;
    const int timing_keep = plan->timing;
    plan->timing = 0;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        if (e0) cudaEventDestroy(e0);
        plan->timing = timing_keep;
        return FFTCONV_ECUDA;
    }
    int best = -1, rc = FFTCONV_OK;
    float best_ms = 0.0f;
    for (int i = 0; i < FFTCONV_TUNE_CANDIDATES; ++i) {
        if (step_ms) step_ms[i] = -1.0f;
        const int cand = kTuneCand[i];
        if (cand != 0 && cand >= plan->n_full) continue;
        if (conv_plan_set_tiling(plan, cand) != FFTCONV_OK) continue;                  // not admissible
        if (conv_plan_set_workspace(plan, workspace, workspace_bytes) != FFTCONV_OK) continue;
        bool ok = true;
        for (int r = -1; r < reps && ok; ++r) {                                       // r = -1: warm-up
            if (r == 0) ok = cudaEventRecord(e0, st) == cudaSuccess;
            ok = ok && run_pass(plan, PASS_FPROP, x, w, y, 0, st) == FFTCONV_OK
                    && run_pass(plan, PASS_BPROP, dy, w, dx, 0, st) == FFTCONV_OK
                    && run_pass(plan, PASS_ACCGRAD, dy, x, dw, 0, st) == FFTCONV_OK;
        }
        float ms = 0.0f;
        ok = ok && cudaEventRecord(e1, st) == cudaSuccess && cudaEventSynchronize(e1) == cudaSuccess
                && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess && conv_plan_status(plan) == FFTCONV_OK;
        if (!ok) { rc = FFTCONV_ECUDA; break; }
        ms /= (float)reps;
        if (step_ms) step_ms[i] = ms;
        if (best < 0 || ms < best_ms) { best = cand; best_ms = ms; }
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    plan->timing = timing_keep;
    if (rc == FFTCONV_OK && best < 0) rc = FFTCONV_EUNSUPPORTED;
    // leave the plan on the fastest basis (on the one it had, after a failure) with the caller's workspace
    if (conv_plan_set_tiling(plan, rc == FFTCONV_OK ? best : keep) != FFTCONV_OK ||
        conv_plan_set_workspace(plan, workspace, workspace_bytes) != FFTCONV_OK)
        return rc == FFTCONV_OK ? FFTCONV_EWORKSPACE : rc;
    if (rc == FFTCONV_OK && chosen_basis) *chosen_basis = best;
    return rc;
}

FFTCONV_API int conv_plan_tile_basis(const conv_plan_t* plan) {
    if (!plan) return FFTCONV_EINVAL;
    return plan->n != plan->n_full ? plan->n : 0;
}

FFTCONV_API int conv_plan_set_workspace(conv_plan_t* plan, void* dev_ptr, size_t bytes) {
    if (!plan) return FFTCONV_EINVAL;
    if (!dev_ptr || (reinterpret_cast<uintptr_t>(dev_ptr) % kAlign) != 0 ||
        bytes < conv_plan_workspace_bytes(plan))
        return FFTCONV_EWORKSPACE;
    if (cudaMemset(dev_ptr, 0, kHeaderBytes) != cudaSuccess) return FFTCONV_ECUDA;
    plan->ws = dev_ptr;
    plan->ws_bytes = bytes;
    plan->cached[0] = plan->cached[1] = plan->cached[2] = nullptr;
    return FFTCONV_OK;
}

FFTCONV_API int conv_plan_set_spectrum_reuse(conv_plan_t* plan, int enable) {
    if (!plan) return FFTCONV_EINVAL;
    if (enable && plan->n != plan->n_full) return FFTCONV_EUNSUPPORTED;   // not with tiling
    plan->reuse = enable ? 1 : 0;
    plan->cached[0] = plan->cached[1] = plan->cached[2] = nullptr;
    return FFTCONV_OK;
}

FFTCONV_API int conv_plan_invalidate_spectra(conv_plan_t* plan) {
    if (!plan) return FFTCONV_EINVAL;
    plan->cached[0] = plan->cached[1] = plan->cached[2] = nullptr;
    return FFTCONV_OK;
}

FFTCONV_API int conv_fprop(conv_plan_t* plan, const float* x, const float* w, float* y,
                           void* cuda_stream) {
    return run_pass(plan, PASS_FPROP, x, w, y, 0, static_cast<cudaStream_t>(cuda_stream));
}

// ---------------------------------------------------------------------------
// fprop on the library's own fixed scratch array: for callers that cannot
// allocate (see the header).  The array is a file-scope device symbol; in host
// code its name is only a handle, so its device address is looked up once per
// device with cudaGetSymbolAddress and that pointer is what the kernels get.
// ---------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_noalloc_scratch[FFTCONV_NOALLOC_BYTES];

namespace {
constexpr int kMaxDevices = 64;
// Written at most once per device with one and the same value (the array's address on that
// device), so concurrent first calls from several host threads agree; atomic so that the
// race is a defined one.
std::atomic<void*> g_noalloc_ptr[kMaxDevices];

// Device address of the scratch array on the current device (nullptr on failure).
void* noalloc_scratch_address() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    void* ptr = g_noalloc_ptr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess) return nullptr;
        g_noalloc_ptr[dev].store(ptr, std::memory_order_release);
    }
    return ptr;
}
}  // namespace

FFTCONV_API int conv_fprop_noalloc(conv_plan_t* plan, const float* x, const float* w, float* y,
                                   void* cuda_stream) {
    if (!plan || !x || !w || !y) return FFTCONV_EINVAL;
    {
        conv_plan_s sized = *plan;      // the size of the ordinary (no-reuse) workspace layout
        sized.reuse = 0;
        if (conv_plan_workspace_bytes(&sized) > (size_t)FFTCONV_NOALLOC_BYTES) return FFTCONV_EWORKSPACE;
    }
    void* scratch = noalloc_scratch_address();
    if (!scratch) return FFTCONV_ECUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // the header (device status word) must start at zero; the spectra need no clearing
    // because every element the contraction and the inverse transform read is written first
    if (cudaMemsetAsync(scratch, 0, kHeaderBytes, st) != cudaSuccess) return FFTCONV_ECUDA;
    conv_plan_s local = *plan;          // same shape and math mode, library-owned scratch
    local.ws = scratch;
    local.ws_bytes = FFTCONV_NOALLOC_BYTES;
    local.reuse = 0;
    local.timing = 0;
    local.timed = false;
    local.ev_made = false;
    return run_pass(&local, PASS_FPROP, x, w, y, 0, st);
}

FFTCONV_API int conv_bprop(conv_plan_t* plan, const float* dy, const float* w, float* dx,
                           void* cuda_stream) {
    return run_pass(plan, PASS_BPROP, dy, w, dx, 0, static_cast<cudaStream_t>(cuda_stream));
}

FFTCONV_API int conv_accgrad(conv_plan_t* plan, const float* dy, const float* x, float* dw,
                             int accumulate, void* cuda_stream) {
    return run_pass(plan, PASS_ACCGRAD, dy, x, dw, accumulate,
                    static_cast<cudaStream_t>(cuda_stream));
}

FFTCONV_API int conv_plan_status(conv_plan_t* plan) {
    if (!plan) return FFTCONV_EINVAL;
    if (!plan->ws) return FFTCONV_EWORKSPACE;
    if (cudaDeviceSynchronize() != cudaSuccess) return FFTCONV_ECUDA;
    int word = 0;
    if (cudaMemcpy(&word, plan->ws, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
        return FFTCONV_ECUDA;
    if (word != 0) {
        cudaMemset(plan->ws, 0, sizeof(int));
        return FFTCONV_EDEVICE_TIMEOUT;
    }
    return FFTCONV_OK;
}

FFTCONV_API int conv_plan_set_wait_limit(conv_plan_t* plan, long long sm_cycles) {
    if (!plan || sm_cycles < 0) return FFTCONV_EINVAL;
    plan->wait_cycles = sm_cycles;
    return FFTCONV_OK;
}

FFTCONV_API int conv_plan_set_filter_chunks(conv_plan_t* plan, int chunks) {
    if (!plan || chunks < 0) return FFTCONV_EINVAL;
    plan->filter_chunks = chunks < 1 ? 1 : chunks;
    return FFTCONV_OK;
}

FFTCONV_API int conv_plan_set_small_plane_kernel(conv_plan_t* plan, int enable) {
    if (!plan) return FFTCONV_EINVAL;
    plan->small_planes = enable <= 0 ? 0 : (enable >= 2 ? 2 : 1);
    return FFTCONV_OK;
}

FFTCONV_API int conv_plan_destroy(conv_plan_t* plan) {
    if (plan && plan->ev_made)
        for (int i = 0; i < 5; ++i) cudaEventDestroy(plan->ev[i]);
    delete plan;
    return FFTCONV_OK;
}

FFTCONV_API int conv_plan_enable_stage_timing(conv_plan_t* plan, int enable) {
    if (!plan) return FFTCONV_EINVAL;
    if (enable && !plan->ev_made) {
        for (int i = 0; i < 5; ++i)
            if (cudaEventCreate(&plan->ev[i]) != cudaSuccess) {
                for (int j = 0; j < i; ++j) cudaEventDestroy(plan->ev[j]);
                return FFTCONV_ECUDA;
            }
        plan->ev_made = true;
    }
    plan->timing = enable ? (enable == 2 ? 2 : 1) : 0;
    plan->timed = false;
    return FFTCONV_OK;
}

FFTCONV_API int conv_plan_stage_times_ms(conv_plan_t* plan, float* out_ms) {
    if (!plan || !out_ms || !plan->timing || !plan->timed) return FFTCONV_EINVAL;
    if (cudaEventSynchronize(plan->ev[4]) != cudaSuccess) return FFTCONV_ECUDA;
    for (int i = 0; i < 4; ++i)
        if (cudaEventElapsedTime(&out_ms[i], plan->ev[i], plan->ev[i + 1]) != cudaSuccess)
            return FFTCONV_ECUDA;
    if (!plan->second_stage_used) out_ms[1] = 0.0f;      // nothing was launched there: two adjacent events
    return FFTCONV_OK;
}

FFTCONV_API int fft2d_r2c(const float* in, void* out_c, int batch, int h, int w, int n,
                          void* cuda_stream) {
    if (!in || !out_c || batch < 1 || h < 1 || w < 1) return FFTCONV_EINVAL;
    if (!valid_n(n)) return FFTCONV_EUNSUPPORTED;
    if (n < h || n < w) return FFTCONV_EINVAL;
    fc::FftParams p{};
    p.real_in = in; p.spec_out = static_cast<float*>(out_c);
    p.h = h; p.w = w; p.R = 1; p.C = batch; p.ld = batch;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return fc::launch_r2c<false>(n, p, nullptr, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
               ? FFTCONV_OK : FFTCONV_ECUDA;
}

FFTCONV_API int fft2d_c2r(const void* in_c, float* out, int batch, int n, int oh, int ow,
                          float scale, int accumulate, void* cuda_stream) {
    if (!in_c || !out || batch < 1 || oh < 1 || ow < 1) return FFTCONV_EINVAL;
    if (!valid_n(n)) return FFTCONV_EUNSUPPORTED;
    if (oh > n || ow > n) return FFTCONV_EINVAL;
    fc::FftParams p{};
    p.spec_in = static_cast<const float*>(in_c); p.real_out = out;
    p.h = oh; p.w = ow; p.R = 1; p.C = batch; p.ld = batch;
    p.scale = scale; p.accumulate = accumulate ? 1 : 0;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return fc::launch_c2r<false>(n, p, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
               ? FFTCONV_OK : FFTCONV_ECUDA;
}

FFTCONV_API int fft1d_r2c(const float* in, void* out_c, long long batch, int len, int n,
                          void* cuda_stream) {
    if (!in || !out_c || batch < 1 || len < 1) return FFTCONV_EINVAL;
    if (n < 2 || n > 256 || (n & (n - 1)) != 0) return FFTCONV_EUNSUPPORTED;
    if (len > n) return FFTCONV_EINVAL;
    if ((reinterpret_cast<uintptr_t>(out_c) & 7) != 0) return FFTCONV_EINVAL;
    fc::Fft1dParams p{};
    p.real_in = in; p.spec_out = static_cast<float2*>(out_c);
    p.batch = batch; p.len = len;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return fc::launch_fft1d(n, p, false, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
               ? FFTCONV_OK : FFTCONV_ECUDA;
}

FFTCONV_API int fft1d_c2r(const void* in_c, float* out, long long batch, int n, int olen,
                          float scale, int accumulate, void* cuda_stream) {
    if (!in_c || !out || batch < 1 || olen < 1) return FFTCONV_EINVAL;
    if (n < 2 || n > 256 || (n & (n - 1)) != 0) return FFTCONV_EUNSUPPORTED;
    if (olen > n) return FFTCONV_EINVAL;
    if ((reinterpret_cast<uintptr_t>(in_c) & 7) != 0) return FFTCONV_EINVAL;
    fc::Fft1dParams p{};
    p.spec_in = static_cast<const float2*>(in_c); p.real_out = out;
    p.batch = batch; p.len = olen; p.scale = scale; p.accumulate = accumulate ? 1 : 0;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return fc::launch_fft1d(n, p, true, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
               ? FFTCONV_OK : FFTCONV_ECUDA;
}

FFTCONV_API int fftconv_bin_contract(const float* A, const float* B, float* C, int bins, int M,
                                     int N, int K, int lda, int ldb, int ldc, int transA,
                                     int transB, int conjA, int conjB, int math,
                                     int* status_word, void* cuda_stream) {
    if (!A || !B || !C || bins < 1 || M < 1 || N < 1 || K < 1) return FFTCONV_EINVAL;
    if (lda < (transA ? M : K) || ldb < (transB ? N : K) || ldc < N || (lda & 3) || (ldb & 3) ||
        (ldc & 3))
        return FFTCONV_EINVAL;
    if (((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B) |
          reinterpret_cast<uintptr_t>(C)) & 15) != 0)
        return FFTCONV_EINVAL;
    if (bins > 65535) return FFTCONV_EUNSUPPORTED;
    fc::GemmParams gp{};
    gp.A = A; gp.B = B; gp.C = C;
    gp.bins = bins; gp.M = M; gp.N = N; gp.K = K;
    gp.lda = lda; gp.ldb = ldb; gp.ldc = ldc;
    gp.transA = transA ? 1 : 0; gp.transB = transB ? 1 : 0;
    gp.conjA = conjA ? 1 : 0; gp.conjB = conjB ? 1 : 0;
    int eff = math;
    if (math == FFTCONV_MATH_AUTO)
        eff = (fc::tc_shape_supported(M, N, K) && fc::tc_shape_profitable(M, N, K))
                  ? FFTCONV_MATH_TF32 : FFTCONV_MATH_FP32;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e;
    if (eff == FFTCONV_MATH_TF32) {
        if (!fc::tc_shape_supported(M, N, K)) return FFTCONV_EUNSUPPORTED;
        if (!status_word) return FFTCONV_EINVAL;
        g_launches.fetch_add(1, std::memory_order_relaxed);
        e = fc::launch_cgemm_tc(gp, status_word, st);
    } else if (eff == FFTCONV_MATH_FP32) {
        g_launches.fetch_add(1, std::memory_order_relaxed);
        e = fc::launch_cgemm_ffma(gp, st);
    } else {
        return FFTCONV_EUNSUPPORTED;
    }
    return e == cudaSuccess ? FFTCONV_OK : FFTCONV_ECUDA;
}

FFTCONV_API const char* fftconv_status_string(int status) {
    switch (status) {
        case FFTCONV_OK: return "ok";
        case FFTCONV_EINVAL: return "invalid argument";
        case FFTCONV_EUNSUPPORTED: return "unsupported size or mode";
        case FFTCONV_EWORKSPACE: return "workspace missing, misaligned or too small";
        case FFTCONV_ECUDA: return "CUDA call failed";
        case FFTCONV_EDEVICE_TIMEOUT: return "bounded device-side wait ran out";
    }
    return "unknown status";
}

FFTCONV_API unsigned long long fftconv_launch_count(void) {
    return g_launches.load(std::memory_order_relaxed);
}
