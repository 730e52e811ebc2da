"""Thin ctypes binding of libfftconv.so: same names as the C ABI, argument
marshalling only.  Tensors are torch CUDA tensors (torch supplies device memory
and streams, nothing else); every step of the computation runs inside the
library's CUDA kernels.  There is no fallback: if the library is missing or a
call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfftconv.so")

OK = 0
EINVAL, EUNSUPPORTED, EWORKSPACE, ECUDA, EDEVICE_TIMEOUT = -1, -2, -3, -4, -5
MATH_AUTO, MATH_FP32, MATH_TF32 = 0, 1, 2
TILE_AUTO = -1

EXPORTS = (
    "conv_plan", "conv_plan_set_math", "conv_plan_effective_math", "conv_plan_pass_math",
    "conv_plan_workspace_bytes",
    "conv_plan_set_workspace", "conv_plan_set_spectrum_reuse", "conv_plan_invalidate_spectra",
    "conv_plan_set_tiling", "conv_plan_tile_basis", "conv_plan_tune_tiling", "conv_plan_tune_workspace_bytes",
    "conv_fprop", "conv_fprop_noalloc", "conv_bprop", "conv_accgrad", "conv_plan_status",
    "conv_plan_set_wait_limit", "conv_plan_set_small_plane_kernel", "conv_plan_set_filter_chunks",
    "conv_plan_destroy", "conv_plan_enable_stage_timing", "conv_plan_stage_times_ms", "fft2d_r2c", "fft2d_c2r", "fft1d_r2c", "fft1d_c2r", "fftconv_bin_contract",
    "fftconv_status_string", "fftconv_launch_count",
)

_lib = None


class FftConvError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__("%s failed: %s (%d)" % (where, status_string(status), status))


def lib():
    """Load libfftconv.so (built by paper_1412_7580_b200.build); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                "libfftconv.so is not built: run `python -m paper_1412_7580_b200.build` "
                "(needs nvcc); there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        i, p, z, fl = ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_float
        L.conv_plan.argtypes = [ctypes.POINTER(p)] + [i] * 8
        L.conv_plan_set_math.argtypes = [p, i]
        L.conv_plan_effective_math.argtypes = [p]
        L.conv_plan_pass_math.argtypes = [p, i]
        L.conv_plan_workspace_bytes.argtypes = [p]
        L.conv_plan_workspace_bytes.restype = z
        L.conv_plan_set_workspace.argtypes = [p, p, z]
        L.conv_plan_set_spectrum_reuse.argtypes = [p, i]
        L.conv_plan_invalidate_spectra.argtypes = [p]
        L.conv_plan_set_tiling.argtypes = [p, i]
        L.conv_plan_tile_basis.argtypes = [p]
        L.conv_plan_tune_workspace_bytes.argtypes = [p]
        L.conv_plan_tune_workspace_bytes.restype = z
        L.conv_plan_tune_tiling.argtypes = [p, p, p, p, p, p, p, p, z, i, p, ctypes.POINTER(i),
                                            ctypes.POINTER(fl)]
        L.conv_fprop.argtypes = [p, p, p, p, p]
        L.conv_fprop_noalloc.argtypes = [p, p, p, p, p]
        L.conv_bprop.argtypes = [p, p, p, p, p]
        L.conv_accgrad.argtypes = [p, p, p, p, i, p]
        L.conv_plan_status.argtypes = [p]
        L.conv_plan_set_wait_limit.argtypes = [p, ctypes.c_longlong]
        L.conv_plan_set_small_plane_kernel.argtypes = [p, i]
        L.conv_plan_set_filter_chunks.argtypes = [p, i]
        L.conv_plan_destroy.argtypes = [p]
        L.conv_plan_enable_stage_timing.argtypes = [p, i]
        L.conv_plan_stage_times_ms.argtypes = [p, p]
        L.fft2d_r2c.argtypes = [p, p, i, i, i, i, p]
        L.fft2d_c2r.argtypes = [p, p, i, i, i, i, fl, i, p]
        L.fft1d_r2c.argtypes = [p, p, ctypes.c_longlong, i, i, p]
        L.fft1d_c2r.argtypes = [p, p, ctypes.c_longlong, i, i, fl, i, p]
        L.fftconv_bin_contract.argtypes = [p, p, p] + [i] * 12 + [p, p]
        L.fftconv_status_string.argtypes = [i]
        L.fftconv_status_string.restype = ctypes.c_char_p
        L.fftconv_launch_count.argtypes = []
        L.fftconv_launch_count.restype = ctypes.c_ulonglong
        for name in EXPORTS:
            fn = getattr(L, name)
            if name not in ("conv_plan_workspace_bytes", "conv_plan_tune_workspace_bytes",
                            "fftconv_status_string", "fftconv_launch_count"):
                fn.restype = i
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().fftconv_status_string(int(status)).decode()


def fftconv_launch_count() -> int:
    return int(lib().fftconv_launch_count())


def _check(status, where):
    if status != OK:
        raise FftConvError(status, where)


def _stream_ptr(stream):
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _dev(t, dims=None, what="tensor"):
    import torch
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32
            and t.is_contiguous()):
        raise TypeError("%s must be a contiguous float32 CUDA tensor" % what)
    if dims is not None and tuple(t.shape) != tuple(dims):
        raise ValueError("%s has shape %s, expected %s" % (what, tuple(t.shape), tuple(dims)))
    return ctypes.c_void_p(t.data_ptr())


class Plan:
    """Handle of a conv_plan_t plus the workspace tensor that was lent to it."""

    def __init__(self, handle, dims):
        self._h = handle
        (self.S, self.f, self.fp, self.h, self.w, self.kh, self.kw, self.n) = dims
        self.oh, self.ow = self.h - self.kh + 1, self.w - self.kw + 1
        self.workspace = None

    @property
    def handle(self):
        if self._h is None:
            raise ValueError("plan destroyed")
        return self._h

    def __del__(self):
        try:
            if self._h is not None and _lib is not None:
                _lib.conv_plan_destroy(self._h)
                self._h = None
        except Exception:
            pass


def conv_plan(S, f, fprime, h, w, kh, kw, n) -> Plan:
    out = ctypes.c_void_p()
    dims = tuple(int(v) for v in (S, f, fprime, h, w, kh, kw, n))
    _check(lib().conv_plan(ctypes.byref(out), *dims), "conv_plan")
    return Plan(out, dims)


def conv_plan_set_math(plan: Plan, math: int) -> None:
    _check(lib().conv_plan_set_math(plan.handle, int(math)), "conv_plan_set_math")


def conv_plan_effective_math(plan: Plan) -> int:
    return int(lib().conv_plan_effective_math(plan.handle))


def conv_plan_pass_math(plan: Plan, which: int) -> int:
    """Math mode of pass 0 (fprop), 1 (bprop) or 2 (accGrad) once AUTO is resolved."""
    r = int(lib().conv_plan_pass_math(plan.handle, int(which)))
    if r < 0:
        raise FftConvError(r, "conv_plan_pass_math")
    return r


def conv_plan_workspace_bytes(plan: Plan) -> int:
    return int(lib().conv_plan_workspace_bytes(plan.handle))


def conv_plan_set_workspace(plan: Plan, workspace) -> None:
    """`workspace`: a uint8 / any-dtype CUDA tensor the caller keeps alive."""
    nbytes = workspace.numel() * workspace.element_size()
    _check(lib().conv_plan_set_workspace(plan.handle, ctypes.c_void_p(workspace.data_ptr()),
                                         nbytes), "conv_plan_set_workspace")
    plan.workspace = workspace


def conv_plan_set_spectrum_reuse(plan: Plan, enable=True) -> None:
    """Keep the forward spectra between fprop / bprop / accGrad of one step (changes the
    workspace size: size and lend the workspace after this call)."""
    _check(lib().conv_plan_set_spectrum_reuse(plan.handle, int(bool(enable))),
           "conv_plan_set_spectrum_reuse")


def conv_plan_set_tiling(plan: Plan, n_tile: int) -> None:
    """Spatial tiling with an n_tile x n_tile basis (0 = off); changes the workspace size:
    size and lend the workspace after this call."""
    _check(lib().conv_plan_set_tiling(plan.handle, int(n_tile)), "conv_plan_set_tiling")
    plan.workspace = None


def conv_plan_tile_basis(plan: Plan) -> int:
    return lib().conv_plan_tile_basis(plan.handle)


TUNE_CANDIDATES = (0, 8, 16, 32, 64)


def conv_plan_tune_workspace_bytes(plan: Plan) -> int:
    """Bytes of the largest workspace any candidate basis of conv_plan_tune_tiling needs."""
    return int(lib().conv_plan_tune_workspace_bytes(plan.handle))


def conv_plan_tune_tiling(plan: Plan, x, w, dy, y, dx, dw, workspace, reps=3, stream=None):
    """Measured choice of the tile basis: times a training step for the untiled basis and every
    admissible tile basis on the given CUDA tensors and leaves the plan on the fastest, with
    `workspace` lent to it (a CUDA tensor; conv_plan_tune_workspace_bytes(plan) bytes hold every
    candidate, a candidate that needs more than the tensor has is left out).  Returns (chosen basis, {basis: step time in ms}) with 0 for the untiled basis."""
    nbytes = workspace.numel() * workspace.element_size()
    chosen = ctypes.c_int(-1)
    ms = (ctypes.c_float * len(TUNE_CANDIDATES))()
    _check(lib().conv_plan_tune_tiling(plan.handle,
                                       _dev(x, (plan.S, plan.f, plan.h, plan.w), "x"),
                                       _dev(w, (plan.fp, plan.f, plan.kh, plan.kw), "w"),
                                       _dev(dy, (plan.S, plan.fp, plan.oh, plan.ow), "dy"),
                                       _dev(y, (plan.S, plan.fp, plan.oh, plan.ow), "y"),
                                       _dev(dx, (plan.S, plan.f, plan.h, plan.w), "dx"),
                                       _dev(dw, (plan.fp, plan.f, plan.kh, plan.kw), "dw"),
                                       ctypes.c_void_p(workspace.data_ptr()), nbytes, int(reps),
                                       _stream_ptr(stream), ctypes.byref(chosen), ms),
           "conv_plan_tune_tiling")
    plan.workspace = workspace
    return int(chosen.value), {b: float(ms[i]) for i, b in enumerate(TUNE_CANDIDATES) if ms[i] >= 0.0}


def conv_plan_invalidate_spectra(plan: Plan) -> None:
    _check(lib().conv_plan_invalidate_spectra(plan.handle), "conv_plan_invalidate_spectra")


def conv_plan_alloc_workspace(plan: Plan, device="cuda"):
    """Convenience: allocate the workspace with torch and lend it to the plan."""
    import torch
    ws = torch.empty(conv_plan_workspace_bytes(plan), dtype=torch.uint8, device=device)
    conv_plan_set_workspace(plan, ws)
    return ws


def conv_fprop(plan: Plan, x, w, y, stream=None) -> None:
    _check(lib().conv_fprop(plan.handle,
                            _dev(x, (plan.S, plan.f, plan.h, plan.w), "x"),
                            _dev(w, (plan.fp, plan.f, plan.kh, plan.kw), "w"),
                            _dev(y, (plan.S, plan.fp, plan.oh, plan.ow), "y"),
                            _stream_ptr(stream)), "conv_fprop")


NOALLOC_BYTES = 32 << 20


def conv_fprop_noalloc(plan: Plan, x, w, y, stream=None) -> None:
    """conv_fprop on the library's built-in 32 MiB scratch array: for callers that
    hold tensors but cannot allocate a workspace.  The plan needs no workspace; plans
    that need more than NOALLOC_BYTES are refused (FftConvError, EWORKSPACE).  Calls
    share the array, so do not let two of them overlap on the GPU; make the first call
    on a device outside any stream capture."""
    _check(lib().conv_fprop_noalloc(plan.handle,
                                    _dev(x, (plan.S, plan.f, plan.h, plan.w), "x"),
                                    _dev(w, (plan.fp, plan.f, plan.kh, plan.kw), "w"),
                                    _dev(y, (plan.S, plan.fp, plan.oh, plan.ow), "y"),
                                    _stream_ptr(stream)), "conv_fprop_noalloc")


def conv_bprop(plan: Plan, dy, w, dx, stream=None) -> None:
    _check(lib().conv_bprop(plan.handle,
                            _dev(dy, (plan.S, plan.fp, plan.oh, plan.ow), "dy"),
                            _dev(w, (plan.fp, plan.f, plan.kh, plan.kw), "w"),
                            _dev(dx, (plan.S, plan.f, plan.h, plan.w), "dx"),
                            _stream_ptr(stream)), "conv_bprop")


def conv_accgrad(plan: Plan, dy, x, dw, accumulate=False, stream=None) -> None:
    _check(lib().conv_accgrad(plan.handle,
                              _dev(dy, (plan.S, plan.fp, plan.oh, plan.ow), "dy"),
                              _dev(x, (plan.S, plan.f, plan.h, plan.w), "x"),
                              _dev(dw, (plan.fp, plan.f, plan.kh, plan.kw), "dw"),
                              int(bool(accumulate)), _stream_ptr(stream)), "conv_accgrad")


def conv_plan_status(plan: Plan) -> int:
    return int(lib().conv_plan_status(plan.handle))


def conv_plan_set_small_plane_kernel(plan: Plan, enable=1) -> None:
    """Pruned-DFT kernels for small planes: 0 never, 1 where measured to pay (default), 2 wherever they apply."""
    _check(lib().conv_plan_set_small_plane_kernel(plan.handle, int(enable)),
           "conv_plan_set_small_plane_kernel")


def conv_plan_set_filter_chunks(plan: Plan, chunks: int) -> None:
    """fprop / bprop: transform and contract the filters in this many ranges of frequency rows."""
    _check(lib().conv_plan_set_filter_chunks(plan.handle, int(chunks)), "conv_plan_set_filter_chunks")


def conv_plan_set_wait_limit(plan: Plan, sm_cycles: int) -> None:
    """Limit of one bounded device-side wait in SM cycles (0 = default, about a second)."""
    _check(lib().conv_plan_set_wait_limit(plan.handle, int(sm_cycles)), "conv_plan_set_wait_limit")


def conv_plan_enable_stage_timing(plan: Plan, enable=1) -> None:
    """0 off; 1 time the normal launch sequence; 2 launch the two forward FFTs apart."""
    _check(lib().conv_plan_enable_stage_timing(plan.handle, int(enable)),
           "conv_plan_enable_stage_timing")


def conv_plan_stage_times_ms(plan: Plan):
    """Milliseconds of the last timed pass: forward FFT A (mode 1: A and B fused), forward
    FFT B (mode 1: 0), contraction, inverse FFT."""
    buf = (ctypes.c_float * 4)()
    _check(lib().conv_plan_stage_times_ms(plan.handle, ctypes.cast(buf, ctypes.c_void_p)),
           "conv_plan_stage_times_ms")
    return [float(v) for v in buf]


def conv_plan_destroy(plan: Plan) -> None:
    if plan._h is not None:
        lib().conv_plan_destroy(plan._h)
        plan._h = None


def fft2d_r2c(inp, out_c, n, stream=None) -> None:
    """inp: [batch, h, w] float32; out_c: [batch, n, n/2+1, 2] float32 (re, im)."""
    batch, h, w = inp.shape
    _check(lib().fft2d_r2c(_dev(inp, None, "in"), _dev(out_c, (batch, n, n // 2 + 1, 2), "out_c"),
                           batch, h, w, int(n), _stream_ptr(stream)), "fft2d_r2c")


def fft2d_c2r(in_c, out, n, scale, accumulate=False, stream=None) -> None:
    """in_c: [batch, n, n/2+1, 2] float32; out: [batch, oh, ow] float32."""
    batch, oh, ow = out.shape
    _check(lib().fft2d_c2r(_dev(in_c, (batch, n, n // 2 + 1, 2), "in_c"), _dev(out, None, "out"),
                           batch, int(n), oh, ow, float(scale), int(bool(accumulate)),
                           _stream_ptr(stream)), "fft2d_c2r")


def fft1d_r2c(inp, out_c, n, stream=None) -> None:
    """inp: [batch, len] float32; out_c: [batch, n/2+1, 2] float32 (re, im)."""
    batch, ln = inp.shape
    _check(lib().fft1d_r2c(_dev(inp, None, "in"), _dev(out_c, (batch, n // 2 + 1, 2), "out_c"),
                           batch, ln, int(n), _stream_ptr(stream)), "fft1d_r2c")


def fft1d_c2r(in_c, out, n, scale, accumulate=False, stream=None) -> None:
    """in_c: [batch, n/2+1, 2] float32; out: [batch, olen] float32."""
    batch, olen = out.shape
    _check(lib().fft1d_c2r(_dev(in_c, (batch, n // 2 + 1, 2), "in_c"), _dev(out, None, "out"),
                           batch, int(n), olen, float(scale), int(bool(accumulate)),
                           _stream_ptr(stream)), "fft1d_c2r")


def fftconv_bin_contract(A, B, C, M, N, K, transA=False, transB=False, conjA=False, conjB=False,
                         math=MATH_FP32, status_word=None, stream=None) -> None:
    """Planar float32 operands: A [2, bins, M, lda] (or [2, bins, K, lda] with transA),
    B [2, bins, N, ldb] (or [2, bins, K, ldb] with transB), C [2, bins, M, ldc]."""
    bins = A.shape[1]
    assert A.shape[0] == 2 and B.shape[:2] == (2, bins) and C.shape[:3] == (2, bins, M)
    assert A.shape[2] == (K if transA else M) and B.shape[2] == (K if transB else N)
    lda, ldb, ldc = A.shape[3], B.shape[3], C.shape[3]
    sw = ctypes.c_void_p(status_word.data_ptr()) if status_word is not None else ctypes.c_void_p()
    _check(lib().fftconv_bin_contract(_dev(A, None, "A"), _dev(B, None, "B"), _dev(C, None, "C"),
                                      bins, int(M), int(N), int(K), lda, ldb, ldc,
                                      int(bool(transA)), int(bool(transB)), int(bool(conjA)),
                                      int(bool(conjB)), int(math), sw, _stream_ptr(stream)),
           "fftconv_bin_contract")
