"""CPU oracle (float64, plain definitions) -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  The product package never does.  The arithmetic lives in
``oracle.c`` (plain C, nested sums, OpenMP over independent outputs); this file
only builds that C file with gcc, loads it with ctypes and marshals numpy
arrays.

Functions (paper notation: S, f, fp = f', h, w, kh, kw, n):
  fprop(x, w)            -> y   float64 [S, fp, oh, ow]   (Section 2, eq. 1)
  bprop(dy, w, h, w_)    -> dx  float64 [S, f, h, w]      (Section 2, eq. 2)
  accgrad(dy, x, kh, kw) -> dw  float64 [fp, f, kh, kw]   (Section 2, eq. 3)
  *_at(..., coords)      -> the same elements at sampled coordinates
  dft2d_r2c(x, n)        -> complex128 [batch, n, n/2+1]  (Supplement 8.2)
  idft2d_c2r(X, n, oh, ow, scale) -> float64 [batch, oh, ow]
  dft1d_r2c(x, n)        -> complex128 [batch, n/2+1]     (Supplement 8.2)
  idft1d_c2r(X, n, olen, scale)   -> float64 [batch, olen]
  bin_contract(A, B, conjA, conjB) -> complex128 [bins, M, N] (Table 1, Cgemm)
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile oracle.c into liboracle.so with gcc (no CUDA involved)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
           "-fvisibility=hidden", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i, l, d = ctypes.c_int, ctypes.c_long, ctypes.c_double
        p = ctypes.c_void_p
        lib.oracle_num_threads.restype = i
        lib.oracle_fprop.argtypes = [p, p, p] + [i] * 7
        lib.oracle_bprop.argtypes = [p, p, p] + [i] * 7
        lib.oracle_accgrad.argtypes = [p, p, p] + [i] * 7
        for name in ("oracle_fprop_at", "oracle_bprop_at", "oracle_accgrad_at"):
            getattr(lib, name).argtypes = [p, p, p, l, p] + [i] * 7
        lib.oracle_dft2d_r2c.argtypes = [p, p, l, i, i, i]
        lib.oracle_idft2d_c2r.argtypes = [p, p, l, i, i, i, d]
        lib.oracle_dft1d_r2c.argtypes = [p, p, l, i, i]
        lib.oracle_idft1d_c2r.argtypes = [p, p, l, i, i, d]
        lib.oracle_bin_contract.argtypes = [p, p, p, l, i, i, i, i, i]
        for name in ("oracle_fprop", "oracle_bprop", "oracle_accgrad",
                     "oracle_fprop_at", "oracle_bprop_at", "oracle_accgrad_at",
                     "oracle_dft2d_r2c", "oracle_idft2d_c2r", "oracle_bin_contract"):
            getattr(lib, name).restype = None
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def fprop(x, w):
    x, w = _f32(x), _f32(w)
    S, f, h, wd = x.shape
    fp, f2, kh, kw = w.shape
    assert f2 == f and kh <= h and kw <= wd
    y = np.empty((S, fp, h - kh + 1, wd - kw + 1), dtype=np.float64)
    _load().oracle_fprop(_ptr(x), _ptr(w), _ptr(y), S, f, fp, h, wd, kh, kw)
    return y


def bprop(dy, w, h, wd):
    dy, w = _f32(dy), _f32(w)
    S, fp, oh, ow = dy.shape
    fp2, f, kh, kw = w.shape
    assert fp2 == fp and oh == h - kh + 1 and ow == wd - kw + 1
    dx = np.empty((S, f, h, wd), dtype=np.float64)
    _load().oracle_bprop(_ptr(dy), _ptr(w), _ptr(dx), S, f, fp, h, wd, kh, kw)
    return dx


def accgrad(dy, x, kh, kw):
    dy, x = _f32(dy), _f32(x)
    S, fp, oh, ow = dy.shape
    S2, f, h, wd = x.shape
    assert S2 == S and oh == h - kh + 1 and ow == wd - kw + 1
    dw = np.empty((fp, f, kh, kw), dtype=np.float64)
    _load().oracle_accgrad(_ptr(dy), _ptr(x), _ptr(dw), S, f, fp, h, wd, kh, kw)
    return dw


def _coords(c):
    c = np.ascontiguousarray(c, dtype=np.int32)
    assert c.ndim == 2 and c.shape[1] == 4
    return c


def fprop_at(x, w, coords):
    """coords rows are (s, j, a, b)."""
    x, w, c = _f32(x), _f32(w), _coords(coords)
    S, f, h, wd = x.shape
    fp, _, kh, kw = w.shape
    out = np.empty(len(c), dtype=np.float64)
    _load().oracle_fprop_at(_ptr(x), _ptr(w), _ptr(c), len(c), _ptr(out),
                            S, f, fp, h, wd, kh, kw)
    return out


def bprop_at(dy, w, h, wd, coords):
    """coords rows are (s, i, p, q)."""
    dy, w, c = _f32(dy), _f32(w), _coords(coords)
    S, fp, oh, ow = dy.shape
    _, f, kh, kw = w.shape
    assert oh == h - kh + 1 and ow == wd - kw + 1
    out = np.empty(len(c), dtype=np.float64)
    _load().oracle_bprop_at(_ptr(dy), _ptr(w), _ptr(c), len(c), _ptr(out),
                            S, f, fp, h, wd, kh, kw)
    return out


def accgrad_at(dy, x, kh, kw, coords):
    """coords rows are (j, i, u, v)."""
    dy, x, c = _f32(dy), _f32(x), _coords(coords)
    S, fp, oh, ow = dy.shape
    _, f, h, wd = x.shape
    assert oh == h - kh + 1 and ow == wd - kw + 1
    out = np.empty(len(c), dtype=np.float64)
    _load().oracle_accgrad_at(_ptr(dy), _ptr(x), _ptr(c), len(c), _ptr(out),
                              S, f, fp, h, wd, kh, kw)
    return out


def dft2d_r2c(x, n):
    x = _f32(x)
    batch, h, wd = x.shape
    assert n >= h and n >= wd
    out = np.empty((batch, n, n // 2 + 1), dtype=np.complex128)
    _load().oracle_dft2d_r2c(_ptr(x), _ptr(out), batch, h, wd, n)
    return out


def idft2d_c2r(X, n, oh, ow, scale):
    X = np.ascontiguousarray(X, dtype=np.complex128)
    batch = X.shape[0]
    assert X.shape[1:] == (n, n // 2 + 1)
    out = np.empty((batch, oh, ow), dtype=np.float64)
    _load().oracle_idft2d_c2r(_ptr(X), _ptr(out), batch, n, oh, ow, float(scale))
    return out


def dft1d_r2c(x, n):
    x = _f32(x)
    batch, ln = x.shape
    assert n >= ln
    out = np.empty((batch, n // 2 + 1), dtype=np.complex128)
    _load().oracle_dft1d_r2c(_ptr(x), _ptr(out), batch, ln, n)
    return out


def idft1d_c2r(X, n, olen, scale):
    X = np.ascontiguousarray(X, dtype=np.complex128)
    batch = X.shape[0]
    assert X.shape[1:] == (n // 2 + 1,)
    out = np.empty((batch, olen), dtype=np.float64)
    _load().oracle_idft1d_c2r(_ptr(X), _ptr(out), batch, n, olen, float(scale))
    return out


def bin_contract(A, B, conjA=False, conjB=False):
    """C[b,m,n] = sum_k op(A[b,m,k]) * op(B[b,n,k])."""
    A = np.ascontiguousarray(A, dtype=np.complex128)
    B = np.ascontiguousarray(B, dtype=np.complex128)
    bins, M, K = A.shape
    bins2, N, K2 = B.shape
    assert bins2 == bins and K2 == K
    C = np.empty((bins, M, N), dtype=np.complex128)
    _load().oracle_bin_contract(_ptr(A), _ptr(B), _ptr(C), bins, M, N, K,
                                int(conjA), int(conjB))
    return C
