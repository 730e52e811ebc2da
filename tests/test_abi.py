"""Host-side checks that need no GPU: the library builds, loads and exports
every symbol the public header declares; plan validation and workspace sizing."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_1412_7580_b200 import build, binding
    build.build()
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fftconv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b([a-z_0-9]+)\s*\([^;{]*\)\s*;", text)
    return sorted(set(names))


def test_header_symbols_are_exported(L):
    names = declared_functions()
    assert {"conv_plan", "conv_fprop", "conv_bprop", "conv_accgrad", "fft2d_r2c",
            "fft2d_c2r"} <= set(names)
    for n in names:
        assert hasattr(L, n), "libfftconv.so does not export %s" % n
    from paper_1412_7580_b200 import binding
    assert set(binding.EXPORTS) == set(names)


def test_binding_has_same_names():
    import paper_1412_7580_b200 as pkg
    for n in ("conv_plan", "conv_fprop", "conv_bprop", "conv_accgrad", "fft2d_r2c", "fft2d_c2r"):
        assert callable(getattr(pkg, n))


def test_no_torch_or_oracle_in_library_link():
    # the product library may not depend on the oracle or on torch
    from paper_1412_7580_b200 import binding
    out = os.popen("ldd %s" % binding.LIB_PATH).read()
    assert "oracle" not in out and "torch" not in out and "libcuda.so" not in out


def test_plan_validation(L):
    from paper_1412_7580_b200 import binding as b
    h = ctypes.c_void_p()

    def plan(*a):
        return L.conv_plan(ctypes.byref(h), *a)

    assert plan(8, 4, 8, 16, 16, 3, 3, 16) == b.OK
    assert L.conv_plan_workspace_bytes(h) > 0
    assert L.conv_plan_destroy(h) == b.OK
    assert L.conv_plan(None, 8, 4, 8, 16, 16, 3, 3, 16) == b.EINVAL
    assert plan(0, 4, 8, 16, 16, 3, 3, 16) == b.EINVAL
    assert plan(8, 4, 8, 16, 16, 17, 3, 16) == b.EINVAL       # kh > h
    assert plan(8, 4, 8, 16, 16, 3, 3, 8) == b.EINVAL         # n < h
    assert plan(8, 4, 8, 16, 16, 3, 3, 24) == b.EUNSUPPORTED  # not a power of two
    assert plan(8, 4, 8, 16, 16, 3, 3, 2048) == b.EUNSUPPORTED
    # 256, 512, 1024: accepted as the frame of a tiled plan, which cannot be untiled
    assert plan(2, 4, 8, 200, 200, 3, 3, 256) == b.OK
    assert L.conv_plan_tile_basis(h) in (8, 16, 32, 64)
    assert L.conv_plan_set_tiling(h, 0) == b.EUNSUPPORTED
    assert L.conv_plan_set_tiling(h, b.TILE_AUTO) == b.OK and L.conv_plan_tile_basis(h) > 0
    # the measured tuner: workspace of the largest candidate, plan left on the basis it had;
    # null tensors are refused before anything runs
    basis = L.conv_plan_tile_basis(h)
    assert L.conv_plan_tune_workspace_bytes(h) >= L.conv_plan_workspace_bytes(h)
    assert L.conv_plan_tile_basis(h) == basis
    assert L.conv_plan_tune_tiling(h, None, None, None, None, None, None, None, 0, 1, None, None, None) == b.EINVAL
    assert L.conv_plan_destroy(h) == b.OK
    assert plan(8, 4, 8, 4, 4, 3, 3, 4) == b.EUNSUPPORTED
    # rectangular planes and kernels are accepted
    assert plan(2, 3, 4, 13, 9, 5, 2, 16) == b.OK
    assert L.conv_plan_destroy(h) == b.OK


def test_workspace_bytes_cover_all_three_spectra(L):
    from paper_1412_7580_b200 import binding as b
    S, f, fp, hh, ww, k, n = 128, 96, 256, 31, 31, 5, 32
    p = b.conv_plan(S, f, fp, hh, ww, k, k, n)
    b.conv_plan_set_math(p, b.MATH_FP32)
    bins = n * (n // 2 + 1)
    need = bins * 8 * (S * f + fp * f + S * fp)    # complex fp32 per bin per plane
    got = b.conv_plan_workspace_bytes(p)
    assert need <= got <= need * 1.05 + 4096
    assert b.conv_plan_set_math(p, b.MATH_TF32) is None
    with pytest.raises(b.FftConvError):
        b.conv_plan_set_math(p, 7)
    b.conv_plan_destroy(p)


def test_calls_without_workspace_or_pointers_fail_cleanly(L):
    from paper_1412_7580_b200 import binding as b
    p = b.conv_plan(2, 2, 2, 8, 8, 3, 3, 8)
    z = ctypes.c_void_p(0)
    assert L.conv_fprop(p.handle, z, z, z, z) == b.EINVAL
    one = ctypes.c_void_p(256)
    assert L.conv_fprop(p.handle, one, one, one, z) == b.EWORKSPACE
    assert L.conv_plan_set_workspace(p.handle, ctypes.c_void_p(3), 1 << 30) == b.EWORKSPACE
    assert L.conv_plan_status(p.handle) == b.EWORKSPACE
    assert L.fft2d_r2c(one, one, 1, 9, 9, 8, z) == b.EINVAL
    assert L.fft2d_r2c(one, one, 1, 8, 8, 12, z) == b.EUNSUPPORTED
    assert L.fft2d_c2r(one, one, 1, 8, 9, 8, 1.0, 0, z) == b.EINVAL
    assert b.status_string(b.EWORKSPACE).startswith("workspace")
    b.conv_plan_destroy(p)


def test_tiling_argument_checks(L):
    import paper_1412_7580_b200 as fc
    p = fc.conv_plan(2, 3, 4, 31, 31, 9, 9, 32)
    with pytest.raises(fc.FftConvError) as e:
        fc.conv_plan_set_tiling(p, 12)                 # not a supported basis
    assert e.value.status == fc.binding.EUNSUPPORTED
    with pytest.raises(fc.FftConvError) as e:
        fc.conv_plan_set_tiling(p, 8)                  # smaller than the kernel
    assert e.value.status == fc.binding.EINVAL
    with pytest.raises(fc.FftConvError) as e:
        fc.conv_plan_set_tiling(p, 64)                 # larger than the plan's basis
    assert e.value.status == fc.binding.EINVAL
    before = fc.conv_plan_workspace_bytes(p)
    fc.conv_plan_set_tiling(p, 16)
    assert fc.conv_plan_tile_basis(p) == 16 and fc.conv_plan_workspace_bytes(p) != before
    with pytest.raises(fc.FftConvError) as e:
        fc.conv_plan_set_spectrum_reuse(p, True)       # the passes use different windows
    assert e.value.status == fc.binding.EUNSUPPORTED
    fc.conv_plan_set_tiling(p, 0)
    assert fc.conv_plan_tile_basis(p) == 0 and fc.conv_plan_workspace_bytes(p) == before
    fc.conv_plan_destroy(p)
