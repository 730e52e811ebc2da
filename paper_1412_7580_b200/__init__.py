"""FFT-domain convolution for CNN layers on NVIDIA B200 (sm_100a).

`binding` wraps the C ABI of libfftconv.so (include/fftconv.h); `workloads`
holds the seeded synthetic inputs; `build` compiles the library with nvcc.
The compute path is the CUDA library only -- there is no CPU fallback.
"""
from . import workloads  # noqa: F401
from .binding import (  # noqa: F401
    MATH_AUTO, MATH_FP32, MATH_TF32, TILE_AUTO, FftConvError, Plan, conv_accgrad, conv_bprop, conv_fprop, conv_fprop_noalloc,
    conv_plan, conv_plan_alloc_workspace, conv_plan_destroy, conv_plan_effective_math, conv_plan_pass_math, conv_plan_enable_stage_timing,
    conv_plan_stage_times_ms,
    conv_plan_set_math, conv_plan_set_tiling, conv_plan_tile_basis, conv_plan_tune_tiling, conv_plan_tune_workspace_bytes, conv_plan_set_spectrum_reuse, conv_plan_invalidate_spectra, conv_plan_set_workspace, conv_plan_set_wait_limit, conv_plan_set_small_plane_kernel, conv_plan_set_filter_chunks, conv_plan_status, conv_plan_workspace_bytes,
    fft1d_c2r, fft1d_r2c, fft2d_c2r, fft2d_r2c, fftconv_bin_contract, fftconv_launch_count, status_string,
)
