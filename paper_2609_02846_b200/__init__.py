"""UE5M3-FP4 quantize-and-multiply hot path for NVIDIA B200 (sm_100a).

The work is done by hand-written CUDA kernels behind the C ABI declared in ``include/ue5m3.h``
(``libue5m3.so``).  This package only marshals arguments: torch supplies device memory and streams.
There is no CPU or library fallback: importing :mod:`.binding` without the built library, or calling
an entry point without an sm_100 device, raises.
"""
from .binding import (  # noqa: F401
    BF16, BLOCK_32, F32, FPROP, DGRAD, WGRAD, LAYOUT_1D_COL, LAYOUT_1D_ROW, LAYOUT_2D, ROUND_RNE, ROUND_SR,
    SCALE_1D, SCALE_1D_TILED, SCALE_2D, SCALES_ROWMAJOR, SCALES_TILED,
    AmaxCache, QuantizedOperand, Ue5m3Error, gemm, gemm_fp16, gemm_native, gemm_native_workspace, gemm_static, native_windows, gemm_probe_matched, gemm_stall_selftest, last_device_status, library_path, linear_backward,
    linear_forward, quantize, quantize_current, quantize_dual, sample_amax, scales_bytes, status_string, unswizzle_scales,
)
