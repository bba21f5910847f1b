"""B200-native Winograd convolution F(m x m, 3 x 3) for arbitrary point sets.

Thin Python binding over the C ABI in include/nova.h (libnova.so, built by
paper_2512_18453_b200.build).  PyTorch is used for device memory and streams
only; every step of the computation runs in the library's CUDA kernels.
"""
from .binding import (  # noqa: F401
    NovaError, Plan, lib, status_string, maxpool2x2, snap_to_rational, verify_decomposition, symmetric_search,
    FP32, FP16_F32ACC, COEF_ROUND_TO_MODE, COEF_FP32, RELU, GEMM_SIMT, GEMM_TCGEN05, TRANSFORM_SIMT, PROFILE_WAITS, POOL2X2,
    EXPORTED_SYMBOLS, STATIC_SCRATCH_BYTES, QUANT_PER_TENSOR, QUANT_PER_CHANNEL, QUANT_GIVEN,
)
