"""FP4-quantized linear layer for NVIDIA B200 (sm_100a): Python binding of libfp4linear.so.

The library is the product; this package marshals arguments to its C ABI
(include/fp4_linear.h).  Importing the package does not load the library, so the
seeded workload generators stay usable on a machine without CUDA; every compute
entry point loads it on first use and raises if it has not been built.
"""
from .binding import (  # noqa: F401
    FP4_DEV_NONFINITE, FP4_DEV_TIMEOUT, FP4_GEMM_F8F6F4, FP4_GEMM_F8F6F4_A8, FP4_GEMM_F8F6F4_A8B8, FP4_GEMM_F8F6F4_B8, FP4_GEMM_MXF4,
    FP4_BWD_DY_E4M3, FP4_BWD_DY_E5M2, FP4_FORMAT_E2M1, FP4_FORMAT_E4M3, FP4_FORMAT_E5M2, FP4_GEMM_A_E5M2, FP4_GEMM_B_E5M2, FP4_QUANTILE_ABS, FP4_QUANTILE_SIGNED, FP4_QUANTILE_TOKEN, EXPORTS,
    Context, Fp4Error, QTensor, fp4_gemm, fp4_linear_bwd, fp4_linear_fwd, fp4_linear_step_host, fp4_quantile_thresholds_static, fp4_quantize, fp4_l2_read_probe, load_library,
    tail_capacity, KERNEL_CLASSES,
)
from . import workloads  # noqa: F401
