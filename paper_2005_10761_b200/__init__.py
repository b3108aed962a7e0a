"""rTop-k sparsification + aggregation for NVIDIA B200: Python binding of librtopk.so.

The work is done by the CUDA library behind the C ABI in ``include/rtopk.h``; this package only
marshals arguments (torch tensors -> device pointers, the current CUDA stream).  There is no CPU
fallback: using the binding without the built library or without a CUDA device raises.
"""
from .workloads import Workload, configs, gradient, zero_residual  # noqa: F401
from .binding import (RTopK, RTopKError, library_path, load_library, packed_layout, tiled_layout, warmup_sizes, GRAD_F32, GRAD_BF16,  # noqa: F401
                      SCALE_MEAN, SCALE_SUM, SCALE_UNBIASED, SCALE_COUNT, EXPORTS)

__all__ = ["RTopK", "RTopKError", "library_path", "load_library", "packed_layout", "tiled_layout", "warmup_sizes", "Workload", "configs", "gradient",
           "zero_residual", "GRAD_F32", "GRAD_BF16", "SCALE_MEAN", "SCALE_SUM", "SCALE_UNBIASED", "SCALE_COUNT", "EXPORTS"]
