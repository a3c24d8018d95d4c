"""LLMA reference-copy decoding on one B200: Python binding of the C-ABI library.

The binding only marshals arguments; every step of the decoding path runs in the
CUDA kernels of ``libllma_b200.so``.  Importing the package does not load the
library; the first call does, and fails loudly if it is missing.
"""
from .binding import (  # noqa: F401
    Engine,
    LlmaError,
    LlmaConfig,
    LlmaStats,
    LlmaStepInfo,
    lib,
    llma_gemm_rows32_bf16,
    llma_gemm_rows32_bf16_noalloc,
    llma_microbench_mma,
    LIB_PATH,
)
