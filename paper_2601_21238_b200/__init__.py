"""B200-native STWQ quantized linear layer (PTQ4ARVG inference hot path).

Importing the package does not load the CUDA library; the first `Context()` does, and it
raises if libstwq.so has not been built (`python -m paper_2601_21238_b200.build`) or if no
sm_100 GPU is present. There is no CPU fallback.
"""
from .binding import (ACT_GELU_ERF, ACT_GELU_FAST, ACT_GELU_TANH, ACT_NONE, OPT_GEMM_PATH, OPT_KSPLIT, OPT_TILE_N,
                      OPT_VARIANT, OPT_WAIT_LIMIT_MS, OUT_BF16, OUT_F32, OUT_INT32, Context,
                      StwqError, check_args, exported_symbols, library_path, load_library, qlinear_static)

__all__ = ["Context", "StwqError", "load_library", "library_path", "exported_symbols", "qlinear_static", "check_args", "ACT_NONE",
           "ACT_GELU_ERF", "ACT_GELU_TANH", "ACT_GELU_FAST", "OUT_F32", "OUT_BF16", "OUT_INT32", "OPT_GEMM_PATH",
           "OPT_WAIT_LIMIT_MS", "OPT_TILE_N", "OPT_VARIANT", "OPT_KSPLIT"]
