"""B200-native split feed-forward network (FFSplit, arXiv 2401.04044).

The product is libffsplit.so (C ABI in include/ffsplit.h, CUDA sources in
csrc/); this package holds its ctypes binding and the in-tree build step.
"""
from .binding import (BF16, F32, GELU_ERF, GELU_TANH, SWIGLU, SCORE_ACT_ONLY, SCORE_EQ3, SCORE_SUM_NORM, Context,
                      FFSplitError, Shape, load_library, make_shape, read_section)

__all__ = ["BF16", "F32", "GELU_ERF", "GELU_TANH", "SWIGLU", "SCORE_ACT_ONLY", "SCORE_EQ3", "SCORE_SUM_NORM",
           "Context", "FFSplitError", "Shape", "load_library", "make_shape", "read_section"]
