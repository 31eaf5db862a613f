"""B200-native library for progressive stochastic binarization (PSB) inference layers.

The product is the CUDA library ``libpsb_b200.so`` (C ABI in ``include/psb.h``);
this package only loads it and marshals arguments.
"""
from .binding import (  # noqa: F401
    Context, Weights, PsbError, load_library, EXPORTS, LIB_PATH,
    PSB_OK, PSB_ERR_INVALID_ARG, PSB_ERR_BAD_K, PSB_ERR_UNSUPPORTED, PSB_ERR_ALLOC, PSB_ERR_CUDA,
    PSB_ERR_TIMEOUT, PSB_ERR_NONFINITE_WEIGHT, PSB_ERR_RANGE, PSB_CHECK_RANGE, PSB_LAYOUT_NCHW, PSB_LAYOUT_NHWC, PSB_DT_U8, PSB_DT_S8,
    PSB_PATH_AUTO, PSB_PATH_SHIFT_ADD, PSB_PATH_TENSOR, PSB_STATIC_MAX_OUT_CH, sample_level_static,
)
