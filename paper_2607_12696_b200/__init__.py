"""B200-native MoE verification layer (sm_100a): thin Python binding over ``libmoev.so``.

The package is argument marshalling only -- every step of the path (router top-k, expert
union and grouping, grouped SwiGLU expert FFN, weighted combine) runs in the CUDA kernels
behind the C ABI declared in ``include/moev.h``.  There is no CPU fallback: if the library
is missing or fails to load, importing :mod:`paper_2607_12696_b200.binding` raises.
"""
from .binding import (ACT_BF16, ACT_FP32, ACTQ_FP8_B128, ACTQ_FP8_B128_POW2, ACTQ_NONE, IMPL_AUTO, IMPL_SIMT, IMPL_TCGEN05, SCORE_SIGMOID,  # noqa: F401
                      SCORE_SOFTMAX, W_BF16, W_FP32, W_FP8E4M3_B128, W_MXFP4, MoevConfig,
                      MoevError, MoeVerifier, expert_bytes, expert_code_bytes, lib, lib_path,
                      route_topk_static, select_drafts, static_scratch_floats)
