"""CPU oracle (fp64, plain loops) for the fused attention / fused linear patterns.

Test infrastructure only: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA product path never imports this package.
"""
from .ref import (  # noqa: F401
    attn,
    attn_probs,
    attn_bias,
    attn_decode,
    linear_bias_gelu,
    linear_act,
    linear_swiglu,
    linear_w8,
    ACT_GELU_TANH,
    ACT_GELU_ERF,
    ACT_RELU,
    ACT_SILU,
    ACT_NONE,
    gelu_tanh,
    num_threads,
    build,
)
from . import planner, layer  # noqa: F401,E402
