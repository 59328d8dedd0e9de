"""Seeded synthetic inputs and layer shapes for the HLQ LUT-GEMM path.

This package holds no arithmetic of the method itself: it only draws the
tensors (activations, bit-planes, scales, offsets) that both the CPU oracle
and the CUDA library are fed, so that the two sides see identical bits.
"""

from .synth import (  # noqa: F401
    HlqLayer,
    activations,
    hlq_layer,
    bit_planes,
    scales,
    offsets,
    outlier_columns,
    dense_weights,
)
from . import shapes  # noqa: F401
from .shapes import (  # noqa: F401
    LLAMA31_8B,
    LLAMA31_70B,
    config0,
    config1_calls,
    config2_calls,
    config3_calls,
    config4_prefill_calls,
    config4_stack_calls,
    algorithmic_bytes,
)
