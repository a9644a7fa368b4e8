"""Seeded synthetic inputs and problem-shape lists for the GEMM hot path.

This package is the only code that both the CPU oracle's tests and the CUDA
path's tests/bench import.  It holds no GEMM arithmetic: only a counter-based
random generator, the value distributions of the workloads, dtype encoding of
the generated values, and the lists of problem shapes.
"""
from .generators import (  # noqa: F401
    Matrix,
    make_matrix,
    encode_f16,
    encode_bf16,
    DTYPE_F32,
    DTYPE_F16,
    DTYPE_BF16,
    DTYPE_NAMES,
)
from .shapes import (  # noqa: F401
    RESNET50_V15_BATCH1,
    VGG16_BATCH1,
    im2row_shapes,
    square_fp32_sweep,
    nonsquarish_fp32,
    square_half_sweep,
    Problem,
    config_problems,
    im2row_problems,
    ConvProblem,
    conv_layer_problems,
)
