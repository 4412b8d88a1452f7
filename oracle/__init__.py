"""CPU oracle for the gradient-quantization path (test infrastructure only).

Nothing in the product package imports this; only the tests, the smoke check
and the benchmark's CPU-baseline leg do.
"""
from .oracle import (  # noqa: F401
    PB,
    B,
    ORQ,
    build,
    lib,
    stats,
    levels_bingrad_b,
    levels_bingrad_pb,
    levels_orq,
    qstar,
    philox4x32_10,
    quantize,
    packed_words,
    pack,
    unpack,
    unpack_sum,
    bits_for,
    bucket_levels_orq,
    bucket_levels_bingrad,
    bucket_quantize_pack,
    bucket_unpack_sum,
    packed_layout,
)
