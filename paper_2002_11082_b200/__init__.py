"""B200 (sm_100a) gradient quantization: BinGrad-b / BinGrad-pb / ORQ level
solvers, quantize + bit-pack, unpack + sum, behind a C ABI (``include/ogq.h``).

This package is a thin ctypes binding over ``libogq.so``: it only marshals
arguments (torch tensors supply device memory and streams); every step of the
path runs in the library's CUDA kernels.  There is no CPU fallback: importing
the binding fails if the library has not been built.
"""
from .binding import (  # noqa: F401
    OGQ_BINGRAD_PB,
    OGQ_BINGRAD_B,
    OGQ_ORQ,
    OGQ_ST_EMPTY,
    OGQ_ST_NONFINITE,
    OGQ_ST_CONSTANT,
    OGQ_ST_ITER_CAP,
    OGQ_ST_INTERNAL,
    OgqError,
    lib,
    lib_path,
    ogq_version,
    ogq_bits_for_levels,
    ogq_packed_layout,
    ogq_workspace_bytes,
    ogq_levels_bingrad,
    ogq_levels_bingrad_b_noalloc,
    ogq_levels_orq,
    ogq_quantize_pack,
    ogq_unpack_sum,
    ogq_quant_error,
    ogq_expected_error,
    ogq_dense_digits,
    ogq_dense_layout,
    ogq_quantize_pack_dense,
    ogq_unpack_sum_dense,
    ogq_clip_threshold,
    ogq_levels_orq_clipped,
    ogq_levels_bingrad_clipped,
    ogq_quantize_pack_clipped,
    ogq_bucket_packed_words,
    ogq_bucket_encode,
    ogq_bucket_decode_sum,
    ogq_launch_count,
    ogq_profile_enable,
    ogq_profile_collect,
    device_pointer_array,
)
