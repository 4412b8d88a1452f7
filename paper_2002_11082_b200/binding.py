"""ctypes binding of libogq.so: same names and argument order as include/ogq.h."""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libogq.so")

OGQ_BINGRAD_PB, OGQ_BINGRAD_B, OGQ_ORQ = 0, 1, 2
OGQ_ST_EMPTY, OGQ_ST_NONFINITE, OGQ_ST_CONSTANT, OGQ_ST_ITER_CAP, OGQ_ST_INTERNAL = 1, 2, 4, 8, 16

_STATUS_NAMES = {1: "OGQ_ERR_INVALID_ARG", 2: "OGQ_ERR_UNSUPPORTED", 3: "OGQ_ERR_WORKSPACE", 4: "OGQ_ERR_CUDA",
                 5: "OGQ_ERR_LIMIT"}


class OgqError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where} failed: {_STATUS_NAMES.get(code, code)}")
        self.code = code


_lib: Optional[ctypes.CDLL] = None


def lib_path() -> str:
    return _LIB_PATH


def lib() -> ctypes.CDLL:
    """The loaded library.  Raises if libogq.so has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2002_11082_b200.build` "
                "(nvcc, sm_100a); there is no CPU fallback"
            )
        L = ctypes.CDLL(_LIB_PATH)
        vp, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
        L.ogq_version.restype = ctypes.c_char_p
        L.ogq_version.argtypes = []
        L.ogq_bits_for_levels.restype = i32
        L.ogq_bits_for_levels.argtypes = [i32]
        L.ogq_packed_layout.restype = i32
        L.ogq_packed_layout.argtypes = [vp, i32, i32, vp]
        L.ogq_workspace_bytes.restype = sz
        L.ogq_workspace_bytes.argtypes = [i32, i64, i32]
        L.ogq_levels_bingrad.restype = i32
        L.ogq_levels_bingrad.argtypes = [vp, vp, i32, i64, i32, i32, vp, vp, vp, vp, sz, vp]
        L.ogq_levels_bingrad_b_noalloc.restype = i32
        L.ogq_levels_bingrad_b_noalloc.argtypes = [vp, vp, i32, i64, i32, vp, vp, vp, vp]
        L.ogq_levels_orq.restype = i32
        L.ogq_levels_orq.argtypes = [vp, vp, i32, i64, i32, vp, vp, vp, sz, vp]
        L.ogq_quantize_pack.restype = i32
        L.ogq_quantize_pack.argtypes = [vp, vp, i32, i64, i32, i32, vp, vp, ctypes.c_uint64, ctypes.c_uint32, vp, vp, vp]
        L.ogq_unpack_sum.restype = i32
        L.ogq_unpack_sum.argtypes = [vp, vp, i32, vp, vp, i32, i64, i32, ctypes.c_float, vp, vp]
        L.ogq_bucket_packed_words.restype = i64
        L.ogq_bucket_packed_words.argtypes = [i64, i32, i32]
        L.ogq_bucket_encode.restype = i32
        L.ogq_bucket_encode.argtypes = [vp, i64, i32, i32, i32, i32, ctypes.c_float, ctypes.c_uint64, ctypes.c_uint32,
                                        vp, vp, vp, vp, vp]
        L.ogq_clip_threshold.restype = i32
        L.ogq_clip_threshold.argtypes = [vp, vp, i32, i64, ctypes.c_float, vp, vp, vp, sz, vp]
        L.ogq_levels_orq_clipped.restype = i32
        L.ogq_levels_orq_clipped.argtypes = [vp, vp, i32, i64, i32, vp, vp, vp, vp, sz, vp]
        L.ogq_quant_error.restype = i32
        L.ogq_quant_error.argtypes = [vp, vp, i32, i64, i32, vp, vp, vp, vp, vp]
        L.ogq_expected_error.restype = i32
        L.ogq_expected_error.argtypes = [vp, vp, i32, i64, i32, vp, vp, vp]
        L.ogq_dense_digits.restype = i32
        L.ogq_dense_digits.argtypes = [i32]
        L.ogq_dense_layout.restype = i32
        L.ogq_dense_layout.argtypes = [vp, i32, i32, vp]
        L.ogq_quantize_pack_dense.restype = i32
        L.ogq_quantize_pack_dense.argtypes = [vp, vp, i32, i64, i32, vp, ctypes.c_uint64, ctypes.c_uint32, vp, vp, vp]
        L.ogq_unpack_sum_dense.restype = i32
        L.ogq_unpack_sum_dense.argtypes = [vp, vp, i32, vp, vp, i32, i64, i32, ctypes.c_float, vp, vp]
        L.ogq_quantize_pack_clipped.restype = i32
        L.ogq_quantize_pack_clipped.argtypes = [vp, vp, i32, i64, i32, i32, vp, vp, vp, ctypes.c_uint64, ctypes.c_uint32,
                                                vp, vp, vp]
        L.ogq_levels_bingrad_clipped.restype = i32
        L.ogq_levels_bingrad_clipped.argtypes = [vp, vp, i32, i64, i32, i32, vp, vp, vp, vp, vp, sz, vp]
        L.ogq_bucket_decode_sum.restype = i32
        L.ogq_bucket_decode_sum.argtypes = [vp, vp, i32, i64, i32, i32, ctypes.c_float, vp, vp]
        L.ogq_launch_count.restype = ctypes.c_ulonglong
        L.ogq_launch_count.argtypes = []
        L.ogq_profile_enable.restype = i32
        L.ogq_profile_enable.argtypes = [i32]
        L.ogq_profile_collect.restype = i32
        L.ogq_profile_collect.argtypes = [vp, vp, i32, i32]
        _lib = L
    return _lib


def _ptr(t) -> Optional[int]:
    """Address of a torch tensor's storage, a raw integer address, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(code: int, where: str) -> None:
    if code != 0:
        raise OgqError(code, where)


def ogq_version() -> str:
    return lib().ogq_version().decode()


def ogq_bits_for_levels(s: int) -> int:
    return int(lib().ogq_bits_for_levels(int(s)))


def ogq_packed_layout(h_off, bits: int) -> np.ndarray:
    """Host helper: word offsets [T+1] of the packed regions for element offsets h_off [T+1]."""
    h = np.ascontiguousarray(np.asarray(h_off), dtype=np.int64)
    out = np.zeros_like(h)
    _check(lib().ogq_packed_layout(h.ctypes.data, h.size - 1, int(bits), out.ctypes.data), "ogq_packed_layout")
    return out


def ogq_workspace_bytes(num_tensors: int, total_elems: int, max_levels: int) -> int:
    return int(lib().ogq_workspace_bytes(int(num_tensors), int(total_elems), int(max_levels)))


def ogq_levels_bingrad(d_grad, d_off, T: int, total_elems: int, variant: int, lloyd_iters: int,
                       d_levels, d_thresh, d_status, d_ws, ws_bytes: int, stream=None) -> None:
    _check(
        lib().ogq_levels_bingrad(_ptr(d_grad), _ptr(d_off), int(T), int(total_elems), int(variant),
                                 int(lloyd_iters), _ptr(d_levels), _ptr(d_thresh), _ptr(d_status),
                                 _ptr(d_ws), int(ws_bytes), _stream(stream)),
        "ogq_levels_bingrad",
    )


def ogq_levels_bingrad_b_noalloc(d_grad, d_off, T: int, total_elems: int, lloyd_iters: int, d_levels, d_thresh,
                                 d_status, stream=None) -> None:
    """BinGrad-b levels with the solver's scratch held inside the library (no workspace argument).

    For callers that may not allocate device memory; at most 1024 tensors per call, and calls that
    overlap on the GPU must be ordered because they share the one built-in scratch array."""
    _check(
        lib().ogq_levels_bingrad_b_noalloc(_ptr(d_grad), _ptr(d_off), int(T), int(total_elems), int(lloyd_iters),
                                           _ptr(d_levels), _ptr(d_thresh), _ptr(d_status), _stream(stream)),
        "ogq_levels_bingrad_b_noalloc",
    )


def ogq_levels_orq(d_grad, d_off, T: int, total_elems: int, s: int, d_levels, d_status, d_ws,
                   ws_bytes: int, stream=None) -> None:
    _check(
        lib().ogq_levels_orq(_ptr(d_grad), _ptr(d_off), int(T), int(total_elems), int(s), _ptr(d_levels),
                             _ptr(d_status), _ptr(d_ws), int(ws_bytes), _stream(stream)),
        "ogq_levels_orq",
    )


def ogq_quantize_pack(d_grad, d_off, T: int, total_elems: int, scheme: int, s: int, d_levels, d_thresh,
                      seed: int, stream_id: int, d_packed_off, d_packed, stream=None) -> None:
    _check(
        lib().ogq_quantize_pack(_ptr(d_grad), _ptr(d_off), int(T), int(total_elems), int(scheme), int(s),
                                _ptr(d_levels), _ptr(d_thresh), int(seed) & 0xFFFFFFFFFFFFFFFF,
                                int(stream_id) & 0xFFFFFFFF, _ptr(d_packed_off), _ptr(d_packed),
                                _stream(stream)),
        "ogq_quantize_pack",
    )


def ogq_unpack_sum(d_packed_k, d_levels_k, K: int, d_off, d_packed_off, T: int, total_elems: int, s: int,
                   scale: float, d_out, stream=None) -> None:
    _check(
        lib().ogq_unpack_sum(_ptr(d_packed_k), _ptr(d_levels_k), int(K), _ptr(d_off), _ptr(d_packed_off),
                             int(T), int(total_elems), int(s), float(scale), _ptr(d_out), _stream(stream)),
        "ogq_unpack_sum",
    )


def ogq_bucket_packed_words(total_elems: int, d: int, bits: int) -> int:
    return int(lib().ogq_bucket_packed_words(int(total_elems), int(d), int(bits)))


def ogq_clip_threshold(d_grad, d_off, T: int, total_elems: int, c: float, d_tau, d_status, d_ws, ws_bytes: int,
                       stream=None) -> None:
    _check(
        lib().ogq_clip_threshold(_ptr(d_grad), _ptr(d_off), int(T), int(total_elems), float(c), _ptr(d_tau),
                                 _ptr(d_status), _ptr(d_ws), int(ws_bytes), _stream(stream)),
        "ogq_clip_threshold",
    )


def ogq_levels_orq_clipped(d_grad, d_off, T: int, total_elems: int, s: int, d_tau, d_levels, d_status, d_ws,
                           ws_bytes: int, stream=None) -> None:
    _check(
        lib().ogq_levels_orq_clipped(_ptr(d_grad), _ptr(d_off), int(T), int(total_elems), int(s), _ptr(d_tau),
                                     _ptr(d_levels), _ptr(d_status), _ptr(d_ws), int(ws_bytes), _stream(stream)),
        "ogq_levels_orq_clipped",
    )


def ogq_levels_bingrad_clipped(d_grad, d_off, T: int, total_elems: int, variant: int, lloyd_iters: int, d_tau,
                               d_levels, d_thresh, d_status, d_ws, ws_bytes: int, stream=None) -> None:
    _check(
        lib().ogq_levels_bingrad_clipped(_ptr(d_grad), _ptr(d_off), int(T), int(total_elems), int(variant),
                                         int(lloyd_iters), _ptr(d_tau), _ptr(d_levels), _ptr(d_thresh),
                                         _ptr(d_status), _ptr(d_ws), int(ws_bytes), _stream(stream)),
        "ogq_levels_bingrad_clipped",
    )


def ogq_quant_error(d_grad, d_off, T: int, total_elems: int, s: int, d_levels, d_packed_off, d_packed, d_err,
                    stream=None) -> None:
    _check(
        lib().ogq_quant_error(_ptr(d_grad), _ptr(d_off), int(T), int(total_elems), int(s), _ptr(d_levels),
                              _ptr(d_packed_off), _ptr(d_packed), _ptr(d_err), _stream(stream)),
        "ogq_quant_error",
    )


def ogq_expected_error(d_grad, d_off, T: int, total_elems: int, s: int, d_levels, d_err, stream=None) -> None:
    _check(
        lib().ogq_expected_error(_ptr(d_grad), _ptr(d_off), int(T), int(total_elems), int(s), _ptr(d_levels),
                                 _ptr(d_err), _stream(stream)),
        "ogq_expected_error",
    )


def ogq_dense_digits(s: int) -> int:
    return int(lib().ogq_dense_digits(int(s)))


def ogq_dense_layout(h_off, s: int) -> np.ndarray:
    """Host helper: word offsets [T+1] of the base-s packed regions for element offsets h_off [T+1]."""
    h = np.ascontiguousarray(np.asarray(h_off), dtype=np.int64)
    out = np.zeros_like(h)
    _check(lib().ogq_dense_layout(h.ctypes.data, h.size - 1, int(s), out.ctypes.data), "ogq_dense_layout")
    return out


def ogq_quantize_pack_dense(d_grad, d_off, T: int, total_elems: int, s: int, d_levels, seed: int, stream_id: int,
                            d_packed_off, d_packed, stream=None) -> None:
    _check(
        lib().ogq_quantize_pack_dense(_ptr(d_grad), _ptr(d_off), int(T), int(total_elems), int(s), _ptr(d_levels),
                                      int(seed) & 0xFFFFFFFFFFFFFFFF, int(stream_id) & 0xFFFFFFFF,
                                      _ptr(d_packed_off), _ptr(d_packed), _stream(stream)),
        "ogq_quantize_pack_dense",
    )


def ogq_unpack_sum_dense(d_packed_k, d_levels_k, K: int, d_off, d_packed_off, T: int, total_elems: int, s: int,
                         scale: float, d_out, stream=None) -> None:
    _check(
        lib().ogq_unpack_sum_dense(_ptr(d_packed_k), _ptr(d_levels_k), int(K), _ptr(d_off), _ptr(d_packed_off),
                                   int(T), int(total_elems), int(s), float(scale), _ptr(d_out), _stream(stream)),
        "ogq_unpack_sum_dense",
    )


def ogq_quantize_pack_clipped(d_grad, d_off, T: int, total_elems: int, scheme: int, s: int, d_levels, d_thresh,
                              d_tau, seed: int, stream_id: int, d_packed_off, d_packed, stream=None) -> None:
    _check(
        lib().ogq_quantize_pack_clipped(_ptr(d_grad), _ptr(d_off), int(T), int(total_elems), int(scheme), int(s),
                                        _ptr(d_levels), _ptr(d_thresh), _ptr(d_tau), int(seed) & 0xFFFFFFFFFFFFFFFF,
                                        int(stream_id) & 0xFFFFFFFF, _ptr(d_packed_off), _ptr(d_packed),
                                        _stream(stream)),
        "ogq_quantize_pack_clipped",
    )


def ogq_bucket_encode(d_grad, total_elems: int, d: int, scheme: int, s: int, iters: int, clip_c: float, seed: int,
                      stream_id: int, d_levels, d_thresh, d_status, d_packed, stream=None) -> None:
    _check(
        lib().ogq_bucket_encode(_ptr(d_grad), int(total_elems), int(d), int(scheme), int(s), int(iters), float(clip_c),
                                int(seed) & 0xFFFFFFFFFFFFFFFF, int(stream_id) & 0xFFFFFFFF, _ptr(d_levels),
                                _ptr(d_thresh), _ptr(d_status), _ptr(d_packed), _stream(stream)),
        "ogq_bucket_encode",
    )


def ogq_bucket_decode_sum(d_packed_k, d_levels_k, K: int, total_elems: int, d: int, s: int, scale: float, d_out,
                          stream=None) -> None:
    _check(
        lib().ogq_bucket_decode_sum(_ptr(d_packed_k), _ptr(d_levels_k), int(K), int(total_elems), int(d), int(s),
                                    float(scale), _ptr(d_out), _stream(stream)),
        "ogq_bucket_decode_sum",
    )


def ogq_launch_count() -> int:
    return int(lib().ogq_launch_count())


def ogq_profile_enable(on: bool) -> None:
    lib().ogq_profile_enable(1 if on else 0)


def ogq_profile_collect(max_records: int = 65536):
    """Returns [(kernel name, milliseconds), ...] for the launches recorded since profiling was enabled."""
    ms = np.zeros(max_records, dtype=np.float32)
    stride = 48
    names = ctypes.create_string_buffer(max_records * stride)
    n = lib().ogq_profile_collect(ms.ctypes.data, ctypes.cast(names, ctypes.c_void_p), stride, max_records)
    raw = names.raw
    return [(raw[i * stride : (i + 1) * stride].split(b"\0", 1)[0].decode(), float(ms[i])) for i in range(n)]


def device_pointer_array(tensors: Sequence, device=None):
    """An int64 device tensor holding the data pointers of `tensors` (for ogq_unpack_sum)."""
    import torch

    dev = device if device is not None else tensors[0].device
    return torch.tensor([t.data_ptr() for t in tensors], dtype=torch.int64, device=dev)
