"""ctypes front end of the C oracle (test infrastructure only).

The arithmetic lives in ``ogq_oracle.c``; this file compiles it on demand,
marshals numpy arrays and loops over the tensors of a bucket.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ogq_oracle.c")
_SO = os.path.join(_HERE, "libogq_oracle.so")

PB, B, ORQ = 0, 1, 2

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared object next to its source."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = [
            "gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fexcess-precision=standard",
            "-shared", "-fPIC", _SRC, "-o", _SO, "-lm",
        ]
        subprocess.run(cmd, check=True)
    return _SO


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        L = _lib
        fp = ctypes.POINTER(ctypes.c_float)
        dp = ctypes.POINTER(ctypes.c_double)
        u8 = ctypes.POINTER(ctypes.c_uint8)
        u32 = ctypes.POINTER(ctypes.c_uint32)
        i64 = ctypes.c_int64
        L.ogq_oracle_stats.argtypes = [fp, i64, dp]
        L.ogq_oracle_stats.restype = ctypes.c_int
        L.ogq_oracle_levels_bingrad_b.argtypes = [fp, i64, ctypes.c_int, fp, fp]
        L.ogq_oracle_levels_bingrad_b.restype = ctypes.c_int
        L.ogq_oracle_levels_bingrad_pb.argtypes = [fp, i64, fp]
        L.ogq_oracle_levels_bingrad_pb.restype = ctypes.c_int
        L.ogq_oracle_qstar.argtypes = [fp, i64, ctypes.c_double, ctypes.c_double]
        L.ogq_oracle_qstar.restype = ctypes.c_double
        L.ogq_oracle_levels_orq.argtypes = [fp, i64, ctypes.c_int, fp]
        L.ogq_oracle_levels_orq.restype = ctypes.c_int
        L.ogq_oracle_philox4x32_10.argtypes = [u32, u32, u32]
        L.ogq_oracle_philox4x32_10.restype = None
        L.ogq_oracle_quantize.argtypes = [
            fp, i64, ctypes.c_int, ctypes.c_int, fp, ctypes.c_float,
            ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, u8,
        ]
        L.ogq_oracle_quantize.restype = None
        L.ogq_oracle_packed_words.argtypes = [i64, ctypes.c_int]
        L.ogq_oracle_packed_words.restype = i64
        L.ogq_oracle_pack.argtypes = [u8, i64, ctypes.c_int, u32]
        L.ogq_oracle_pack.restype = None
        L.ogq_oracle_unpack.argtypes = [u32, i64, ctypes.c_int, u8]
        L.ogq_oracle_unpack.restype = None
        L.ogq_oracle_unpack_sum.argtypes = [
            ctypes.POINTER(u32), ctypes.POINTER(fp), ctypes.c_int, i64, ctypes.c_int,
            ctypes.c_float, fp,
        ]
        L.ogq_oracle_unpack_sum.restype = None
        L.ogq_oracle_clip_threshold.argtypes = [fp, i64, ctypes.c_double, fp]
        L.ogq_oracle_clip_threshold.restype = ctypes.c_int
        L.ogq_oracle_clip.argtypes = [fp, i64, ctypes.c_float, fp]
        L.ogq_oracle_clip.restype = None
        L.ogq_oracle_dense_digits.argtypes = [ctypes.c_int]
        L.ogq_oracle_dense_digits.restype = ctypes.c_int
        L.ogq_oracle_dense_words.argtypes = [i64, ctypes.c_int]
        L.ogq_oracle_dense_words.restype = i64
        L.ogq_oracle_pack_dense.argtypes = [u8, i64, ctypes.c_int, u32]
        L.ogq_oracle_pack_dense.restype = None
        L.ogq_oracle_unpack_dense.argtypes = [u32, i64, ctypes.c_int, u8]
        L.ogq_oracle_unpack_dense.restype = None
        L.ogq_oracle_unpack_sum_dense.argtypes = [
            ctypes.POINTER(u32), ctypes.POINTER(fp), ctypes.c_int, i64, ctypes.c_int,
            ctypes.c_float, fp,
        ]
        L.ogq_oracle_unpack_sum_dense.restype = None
        L.ogq_oracle_quant_error.argtypes = [fp, i64, fp, u8]
        L.ogq_oracle_quant_error.restype = ctypes.c_double
        L.ogq_oracle_expected_error.argtypes = [fp, i64, ctypes.c_int, fp]
        L.ogq_oracle_expected_error.restype = ctypes.c_double
        L.ogq_oracle_refine_orq.argtypes = [fp, i64, ctypes.c_int, fp, ctypes.c_int]
        L.ogq_oracle_refine_orq.restype = ctypes.c_int
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def bits_for(s: int) -> int:
    """Code width: 1 bit for two levels, ceil(log2 s) bits otherwise."""
    return max(1, int(s - 1).bit_length())


# ---------------------------------------------------------------- per tensor


def stats(v) -> Tuple[dict, int]:
    v = _f32(v)
    out = np.zeros(4, dtype=np.float64)
    st = lib().ogq_oracle_stats(_ptr(v, ctypes.c_float), v.size, _ptr(out, ctypes.c_double))
    return {"n": v.size, "sum": out[0], "min": out[1], "max": out[2], "abs_sum": out[3]}, st


def levels_bingrad_b(v, lloyd_iters: int = 0) -> Tuple[np.ndarray, float, int]:
    v = _f32(v)
    lv = np.zeros(2, dtype=np.float32)
    th = ctypes.c_float(0.0)
    st = lib().ogq_oracle_levels_bingrad_b(
        _ptr(v, ctypes.c_float), v.size, int(lloyd_iters), _ptr(lv, ctypes.c_float), ctypes.byref(th)
    )
    return lv, np.float32(th.value), st


def levels_bingrad_pb(v) -> Tuple[np.ndarray, int]:
    v = _f32(v)
    b1 = ctypes.c_float(0.0)
    st = lib().ogq_oracle_levels_bingrad_pb(_ptr(v, ctypes.c_float), v.size, ctypes.byref(b1))
    b = np.float32(b1.value)
    return np.array([-b, b], dtype=np.float32), st


def qstar(v, L: float, R: float) -> float:
    v = _f32(v)
    return float(lib().ogq_oracle_qstar(_ptr(v, ctypes.c_float), v.size, float(L), float(R)))


def levels_orq(v, s: int) -> Tuple[np.ndarray, int]:
    v = _f32(v)
    lv = np.zeros(s, dtype=np.float32)
    st = lib().ogq_oracle_levels_orq(_ptr(v, ctypes.c_float), v.size, int(s), _ptr(lv, ctypes.c_float))
    return lv, st


def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().ogq_oracle_philox4x32_10(
        _ptr(c, ctypes.c_uint32), _ptr(k, ctypes.c_uint32), _ptr(out, ctypes.c_uint32)
    )
    return out


def quantize(v, scheme: int, s: int, levels, thresh: float, seed: int, tensor_id: int, stream_id: int) -> np.ndarray:
    v = _f32(v)
    lv = _f32(levels)
    codes = np.zeros(v.size, dtype=np.uint8)
    lib().ogq_oracle_quantize(
        _ptr(v, ctypes.c_float), v.size, int(scheme), int(s), _ptr(lv, ctypes.c_float),
        ctypes.c_float(float(thresh)), ctypes.c_uint64(int(seed)), ctypes.c_uint32(int(tensor_id)),
        ctypes.c_uint32(int(stream_id)), _ptr(codes, ctypes.c_uint8),
    )
    return codes


def packed_words(n: int, bits: int) -> int:
    return int(lib().ogq_oracle_packed_words(int(n), int(bits)))


def pack(codes, bits: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    words = np.zeros(packed_words(codes.size, bits), dtype=np.uint32)
    lib().ogq_oracle_pack(_ptr(codes, ctypes.c_uint8), codes.size, int(bits), _ptr(words, ctypes.c_uint32))
    return words


def unpack(words, n: int, bits: int) -> np.ndarray:
    words = np.ascontiguousarray(words, dtype=np.uint32)
    codes = np.zeros(n, dtype=np.uint8)
    lib().ogq_oracle_unpack(_ptr(words, ctypes.c_uint32), int(n), int(bits), _ptr(codes, ctypes.c_uint8))
    return codes


def unpack_sum(packed: Sequence[np.ndarray], levels: Sequence[np.ndarray], n: int, bits: int, scale: float) -> np.ndarray:
    K = len(packed)
    pk = [np.ascontiguousarray(p, dtype=np.uint32) for p in packed]
    lv = [_f32(l) for l in levels]
    pp = (ctypes.POINTER(ctypes.c_uint32) * K)(*[_ptr(p, ctypes.c_uint32) for p in pk])
    lp = (ctypes.POINTER(ctypes.c_float) * K)(*[_ptr(l, ctypes.c_float) for l in lv])
    out = np.zeros(n, dtype=np.float32)
    lib().ogq_oracle_unpack_sum(pp, lp, K, int(n), int(bits), ctypes.c_float(float(scale)), _ptr(out, ctypes.c_float))
    return out


def clip_threshold(v, c: float) -> Tuple[np.float32, int]:
    """tau = fp32(c * sigma), sigma^2 the variance of v about its mean (1/n)."""
    v = _f32(v)
    tau = ctypes.c_float(0.0)
    st = lib().ogq_oracle_clip_threshold(_ptr(v, ctypes.c_float), v.size, float(c), ctypes.byref(tau))
    return np.float32(tau.value), st


def clip(v, tau: float) -> np.ndarray:
    """sign(v) * min(|v|, tau), element by element."""
    v = _f32(v)
    out = np.zeros_like(v)
    lib().ogq_oracle_clip(_ptr(v, ctypes.c_float), v.size, ctypes.c_float(float(tau)), _ptr(out, ctypes.c_float))
    return out


def dense_digits(s: int) -> int:
    return int(lib().ogq_oracle_dense_digits(int(s)))


def dense_words(n: int, s: int) -> int:
    return int(lib().ogq_oracle_dense_words(int(n), int(s)))


def pack_dense(codes, s: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    words = np.zeros(dense_words(codes.size, s), dtype=np.uint32)
    lib().ogq_oracle_pack_dense(_ptr(codes, ctypes.c_uint8), codes.size, int(s), _ptr(words, ctypes.c_uint32))
    return words


def unpack_dense(words, n: int, s: int) -> np.ndarray:
    words = np.ascontiguousarray(words, dtype=np.uint32)
    codes = np.zeros(n, dtype=np.uint8)
    lib().ogq_oracle_unpack_dense(_ptr(words, ctypes.c_uint32), int(n), int(s), _ptr(codes, ctypes.c_uint8))
    return codes


def unpack_sum_dense(packed: Sequence[np.ndarray], levels: Sequence[np.ndarray], n: int, s: int, scale: float) -> np.ndarray:
    K = len(packed)
    pk = [np.ascontiguousarray(p, dtype=np.uint32) for p in packed]
    lv = [_f32(l) for l in levels]
    pp = (ctypes.POINTER(ctypes.c_uint32) * K)(*[_ptr(p, ctypes.c_uint32) for p in pk])
    lp = (ctypes.POINTER(ctypes.c_float) * K)(*[_ptr(l, ctypes.c_float) for l in lv])
    out = np.zeros(n, dtype=np.float32)
    lib().ogq_oracle_unpack_sum_dense(pp, lp, K, int(n), int(s), ctypes.c_float(float(scale)), _ptr(out, ctypes.c_float))
    return out


def quant_error(v, levels, codes) -> float:
    """sum_i (levels[code_i] - v_i)^2."""
    v = _f32(v)
    lv = _f32(levels)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    return float(lib().ogq_oracle_quant_error(_ptr(v, ctypes.c_float), v.size, _ptr(lv, ctypes.c_float),
                                              _ptr(codes, ctypes.c_uint8)))


def expected_error(v, levels) -> float:
    """Expectation of the random-rounding error over the draws: sum_i (v_i - lo_i)(hi_i - v_i)."""
    v = _f32(v)
    lv = _f32(levels)
    return float(lib().ogq_oracle_expected_error(_ptr(v, ctypes.c_float), v.size, lv.size, _ptr(lv, ctypes.c_float)))


def refine_orq(v, levels, max_sweeps: int) -> Tuple[np.ndarray, int]:
    """Refinement sweeps b_k <- Q*(b_{k-1}, b_{k+1}) over the interior levels; returns (levels, sweeps that changed something)."""
    v = _f32(v)
    lv = _f32(levels).copy()
    n = lib().ogq_oracle_refine_orq(_ptr(v, ctypes.c_float), v.size, lv.size, _ptr(lv, ctypes.c_float), int(max_sweeps))
    return lv, int(n)


# ---------------------------------------------------------------- per bucket


def dense_layout(offsets, s: int) -> np.ndarray:
    """Word offset of every tensor's region in the base-s format."""
    offsets = np.asarray(offsets, dtype=np.int64)
    T = offsets.size - 1
    po = np.zeros(T + 1, dtype=np.int64)
    for t in range(T):
        po[t + 1] = po[t] + dense_words(int(offsets[t + 1] - offsets[t]), s)
    return po


def bucket_clip_thresholds(values, offsets, c: float) -> Tuple[np.ndarray, np.ndarray]:
    offsets = np.asarray(offsets, dtype=np.int64)
    T = offsets.size - 1
    tau = np.zeros(T, dtype=np.float32)
    st = np.zeros(T, dtype=np.int32)
    for t in range(T):
        tau[t], st[t] = clip_threshold(values[offsets[t] : offsets[t + 1]], c)
    return tau, st


def bucket_clip(values, offsets, tau) -> np.ndarray:
    offsets = np.asarray(offsets, dtype=np.int64)
    out = np.array(values, dtype=np.float32, copy=True)
    for t in range(offsets.size - 1):
        out[offsets[t] : offsets[t + 1]] = clip(values[offsets[t] : offsets[t + 1]], float(tau[t]))
    return out


def bucket_pack_dense(codes_per_tensor: Sequence[np.ndarray], offsets, s: int) -> Tuple[np.ndarray, np.ndarray]:
    po = dense_layout(offsets, s)
    out = np.zeros(int(po[-1]), dtype=np.uint32)
    for t, codes in enumerate(codes_per_tensor):
        out[po[t] : po[t + 1]] = pack_dense(codes, s)
    return out, po


def bucket_unpack_sum_dense(packed_k: Sequence[np.ndarray], levels_k: Sequence[np.ndarray], offsets, s: int, scale: float) -> np.ndarray:
    offsets = np.asarray(offsets, dtype=np.int64)
    T = offsets.size - 1
    po = dense_layout(offsets, s)
    out = np.zeros(int(offsets[-1]), dtype=np.float32)
    for t in range(T):
        n = int(offsets[t + 1] - offsets[t])
        out[offsets[t] : offsets[t + 1]] = unpack_sum_dense(
            [p[po[t] : po[t + 1]] for p in packed_k], [l[t] for l in levels_k], n, s, scale
        )
    return out


def packed_layout(offsets, bits: int) -> np.ndarray:
    """Word offset of every tensor's packed region (regions are multiples of 4 words)."""
    offsets = np.asarray(offsets, dtype=np.int64)
    T = offsets.size - 1
    po = np.zeros(T + 1, dtype=np.int64)
    for t in range(T):
        po[t + 1] = po[t] + packed_words(int(offsets[t + 1] - offsets[t]), bits)
    return po


def bucket_levels_orq(values, offsets, s: int) -> Tuple[np.ndarray, np.ndarray]:
    offsets = np.asarray(offsets, dtype=np.int64)
    T = offsets.size - 1
    lv = np.zeros((T, s), dtype=np.float32)
    st = np.zeros(T, dtype=np.int32)
    for t in range(T):
        lv[t], st[t] = levels_orq(values[offsets[t] : offsets[t + 1]], s)
    return lv, st


def bucket_levels_bingrad(values, offsets, variant: int, lloyd_iters: int = 0):
    offsets = np.asarray(offsets, dtype=np.int64)
    T = offsets.size - 1
    lv = np.zeros((T, 2), dtype=np.float32)
    th = np.zeros(T, dtype=np.float32)
    st = np.zeros(T, dtype=np.int32)
    for t in range(T):
        seg = values[offsets[t] : offsets[t + 1]]
        if variant == B:
            lv[t], th[t], st[t] = levels_bingrad_b(seg, lloyd_iters)
        else:
            lv[t], st[t] = levels_bingrad_pb(seg)
    return lv, th, st


def bucket_quantize_pack(values, offsets, scheme: int, s: int, levels, thresh, seed: int, stream_id: int,
                         return_codes: bool = False):
    offsets = np.asarray(offsets, dtype=np.int64)
    T = offsets.size - 1
    bits = bits_for(s)
    po = packed_layout(offsets, bits)
    out = np.zeros(int(po[-1]), dtype=np.uint32)
    all_codes: List[np.ndarray] = []
    for t in range(T):
        seg = values[offsets[t] : offsets[t + 1]]
        th = float(thresh[t]) if thresh is not None else 0.0
        codes = quantize(seg, scheme, s, levels[t], th, seed, t, stream_id)
        out[po[t] : po[t + 1]] = pack(codes, bits)
        if return_codes:
            all_codes.append(codes)
    if return_codes:
        return out, po, all_codes
    return out, po


def bucket_unpack_sum(packed_k: Sequence[np.ndarray], levels_k: Sequence[np.ndarray], offsets, s: int, scale: float) -> np.ndarray:
    offsets = np.asarray(offsets, dtype=np.int64)
    T = offsets.size - 1
    bits = bits_for(s)
    po = packed_layout(offsets, bits)
    out = np.zeros(int(offsets[-1]), dtype=np.float32)
    for t in range(T):
        n = int(offsets[t + 1] - offsets[t])
        out[offsets[t] : offsets[t + 1]] = unpack_sum(
            [p[po[t] : po[t + 1]] for p in packed_k], [l[t] for l in levels_k], n, bits, scale
        )
    return out
