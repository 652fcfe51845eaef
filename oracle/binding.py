"""ctypes marshalling for the C++ checker in ``aq_oracle.cpp`` (no arithmetic here)."""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "aq_oracle.cpp")


def _cpu_tag() -> str:
    """-march=native code only runs on a like CPU: key the library by the CPU's feature flags."""
    import hashlib
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    return hashlib.sha1(flags.encode()).hexdigest()[:10]


_LIB = os.path.join(_DIR, f"libaq_oracle.{_cpu_tag()}.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the checker with g++ (-O3, OpenMP); returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O3", "-march=native", "-fopenmp", "-std=c++17", "-shared",
                               "-fPIC", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        L.orc_half_to_float.restype = C.c_float
        L.orc_half_to_float.argtypes = [C.c_uint16]
        L.orc_double_to_half.restype = C.c_uint16
        L.orc_double_to_half.argtypes = [C.c_double]
        L.orc_float_to_half.restype = C.c_uint16
        L.orc_float_to_half.argtypes = [C.c_float]
        L.orc_pow2_exponent.restype = C.c_int
        L.orc_pow2_exponent.argtypes = [C.c_float, C.c_int]
        L.orc_absmax.restype = C.c_float
        L.orc_layer_exponent.restype = C.c_int
        L.orc_token_select.restype = C.c_int
        L.orc_int_gemm.restype = C.c_longlong
        L.orc_linear.restype = C.c_longlong
        L.orc_progressive_ratio.restype = C.c_double
        L.orc_progressive_ratio.argtypes = [C.c_double, C.c_int]
        L.orc_num_threads.restype = C.c_int
        L.orc_quantize_act_trip.restype = C.c_longlong
        L.orc_log2_quantize.restype = C.c_float
        L.orc_log2_quantize.argtypes = [C.c_void_p, C.c_longlong, C.c_int, C.c_void_p]
        L.orc_attn_v_log2.argtypes = [C.c_void_p, C.c_float, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                      C.c_int, C.c_void_p, C.c_void_p]
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == dtype, (a.dtype, dtype)
    return a


def _half_bits(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.float16
    return a.view(np.uint16)


def num_groups(K: int, group: int) -> int:
    return 1 if group == 0 else K // group


def half_to_float(bits: int) -> float:
    return float(lib().orc_half_to_float(int(bits)))


def double_to_half(d: float) -> int:
    return int(lib().orc_double_to_half(float(d)))


def float_to_half(f: float) -> int:
    return int(lib().orc_float_to_half(float(f)))


def pow2_exponent(a: float, bits: int) -> int:
    return int(lib().orc_pow2_exponent(C.c_float(a), bits))


def progressive_ratio(beta: float, m: int) -> float:
    return float(lib().orc_progressive_ratio(beta, m))


def num_threads() -> int:
    return int(lib().orc_num_threads())


def quantize_weights(w: np.ndarray, group: int) -> Tuple[np.ndarray, np.ndarray]:
    """fp16 [N,K] -> (int8 codes [N,K], fp16 scales [N,G])."""
    N, K = w.shape
    G = num_groups(K, group)
    codes = np.empty((N, K), np.int8)
    scales = np.empty((N, G), np.float16)
    lib().orc_quantize_weights(_p(_half_bits(w)), N, K, group, _p(codes), _p(scales.view(np.uint16)))
    return codes, scales


def pack_w4(codes: np.ndarray) -> np.ndarray:
    codes = _c(codes, np.int8)
    N, K = codes.shape
    out = np.empty((N, K // 2), np.uint8)
    lib().orc_pack_w4(_p(codes), N, K, _p(out))
    return out


def unpack_w4(packed: np.ndarray) -> np.ndarray:
    packed = _c(packed, np.uint8)
    N, K2 = packed.shape
    out = np.empty((N, K2 * 2), np.int8)
    lib().orc_unpack_w4(_p(packed), N, K2 * 2, _p(out))
    return out


def pack_act4(codes: np.ndarray) -> np.ndarray:
    """4-bit activation codes [M, K] -> [M, K/2] bytes; the nibble order is the one of pack_w4."""
    return pack_w4(codes)


def unpack_act4(packed: np.ndarray) -> np.ndarray:
    return unpack_w4(packed)


def token_select(scores: np.ndarray, n_keep: int) -> np.ndarray:
    scores = _c(scores, np.float32)
    idx = np.empty((n_keep,), np.int32)
    rc = lib().orc_token_select(_p(scores), scores.shape[0], n_keep, _p(idx))
    if rc != 0:
        raise ValueError("n_keep out of range")
    return idx


def token_compact(x: np.ndarray, idx: np.ndarray) -> np.ndarray:
    idx = _c(idx, np.int32)
    M, K = x.shape
    out = np.empty((idx.shape[0], K), np.float16)
    lib().orc_token_compact(_p(_half_bits(x)), K, _p(idx), idx.shape[0], _p(out.view(np.uint16)))
    return out


def absmax(x: np.ndarray, row_idx: Optional[np.ndarray] = None) -> float:
    M_in, K = x.shape
    ri = None if row_idx is None else _c(row_idx, np.int32)
    M = M_in if ri is None else ri.shape[0]
    return float(lib().orc_absmax(_p(_half_bits(x)), K, _p(ri), M))


def layer_exponent(x: np.ndarray, bits: int, row_idx: Optional[np.ndarray] = None) -> int:
    M_in, K = x.shape
    ri = None if row_idx is None else _c(row_idx, np.int32)
    M = M_in if ri is None else ri.shape[0]
    return int(lib().orc_layer_exponent(_p(_half_bits(x)), K, _p(ri), M, bits))


def quantize_act(x: np.ndarray, bits: int, e: int, row_idx: Optional[np.ndarray] = None) -> np.ndarray:
    M_in, K = x.shape
    ri = None if row_idx is None else _c(row_idx, np.int32)
    M = M_in if ri is None else ri.shape[0]
    q = np.empty((M, K), np.int8)
    lib().orc_quantize_act(_p(_half_bits(x)), K, _p(ri), M, bits, e, _p(q))
    return q


def quantize_act_trip(x: np.ndarray, bits: int, e: int, alpha: np.ndarray,
                      row_idx: Optional[np.ndarray] = None) -> np.ndarray:
    """Eq. 5 with per-channel factors: int8 values q * 2^alpha_k at base exponent e."""
    M_in, K = x.shape
    ri = None if row_idx is None else _c(row_idx, np.int32)
    M = M_in if ri is None else ri.shape[0]
    al = _c(alpha, np.uint8)
    assert al.shape == (K,)
    v = np.empty((M, K), np.int8)
    misfit = lib().orc_quantize_act_trip(_p(_half_bits(x)), K, _p(ri), M, bits, e, _p(al), _p(v))
    assert misfit == 0, "a shifted code left the int8 range"
    return v


def trip_calibrate(x: np.ndarray, bits: int, e: int, k_max: int, row_idx: Optional[np.ndarray] = None) -> np.ndarray:
    """Eq. 8: per-channel factor in {0..k_max} with the least squared error at base exponent e."""
    M_in, K = x.shape
    ri = None if row_idx is None else _c(row_idx, np.int32)
    M = M_in if ri is None else ri.shape[0]
    out = np.empty((K,), np.uint8)
    lib().orc_trip_calibrate(_p(_half_bits(x)), K, _p(ri), M, bits, e, k_max, _p(out))
    return out


def trip_base_exponent(x: np.ndarray, bits: int, k_max: int, row_idx: Optional[np.ndarray] = None) -> int:
    """Eq. 6 read as s = 2^(e0 - k_max): channels with the largest factor still reach the layer maximum."""
    return layer_exponent(x, bits, row_idx) - k_max


def asym_params(x: np.ndarray, bits: int, row_idx: Optional[np.ndarray] = None) -> Tuple[int, int]:
    """(e, zp) of the unsigned quantizer of Eq. 2 / Eq. 5-7 with a power-of-two scale."""
    M_in, K = x.shape
    ri = None if row_idx is None else _c(row_idx, np.int32)
    M = M_in if ri is None else ri.shape[0]
    e, zp = C.c_int(0), C.c_int(0)
    lib().orc_asym_params(_p(_half_bits(x)), K, _p(ri), M, bits, C.byref(e), C.byref(zp))
    return e.value, zp.value


def quantize_act_asym(x: np.ndarray, bits: int, e: int, zp: int, row_idx: Optional[np.ndarray] = None) -> np.ndarray:
    """Unsigned codes CLIP(round(x / 2^e) + zp, 0, 2^b - 1)."""
    M_in, K = x.shape
    ri = None if row_idx is None else _c(row_idx, np.int32)
    M = M_in if ri is None else ri.shape[0]
    q = np.empty((M, K), np.uint8)
    lib().orc_quantize_act_asym(_p(_half_bits(x)), K, _p(ri), M, bits, e, zp, _p(q))
    return q


def linear_asym(q: np.ndarray, zp: int, c: np.ndarray, scales: np.ndarray, e: int, group: int):
    """(int64 sums [M,N,G] of (q - zp) * c, fp16 y [M,N])."""
    q = _c(q, np.uint8)
    c = _c(c, np.int8)
    M, K = q.shape
    N = c.shape[0]
    G = num_groups(K, group)
    scales = np.ascontiguousarray(scales)
    assert scales.shape == (N, G) and scales.dtype == np.float16
    acc = np.empty((M, N, G), np.int64)
    y = np.empty((M, N), np.float16)
    lib().orc_linear_asym(_p(q), zp, _p(c), _p(scales.view(np.uint16)), e, M, N, K, group, _p(acc),
                          _p(y.view(np.uint16)))
    return acc, y


def log2_quantize(x: np.ndarray, bits: int) -> Tuple[np.ndarray, float]:
    """Eq. 3: (int8 codes Sign * (k + 1), 0 = zero; the tensor's max|x|)."""
    xb = _half_bits(x)
    codes = np.empty(x.shape, np.int8)
    mx = lib().orc_log2_quantize(_p(xb), xb.size, bits, _p(codes))
    return codes, float(mx)


def attn_v_log2(pcodes: np.ndarray, p_max: float, vq: np.ndarray, e_v: int, bits: int):
    """(int64 sums [H,M,D], fp16 y [H,M,D]) of log2-coded P [H,M,J] times int8-coded V [H,J,D]."""
    assert bits <= 5, "the shift form needs kmax <= 15"
    pcodes = _c(pcodes, np.int8)
    vq = _c(vq, np.int8)
    H, M, J = pcodes.shape
    D = vq.shape[2]
    assert vq.shape == (H, J, D)
    acc = np.empty((H, M, D), np.int64)
    y = np.empty((H, M, D), np.float16)
    lib().orc_attn_v_log2(_p(pcodes), p_max, _p(vq), e_v, H, M, J, D, bits, _p(acc), _p(y.view(np.uint16)))
    return acc, y


def int_gemm(q: np.ndarray, c: np.ndarray, group: int) -> np.ndarray:
    """int8 [M,K] x int8 [N,K] -> int32 [M,N,G]; raises if an int32 sum overflowed."""
    q = _c(q, np.int8)
    c = _c(c, np.int8)
    M, K = q.shape
    N = c.shape[0]
    G = num_groups(K, group)
    acc = np.empty((M, N, G), np.int32)
    ovf = lib().orc_int_gemm(_p(q), _p(c), M, N, K, group, _p(acc))
    if ovf:
        raise OverflowError(f"{ovf} int32 accumulators overflowed")
    return acc


def dequant(acc: np.ndarray, scales: np.ndarray, e: int) -> np.ndarray:
    acc = _c(acc, np.int32)
    M, N, G = acc.shape
    scales = np.ascontiguousarray(scales)
    assert scales.shape == (N, G) and scales.dtype == np.float16
    y = np.empty((M, N), np.float16)
    lib().orc_dequant(_p(acc), _p(scales.view(np.uint16)), e, M, N, G, _p(y.view(np.uint16)))
    return y


def linear_sampled(q, c, scales, e: int, group: int, rows, cols):
    """(int32 acc [count,G], fp16 y [count]) at the given output positions."""
    q = _c(q, np.int8)
    c = _c(c, np.int8)
    rows = _c(rows, np.int32)
    cols = _c(cols, np.int32)
    M, K = q.shape
    N = c.shape[0]
    G = num_groups(K, group)
    scales = np.ascontiguousarray(scales)
    assert scales.shape == (N, G) and scales.dtype == np.float16
    cnt = rows.shape[0]
    acc = np.empty((cnt, G), np.int32)
    y = np.empty((cnt,), np.float16)
    lib().orc_linear_sampled(_p(q), _p(c), _p(scales.view(np.uint16)), e, N, K, group, _p(rows),
                             _p(cols), cnt, _p(acc), _p(y.view(np.uint16)))
    return acc, y


def linear(x, codes, scales, bits: int, group: int, scale_mode: int = 0, clip_shift_or_exp: int = 0,
           row_idx=None, want_acc: bool = False):
    """Whole layer. Returns dict(y fp16 [M,N], q int8 [M,K], e int, acc int32 [M,N,G] or None)."""
    M_in, K = x.shape
    ri = None if row_idx is None else _c(row_idx, np.int32)
    M = M_in if ri is None else ri.shape[0]
    codes = _c(codes, np.int8)
    N = codes.shape[0]
    G = num_groups(K, group)
    scales = np.ascontiguousarray(scales)
    assert scales.shape == (N, G) and scales.dtype == np.float16
    y = np.empty((M, N), np.float16)
    q = np.empty((M, K), np.int8)
    acc = np.empty((M, N, G), np.int32) if want_acc else None
    e = C.c_int32(0)
    ovf = lib().orc_linear(_p(_half_bits(x)), K, _p(ri), M, bits, scale_mode, clip_shift_or_exp,
                           _p(codes), _p(scales.view(np.uint16)), N, group, _p(y.view(np.uint16)),
                           _p(q), _p(acc), C.byref(e))
    if ovf:
        raise OverflowError(f"{ovf} int32 accumulators overflowed")
    return {"y": y, "q": q, "e": int(e.value), "acc": acc}
