"""ctypes binding for libagileq.so: same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors used purely as device memory; every step of the layer runs
in the library's kernels. Nothing here computes, and nothing falls back to another path:
if the library is missing or the device is not a B200 the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
import re
from typing import Optional, Tuple

import torch

_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_DIR, "libagileq.so")
HEADER_PATH = os.path.join(os.path.dirname(_DIR), "include", "agileq.h")

AQ_OK = 0
AQ_ERR_INVALID_ARG, AQ_ERR_SHAPE, AQ_ERR_ALIGNMENT, AQ_ERR_WORKSPACE = -1, -2, -3, -4
AQ_ERR_UNSUPPORTED_DEVICE, AQ_ERR_CUDA, AQ_ERR_DEVICE_TIMEOUT = -5, -6, -7
AQ_ERR_TOO_LARGE = -8
AQ_NOALLOC_SCRATCH_BYTES = 16 * 1024 * 1024 + 65536 + 256
AQ_SCALE_DYNAMIC, AQ_SCALE_STATIC = 0, 1
AQ_KERNEL_AUTO, AQ_KERNEL_TENSOR, AQ_KERNEL_DECODE = 0, 1, 2

_lib = None


class AgileqError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} ({status})")


def declared_symbols() -> list:
    """Names of the functions declared in include/agileq.h."""
    text = open(HEADER_PATH).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aq_[a-z0-9_]+)\s*\(", text)))


def load():
    """Loads the CUDA library; raises if it was not built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2312_05693_b200.build` "
                          "(there is no fallback implementation)")
    L = C.CDLL(LIB_PATH)
    vp, i32, sz = C.c_void_p, C.c_int, C.c_size_t
    L.aq_status_string.restype = C.c_char_p
    L.aq_status_string.argtypes = [i32]
    L.aq_version.restype = i32
    L.aq_create.argtypes = [C.POINTER(vp), i32]
    L.aq_destroy.argtypes = [vp]
    L.aq_last_cuda_error.argtypes = [vp]
    L.aq_set_kernel.argtypes = [vp, i32]
    L.aq_set_weights_stable.argtypes = [vp, i32]
    for f in ("aq_packed_w4_bytes",):
        getattr(L, f).restype = sz
        getattr(L, f).argtypes = [i32, i32]
    L.aq_scales_bytes.restype = sz
    L.aq_scales_bytes.argtypes = [i32, i32, i32]
    L.aq_workspace_bytes.restype = sz
    L.aq_workspace_bytes.argtypes = [i32, i32, i32, i32]
    L.aq_workspace_min_bytes.restype = sz
    L.aq_workspace_min_bytes.argtypes = [i32, i32, i32, i32]
    L.aq_packed_w4_layout_version.restype = i32
    L.aq_linear_host_scratch_bytes.restype = sz
    L.aq_linear_host_scratch_bytes.argtypes = [i32, i32, i32, i32]
    L.aq_pack_w4.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
    L.aq_unpack_w4.argtypes = [vp, vp, i32, i32, vp, vp]
    L.aq_quantize_act.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, sz, vp]
    lin = [vp, vp, i32, i32, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, sz, vp]
    L.aq_linear_w4a8.argtypes = lin
    L.aq_linear_w4a4.argtypes = lin
    L.aq_gemm_w4.argtypes = [vp, vp, i32, i32, vp, vp, i32, i32, vp, vp, vp, vp, sz, vp]
    L.aq_act4_bytes.restype = sz
    L.aq_act4_bytes.argtypes = [i32, i32]
    L.aq_act4_pack.argtypes = [vp, vp, i32, i32, vp, vp]
    L.aq_act4_unpack.argtypes = [vp, vp, i32, i32, vp, vp]
    L.aq_quantize_act4.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, sz, vp]
    L.aq_gemm_w4_act4.argtypes = [vp, vp, i32, i32, vp, vp, i32, i32, vp, vp, vp, vp, sz, vp]
    for f in ("aq_linear_w4a8_chain_act4", "aq_linear_w4a4_chain_act4"):
        getattr(L, f).argtypes = [vp, vp, i32, i32, vp, vp, i32, i32, i32, i32, vp, vp, i32, vp, vp, sz, vp]
    L.aq_weight_offsets.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp]
    L.aq_quantize_act_asym.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp]
    lin_asym = [vp, vp, i32, i32, vp, vp, vp, i32, i32, vp, vp, vp, vp, sz, vp]
    L.aq_linear_w4a8_asym.argtypes = lin_asym
    L.aq_linear_w4a4_asym.argtypes = lin_asym
    lin_chain = [vp, vp, i32, i32, vp, vp, i32, i32, i32, i32, vp, vp, i32, i32, vp, vp, sz, vp]
    L.aq_linear_w4a8_chain.argtypes = lin_chain
    L.aq_linear_w4a4_chain.argtypes = lin_chain
    L.aq_log2_quantize.argtypes = [vp, vp, C.c_longlong, i32, vp, vp, vp, sz, vp]
    L.aq_attn_v_log2.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp]
    L.aq_attn_workspace_bytes.restype = sz
    L.aq_attn_workspace_bytes.argtypes = [i32, i32, i32, i32]
    L.aq_attn_v_log2_tc.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, sz, vp]
    L.aq_log2_quantize_factors.argtypes = [vp, vp, C.c_longlong, vp, vp, vp, sz, vp]
    L.aq_attn_v_factors_tc.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, sz, vp]
    L.aq_attn_qk_tc.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, sz, vp]
    L.aq_prune_schedule.argtypes = [i32, C.c_double, i32, vp, vp]
    L.aq_trip_calibrate.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, vp, sz, vp]
    L.aq_quantize_act_trip.argtypes = [vp, vp, i32, i32, vp, i32, i32, i32, vp, vp, vp, vp, sz, vp]
    L.aq_linear_w4a4_trip.argtypes = [vp, vp, i32, i32, vp, vp, i32, i32, vp, i32, i32, i32, vp, vp, vp, vp, sz, vp]
    L.aq_token_select.argtypes = [vp, vp, i32, i32, vp, vp, sz, vp]
    L.aq_token_compact.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp]
    L.aq_linear_host.argtypes = [vp, i32, vp, i32, i32, vp, vp, i32, i32, i32, i32, vp, vp, sz, vp]
    L.aq_linear_host_async.argtypes = L.aq_linear_host.argtypes
    L.aq_check_workspace.argtypes = [vp, vp, vp]
    L.aq_linear_w4a8_noalloc.argtypes = [vp, vp, i32, i32, vp, vp, i32, i32, i32, i32, vp, vp]
    L.aq_check_noalloc.argtypes = [vp, vp]
    L.aq_probe_int8_mma.argtypes = [vp, i32, i32, vp, vp, sz, vp]
    _lib = L
    return L


def status_string(status: int) -> str:
    return load().aq_status_string(status).decode()


def _check(status: int, what: str):
    if status != AQ_OK:
        raise AgileqError(status, what)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def aq_packed_w4_bytes(N: int, K: int) -> int:
    return load().aq_packed_w4_bytes(N, K)


def aq_scales_bytes(N: int, K: int, group_size: int) -> int:
    return load().aq_scales_bytes(N, K, group_size)


def aq_prune_schedule(M: int, beta: float, m: int):
    """Eq. 9: (tokens kept after each of the m pruning layers, gamma). Host only."""
    out = (C.c_int32 * m)()
    gamma = C.c_double(0.0)
    _check(load().aq_prune_schedule(M, beta, m, C.cast(out, C.c_void_p), C.cast(C.byref(gamma), C.c_void_p)),
           "aq_prune_schedule")
    return list(out), gamma.value


def aq_workspace_bytes(M: int, K: int, N: int, group_size: int) -> int:
    return load().aq_workspace_bytes(M, K, N, group_size)


def aq_workspace_min_bytes(M: int, K: int, N: int, group_size: int) -> int:
    return load().aq_workspace_min_bytes(M, K, N, group_size)


def aq_packed_w4_layout_version() -> int:
    return load().aq_packed_w4_layout_version()


def aq_linear_host_scratch_bytes(M: int, K: int, N: int, group_size: int) -> int:
    return load().aq_linear_host_scratch_bytes(M, K, N, group_size)


class Handle:
    """aq_create / aq_destroy. Methods mirror the C entry points and enqueue on torch's
    current stream."""

    def __init__(self, device: int = 0):
        self._h = C.c_void_p()
        self.device = device
        _check(load().aq_create(C.byref(self._h), device), "aq_create")

    def close(self):
        if self._h:
            load().aq_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- helpers: device memory only
    def _dev(self):
        return torch.device("cuda", self.device)

    def alloc_workspace(self, M: int, K: int, N: int, group_size: int) -> torch.Tensor:
        n = aq_workspace_bytes(M, K, N, group_size)
        if n == 0:
            raise AgileqError(AQ_ERR_SHAPE, "aq_workspace_bytes")
        return torch.empty(n, dtype=torch.uint8, device=self._dev())

    def aq_set_kernel(self, kernel: int):
        _check(load().aq_set_kernel(self._h, kernel), "aq_set_kernel")

    def aq_set_weights_stable(self, enabled: bool):
        _check(load().aq_set_weights_stable(self._h, 1 if enabled else 0), "aq_set_weights_stable")

    def aq_last_cuda_error(self) -> int:
        return load().aq_last_cuda_error(self._h)

    def aq_pack_w4(self, w: torch.Tensor, group_size: int) -> Tuple[torch.Tensor, torch.Tensor]:
        """fp16 [N,K] -> (packed uint8 buffer, fp16 scales [G, Npad])."""
        N, K = w.shape
        nb, ns = aq_packed_w4_bytes(N, K), aq_scales_bytes(N, K, group_size)
        if nb == 0 or ns == 0:
            raise AgileqError(AQ_ERR_SHAPE, "aq_pack_w4")
        packed = torch.empty(nb, dtype=torch.uint8, device=w.device)
        G = K // 128 if group_size else 1
        scales = torch.empty((G, ns // (2 * G)), dtype=torch.float16, device=w.device)
        _check(load().aq_pack_w4(self._h, _ptr(w), N, K, group_size, _ptr(packed), _ptr(scales), _stream()),
               "aq_pack_w4")
        return packed, scales

    def aq_unpack_w4(self, packed: torch.Tensor, N: int, K: int) -> torch.Tensor:
        codes = torch.empty((N, K), dtype=torch.int8, device=packed.device)
        _check(load().aq_unpack_w4(self._h, _ptr(packed), N, K, _ptr(codes), _stream()), "aq_unpack_w4")
        return codes

    def aq_quantize_act(self, x: torch.Tensor, bits: int, scale_mode: int = AQ_SCALE_DYNAMIC,
                        clip_shift_or_exp: int = 0, row_idx: Optional[torch.Tensor] = None,
                        workspace: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
        M_in, K = x.shape
        M = M_in if row_idx is None else row_idx.shape[0]
        q = torch.empty((M, K), dtype=torch.int8, device=x.device)
        e = torch.empty(1, dtype=torch.int32, device=x.device)
        ws = workspace if workspace is not None else torch.empty(256, dtype=torch.uint8, device=x.device)
        _check(load().aq_quantize_act(self._h, _ptr(x), M, K, bits, scale_mode, clip_shift_or_exp,
                                      _ptr(row_idx), _ptr(q), _ptr(e), _ptr(ws), ws.numel(), _stream()),
               "aq_quantize_act")
        return q, e

    def _linear(self, fn, name, x, packed, scales, N, group_size, scale_mode, clip_shift_or_exp, row_idx,
                y, acc_dump, workspace):
        M_in, K = x.shape
        M = M_in if row_idx is None else row_idx.shape[0]
        if y is None:
            y = torch.empty((M, N), dtype=torch.float16, device=x.device)
        if workspace is None:
            workspace = self.alloc_workspace(M, K, N, group_size)
        _check(fn(self._h, _ptr(x), M, K, _ptr(packed), _ptr(scales), N, group_size, scale_mode,
                  clip_shift_or_exp, _ptr(row_idx), _ptr(y), _ptr(acc_dump), _ptr(workspace),
                  workspace.numel(), _stream()), name)
        return y

    def aq_linear_w4a8(self, x, packed, scales, N, group_size, scale_mode=AQ_SCALE_DYNAMIC,
                       clip_shift_or_exp=0, row_idx=None, y=None, acc_dump=None, workspace=None):
        return self._linear(load().aq_linear_w4a8, "aq_linear_w4a8", x, packed, scales, N, group_size,
                            scale_mode, clip_shift_or_exp, row_idx, y, acc_dump, workspace)

    def aq_linear_w4a4(self, x, packed, scales, N, group_size, scale_mode=AQ_SCALE_DYNAMIC,
                       clip_shift_or_exp=0, row_idx=None, y=None, acc_dump=None, workspace=None):
        return self._linear(load().aq_linear_w4a4, "aq_linear_w4a4", x, packed, scales, N, group_size,
                            scale_mode, clip_shift_or_exp, row_idx, y, acc_dump, workspace)

    # ---- log2 codes of the softmax output and attention x value (Eq. 3)
    def aq_log2_quantize(self, x: torch.Tensor, bits: int) -> Tuple[torch.Tensor, torch.Tensor]:
        """(int8 codes of x's shape, uint32[1] holding the fp16 bits of max|x|)."""
        codes = torch.empty(x.shape, dtype=torch.int8, device=x.device)
        mx = torch.zeros(1, dtype=torch.int32, device=x.device)
        ws = torch.empty(256, dtype=torch.uint8, device=x.device)
        _check(load().aq_log2_quantize(self._h, _ptr(x), x.numel(), bits, _ptr(codes), _ptr(mx), _ptr(ws), ws.numel(),
                                       _stream()), "aq_log2_quantize")
        return codes, mx

    def aq_attn_v_log2(self, p_codes, p_max_bits, v_codes, v_scale_exp, bits, y=None, acc_dump=None):
        H, M, J = p_codes.shape
        D = v_codes.shape[2]
        if y is None:
            y = torch.empty((H, M, D), dtype=torch.float16, device=p_codes.device)
        _check(load().aq_attn_v_log2(self._h, _ptr(p_codes), _ptr(p_max_bits), _ptr(v_codes), _ptr(v_scale_exp), H, M, J,
                                     D, bits, _ptr(y), _ptr(acc_dump), _stream()), "aq_attn_v_log2")
        return y

    def aq_attn_v_log2_tc(self, p_codes, p_max_bits, v_codes, v_scale_exp, y=None, workspace=None):
        H, M, J = p_codes.shape
        D = v_codes.shape[2]
        if y is None:
            y = torch.empty((H, M, D), dtype=torch.float16, device=p_codes.device)
        if workspace is None:
            workspace = torch.empty(load().aq_attn_workspace_bytes(H, M, J, D), dtype=torch.uint8, device=p_codes.device)
        _check(load().aq_attn_v_log2_tc(self._h, _ptr(p_codes), _ptr(p_max_bits), _ptr(v_codes), _ptr(v_scale_exp), H, M,
                                        J, D, _ptr(y), _ptr(workspace), workspace.numel(), _stream()),
               "aq_attn_v_log2_tc")
        return y, workspace

    def aq_log2_quantize_factors(self, x: torch.Tensor, factors: Optional[torch.Tensor] = None,
                                 workspace: Optional[torch.Tensor] = None):
        """(uint8 byte factors 128 >> k of x's shape, uint32[1] holding the fp16 bits of max|x|, workspace)."""
        if factors is None:
            factors = torch.empty(x.shape, dtype=torch.uint8, device=x.device)
        mx = torch.zeros(1, dtype=torch.int32, device=x.device)
        ws = workspace if workspace is not None else torch.empty(256, dtype=torch.uint8, device=x.device)
        _check(load().aq_log2_quantize_factors(self._h, _ptr(x), x.numel(), _ptr(factors), _ptr(mx), _ptr(ws), ws.numel(),
                                               _stream()), "aq_log2_quantize_factors")
        return factors, mx, ws

    def aq_attn_v_factors_tc(self, p_factors, p_max_bits, v_codes, v_scale_exp, y=None, workspace=None):
        H, M, J = p_factors.shape
        D = v_codes.shape[2]
        if y is None:
            y = torch.empty((H, M, D), dtype=torch.float16, device=p_factors.device)
        if workspace is None:
            workspace = torch.empty(load().aq_attn_workspace_bytes(H, M, J, D), dtype=torch.uint8, device=p_factors.device)
        _check(load().aq_attn_v_factors_tc(self._h, _ptr(p_factors), _ptr(p_max_bits), _ptr(v_codes), _ptr(v_scale_exp), H,
                                           M, J, D, _ptr(y), _ptr(workspace), workspace.numel(), _stream()),
               "aq_attn_v_factors_tc")
        return y, workspace

    def aq_attn_qk_tc(self, q_codes, q_exp, k_codes, k_exp, s=None, workspace=None):
        H, M, D = q_codes.shape
        J = k_codes.shape[1]
        if s is None:
            s = torch.empty((H, M, J), dtype=torch.float16, device=q_codes.device)
        if workspace is None:
            workspace = torch.empty(256, dtype=torch.uint8, device=q_codes.device)
        _check(load().aq_attn_qk_tc(self._h, _ptr(q_codes), _ptr(q_exp), _ptr(k_codes), _ptr(k_exp), H, M, J, D, _ptr(s),
                                    _ptr(workspace), workspace.numel(), _stream()), "aq_attn_qk_tc")
        return s, workspace

    # ---- chaining: the next layer's codes instead of fp16 outputs (Sec. 4.4)
    def aq_linear_chain(self, bits, x, packed, scales, N, group_size, next_bits, next_exp,
                        scale_mode=AQ_SCALE_DYNAMIC, clip_shift_or_exp=0, row_idx=None, q_next=None, acc_dump=None,
                        workspace=None):
        M_in, K = x.shape
        M = M_in if row_idx is None else row_idx.shape[0]
        if q_next is None:
            q_next = torch.empty((M, N), dtype=torch.int8, device=x.device)
        if workspace is None:
            workspace = self.alloc_workspace(M, K, N, group_size)
        fn = load().aq_linear_w4a8_chain if bits == 8 else load().aq_linear_w4a4_chain
        _check(fn(self._h, _ptr(x), M, K, _ptr(packed), _ptr(scales), N, group_size, scale_mode, clip_shift_or_exp,
                  _ptr(row_idx), _ptr(q_next), next_bits, next_exp, _ptr(acc_dump), _ptr(workspace),
                  workspace.numel(), _stream()), "aq_linear_chain")
        return q_next

    # ---- activations with a zero point (Eq. 2, Eq. 5-7)
    def aq_weight_offsets(self, packed: torch.Tensor, scales: torch.Tensor, N: int, K: int, group_size: int
                          ) -> torch.Tensor:
        r = torch.empty(N, dtype=torch.float32, device=packed.device)
        _check(load().aq_weight_offsets(self._h, _ptr(packed), _ptr(scales), N, K, group_size, _ptr(r), _stream()),
               "aq_weight_offsets")
        return r

    def aq_quantize_act_asym(self, x: torch.Tensor, bits: int, row_idx: Optional[torch.Tensor] = None):
        """(int8 codes q - 2^(b-1), e, zp)."""
        M_in, K = x.shape
        M = M_in if row_idx is None else row_idx.shape[0]
        q = torch.empty((M, K), dtype=torch.int8, device=x.device)
        e = torch.empty(1, dtype=torch.int32, device=x.device)
        zp = torch.empty(1, dtype=torch.int32, device=x.device)
        ws = torch.empty(256, dtype=torch.uint8, device=x.device)
        _check(load().aq_quantize_act_asym(self._h, _ptr(x), M, K, bits, _ptr(row_idx), _ptr(q), _ptr(e), _ptr(zp),
                                           _ptr(ws), ws.numel(), _stream()), "aq_quantize_act_asym")
        return q, e, zp

    def aq_linear_asym(self, bits, x, packed, scales, w_offsets, N, group_size, row_idx=None, y=None, acc_dump=None,
                       workspace=None):
        M_in, K = x.shape
        M = M_in if row_idx is None else row_idx.shape[0]
        if y is None:
            y = torch.empty((M, N), dtype=torch.float16, device=x.device)
        if workspace is None:
            workspace = self.alloc_workspace(M, K, N, group_size)
        fn = load().aq_linear_w4a8_asym if bits == 8 else load().aq_linear_w4a4_asym
        _check(fn(self._h, _ptr(x), M, K, _ptr(packed), _ptr(scales), _ptr(w_offsets), N, group_size, _ptr(row_idx),
                  _ptr(y), _ptr(acc_dump), _ptr(workspace), workspace.numel(), _stream()), "aq_linear_asym")
        return y

    # ---- per-channel TRIP factors (Eq. 5-8)
    def aq_trip_calibrate(self, x: torch.Tensor, k_max: int, row_idx: Optional[torch.Tensor] = None
                          ) -> Tuple[torch.Tensor, torch.Tensor]:
        M_in, K = x.shape
        M = M_in if row_idx is None else row_idx.shape[0]
        alpha = torch.empty(K, dtype=torch.uint8, device=x.device)
        e = torch.empty(1, dtype=torch.int32, device=x.device)
        ws = torch.empty(256, dtype=torch.uint8, device=x.device)
        _check(load().aq_trip_calibrate(self._h, _ptr(x), M, K, k_max, _ptr(row_idx), _ptr(alpha), _ptr(e),
                                        _ptr(ws), ws.numel(), _stream()), "aq_trip_calibrate")
        return alpha, e

    def aq_quantize_act_trip(self, x: torch.Tensor, alpha: torch.Tensor, k_max: int,
                             scale_mode: int = AQ_SCALE_DYNAMIC, clip_shift_or_exp: int = 0,
                             row_idx: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
        M_in, K = x.shape
        M = M_in if row_idx is None else row_idx.shape[0]
        q = torch.empty((M, K), dtype=torch.int8, device=x.device)
        e = torch.empty(1, dtype=torch.int32, device=x.device)
        ws = torch.empty(256, dtype=torch.uint8, device=x.device)
        _check(load().aq_quantize_act_trip(self._h, _ptr(x), M, K, _ptr(alpha), k_max, scale_mode,
                                           clip_shift_or_exp, _ptr(row_idx), _ptr(q), _ptr(e), _ptr(ws),
                                           ws.numel(), _stream()), "aq_quantize_act_trip")
        return q, e

    def aq_linear_w4a4_trip(self, x, packed, scales, N, group_size, alpha, k_max, scale_mode=AQ_SCALE_DYNAMIC,
                            clip_shift_or_exp=0, row_idx=None, y=None, acc_dump=None, workspace=None):
        M_in, K = x.shape
        M = M_in if row_idx is None else row_idx.shape[0]
        if y is None:
            y = torch.empty((M, N), dtype=torch.float16, device=x.device)
        if workspace is None:
            workspace = self.alloc_workspace(M, K, N, group_size)
        _check(load().aq_linear_w4a4_trip(self._h, _ptr(x), M, K, _ptr(packed), _ptr(scales), N, group_size,
                                          _ptr(alpha), k_max, scale_mode, clip_shift_or_exp, _ptr(row_idx),
                                          _ptr(y), _ptr(acc_dump), _ptr(workspace), workspace.numel(), _stream()),
               "aq_linear_w4a4_trip")
        return y

    def aq_gemm_w4(self, q, packed, scales, N, group_size, scale_exp, y=None, acc_dump=None, workspace=None):
        M, K = q.shape
        if y is None:
            y = torch.empty((M, N), dtype=torch.float16, device=q.device)
        if workspace is None:
            workspace = self.alloc_workspace(M, K, N, group_size)
        _check(load().aq_gemm_w4(self._h, _ptr(q), M, K, _ptr(packed), _ptr(scales), N, group_size,
                                 _ptr(scale_exp), _ptr(y), _ptr(acc_dump), _ptr(workspace),
                                 workspace.numel(), _stream()), "aq_gemm_w4")
        return y

    def aq_linear_chain_act4(self, bits, x, packed, scales, N, group_size, next_exp, scale_mode=AQ_SCALE_DYNAMIC,
                             clip_shift_or_exp=0, row_idx=None, q4_next=None, acc_dump=None, workspace=None):
        M_in, K = x.shape
        M = M_in if row_idx is None else row_idx.shape[0]
        if q4_next is None:
            q4_next = torch.empty((M, N // 2), dtype=torch.uint8, device=x.device)
        if workspace is None:
            workspace = self.alloc_workspace(M, K, N, group_size)
        fn = load().aq_linear_w4a8_chain_act4 if bits == 8 else load().aq_linear_w4a4_chain_act4
        _check(fn(self._h, _ptr(x), M, K, _ptr(packed), _ptr(scales), N, group_size, scale_mode, clip_shift_or_exp,
                  _ptr(row_idx), _ptr(q4_next), next_exp, _ptr(acc_dump), _ptr(workspace), workspace.numel(),
                  _stream()), "aq_linear_chain_act4")
        return q4_next

    def aq_act4_pack(self, q: torch.Tensor, q4: Optional[torch.Tensor] = None) -> torch.Tensor:
        M, K = q.shape
        if q4 is None:
            q4 = torch.empty((M, K // 2), dtype=torch.uint8, device=q.device)
        _check(load().aq_act4_pack(self._h, _ptr(q), M, K, _ptr(q4), _stream()), "aq_act4_pack")
        return q4

    def aq_act4_unpack(self, q4: torch.Tensor) -> torch.Tensor:
        M, K2 = q4.shape
        q = torch.empty((M, 2 * K2), dtype=torch.int8, device=q4.device)
        _check(load().aq_act4_unpack(self._h, _ptr(q4), M, 2 * K2, _ptr(q), _stream()), "aq_act4_unpack")
        return q

    def aq_quantize_act4(self, x: torch.Tensor, scale_mode: int = AQ_SCALE_DYNAMIC, clip_shift_or_exp: int = 0,
                         row_idx: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None):
        M_in, K = x.shape
        M = M_in if row_idx is None else row_idx.shape[0]
        q4 = torch.empty((M, K // 2), dtype=torch.uint8, device=x.device)
        e = torch.empty(1, dtype=torch.int32, device=x.device)
        if workspace is None:
            workspace = self.alloc_workspace(M, K, 1, 0)
        _check(load().aq_quantize_act4(self._h, _ptr(x), M, K, scale_mode, clip_shift_or_exp, _ptr(row_idx),
                                       _ptr(q4), _ptr(e), _ptr(workspace), workspace.numel(), _stream()),
               "aq_quantize_act4")
        return q4, e

    def aq_gemm_w4_act4(self, q4, packed, scales, N, group_size, scale_exp, y=None, acc_dump=None, workspace=None):
        M, K2 = q4.shape
        K = 2 * K2
        if y is None:
            y = torch.empty((M, N), dtype=torch.float16, device=q4.device)
        if workspace is None:
            workspace = self.alloc_workspace(M, K, N, group_size)
        _check(load().aq_gemm_w4_act4(self._h, _ptr(q4), M, K, _ptr(packed), _ptr(scales), N, group_size,
                                      _ptr(scale_exp), _ptr(y), _ptr(acc_dump), _ptr(workspace),
                                      workspace.numel(), _stream()), "aq_gemm_w4_act4")
        return y

    def aq_token_select(self, scores: torch.Tensor, n_keep: int, workspace=None) -> torch.Tensor:
        M = scores.shape[0]
        idx = torch.empty(max(n_keep, 1), dtype=torch.int32, device=scores.device)[:n_keep]
        if workspace is None:
            workspace = torch.empty(256 + ((M + 255) // 256) * 256, dtype=torch.uint8, device=scores.device)
        _check(load().aq_token_select(self._h, _ptr(scores), M, n_keep, _ptr(idx), _ptr(workspace),
                                      workspace.numel(), _stream()), "aq_token_select")
        return idx

    def aq_token_compact(self, x: torch.Tensor, idx: torch.Tensor, out=None) -> torch.Tensor:
        M, K = x.shape
        n_keep = idx.shape[0]
        if out is None:
            out = torch.empty((n_keep, K), dtype=torch.float16, device=x.device)
        _check(load().aq_token_compact(self._h, _ptr(x), M, K, _ptr(idx), n_keep, _ptr(out), _stream()),
               "aq_token_compact")
        return out

    def aq_linear_host(self, bits: int, x_host: torch.Tensor, packed, scales, N, group_size,
                       y_host: torch.Tensor, device_scratch: torch.Tensor,
                       scale_mode=AQ_SCALE_DYNAMIC, clip_shift_or_exp=0):
        """x_host / y_host are CPU (ideally pinned) fp16 tensors; synchronizes the stream."""
        M, K = x_host.shape
        _check(load().aq_linear_host(self._h, bits, _ptr(x_host), M, K, _ptr(packed), _ptr(scales), N,
                                     group_size, scale_mode, clip_shift_or_exp, _ptr(y_host),
                                     _ptr(device_scratch), device_scratch.numel(), _stream()),
               "aq_linear_host")
        return y_host

    def aq_linear_host_async(self, bits: int, x_host: torch.Tensor, packed, scales, N, group_size,
                             y_host: torch.Tensor, device_scratch: torch.Tensor,
                             scale_mode=AQ_SCALE_DYNAMIC, clip_shift_or_exp=0):
        """As aq_linear_host, but only enqueues on torch's current stream: y_host is valid once that
        stream has been synchronised; the buffers belong to the call until then."""
        M, K = x_host.shape
        _check(load().aq_linear_host_async(self._h, bits, _ptr(x_host), M, K, _ptr(packed), _ptr(scales), N,
                                           group_size, scale_mode, clip_shift_or_exp, _ptr(y_host),
                                           _ptr(device_scratch), device_scratch.numel(), _stream()),
               "aq_linear_host_async")
        return y_host

    def aq_linear_w4a8_noalloc(self, x, packed, scales, N, group_size, y, scale_mode=AQ_SCALE_DYNAMIC,
                               clip_shift_or_exp=0):
        """The W4A8 layer using the library's built-in scratch buffer. The binding itself allocates
        nothing either: the caller passes the output tensor `y` [M, N] fp16."""
        M, K = x.shape
        _check(load().aq_linear_w4a8_noalloc(self._h, _ptr(x), M, K, _ptr(packed), _ptr(scales), N, group_size,
                                             scale_mode, clip_shift_or_exp, _ptr(y), _stream()),
               "aq_linear_w4a8_noalloc")
        return y

    def aq_check_workspace(self, workspace: torch.Tensor) -> int:
        return load().aq_check_workspace(self._h, _ptr(workspace), _stream())

    def aq_probe_int8_mma(self, iters: int, a_from_tmem: bool, workspace: torch.Tensor) -> float:
        """Enqueues the tensor-core rate probe; returns the integer operations of the launch."""
        ops = C.c_double(0.0)
        _check(load().aq_probe_int8_mma(self._h, iters, 1 if a_from_tmem else 0, C.cast(C.byref(ops), C.c_void_p),
                                        _ptr(workspace), workspace.numel(), _stream()), "aq_probe_int8_mma")
        return ops.value

    def aq_check_noalloc(self) -> int:
        return load().aq_check_noalloc(self._h, _stream())
