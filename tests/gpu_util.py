"""Helpers shared by the GPU parity tests: move seeded inputs to the device, run the CPU
checker on the same bits, compare."""
import numpy as np
import torch

import oracle
from paper_2312_05693_b200 import binding

_handle = None


def handle():
    global _handle
    if _handle is None:
        _handle = binding.Handle(0)
    return _handle


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def scales_to_oracle_layout(scales: torch.Tensor, N: int) -> np.ndarray:
    """library [G, Npad] -> checker [N, G]"""
    return np.ascontiguousarray(scales.cpu().numpy()[:, :N].T)


def assert_y_close(y_gpu: np.ndarray, y_ref: np.ndarray, tol: float = 1e-3):
    """max |y_gpu - y_ref| <= tol * max |y_ref| (the layer's stated fp16 tolerance)."""
    a = y_gpu.astype(np.float64)
    b = y_ref.astype(np.float64)
    scale = np.abs(b).max()
    err = np.abs(a - b).max()
    assert err <= tol * scale + 1e-30, (err, scale, err / max(scale, 1e-30))


def run_layer_both(x, w, bits, group, kernel, scale_mode=0, clip=0, row_idx=None, want_acc=True):
    """Runs the library and the checker on the same inputs. Returns (gpu dict, ref dict)."""
    h = handle()
    N, K = w.shape
    M = x.shape[0] if row_idx is None else len(row_idx)
    G = K // 128 if group else 1
    packed, scales = h.aq_pack_w4(dev(w), group)
    h.aq_set_kernel(kernel)
    try:
        acc = torch.full((M, N, G), -123456789, dtype=torch.int32, device="cuda") if want_acc else None
        ws = h.alloc_workspace(M, K, N, group)
        fn = h.aq_linear_w4a8 if bits == 8 else h.aq_linear_w4a4
        ri = None if row_idx is None else dev(row_idx.astype(np.int32))
        y = fn(dev(x), packed, scales, N, group, scale_mode, clip, row_idx=ri, acc_dump=acc, workspace=ws)
        assert h.aq_check_workspace(ws) == binding.AQ_OK
        e_gpu = int(ws[4:8].view(torch.int32).item())
        q_gpu = ws[256:256 + M * K].view(torch.int8).reshape(M, K).cpu().numpy()
    finally:
        h.aq_set_kernel(binding.AQ_KERNEL_AUTO)
    codes, sc = oracle.quantize_weights(w, group)
    ref = oracle.linear(x, codes, sc, bits, group, scale_mode, clip,
                        row_idx=None if row_idx is None else row_idx.astype(np.int32), want_acc=want_acc)
    gpu = {"y": y.cpu().numpy(), "acc": None if acc is None else acc.cpu().numpy(), "e": e_gpu, "q": q_gpu}
    return gpu, ref
