"""The layer at the limits of what the library accepts: the longest reduction (K = 65536, where the integer
sums with their factor 16 come closest to the int32 range) in every product kernel, and the smallest shapes.
Large cases are checked against closed forms (every code extreme), small ones against the CPU checker."""
import numpy as np
import pytest
import torch

import oracle
from paper_2312_05693_b200 import binding, inputs
from gpu_util import assert_y_close, dev, handle, run_layer_both

pytestmark = pytest.mark.gpu

K_MAX = 65536


@pytest.mark.parametrize("M,N,group,kernel", [
    (1, 128, 0, binding.AQ_KERNEL_AUTO),        # single-row streaming kernel (quantizes the row itself: falls back when its code buffer is too small)
    (16, 136, 0, binding.AQ_KERNEL_AUTO),       # 16-row streaming kernel
    (3, 128, 128, binding.AQ_KERNEL_AUTO),      # per-group scales, few rows
    (70, 128, 0, binding.AQ_KERNEL_TENSOR),     # tensor cores, 128-channel tiles
    (200, 256, 0, binding.AQ_KERNEL_TENSOR),    # tensor cores, 256-channel tiles
    (150, 128, 128, binding.AQ_KERNEL_TENSOR),  # tensor cores, per-group scales (512 groups)
])
def test_longest_reduction_with_extreme_codes(M, N, group, kernel):
    """x = -128 everywhere with the static exponent 0 and w = -0.01 everywhere give the codes -128 and -7: every
    sum is 128 * 7 * (terms), the largest the 8-bit layer can produce; with the factor 16 the per-channel sum is
    0.94e9, inside int32. The outputs follow in closed form."""
    h = handle()
    K = K_MAX
    x = torch.full((M, K), -128.0, dtype=torch.float16, device="cuda")
    w = torch.full((N, K), -0.01, dtype=torch.float16, device="cuda")
    packed, scales = h.aq_pack_w4(w, group)
    G = K // 128 if group else 1
    acc = torch.full((M, N, G), -1, dtype=torch.int32, device="cuda")
    ws = h.alloc_workspace(M, K, N, group)
    h.aq_set_kernel(kernel)
    try:
        y = h.aq_linear_w4a8(x, packed, scales, N, group, binding.AQ_SCALE_STATIC, 0, acc_dump=acc, workspace=ws)
        assert h.aq_check_workspace(ws) == binding.AQ_OK
    finally:
        h.aq_set_kernel(binding.AQ_KERNEL_AUTO)
    terms = K // G
    assert torch.all(acc == 128 * 7 * terms).item()
    s = float(np.float16(np.float32(np.float16(0.01)) / np.float32(7.0)))      # the stored scale: fp16(a / 7), a = fp16(0.01)
    exact = 128.0 * 7.0 * K * s                                          # all groups have the same scale
    with np.errstate(over="ignore"):
        expect = np.float16(exact)
    yn = y.cpu().numpy()
    if np.isinf(expect):
        assert np.all(np.isinf(yn)) and np.all(yn > 0)
    else:
        assert np.abs(yn.astype(np.float64) - float(expect)).max() <= 1e-3 * abs(float(expect))


@pytest.mark.parametrize("M", [1, 16])
def test_longest_reduction_against_the_checker(M):
    K, N = K_MAX, 136
    x = inputs.activations(M, K, seed=70 + M, outlier_frac=0.001, outlier_mult=20.0)
    w = inputs.weights(N, K, seed=71)
    gpu, ref = run_layer_both(x, w, 8, 0, binding.AQ_KERNEL_AUTO)
    assert gpu["e"] == ref["e"] and np.array_equal(gpu["q"], ref["q"])
    assert np.array_equal(gpu["acc"], ref["acc"])
    assert_y_close(gpu["y"], ref["y"])


@pytest.mark.parametrize("M,K,N,group", [(1, 32, 1, 0), (1, 128, 1, 128), (2, 32, 3, 0), (129, 32, 1, 0), (1, 64, 257, 0)])
def test_smallest_shapes(M, K, N, group):
    x = inputs.activations(M, K, seed=80 + M + N, outlier_frac=0.05, outlier_mult=10.0)
    w = inputs.weights(N, K, seed=81)
    for kernel in (binding.AQ_KERNEL_DECODE, binding.AQ_KERNEL_TENSOR):
        gpu, ref = run_layer_both(x, w, 8, group, kernel)
        assert gpu["e"] == ref["e"] and np.array_equal(gpu["q"], ref["q"])
        assert np.array_equal(gpu["acc"], ref["acc"])
        assert_y_close(gpu["y"], ref["y"])


def test_sizes_beyond_the_limits_are_refused():
    h = handle()
    for (M, K, N, g) in [(1, K_MAX + 32, 128, 0), (1, 16, 128, 0), (0, 128, 128, 0), (1, 128, 0, 0), (4, 160, 128, 128)]:
        assert binding.aq_workspace_bytes(M, K, N, g) == 0
    x = torch.zeros((1, K_MAX + 32), dtype=torch.float16, device="cuda")
    with pytest.raises(binding.AgileqError) as ei:
        h.aq_quantize_act(x, 8)
    assert ei.value.status == binding.AQ_ERR_SHAPE
