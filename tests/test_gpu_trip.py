"""Per-channel TRIP factors (paper Eq. 5-8, Sec. 4.4) on the GPU against the CPU checker: the Eq. 8
search, the Eq. 5 quantizer with factors (all three quantize kernels: small, one-pass cooperative,
given exponent) and the whole W4A4 layer through both product kernels."""
import numpy as np
import pytest
import torch

import oracle
from paper_2312_05693_b200 import binding, inputs
from gpu_util import assert_y_close, dev, handle

pytestmark = pytest.mark.gpu


def _acts(M, K, seed):
    # N(0,1) body, 1 % of the channels 25x larger: the channels Eq. 8 should give a factor to
    return inputs.activations(M, K, seed=seed, outlier_frac=0.01, outlier_mult=25.0)


@pytest.mark.parametrize("M,K", [(64, 256), (300, 1152)])
@pytest.mark.parametrize("k_max", [0, 2, 4])
def test_trip_calibrate_matches_checker(M, K, k_max):
    x = _acts(M, K, 21)
    x[:, 7] = 0
    x[1, 9] = np.nan
    x[2, 9] = np.inf                 # skipped by the search; +Inf counts as 65504 for the exponent
    h = handle()
    alpha, e = h.aq_trip_calibrate(dev(x), k_max)
    e_ref = oracle.trip_base_exponent(x, 4, k_max)
    assert int(e.item()) == e_ref
    assert np.array_equal(alpha.cpu().numpy(), oracle.trip_calibrate(x, 4, e_ref, k_max))
    rows = np.array(sorted(set(range(0, M, 3)) - {2}), np.int32)
    alpha, e = h.aq_trip_calibrate(dev(x), k_max, row_idx=dev(rows))
    e_ref = oracle.trip_base_exponent(x, 4, k_max, rows)
    assert int(e.item()) == e_ref
    assert np.array_equal(alpha.cpu().numpy(), oracle.trip_calibrate(x, 4, e_ref, k_max, rows))


@pytest.mark.parametrize("M,K", [(1, 128), (16, 768), (701, 1152)])     # small kernel twice, one-pass kernel
def test_quantize_act_trip_matches_checker(M, K):
    g = np.random.Generator(np.random.Philox(key=5 + M))
    x = _acts(M, K, 22)
    if M > 4:
        x[3, 5] = np.nan
        x[4, 6] = -np.inf
    h = handle()
    for k_max in (0, 3, 4):
        alpha = g.integers(0, k_max + 1, size=K).astype(np.uint8)
        for clip in (0, 1):
            q, e = h.aq_quantize_act_trip(dev(x), dev(alpha), k_max, binding.AQ_SCALE_DYNAMIC, clip)
            e_ref = oracle.trip_base_exponent(x, 4, k_max) - clip
            assert int(e.item()) == e_ref
            assert np.array_equal(q.cpu().numpy(), oracle.quantize_act_trip(x, 4, e_ref, alpha))
        # magnitudes whose exponent is outside the half-precision route
        xs = (np.nan_to_num(x.astype(np.float32), nan=0.0, posinf=0.0, neginf=0.0) * np.float32(2.0 ** -21)).astype(np.float16)
        q, e = h.aq_quantize_act_trip(dev(xs), dev(alpha), k_max)
        e_ref = oracle.trip_base_exponent(xs, 4, k_max)
        assert int(e.item()) == e_ref and e_ref < -14
        assert np.array_equal(q.cpu().numpy(), oracle.quantize_act_trip(xs, 4, e_ref, alpha))
        rows = g.integers(0, M, size=max(1, M // 2)).astype(np.int32)
        q, e = h.aq_quantize_act_trip(dev(x), dev(alpha), k_max, binding.AQ_SCALE_STATIC, -1, row_idx=dev(rows))
        assert int(e.item()) == -1
        assert np.array_equal(q.cpu().numpy(), oracle.quantize_act_trip(x, 4, -1, alpha, rows))


@pytest.mark.parametrize("kernel", [binding.AQ_KERNEL_DECODE, binding.AQ_KERNEL_TENSOR])
@pytest.mark.parametrize("M,K,N,group", [(16, 768, 768, 0), (129, 384, 200, 128), (700, 1152, 520, 128)])
def test_linear_w4a4_trip_matches_checker(kernel, M, K, N, group):
    x = _acts(M, K, 23)
    w = inputs.weights(N, K, 23)
    h = handle()
    k_max = 4
    alpha_t, _ = h.aq_trip_calibrate(dev(x), k_max)          # factors from the data itself
    alpha = alpha_t.cpu().numpy()
    e_ref = oracle.trip_base_exponent(x, 4, k_max)
    assert np.array_equal(alpha, oracle.trip_calibrate(x, 4, e_ref, k_max))
    assert alpha.max() >= 1                                   # the outlier channels got a factor
    packed, scales = h.aq_pack_w4(dev(w), group)
    G = K // 128 if group else 1
    acc = torch.full((M, N, G), -1, dtype=torch.int32, device="cuda")
    ws = h.alloc_workspace(M, K, N, group)
    h.aq_set_kernel(kernel)
    try:
        y = h.aq_linear_w4a4_trip(dev(x), packed, scales, N, group, alpha_t, k_max, acc_dump=acc, workspace=ws)
        assert h.aq_check_workspace(ws) == binding.AQ_OK
    finally:
        h.aq_set_kernel(binding.AQ_KERNEL_AUTO)
    assert int(ws[4:8].view(torch.int32).item()) == e_ref
    v_ref = oracle.quantize_act_trip(x, 4, e_ref, alpha)
    assert np.array_equal(ws[256:256 + M * K].view(torch.int8).reshape(M, K).cpu().numpy(), v_ref)
    codes, sc = oracle.quantize_weights(w, group)
    acc_ref = oracle.int_gemm(v_ref, codes, group)
    assert np.array_equal(acc.cpu().numpy(), acc_ref.reshape(M, N, G))
    assert_y_close(y.cpu().numpy(), oracle.dequant(acc_ref.reshape(M, N, G), sc, e_ref))
    # the factors pay: reconstruction error of the activations against the plain 4-bit layer scale
    xf = x.astype(np.float64)
    e_plain = oracle.layer_exponent(x, 4)
    err_plain = np.square(xf - oracle.quantize_act(x, 4, e_plain).astype(np.float64) * 2.0 ** e_plain).sum()
    err_trip = np.square(xf - v_ref.astype(np.float64) * 2.0 ** e_ref).sum()
    assert err_trip < 0.5 * err_plain


def test_trip_bad_arguments_are_refused():
    h = handle()
    x = dev(_acts(8, 128, 1))
    alpha = torch.zeros(128, dtype=torch.uint8, device="cuda")
    L = binding.load()
    q = torch.empty((8, 128), dtype=torch.int8, device="cuda")
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    args = lambda a, k: (h._h, x.data_ptr(), 8, 128, a, k, 0, 0, None, q.data_ptr(), None, ws.data_ptr(), 256, None)
    assert L.aq_quantize_act_trip(*args(alpha.data_ptr(), 5)) == binding.AQ_ERR_INVALID_ARG      # k_max > 4
    assert L.aq_quantize_act_trip(*args(None, 2)) == binding.AQ_ERR_INVALID_ARG                  # no factors
    assert L.aq_quantize_act_trip(*args(alpha.data_ptr() + 1, 2)) == binding.AQ_ERR_ALIGNMENT
