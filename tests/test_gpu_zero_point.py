"""Activations with a zero point (paper Eq. 2, Eq. 5-7) on the GPU against the CPU checker: parameters
and codes, the per-channel weight term, and the whole layer through both product kernels."""
import numpy as np
import pytest
import torch

import oracle
from paper_2312_05693_b200 import binding, inputs
from gpu_util import assert_y_close, dev, handle, scales_to_oracle_layout

pytestmark = pytest.mark.gpu


def _acts(M, K, seed, shift):
    x = inputs.activations(M, K, seed=seed, outlier_frac=0.01, outlier_mult=10.0).astype(np.float32)
    return (x + np.float32(shift)).astype(np.float16)          # not centred: the zero point moves off the middle


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("M,K", [(1, 128), (37, 1152), (300, 4096)])
def test_quantize_act_asym_matches_checker(bits, M, K):
    h = handle()
    for shift in (0.0, 3.0, -40.0, 200.0):                     # 200: every value positive, min' = 0
        x = _acts(M, K, 31, shift)
        if M > 4:
            x[2, 5] = np.nan
            x[3, 6] = np.inf
        q, e, zp = h.aq_quantize_act_asym(dev(x), bits)
        e_ref, zp_ref = oracle.asym_params(x, bits)
        assert (int(e.item()), int(zp.item())) == (e_ref, zp_ref)
        ref = oracle.quantize_act_asym(x, bits, e_ref, zp_ref).astype(np.int64) - (1 << (bits - 1))
        assert np.array_equal(q.cpu().numpy().astype(np.int64), ref)
    x = _acts(M, K, 32, 1.0)
    rows = np.random.Generator(np.random.Philox(key=3)).integers(0, M, size=max(1, M // 2)).astype(np.int32)
    q, e, zp = h.aq_quantize_act_asym(dev(x), bits, row_idx=dev(rows))
    e_ref, zp_ref = oracle.asym_params(x, bits, rows)
    assert (int(e.item()), int(zp.item())) == (e_ref, zp_ref)
    ref = oracle.quantize_act_asym(x, bits, e_ref, zp_ref, rows).astype(np.int64) - (1 << (bits - 1))
    assert np.array_equal(q.cpu().numpy().astype(np.int64), ref)
    z = np.zeros((2, 128), np.float16)
    q, e, zp = h.aq_quantize_act_asym(dev(z), bits)
    assert (int(e.item()), int(zp.item())) == oracle.asym_params(z, bits) == (0, 0)


@pytest.mark.parametrize("N,K,group", [(200, 384, 128), (768, 768, 0), (77, 256, 0)])
def test_weight_offsets_match_exact_sums(N, K, group):
    w = inputs.weights(N, K, 33)
    h = handle()
    packed, scales = h.aq_pack_w4(dev(w), group)
    r = h.aq_weight_offsets(packed, scales, N, K, group).cpu().numpy()
    codes, sc = oracle.quantize_weights(w, group)
    G = 1 if group == 0 else K // 128
    colsum = codes.astype(np.int64).reshape(N, G, K // G).sum(axis=2)
    ref = (colsum.astype(np.float64) * sc.astype(np.float64)).sum(axis=1)
    assert np.array_equal(r, ref.astype(np.float32))


@pytest.mark.parametrize("kernel", [binding.AQ_KERNEL_DECODE, binding.AQ_KERNEL_TENSOR])
@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("M,K,N,group", [(16, 768, 768, 0), (129, 384, 200, 128), (300, 1024, 384, 0),
                                         (260, 1152, 520, 128), (300, 1024, 512, 0), (900, 256, 5120, 0)])
def test_linear_asym_matches_checker(kernel, bits, M, K, N, group):
    x = _acts(M, K, 34, 2.5)
    w = inputs.weights(N, K, 34)
    h = handle()
    packed, scales = h.aq_pack_w4(dev(w), group)
    r = h.aq_weight_offsets(packed, scales, N, K, group)
    G = 1 if group == 0 else K // 128
    acc = torch.full((M, N, G), -1, dtype=torch.int32, device="cuda")
    ws = h.alloc_workspace(M, K, N, group)
    h.aq_set_kernel(kernel)
    try:
        y = h.aq_linear_asym(bits, dev(x), packed, scales, r, N, group, acc_dump=acc, workspace=ws)
        assert h.aq_check_workspace(ws) == binding.AQ_OK
    finally:
        h.aq_set_kernel(binding.AQ_KERNEL_AUTO)
    e_ref, zp_ref = oracle.asym_params(x, bits)
    q_ref = oracle.quantize_act_asym(x, bits, e_ref, zp_ref)
    half = 1 << (bits - 1)
    assert np.array_equal(ws[256:256 + M * K].view(torch.int8).reshape(M, K).cpu().numpy().astype(np.int64),
                          q_ref.astype(np.int64) - half)
    codes, sc = oracle.quantize_weights(w, group)
    acc_ref, y_ref = oracle.linear_asym(q_ref, zp_ref, codes, sc, e_ref, group)
    # the dump holds the signed product; the zero-point term is one constant per (channel, group)
    colsum = codes.astype(np.int64).reshape(N, G, K // G).sum(axis=2)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64) - (zp_ref - half) * colsum[None, :, :], acc_ref)
    assert_y_close(y.cpu().numpy(), y_ref)
    assert zp_ref != half                                        # the data really was off-centre
