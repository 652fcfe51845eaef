"""Chained layers (paper Sec. 4.4: outputs quantized back for the next operation): the call that
writes the next layer's codes instead of fp16 must give exactly the codes that the quantizer gives
the plain call's fp16 outputs, and a second layer fed with them must match the CPU checker run on
those codes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2312_05693_b200 import binding, inputs
from gpu_util import assert_y_close, dev, handle

pytestmark = pytest.mark.gpu

KERNELS = [binding.AQ_KERNEL_DECODE, binding.AQ_KERNEL_TENSOR]


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("next_bits", [8, 4])
@pytest.mark.parametrize("M,K,N,group", [(16, 768, 768, 0), (129, 384, 200, 128), (300, 1024, 384, 0),
                                         (260, 1152, 520, 128), (130, 256, 203, 128), (300, 1024, 512, 0), (900, 256, 5120, 0)])
def test_chain_codes_equal_quantized_plain_output(kernel, next_bits, M, K, N, group):
    x = inputs.activations(M, K, seed=41, outlier_frac=0.01, outlier_mult=20.0)
    w = inputs.weights(N, K, 41)
    h = handle()
    packed, scales = h.aq_pack_w4(dev(w), group)
    h.aq_set_kernel(kernel)
    try:
        y = h.aq_linear_w4a8(dev(x), packed, scales, N, group).cpu().numpy()
        # an exponent that makes the codes use their range and clip a little
        e_next = oracle.layer_exponent(y, next_bits) - 1
        q_next = h.aq_linear_chain(8, dev(x), packed, scales, N, group, next_bits, e_next)
        torch.cuda.synchronize()
    finally:
        h.aq_set_kernel(binding.AQ_KERNEL_AUTO)
    ref = oracle.quantize_act(y, next_bits, e_next)
    assert np.array_equal(q_next.cpu().numpy(), ref)
    assert ref.min() == -(1 << (next_bits - 1)) or ref.max() == (1 << (next_bits - 1)) - 1   # it did clip


def test_two_chained_layers_match_checker_on_the_codes():
    M, K, N1, N2, group = 200, 512, 384, 256, 128
    x = inputs.activations(M, K, seed=42, outlier_frac=0.01, outlier_mult=20.0)
    w1 = inputs.weights(N1, K, 42)
    w2 = inputs.weights(N2, N1, 43)
    h = handle()
    p1, s1 = h.aq_pack_w4(dev(w1), group)
    p2, s2 = h.aq_pack_w4(dev(w2), group)
    y1 = h.aq_linear_w4a8(dev(x), p1, s1, N1, group).cpu().numpy()
    e_next = oracle.layer_exponent(y1, 8)
    q1 = h.aq_linear_chain(8, dev(x), p1, s1, N1, group, 8, e_next)
    e_dev = torch.tensor([e_next], dtype=torch.int32, device="cuda")
    y2 = h.aq_gemm_w4(q1, p2, s2, N2, group, e_dev).cpu().numpy()
    # the checker on the same codes
    c2, sc2 = oracle.quantize_weights(w2, group)
    acc = oracle.int_gemm(q1.cpu().numpy(), c2, group)
    assert_y_close(y2, oracle.dequant(acc.reshape(M, N2, N1 // 128), sc2, e_next))
    # and the chain equals the unchained path: quantize the fp16 output with the same exponent, then the product
    q_plain, _ = h.aq_quantize_act(dev(y1), 8, binding.AQ_SCALE_STATIC, e_next)
    assert torch.equal(q_plain, q1)


def test_chain_bad_arguments_are_refused():
    h = handle()
    x = dev(inputs.activations(8, 128, seed=1))
    p, s = h.aq_pack_w4(dev(inputs.weights(128, 128, 1)), 0)
    with pytest.raises(binding.AgileqError):
        h.aq_linear_chain(8, x, p, s, 128, 0, 5, 0)            # next_bits must be 8 or 4
    with pytest.raises(binding.AgileqError):
        h.aq_linear_chain(8, x, p, s, 128, 0, 8, 41)           # exponent out of range
