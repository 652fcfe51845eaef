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


@pytest.mark.parametrize("M", [1, 4, 16])
def test_three_layers_in_graph_replay_with_the_stable_weights_promise(M):
    """aq_set_weights_stable lets consecutive few-row calls overlap (the next launch is set up early and fetches
    weights before it waits). Three layers x -> y1 -> y2 -> y3, each reading the previous one's fp16 output,
    captured in a CUDA graph and replayed several times: outputs equal bit for bit with the promise on and
    off, every replay gives the same bits, and each layer matches the CPU checker run on its actual input."""
    dims = [(768, 1280), (1280, 640), (640, 896)]          # (K, N) per layer
    h = handle()
    x = inputs.activations(M, dims[0][0], seed=77, outlier_frac=0.01, outlier_mult=20.0)
    ws, layers = [], []
    for li, (K, N) in enumerate(dims):
        w = inputs.weights(N, K, 78 + li) * 8.0             # keeps the activations of later layers well scaled
        packed, scales = h.aq_pack_w4(dev(w), 0)
        layers.append((w, packed, scales, K, N))
        ws.append(h.alloc_workspace(M, K, N, 0))
    xd = dev(x)
    ys = [torch.empty((M, N), dtype=torch.float16, device="cuda") for _, N in dims]

    def run():
        src = xd
        for li, (_, packed, scales, K, N) in enumerate(layers):
            h.aq_linear_w4a8(src, packed, scales, N, 0, y=ys[li], workspace=ws[li])
            src = ys[li]

    results = {}
    try:
        for promise in (False, True):
            h.aq_set_weights_stable(promise)
            run()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                run()
            outs = []
            for _ in range(4):
                for y in ys:
                    y.zero_()
                g.replay()
                torch.cuda.synchronize()
                outs.append([y.cpu().numpy().copy() for y in ys])
            for o in outs[1:]:
                for a, b in zip(o, outs[0]):
                    assert np.array_equal(a.view(np.uint16), b.view(np.uint16))
            for wsp in ws:
                assert h.aq_check_workspace(wsp) == binding.AQ_OK
            results[promise] = outs[0]
    finally:
        h.aq_set_weights_stable(False)
    for a, b in zip(results[False], results[True]):
        assert np.array_equal(a.view(np.uint16), b.view(np.uint16))
    src = x
    for li, (w, _, _, K, N) in enumerate(layers):
        codes, sc = oracle.quantize_weights(w, 0)
        assert_y_close(results[True][li], oracle.linear(src, codes, sc, 8, 0)["y"])
        src = results[True][li]
