"""Packed storage of 4-bit activation codes (paper Sec. 4.4: two adjacent 4-bit values share a
byte): packing, unpacking, the quantizer that writes packed codes and the product that reads them
must be bit-exact against the CPU checker, and a chained pair of layers that stores its
intermediate codes packed must equal the same pair with one-byte containers."""
import numpy as np
import pytest
import torch

import oracle
from paper_2312_05693_b200 import binding, inputs
from gpu_util import assert_y_close, dev, handle

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,K", [(1, 32), (3, 96), (16, 768), (257, 160), (300, 4096)])
def test_pack_and_unpack_are_bit_exact(M, K):
    rng = np.random.default_rng(100 + M + K)
    q = rng.integers(-8, 8, size=(M, K), dtype=np.int8)
    q[0, :4] = [-8, 7, -1, 0]
    h = handle()
    q4 = h.aq_act4_pack(dev(q))
    assert q4.shape == (M, K // 2) and q4.dtype == torch.uint8
    assert np.array_equal(q4.cpu().numpy(), oracle.pack_act4(q))
    assert q4.cpu().numpy()[0, :2].tolist() == [0x78, 0x0F]
    back = h.aq_act4_unpack(q4)
    assert np.array_equal(back.cpu().numpy(), q)
    # every byte value decodes as the checker says
    allb = np.arange(256, dtype=np.uint8).reshape(8, 32)
    assert np.array_equal(h.aq_act4_unpack(dev(allb)).cpu().numpy(), oracle.unpack_act4(allb))


@pytest.mark.parametrize("M,K,clip", [(16, 768, 0), (130, 256, 2), (300, 1024, 3)])
def test_quantizer_writes_the_packed_codes_of_the_plain_quantizer(M, K, clip):
    x = inputs.activations(M, K, seed=61, outlier_frac=0.01, outlier_mult=20.0)
    h = handle()
    q4, e = h.aq_quantize_act4(dev(x), clip_shift_or_exp=clip)
    e_ref = oracle.layer_exponent(x, 4) - clip
    assert int(e.item()) == e_ref
    assert np.array_equal(q4.cpu().numpy(), oracle.pack_act4(oracle.quantize_act(x, 4, e_ref)))
    # static exponent and a row gather
    rows = np.sort(np.random.default_rng(5).choice(M, size=max(1, M // 2), replace=False)).astype(np.int32)
    q4s, es = h.aq_quantize_act4(dev(x), binding.AQ_SCALE_STATIC, -1, row_idx=dev(rows))
    assert int(es.item()) == -1
    assert np.array_equal(q4s.cpu().numpy(), oracle.pack_act4(oracle.quantize_act(x, 4, -1, rows)))


@pytest.mark.parametrize("kernel", [binding.AQ_KERNEL_DECODE, binding.AQ_KERNEL_TENSOR])
@pytest.mark.parametrize("M,K,N,group", [(16, 768, 768, 0), (129, 384, 200, 128), (300, 1024, 384, 0),
                                         (260, 1152, 520, 128)])
def test_product_on_packed_codes_matches_checker(kernel, M, K, N, group):
    x = inputs.activations(M, K, seed=62, outlier_frac=0.01, outlier_mult=20.0)
    w = inputs.weights(N, K, 62)
    h = handle()
    packed, scales = h.aq_pack_w4(dev(w), group)
    q4, e = h.aq_quantize_act4(dev(x), clip_shift_or_exp=2)
    G = K // 128 if group else 1
    dump = torch.empty((M, N, G), dtype=torch.int32, device="cuda")
    h.aq_set_kernel(kernel)
    try:
        y = h.aq_gemm_w4_act4(q4, packed, scales, N, group, e, acc_dump=dump)
        torch.cuda.synchronize()
    finally:
        h.aq_set_kernel(binding.AQ_KERNEL_AUTO)
    e_ref = oracle.layer_exponent(x, 4) - 2
    q_ref = oracle.quantize_act(x, 4, e_ref)
    c, sc = oracle.quantize_weights(w, group)
    acc = oracle.int_gemm(q_ref, c, group)
    assert np.array_equal(dump.cpu().numpy().reshape(acc.shape), acc)
    assert_y_close(y.cpu().numpy(), oracle.dequant(acc.reshape(M, N, G), sc, e_ref))


def test_chained_layers_with_packed_intermediate_codes():
    M, K, N1, N2, group = 200, 512, 384, 256, 128
    x = inputs.activations(M, K, seed=63, outlier_frac=0.01, outlier_mult=20.0)
    h = handle()
    p1, s1 = h.aq_pack_w4(dev(inputs.weights(N1, K, 63)), group)
    p2, s2 = h.aq_pack_w4(dev(inputs.weights(N2, N1, 64)), group)
    y1 = h.aq_linear_w4a4(dev(x), p1, s1, N1, group, clip_shift_or_exp=2).cpu().numpy()
    e_next = oracle.layer_exponent(y1, 4) - 1
    q1 = h.aq_linear_chain(4, dev(x), p1, s1, N1, group, 4, e_next, clip_shift_or_exp=2)   # int8 containers
    q1_packed = h.aq_linear_chain_act4(4, dev(x), p1, s1, N1, group, e_next, clip_shift_or_exp=2)   # what is stored
    assert q1_packed.numel() * 2 == q1.numel()
    assert torch.equal(q1_packed, h.aq_act4_pack(q1))
    e_dev = torch.tensor([e_next], dtype=torch.int32, device="cuda")
    y2_packed = h.aq_gemm_w4_act4(q1_packed, p2, s2, N2, group, e_dev)
    y2_plain = h.aq_gemm_w4(q1, p2, s2, N2, group, e_dev)
    assert torch.equal(y2_packed, y2_plain)
    c2, sc2 = oracle.quantize_weights(inputs.weights(N2, N1, 64), group)
    acc = oracle.int_gemm(oracle.quantize_act(y1, 4, e_next), c2, group)
    assert_y_close(y2_packed.cpu().numpy(), oracle.dequant(acc.reshape(M, N2, N1 // 128), sc2, e_next))


@pytest.mark.parametrize("kernel", [binding.AQ_KERNEL_DECODE, binding.AQ_KERNEL_TENSOR])
@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("M,K,N,group", [(1, 256, 128, 0), (16, 768, 768, 0), (129, 384, 224, 128), (300, 1024, 384, 0),
                                         (260, 1152, 544, 128), (300, 1024, 512, 0), (900, 256, 5120, 0)])
def test_chained_epilogue_writes_packed_codes(kernel, bits, M, K, N, group):
    x = inputs.activations(M, K, seed=65, outlier_frac=0.01, outlier_mult=20.0)
    h = handle()
    packed, scales = h.aq_pack_w4(dev(inputs.weights(N, K, 65)), group)
    clip = 0 if bits == 8 else 2
    lin = h.aq_linear_w4a8 if bits == 8 else h.aq_linear_w4a4
    h.aq_set_kernel(kernel)
    try:
        y = lin(dev(x), packed, scales, N, group, clip_shift_or_exp=clip).cpu().numpy()
        e_next = oracle.layer_exponent(y, 4) - 1
        q4 = h.aq_linear_chain_act4(bits, dev(x), packed, scales, N, group, e_next, clip_shift_or_exp=clip)
        torch.cuda.synchronize()
    finally:
        h.aq_set_kernel(binding.AQ_KERNEL_AUTO)
    ref = oracle.quantize_act(y, 4, e_next)
    assert q4.shape == (M, N // 2)
    assert np.array_equal(q4.cpu().numpy(), oracle.pack_act4(ref))
    assert ref.min() == -8 or ref.max() == 7                                  # it did clip


def test_packed_chain_refuses_what_it_cannot_pack():
    h = handle()
    x = dev(inputs.activations(8, 128, seed=1))
    p, s = h.aq_pack_w4(dev(inputs.weights(200, 128, 1)), 0)
    with pytest.raises(binding.AgileqError):
        h.aq_linear_chain_act4(8, x, p, s, 200, 0, 0)                          # N % 32 != 0


def test_bad_arguments_are_refused():
    h = handle()
    with pytest.raises(binding.AgileqError):
        h.aq_act4_pack(torch.zeros((4, 48), dtype=torch.int8, device="cuda"))       # K % 32 != 0
    with pytest.raises(binding.AgileqError):
        h.aq_act4_unpack(torch.zeros((4, 8), dtype=torch.uint8, device="cuda"))     # K = 16
    with pytest.raises(binding.AgileqError):
        h.aq_quantize_act4(torch.zeros((4, 96), dtype=torch.float16, device="cuda"))   # K % 128 != 0
    assert binding.load().aq_act4_bytes(4, 48) == 0 and binding.load().aq_act4_bytes(4, 64) == 128
