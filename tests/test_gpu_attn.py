"""Log2 codes of the softmax output (paper Eq. 3) and attention x value on them, against the CPU checker."""
import numpy as np
import pytest
import torch

import oracle
from paper_2312_05693_b200 import binding, inputs
from gpu_util import assert_y_close, dev, handle

pytestmark = pytest.mark.gpu


def _softmax_rows(H, M, J, seed):
    g = np.random.Generator(np.random.Philox(key=seed))
    s = g.standard_normal((H, M, J)).astype(np.float32) * 3.0
    s -= s.max(axis=2, keepdims=True)
    p = np.exp(s)
    p /= p.sum(axis=2, keepdims=True)
    return p.astype(np.float16)


@pytest.mark.parametrize("bits", [4, 8])
def test_log2_quantize_matches_checker(bits):
    h = handle()
    p = _softmax_rows(3, 37, 200, 51)
    codes, mx = h.aq_log2_quantize(dev(p), bits)
    ref, mref = oracle.log2_quantize(p, bits)
    assert np.float16(mref).view(np.uint16) == (int(mx.item()) & 0xFFFF)
    assert np.array_equal(codes.cpu().numpy(), ref)
    # general values: both signs, zeros, subnormals, NaN, Inf, every binade
    g = np.random.Generator(np.random.Philox(key=52))
    x = (g.standard_normal(70000) * np.exp2(g.integers(-24, 8, size=70000))).astype(np.float16)
    x[:6] = [0.0, -0.0, np.nan, 6e-8, -6e-8, 1.0]
    for extra in (None, np.inf):
        if extra is not None:
            x[10] = extra
        codes, mx = h.aq_log2_quantize(dev(x), bits)
        ref, mref = oracle.log2_quantize(x, bits)
        assert np.float16(mref).view(np.uint16) == (int(mx.item()) & 0xFFFF)
        assert np.array_equal(codes.cpu().numpy(), ref)
    z = np.zeros(64, np.float16)
    codes, mx = h.aq_log2_quantize(dev(z), bits)
    assert int(mx.item()) == 0 and not codes.any().item()


@pytest.mark.parametrize("max_bits", [0x3C00, 0x3DA7, 0x3DA8, 0x3DA9, 0x3A00, 0x7BFF, 0x0400, 0x03FF, 0x0203, 0x0001,
                                      0x2E66, 0x35A8])
def test_log2_quantize_4bit_every_half_below_a_maximum(max_bits):
    """The 4-bit route compares halves against seven bounds derived from the maximum: every half pattern of both
    signs up to the maximum (normal, subnormal, around the sqrt(2) mantissa boundary 0x5A8 of the rounding rule,
    and subnormal maxima), codes and byte factors, against the checker."""
    h = handle()
    mags = np.arange(0, max_bits + 1, dtype=np.uint16)
    bits16 = np.concatenate([mags, mags | np.uint16(0x8000)])
    pad = (-len(bits16)) % 8
    bits16 = np.concatenate([bits16, np.zeros(pad, np.uint16)])
    x = bits16.view(np.float16)
    codes, mx = h.aq_log2_quantize(dev(x), 4)
    ref, mref = oracle.log2_quantize(x, 4)
    assert (int(mx.item()) & 0xFFFF) == max_bits == int(np.float16(mref).view(np.uint16))
    assert np.array_equal(codes.cpu().numpy(), ref)
    xp = np.concatenate([mags, np.zeros((-len(mags)) % 8, np.uint16)]).view(np.float16)      # non-negative only
    f, _, _ = h.aq_log2_quantize_factors(dev(xp))
    rp, _ = oracle.log2_quantize(xp, 4)
    want = np.where(rp > 0, 128 >> np.maximum(rp.astype(np.int32) - 1, 0), 0).astype(np.uint8)
    assert np.array_equal(f.cpu().numpy().view(np.uint8), want)


@pytest.mark.parametrize("H,M,J,D", [(2, 33, 70, 128), (4, 128, 256, 128), (1, 5, 9, 256)])
def test_attn_v_log2_matches_checker(H, M, J, D):
    bits = 4
    h = handle()
    p = _softmax_rows(H, M, J, 53)
    v = inputs.activations(H * J, D, seed=54, outlier_frac=0.01, outlier_mult=8.0)
    pc, pmax = h.aq_log2_quantize(dev(p), bits)
    vq, ev = h.aq_quantize_act(dev(v), 8)
    acc = torch.full((H, M, D), -1, dtype=torch.int32, device="cuda")
    y = h.aq_attn_v_log2(pc, pmax, vq.reshape(H, J, D), ev, bits, acc_dump=acc)
    pc_ref, pmax_ref = oracle.log2_quantize(p, bits)
    e_ref = oracle.layer_exponent(v, 8)
    vq_ref = oracle.quantize_act(v, 8, e_ref).reshape(H, J, D)
    assert np.array_equal(pc.cpu().numpy(), pc_ref) and int(ev.item()) == e_ref
    acc_ref, y_ref = oracle.attn_v_log2(pc_ref, pmax_ref, vq_ref, e_ref, bits)
    assert np.array_equal(acc.cpu().numpy().astype(np.int64), acc_ref)
    assert_y_close(y.cpu().numpy().reshape(H * M, D), y_ref.reshape(H * M, D))
    # and the codes carry the attention: against the unquantized product
    exact = np.einsum("hmj,hjd->hmd", p.astype(np.float64), v.astype(np.float64).reshape(H, J, D))
    err = np.abs(y.cpu().numpy().astype(np.float64) - exact).max()
    assert err < 0.5 * np.abs(exact).max()


def test_attn_bad_shapes_are_refused():
    h = handle()
    pc = torch.zeros((1, 4, 8), dtype=torch.int8, device="cuda")
    mx = torch.zeros(1, dtype=torch.int32, device="cuda")
    ev = torch.zeros(1, dtype=torch.int32, device="cuda")
    for D in (6, 12, 2048):
        vq = torch.zeros((1, 8, D), dtype=torch.int8, device="cuda")
        with pytest.raises(binding.AgileqError):
            h.aq_attn_v_log2(pc, mx, vq, ev, 4)
    with pytest.raises(binding.AgileqError):
        h.aq_attn_v_log2(pc, mx, torch.zeros((1, 8, 128), dtype=torch.int8, device="cuda"), ev, 8)   # 4-bit codes only


# the last four: items of 256 query rows (M a multiple of 256, D = 128), and more items than SMs for both item sizes
@pytest.mark.parametrize("H,M,J,D", [(2, 33, 80, 128), (4, 128, 256, 128), (3, 300, 1040, 64), (1, 5, 16, 64),
                                     (2, 256, 384, 128), (5, 512, 1040, 128), (40, 1024, 256, 128), (20, 1000, 256, 128)])
def test_attn_v_log2_tensor_core_path_matches_checker(H, M, J, D):
    h = handle()
    p = _softmax_rows(H, M, J, 55)
    v = inputs.activations(H * J, 128, seed=56, outlier_frac=0.01, outlier_mult=8.0)[:, :D].copy()
    pc, pmax = h.aq_log2_quantize(dev(p), 4)
    # value codes: the layer quantizer wants rows of 128 values, so quantize a [H*J*D/128, 128] view
    vq, ev = h.aq_quantize_act(dev(v.reshape(-1, 128)), 8)
    vq = vq.reshape(H, J, D)
    y, ws = h.aq_attn_v_log2_tc(pc, pmax, vq, ev)
    assert h.aq_check_workspace(ws) == binding.AQ_OK
    pc_ref, pmax_ref = oracle.log2_quantize(p, 4)
    e_ref = oracle.layer_exponent(v.reshape(-1, 128), 8)
    vq_ref = oracle.quantize_act(v.reshape(-1, 128), 8, e_ref).reshape(H, J, D)
    assert int(ev.item()) == e_ref
    _, y_ref = oracle.attn_v_log2(pc_ref, pmax_ref, vq_ref, e_ref, 4)
    assert_y_close(y.cpu().numpy().reshape(H * M, D), y_ref.reshape(H * M, D))
    # bit for bit the same as the shift kernel (same integer sums, same scaling)
    y_shift = h.aq_attn_v_log2(pc, pmax, vq, ev, 4)
    assert torch.equal(y, y_shift)


@pytest.mark.parametrize("H,M,J,D", [(2, 33, 80, 128), (3, 300, 1040, 64), (1, 5, 16, 64)])
def test_byte_factors_from_the_log2_kernel_feed_the_tensor_core_path(H, M, J, D):
    """aq_log2_quantize_factors writes 128 >> k where aq_log2_quantize writes the code k + 1: the bytes must be that
    function of the checker's codes, and the product on them must be the product on the codes, bit for bit."""
    h = handle()
    p = _softmax_rows(H, M, J, 59)
    p[0, 0, :3] = 0.0                                        # exact zeros: code 0, factor 0
    f, fmax, ws_q = h.aq_log2_quantize_factors(dev(p))
    assert h.aq_check_workspace(ws_q) == binding.AQ_OK
    pc_ref, pmax_ref = oracle.log2_quantize(p, 4)
    assert np.float16(pmax_ref).view(np.uint16) == (int(fmax.item()) & 0xFFFF)
    expect = np.where(pc_ref > 0, 128 >> np.maximum(pc_ref.astype(np.int32) - 1, 0), 0).astype(np.uint8)
    assert np.array_equal(f.cpu().numpy(), expect)
    v = inputs.activations(H * J, 128, seed=60, outlier_frac=0.01, outlier_mult=8.0)[:, :D].copy()
    vq, ev = h.aq_quantize_act(dev(v.reshape(-1, 128)), 8)
    vq = vq.reshape(H, J, D)
    y_f, ws = h.aq_attn_v_factors_tc(f, fmax, vq, ev)
    assert h.aq_check_workspace(ws) == binding.AQ_OK
    pc, pmax = h.aq_log2_quantize(dev(p), 4)
    y_c, _ = h.aq_attn_v_log2_tc(pc, pmax, vq, ev)
    assert torch.equal(y_f, y_c)
    e_ref = oracle.layer_exponent(v.reshape(-1, 128), 8)
    vq_ref = oracle.quantize_act(v.reshape(-1, 128), 8, e_ref).reshape(H, J, D)
    _, y_ref = oracle.attn_v_log2(pc_ref, pmax_ref, vq_ref, e_ref, 4)
    assert_y_close(y_f.cpu().numpy().reshape(H * M, D), y_ref.reshape(H * M, D))
    # a negative input has no byte factor: reported, not silently dropped
    pn = p.copy()
    pn[0, 1, 2] = -0.25
    _, _, ws_n = h.aq_log2_quantize_factors(dev(pn))
    assert h.aq_check_workspace(ws_n) == binding.AQ_ERR_INVALID_ARG


def test_attn_tensor_core_path_reports_negative_codes():
    h = handle()
    pc = torch.ones((1, 8, 16), dtype=torch.int8, device="cuda")
    pc[0, 3, 5] = -2
    mx = torch.full((1,), 0x3C00, dtype=torch.int32, device="cuda")
    ev = torch.zeros(1, dtype=torch.int32, device="cuda")
    vq = torch.ones((1, 16, 64), dtype=torch.int8, device="cuda")
    y, ws = h.aq_attn_v_log2_tc(pc, mx, vq, ev)
    assert h.aq_check_workspace(ws) == binding.AQ_ERR_INVALID_ARG


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("H,M,J", [(2, 33, 80), (3, 300, 1048), (1, 128, 128), (2, 5, 8)])
def test_attn_qk_matches_checker(bits, H, M, J):
    D = 128
    h = handle()
    q = inputs.activations(H * M, D, seed=57, outlier_frac=0.01, outlier_mult=6.0)
    k = inputs.activations(H * J, D, seed=58, outlier_frac=0.01, outlier_mult=6.0)
    qc, eq = h.aq_quantize_act(dev(q), bits)
    kc, ek = h.aq_quantize_act(dev(k), bits)
    s, ws = h.aq_attn_qk_tc(qc.reshape(H, M, D), eq, kc.reshape(H, J, D), ek)
    assert h.aq_check_workspace(ws) == binding.AQ_OK
    eq_ref, ek_ref = oracle.layer_exponent(q, bits), oracle.layer_exponent(k, bits)
    assert (int(eq.item()), int(ek.item())) == (eq_ref, ek_ref)
    qr = oracle.quantize_act(q, bits, eq_ref).reshape(H, M, D)
    kr = oracle.quantize_act(k, bits, ek_ref).reshape(H, J, D)
    ones = np.ones((J, 1), np.float16)
    ref = np.stack([oracle.dequant(oracle.int_gemm(qr[i], kr[i], 0).reshape(M, J, 1), ones, eq_ref + ek_ref)
                    for i in range(H)])
    assert_y_close(s.cpu().numpy().reshape(H * M, J), ref.reshape(H * M, J))
    # the integer sums are below 2^24 here, so the scaled fp16 values are the same bits
    assert np.array_equal(s.cpu().numpy(), ref)
