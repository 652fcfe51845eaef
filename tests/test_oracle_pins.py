"""Pins for the CPU checker: it is compared with things other than itself.

Hand-worked fixtures (tests/golden), closed forms, invariants the quantizers must
satisfy, brute force in Python integers on tiny inputs, library routines that the
special cases reduce to (numpy's fp16 casts, torch's int64 matmul, numpy sorting), and
a restatement of the packed-lane product of Algorithm 1 as a third route to the same
integer sums.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2312_05693_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append(line.split())
    return out


# ----------------------------------------------------------------------------- fp16
def test_half_to_float_all_patterns_match_numpy():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    ref = bits.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(b)) for b in bits], dtype=np.float32)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))


def test_double_to_half_matches_numpy_rne():
    rng = np.random.default_rng(7)
    vals = np.concatenate([
        rng.standard_normal(20000) * 10.0 ** rng.integers(-9, 6, 20000),
        # exact ties between neighbouring halves, subnormals, overflow boundary
        np.array([1.00048828125, 1.00146484375, 2047.5, 2048.5, 65504.0, 65519.999, 65520.0,
                  65536.0, 1e9, 5.960464477539063e-08, 2.9802322387695312e-08,
                  2.98023223876953e-08, 8.940696716308594e-08, 6.097555160522461e-05,
                  6.103515625e-05, 0.0, -0.0, float("inf"), -float("inf")]),
    ])
    vals = np.concatenate([vals, -vals])
    with np.errstate(over="ignore"):
        ref = vals.astype(np.float64).astype(np.float16).view(np.uint16)
    got = np.array([oracle.double_to_half(float(v)) for v in vals], dtype=np.uint16)
    assert np.array_equal(got, ref)


def test_half_round_trip_identity():
    for b in list(range(0, 0x7C01)) + list(range(0x8000, 0xFC01)):
        assert oracle.float_to_half(oracle.half_to_float(b)) == b


# ------------------------------------------------------------------- layer exponent
def test_pow2_exponent_hand_worked():
    for bits, a, e in _rows("pow2_exponent_hand_worked.txt"):
        assert oracle.pow2_exponent(float(a), int(bits)) == int(e), (bits, a, e)


@pytest.mark.parametrize("bits", [8, 4])
def test_pow2_exponent_is_smallest_covering_power(bits):
    rng = np.random.default_rng(1)
    qmax = 2 ** (bits - 1) - 1
    a = (rng.random(20000) * 10.0 ** rng.integers(-6, 5, 20000)).astype(np.float32)
    a = np.minimum(a, np.float32(65504.0))
    for v in a:
        if v == 0:
            continue
        e = oracle.pow2_exponent(float(v), bits)
        assert math.ldexp(qmax, e) >= float(v) > math.ldexp(qmax, e - 1)


def test_layer_exponent_ignores_nan_and_uses_kept_rows_only():
    x = np.zeros((6, 32), np.float16)
    x[1, 3] = 200.0       # dropped row
    x[2, 5] = -3.0
    x[4, 7] = np.nan
    rows = np.array([0, 2, 4, 5], np.int32)
    assert oracle.absmax(x, rows) == 3.0
    assert oracle.layer_exponent(x, 8, rows) == oracle.pow2_exponent(3.0, 8) == -5
    assert oracle.layer_exponent(x, 8) == 1


# ---------------------------------------------------------------- activation quantizer
def test_quantize_act_hand_worked():
    for bits, e, x, code in _rows("quantizer_hand_worked.txt"):
        xs = np.array([[float(x)]], np.float16)
        q = oracle.quantize_act(xs, int(bits), int(e))
        assert int(q[0, 0]) == int(code), (bits, e, x, code, int(q[0, 0]))


@pytest.mark.parametrize("bits,e", [(8, 0), (8, -3), (8, 2), (4, 1), (4, -2), (4, 0)])
def test_quantize_act_invariants(bits, e):
    rng = np.random.default_rng(bits * 100 + e + 50)
    s = 2.0 ** e
    lo, hi = -(2 ** (bits - 1)), 2 ** (bits - 1) - 1
    x = (rng.standard_normal((64, 96)) * s * (hi / 2.0)).astype(np.float16)
    q = oracle.quantize_act(x, bits, e).astype(np.int64)
    xf = x.astype(np.float64)
    assert q.min() >= lo and q.max() <= hi
    inside = (xf >= lo * s) & (xf <= hi * s)
    assert inside.any() and (~inside).any()
    # half a step inside the range (Eq. 2 rounds to the nearest code)
    assert np.all(np.abs(xf[inside] - q[inside] * s) <= s / 2)
    # exact saturation outside
    assert np.all(q[xf > hi * s] == hi)
    assert np.all(q[xf < lo * s] == lo)
    # idempotent: quantizing the dequantized value reproduces the code
    dq = (q * s).astype(np.float16)
    assert np.array_equal(oracle.quantize_act(dq, bits, e).astype(np.int64), q)
    # monotone in x
    order = np.argsort(xf.ravel(), kind="stable")
    assert np.all(np.diff(q.ravel()[order]) >= 0)


def test_quantize_act_ties_go_to_even_and_nonfinite():
    e = -1
    js = np.arange(-20, 20)
    x = ((js + 0.5) * 2.0 ** e).astype(np.float16)[None, :]
    q = oracle.quantize_act(x, 8, e)[0].astype(np.int64)
    expect = np.where(js % 2 == 0, js, js + 1)
    assert np.array_equal(q, expect)
    x = np.array([[np.nan, np.inf, -np.inf]], np.float16)
    assert oracle.quantize_act(x, 8, 0)[0].tolist() == [0, 127, -128]
    assert oracle.quantize_act(x, 4, 3)[0].tolist() == [0, 7, -8]


def test_dynamic_scale_never_clips_and_uses_the_range():
    for seed, bits in [(0, 8), (1, 4), (2, 8)]:
        x = inputs.activations(32, 256, seed, 0.01, 20.0)
        e = oracle.layer_exponent(x, bits)
        q = oracle.quantize_act(x, bits, e).astype(np.int64)
        hi = 2 ** (bits - 1) - 1
        assert np.abs(q).max() <= hi          # -2^(b-1) is never produced without clip_shift
        assert np.abs(q).max() > hi // 2      # one exponent lower would have clipped
        err = np.abs(x.astype(np.float64) - q * 2.0 ** e)
        assert err.max() <= 2.0 ** e / 2


# -------------------------------------------------------------------- weight quantizer
@pytest.mark.parametrize("group", [0, 128])
def test_weight_quantizer_invariants(group):
    w = inputs.weights(24, 384, seed=3)
    w[5, :] = 0                         # an all-zero channel
    w[7, 128:256] = 0                   # an all-zero group
    codes, scales = oracle.quantize_weights(w, group)
    G = 1 if group == 0 else 384 // group
    assert codes.shape == (24, 384) and scales.shape == (24, G)
    assert codes.min() >= -8 and codes.max() <= 7
    gs = 384 // G
    wf = w.astype(np.float64).reshape(24, G, gs)
    cf = codes.astype(np.float64).reshape(24, G, gs)
    sf = scales.astype(np.float64)[:, :, None]
    # every weight is within half a step of its code (the scale is a/7 rounded to fp16,
    # so the largest weight can land a hair beyond code 7 before rounding: allow the
    # clip at 7 to cost at most that rounding)
    amax = np.abs(wf).max(axis=2, keepdims=True)
    slack = np.maximum(amax - 7 * sf, 0)
    assert np.all(np.abs(wf - cf * sf) <= sf / 2 + slack + 1e-12)
    # scale is fp16(absmax/7); the extreme code is used in every non-zero group
    nz = amax[:, :, 0] > 0
    exp_scale = (amax[:, :, 0].astype(np.float32) / np.float32(7.0)).astype(np.float16)
    assert np.array_equal(scales[nz], exp_scale[nz])
    assert np.all(np.abs(cf).max(axis=2)[nz] == 7)
    assert np.all(cf[~nz] == 0) and np.all(scales[~nz] == np.float16(1.0))


def test_weight_codes_match_numpy_rint_of_ieee_division():
    w = inputs.weights(16, 256, seed=11)
    codes, scales = oracle.quantize_weights(w, 128)
    s = np.repeat(scales.astype(np.float32), 128, axis=1)
    ref = np.clip(np.rint(w.astype(np.float32) / s), -8, 7).astype(np.int8)
    assert np.array_equal(codes, ref)


def test_pack_unpack_identity_and_nibble_order():
    allb = np.arange(256, dtype=np.uint8).reshape(1, 256)
    codes = oracle.unpack_w4(allb)
    assert codes.min() == -8 and codes.max() == 7
    assert np.array_equal(oracle.pack_w4(codes), allb)
    # byte 0x8F: low nibble 0xF = -1 is the even k, high nibble 0x8 = -8 the odd k
    assert oracle.unpack_w4(np.array([[0x8F]], np.uint8))[0].tolist() == [-1, -8]
    rng = np.random.default_rng(5)
    c = rng.integers(-8, 8, size=(9, 64)).astype(np.int8)
    assert np.array_equal(oracle.unpack_w4(oracle.pack_w4(c)), c)


def test_packed_activation_codes_by_hand_and_by_arithmetic():
    # Two 4-bit codes per byte (Sec. 4.4), even k in the low nibble: [-8, 7, -1, 0] -> 0x78, 0x0F.
    assert oracle.pack_act4(np.array([[-8, 7, -1, 0]], np.int8))[0].tolist() == [0x78, 0x0F]
    assert oracle.unpack_act4(np.array([[0x78, 0x0F]], np.uint8))[0].tolist() == [-8, 7, -1, 0]
    # against the arithmetic definition byte = (even mod 16) + 16 * (odd mod 16), written with numpy
    rng = np.random.default_rng(11)
    q = rng.integers(-8, 8, size=(7, 96)).astype(np.int8)
    ref = (q[:, 0::2].astype(np.int32) % 16 + 16 * (q[:, 1::2].astype(np.int32) % 16)).astype(np.uint8)
    assert np.array_equal(oracle.pack_act4(q), ref)
    assert np.array_equal(oracle.unpack_act4(ref), q)
    # the product does not care how the codes were stored
    c = rng.integers(-8, 8, size=(5, 128)).astype(np.int8)
    q2 = rng.integers(-8, 8, size=(3, 128)).astype(np.int8)
    assert np.array_equal(oracle.int_gemm(oracle.unpack_act4(oracle.pack_act4(q2)), c, 0), oracle.int_gemm(q2, c, 0))


# --------------------------------------------------------------------- integer product
def _brute(q, c, group):
    M, K = q.shape
    N = c.shape[0]
    gs = K if group == 0 else group
    G = K // gs
    out = np.zeros((M, N, G), dtype=object)
    for g in range(G):
        for k in range(g * gs, (g + 1) * gs):      # k outermost: an unrelated loop order
            for n in range(N):
                for m in range(M):
                    out[m, n, g] += int(q[m, k]) * int(c[n, k])
    return out.astype(np.int64)


@pytest.mark.parametrize("M,N,K,group", [(3, 5, 32, 0), (4, 2, 128, 0), (5, 3, 256, 128),
                                         (1, 4, 384, 128), (2, 5, 160, 0)])
def test_int_gemm_brute_force(M, N, K, group):
    rng = np.random.default_rng(M * 1000 + N * 10 + K)
    q = rng.integers(-128, 128, size=(M, K)).astype(np.int8)
    c = rng.integers(-8, 8, size=(N, K)).astype(np.int8)
    assert np.array_equal(oracle.int_gemm(q, c, group).astype(np.int64), _brute(q, c, group))


def test_int_gemm_closed_forms():
    K = 256
    ones_q = np.ones((3, K), np.int8)
    ones_c = np.ones((4, K), np.int8)
    assert np.all(oracle.int_gemm(ones_q, ones_c, 0) == K)
    assert np.all(oracle.int_gemm(ones_q, ones_c, 128) == 128)
    # c[n,k] = [k == n] picks column n of q
    rng = np.random.default_rng(2)
    q = rng.integers(-128, 128, size=(5, K)).astype(np.int8)
    eye = np.zeros((7, K), np.int8)
    eye[np.arange(7), np.arange(7)] = 1
    assert np.array_equal(oracle.int_gemm(q, eye, 0)[:, :, 0], q[:, :7].astype(np.int32))
    # extremes: (-128)(-8)K, and the largest supported reduction stays inside int32
    lo_q = np.full((1, 13824), -128, np.int8)
    lo_c = np.full((1, 13824), -8, np.int8)
    assert oracle.int_gemm(lo_q, lo_c, 0)[0, 0, 0] == 128 * 8 * 13824
    # transposition would be caught: asymmetric operands
    q2 = np.zeros((2, 32), np.int8)
    c2 = np.zeros((3, 32), np.int8)
    q2[1, 4] = 9
    c2[2, 4] = -3
    acc = oracle.int_gemm(q2, c2, 0)
    assert acc[1, 2, 0] == -27 and np.count_nonzero(acc) == 1


def test_int_gemm_linearity_and_library_matmul():
    rng = np.random.default_rng(9)
    M, N, K = 17, 33, 384
    q1 = rng.integers(-60, 60, size=(M, K)).astype(np.int8)
    q2 = rng.integers(-60, 60, size=(M, K)).astype(np.int8)
    c = rng.integers(-8, 8, size=(N, K)).astype(np.int8)
    a1, a2 = oracle.int_gemm(q1, c, 128), oracle.int_gemm(q2, c, 128)
    assert np.array_equal(oracle.int_gemm((q1 + q2).astype(np.int8), c, 128), a1 + a2)
    # textbook integer matmul from a library, per group and over all of K
    tq, tc = torch.from_numpy(q1).long(), torch.from_numpy(c).long()
    for g in range(3):
        ref = tq[:, g * 128:(g + 1) * 128] @ tc[:, g * 128:(g + 1) * 128].T
        assert np.array_equal(a1[:, :, g].astype(np.int64), ref.numpy())
    assert np.array_equal(oracle.int_gemm(q1, c, 0)[:, :, 0].astype(np.int64), (tq @ tc.T).numpy())
    assert np.array_equal(a1.sum(axis=2), oracle.int_gemm(q1, c, 0)[:, :, 0])


def test_int_gemm_two_sums_share_one_word_without_carry():
    """Sec. 4.4 'INT4 Multiplier': two sums of unsigned 4-bit products can live side by side in one
    32-bit word as long as the reduction is at most 2^8 long. The property behind it, checked here
    against the checker's sums: each sum is at most 15 * 15 * 256 = 57600 < 2^16, so the word
    s0 + 2^16 * s1, built in plain integers, splits back into the two sums with no carry from the low
    field into the high one, also at the extreme (every operand 15); one more doubling of the
    reduction (512 terms of 225 = 115200 > 2^16) would carry, which is why the limit is 2^8."""
    rng = np.random.default_rng(4)
    K = 256
    assert 15 * 15 * K < 1 << 16 <= 15 * 15 * 2 * K
    a = rng.integers(0, 16, size=(4, K))
    w = rng.integers(0, 16, size=(2, K))
    a[0, :] = 15
    w[0, :] = 15                              # row 0 x channel 0 reaches the bound exactly
    sums = oracle.int_gemm(a.astype(np.int8), w.astype(np.int8), 0)[:, :, 0]
    assert int(sums[0, 0]) == 15 * 15 * K
    for m in range(4):
        s0 = sum(int(a[m, k]) * int(w[0, k]) for k in range(K))       # per-field sums, plain integers
        s1 = sum(int(a[m, k]) * int(w[1, k]) for k in range(K))
        word = s0 + (s1 << 16)
        assert word < 1 << 32
        assert (word & 0xFFFF, word >> 16) == (int(sums[m, 0]), int(sums[m, 1]))


# ----------------------------------------------------------------------------- dequant
def test_dequant_per_channel_is_one_rounding_of_the_exact_value():
    rng = np.random.default_rng(12)
    acc = rng.integers(-200000, 200000, size=(6, 10, 1)).astype(np.int32)
    scales = (rng.random((10, 1)) * 0.01 + 1e-4).astype(np.float16)
    for e in (-3, 0, 2):
        y = oracle.dequant(acc, scales, e)
        exact = acc[:, :, 0].astype(np.float64) * scales[:, 0].astype(np.float64)[None, :] * 2.0 ** e
        with np.errstate(over="ignore"):
            assert np.array_equal(y.view(np.uint16), exact.astype(np.float16).view(np.uint16))


def test_dequant_groups_sum_in_double():
    rng = np.random.default_rng(13)
    acc = rng.integers(-100000, 100000, size=(4, 8, 5)).astype(np.int32)
    scales = (rng.random((8, 5)) * 0.02 + 1e-4).astype(np.float16)
    y = oracle.dequant(acc, scales, -1)
    exact = np.einsum("mng,ng->mn", acc.astype(np.float64), scales.astype(np.float64)) * 0.5
    assert np.array_equal(y.view(np.uint16), exact.astype(np.float16).view(np.uint16))


@pytest.mark.parametrize("group,bits", [(0, 8), (128, 8), (128, 4)])
def test_layer_output_within_quantization_error_bound_of_fp_linear(group, bits):
    """With nothing clipped, |y - x w^T| <= sum_k (2^(e-1)|w_k| + (s_w/2)|x_k| + 2^(e-1) s_w/2)
    plus the final fp16 rounding."""
    M, K, N = 8, 256, 12
    x = inputs.activations(M, K, 21, 0.01, 20.0)
    w = inputs.weights(N, K, 21)
    codes, scales = oracle.quantize_weights(w, group)
    out = oracle.linear(x, codes, scales, bits, group)
    e = out["e"]
    xf, wf = x.astype(np.float64), w.astype(np.float64)
    ref = xf @ wf.T
    G = scales.shape[1]
    sw = np.repeat(scales.astype(np.float64), K // G, axis=1)            # [N,K]
    # the scale a/7 is rounded to fp16, so the largest weight of a group may clip by a hair
    werr = np.maximum(sw / 2, np.abs(wf - codes * sw))
    bound = (2.0 ** (e - 1)) * np.abs(wf).sum(axis=1)[None, :] + np.abs(xf) @ werr.T \
        + (2.0 ** (e - 1)) * werr.sum(axis=1)[None, :]
    y = out["y"].astype(np.float64)
    assert np.all(np.abs(y - ref) <= bound + np.abs(ref) * 2.0 ** -10 + 1e-6)
    # and it is not vacuous: the layer tracks the fp result
    assert np.corrcoef(y.ravel(), ref.ravel())[0, 1] > (0.99 if bits == 8 else 0.8)


def test_linear_composite_equals_its_steps():
    M, K, N = 5, 256, 7
    x = inputs.activations(M, K, 31, 0.01, 20.0)
    w = inputs.weights(N, K, 31)
    codes, scales = oracle.quantize_weights(w, 128)
    out = oracle.linear(x, codes, scales, 4, 128, 0, 2, want_acc=True)
    e = oracle.layer_exponent(x, 4) - 2
    q = oracle.quantize_act(x, 4, e)
    acc = oracle.int_gemm(q, codes, 128)
    assert out["e"] == e and np.array_equal(out["q"], q) and np.array_equal(out["acc"], acc)
    assert np.array_equal(out["y"].view(np.uint16), oracle.dequant(acc, scales, e).view(np.uint16))
    assert q.min() == -8 and q.max() == 7      # clip_shift makes the outlier channels saturate
    rows = np.array([0, 4, 2], np.int32)
    cols = np.array([6, 0, 3], np.int32)
    sa, sy = oracle.linear_sampled(q, codes, scales, e, 128, rows, cols)
    assert np.array_equal(sa, acc[rows, cols]) and np.array_equal(sy, out["y"][rows, cols])
    st = oracle.linear(x, codes, scales, 4, 128, 1, e)
    assert np.array_equal(st["y"].view(np.uint16), out["y"].view(np.uint16))


# ----------------------------------------------------------------------- token pruning
def test_token_select_brute_force_with_ties():
    rng = np.random.default_rng(8)
    for M in (1, 2, 7, 33, 64):
        scores = rng.integers(0, 6, size=M).astype(np.float32) / 4      # many duplicates
        for n_keep in sorted({0, 1, M // 2, max(M - 1, 0), M}):
            idx = oracle.token_select(scores, n_keep)
            # brute force: rank = how many tokens beat token i
            rank = [sum(1 for j in range(M) if scores[j] > scores[i] or
                        (scores[j] == scores[i] and j < i)) for i in range(M)]
            ref = [i for i in range(M) if rank[i] < n_keep]
            assert idx.tolist() == ref


def test_token_select_invariants_and_gather():
    M, K = 257, 64
    scores = inputs.token_scores(M, 4)
    n_keep = int(math.ceil(0.6 * M))
    idx = oracle.token_select(scores, n_keep)
    assert len(idx) == n_keep and np.all(np.diff(idx) > 0)
    dropped = np.setdiff1d(np.arange(M), idx)
    assert scores[idx].min() >= scores[dropped].max()
    # numpy's sort as the library routine: same kept set
    ref = np.sort(np.argsort(-scores, kind="stable")[:n_keep])
    assert np.array_equal(idx, ref.astype(np.int32))
    x = inputs.activations(M, K, 4)
    xp = oracle.token_compact(x, idx)
    assert np.array_equal(xp.view(np.uint16), x[idx].view(np.uint16))
    with pytest.raises(ValueError):
        oracle.token_select(scores, M + 1)


def test_progressive_ratio_closed_form():
    # Eq. 9: applying gamma at each of the m pruning layers leaves (1-beta) of the tokens
    for beta, m in [(0.4, 4), (0.16, 8), (0.5, 1), (0.0, 3)]:
        g = oracle.progressive_ratio(beta, m)
        assert abs((1 - g) ** m - (1 - beta)) < 1e-12
    assert abs(oracle.progressive_ratio(0.75, 2) - 0.5) < 1e-15


# ------------------------------------------------------------------------ input recipe
def test_inputs_are_seeded_and_structured():
    a = inputs.activations(64, 512, 1, 0.005, 30.0)
    b = inputs.activations(64, 512, 1, 0.005, 30.0)
    assert np.array_equal(a.view(np.uint16), b.view(np.uint16))
    ch = inputs.outlier_channels(512, 0.005, 1)
    assert len(ch) == 3
    body = np.delete(a.astype(np.float32), ch, axis=1)
    assert 0.9 < body.std() < 1.1 and a.astype(np.float32)[:, ch].std() > 20
    w = inputs.weights(32, 512, 1)
    assert 0.018 < w.astype(np.float32).std() < 0.022
    s = inputs.token_scores(100, 1)
    assert s.min() >= 0 and s.max() < 1 and s.dtype == np.float32


# ------------------------------------------------------------------ TRIP factors (Eq. 5-8)
def _trip_rows():
    rows = []
    for line in open(os.path.join(GOLDEN, "trip_hand_worked.txt")):
        if line.startswith("#") or not line.strip():
            continue
        e, a, x, v = line.split()
        rows.append((int(e), int(a), float(x), int(v)))
    return rows


def test_trip_quantizer_hand_worked_table():
    # Eq. 5 with a per-channel factor, values worked by hand
    for e, a, x, v in _trip_rows():
        xs = np.array([[x]], np.float16)
        got = oracle.quantize_act_trip(xs, 4, e, np.array([a], np.uint8))
        # the table's x are exactly representable in fp16 or far from a rounding boundary
        assert int(got[0, 0]) == v, (e, a, x, v, int(got[0, 0]))


def test_trip_quantizer_invariants_and_special_cases():
    g = np.random.Generator(np.random.Philox(key=4242))
    M, K = 64, 96
    x = (g.standard_normal((M, K)) * 6).astype(np.float16)
    x[:, 5] *= 20
    alpha = g.integers(0, 5, size=K).astype(np.uint8)
    for e in (-3, 0, 2):
        v = oracle.quantize_act_trip(x, 4, e, alpha).astype(np.int64)
        # alpha = 0 everywhere is the plain quantizer of Eq. 2 / Eq. 5
        assert np.array_equal(oracle.quantize_act_trip(x, 4, e, np.zeros(K, np.uint8)), oracle.quantize_act(x, 4, e))
        xf = x.astype(np.float64)
        step = np.exp2(e + alpha.astype(np.float64))[None, :]
        # every value is a multiple of 2^alpha with a 4-bit quotient, and fits int8
        assert np.all(v % (1 << alpha.astype(np.int64))[None, :] == 0)
        qq = v // (1 << alpha.astype(np.int64))[None, :]
        assert qq.min() >= -8 and qq.max() <= 7 and v.min() >= -128 and v.max() <= 127
        # inside the representable range the reconstruction is within half a (coarse) step; outside it saturates
        inside = (xf >= -8 * step) & (xf <= 7 * step)
        assert np.all(np.abs(xf - v * np.exp2(e))[inside] <= step.repeat(M, 0)[inside] / 2 + 1e-12)
        assert np.all(qq[xf > 7 * step] == 7) and np.all(qq[xf < -8 * step] == -8)


def test_trip_factor_on_weights_equals_factor_on_codes():
    # Sec. 4.4: the factor is "transformed over the corresponding weights": shifting weight column k by
    # alpha_k gives the same integer sums as shifting the activation codes of channel k
    g = np.random.Generator(np.random.Philox(key=99))
    M, K, N = 9, 256, 7
    x = (g.standard_normal((M, K)) * 5).astype(np.float16)
    alpha = g.integers(0, 5, size=K).astype(np.uint8)
    c = g.integers(-8, 8, size=(N, K)).astype(np.int8)
    e = -1
    v = oracle.quantize_act_trip(x, 4, e, alpha)
    acc_codes = oracle.int_gemm(v, c, 128)                                 # factor on the codes
    q = v.astype(np.int64) // (1 << alpha.astype(np.int64))[None, :]
    c_shift = c.astype(np.int64) * (1 << alpha.astype(np.int64))[None, :]   # factor on the weights (up to 8 bits)
    ref = np.einsum("mgk,ngk->mng", q.reshape(M, 2, 128), c_shift.reshape(N, 2, 128))
    assert np.array_equal(acc_codes.reshape(M, N, 2).astype(np.int64), ref)


def test_trip_calibration_against_exact_rational_search():
    # Eq. 8 (with the clipping of Eq. 5) by exhaustive search in exact rational arithmetic
    from fractions import Fraction as F
    import math
    def rhe(t):
        f = math.floor(t)
        d = t - f
        return f + 1 if d > F(1, 2) else f if d < F(1, 2) else (f if f % 2 == 0 else f + 1)
    g = np.random.Generator(np.random.Philox(key=31))
    M, K, k_max = 12, 10, 4
    x = (g.standard_normal((M, K)) * 3).astype(np.float16)
    x[:, 2] *= 30                      # an outlier channel
    x[3, 7] = 90                       # a single outlier
    x[:, 4] = 0                        # all zero: every alpha ties at error 0
    x[:, 9] = (g.integers(-7, 8, size=M)).astype(np.float16)   # exactly representable at alpha 0
    for e in (0, -1):
        got = oracle.trip_calibrate(x, 4, e, k_max)
        for k in range(K):
            errs = []
            for a in range(k_max + 1):
                s = F(2) ** (e + a)
                err = F(0)
                for m in range(M):
                    xv = F(float(x[m, k]))
                    q = max(-8, min(7, rhe(xv / s)))
                    err += (xv - q * s) ** 2
                errs.append(err)
            assert int(got[k]) == errs.index(min(errs)), (e, k, errs)
        assert got[4] == 0
        if e == 0:
            assert got[9] == 0 and got[2] >= 3


def test_trip_base_exponent_reaches_the_layer_maximum():
    # Eq. 6 read as s = 2^(e0 - K): with the largest factor the step is the plain layer step again
    x = np.zeros((2, 128), np.float16)
    x[1, 3] = 100.0
    for k_max in (0, 2, 4):
        e = oracle.trip_base_exponent(x, 4, k_max)
        assert e == oracle.layer_exponent(x, 4) - k_max
        alpha = np.full(128, k_max, np.uint8)
        v = oracle.quantize_act_trip(x, 4, e, alpha)
        assert np.array_equal(v.astype(np.int64) >> k_max, oracle.quantize_act(x, 4, e + k_max).astype(np.int64))


# ------------------------------------------- unsigned quantizer with a zero point (Eq. 2, Eq. 5-7)
def test_asym_hand_worked_table():
    for line in open(os.path.join(GOLDEN, "asym_hand_worked.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        if f[0] == "P":
            bits, lo, hi, e, zp = int(f[1]), float(f[2]), float(f[3]), int(f[4]), int(f[5])
            x = np.array([[lo, hi, np.nan, 0.0]], np.float16)          # NaN is ignored
            assert oracle.asym_params(x, bits) == (e, zp), line
        else:
            bits, e, zp, xv, code = int(f[1]), int(f[2]), int(f[3]), float(f[4]), int(f[5])
            got = oracle.quantize_act_asym(np.array([[xv]], np.float16), bits, e, zp)
            assert int(got[0, 0]) == code, line


def test_asym_quantizer_invariants_and_reduction_to_the_signed_one():
    g = np.random.Generator(np.random.Philox(key=808))
    for bits in (8, 4):
        x = (g.standard_normal((50, 64)) * 3 + 2.0).astype(np.float16)       # not centred: zp away from the middle
        e, zp = oracle.asym_params(x, bits)
        qr = (1 << bits) - 1
        xf = x.astype(np.float64)
        lo, hi = min(xf.min(), 0.0), max(xf.max(), 0.0)
        assert qr * 2.0 ** e >= hi - lo > qr * 2.0 ** (e - 1)                # smallest power of two that covers the range
        assert 0 <= zp <= qr and abs(zp - (-lo) / 2.0 ** e) <= 0.5
        q = oracle.quantize_act_asym(x, bits, e, zp).astype(np.int64)
        assert q.min() >= 0 and q.max() <= qr
        deq = (q - zp) * 2.0 ** e
        inside = (xf >= (0 - zp) * 2.0 ** e) & (xf <= (qr - zp) * 2.0 ** e)
        assert np.all(np.abs(xf - deq)[inside] <= 2.0 ** e / 2 + 1e-12)
        assert np.all(q[xf > (qr - zp) * 2.0 ** e] == qr)
        # with zp in the middle of the code range this is the signed quantizer of Eq. 1 moved by 2^(b-1)
        half = 1 << (bits - 1)
        for ee in (e, e - 2):
            assert np.array_equal(oracle.quantize_act_asym(x, bits, ee, half).astype(np.int64) - half,
                                  oracle.quantize_act(x, bits, ee).astype(np.int64))


def test_asym_layer_brute_force_and_zero_point_identity():
    g = np.random.Generator(np.random.Philox(key=909))
    M, K, N = 5, 256, 6
    q = g.integers(0, 256, size=(M, K)).astype(np.uint8)
    c = g.integers(-8, 8, size=(N, K)).astype(np.int8)
    zp, e = 77, -3
    for group in (0, 128):
        G = 1 if group == 0 else K // 128
        sc = (g.random((N, G)) * 0.01 + 0.001).astype(np.float16)
        acc, y = oracle.linear_asym(q, zp, c, sc, e, group)
        ref = np.einsum("mgk,ngk->mng", q.astype(np.int64).reshape(M, G, K // G) - zp,
                        c.astype(np.int64).reshape(N, G, K // G))
        assert np.array_equal(acc, ref)
        # the form the integer product uses: signed codes q - 128 and one correction per (channel, group)
        qs = (q.astype(np.int64) - 128).astype(np.int8)
        raw = oracle.int_gemm(qs, c, group).reshape(M, N, G).astype(np.int64)
        colsum = c.astype(np.int64).reshape(N, G, K // G).sum(axis=2)
        assert np.array_equal(raw - (zp - 128) * colsum[None, :, :], ref)
        # one rounding of the exact value
        exact = (ref.astype(np.float64) * sc.astype(np.float64)[None, :, :]).sum(axis=2) * 2.0 ** e
        assert np.array_equal(y, exact.astype(np.float16))


# ------------------------------------------------------- log2 quantizer and attention x value (Eq. 3)
def test_log2_quantizer_hand_worked_table():
    for line in open(os.path.join(GOLDEN, "log2_hand_worked.txt")):
        if line.startswith("#") or not line.strip():
            continue
        bits, mx, xv, stored = line.split()
        x = np.array([float(mx), float(xv)], np.float16)
        codes, got_max = oracle.log2_quantize(x, int(bits))
        assert got_max == float(np.float16(float(mx)))
        assert int(codes[1]) == int(stored), line
        assert int(codes[0]) == 1                                  # the maximum itself has k = 0


def test_log2_quantizer_against_exact_integer_rule_and_invariants():
    # round(-log2 r) for r = (ma * 2^ea) / (mb * 2^eb) decided with integers only: the fractional part of
    # log2 reaches one half exactly when the mantissa ratio reaches sqrt(2), i.e. when its square reaches 2
    from fractions import Fraction as F
    g = np.random.Generator(np.random.Philox(key=123))
    x = (g.standard_normal(4000) * np.exp2(g.integers(-12, 3, size=4000))).astype(np.float16)
    x[:5] = [0.0, -0.0, np.nan, 6.0, -6.0]
    for bits in (4, 8):
        codes, mx = oracle.log2_quantize(x, bits)
        kmax = (1 << (bits - 1)) - 1
        assert mx == float(np.nanmax(np.abs(x.astype(np.float64))))
        for xv, c in zip(x.tolist(), codes.tolist()):
            if xv != xv or xv == 0.0:
                assert c == 0
                continue
            r = F(abs(xv)) / F(mx)                                 # exact ratio, 0 < r <= 1
            k = 0
            while r * 2 <= 1:                                      # bring r into (1/2, 1]
                r *= 2
                k += 1
            if r * r < F(1, 2):                                    # below 2^-1/2: rounds up to the next k
                k += 1
            k = min(k, kmax)
            assert c == (1 if xv > 0 else -1) * (k + 1), (xv, mx, c, k)
            if k < kmax:                                           # the value lies within half a binade of 2^-k
                assert 2.0 ** (-(k + 0.5)) < abs(xv) / mx <= 2.0 ** (-(k - 0.5))


def test_attn_v_log2_brute_force_and_shift_form():
    g = np.random.Generator(np.random.Philox(key=321))
    H, M, J, D, bits = 2, 5, 40, 16, 4
    kmax = 7
    pc = g.integers(-8, 9, size=(H, M, J)).astype(np.int8)
    vq = g.integers(-128, 128, size=(H, J, D)).astype(np.int8)
    p_max, e_v = 0.8125, -3
    acc, y = oracle.attn_v_log2(pc, p_max, vq, e_v, bits)
    ref = np.zeros((H, M, D), dtype=object)
    for h in range(H):
        for m in range(M):
            for j in range(J):
                c = int(pc[h, m, j])
                if c == 0:
                    continue
                sh = kmax - (abs(c) - 1)
                for d in range(D):
                    t = int(vq[h, j, d]) << sh                     # the product is a shift
                    ref[h, m, d] += t if c > 0 else -t
    assert np.array_equal(acc, ref.astype(np.int64))
    exact = ref.astype(np.float64) * p_max * 2.0 ** (e_v - kmax)
    assert np.array_equal(y, exact.astype(np.float16))
    # the dequantized operands give the same number: p_hat = p_max * sign * 2^-k, v_hat = vq * 2^e_v
    p_hat = np.where(pc == 0, 0.0, np.sign(pc) * p_max * np.exp2(-(np.abs(pc.astype(np.float64)) - 1)))
    assert np.allclose(np.einsum("hmj,hjd->hmd", p_hat, vq.astype(np.float64) * 2.0 ** e_v), exact, rtol=1e-12)
