"""GPU parity: the CUDA library against the CPU checker, element by element, through the
C ABI. Integer results (weight codes, scales' bit patterns, the layer exponent, activation
codes, int32 sums, token indices) must be bit-exact; fp16 outputs must satisfy
max|y_gpu - y_ref| <= 1e-3 * max|y_ref|."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2312_05693_b200 import binding, inputs
from gpu_util import assert_y_close, dev, handle, run_layer_both, scales_to_oracle_layout

pytestmark = pytest.mark.gpu

TENSOR, DECODE = binding.AQ_KERNEL_TENSOR, binding.AQ_KERNEL_DECODE
KERNELS = [pytest.param(DECODE, id="decode"), pytest.param(TENSOR, id="tensor")]


# ------------------------------------------------------------------------------ weights
@pytest.mark.parametrize("N,K,group", [(768, 768, 0), (200, 384, 128), (128, 128, 0), (1, 256, 128),
                                       (384, 1024, 128), (200, 160, 0), (136, 96, 0), (9, 32, 0)])
def test_pack_w4_codes_and_scales_bit_exact(N, K, group):
    w = inputs.weights(N, K, seed=N + K)
    if N > 5:
        w[3, :] = 0
        w[4, :128] = 0
        w[5, 7] = np.float16(6e-8)       # a/7 underflows fp16 in its group when alone
        w[5, :7] = 0
        w[5, 8:128] = 0
    h = handle()
    packed, scales = h.aq_pack_w4(dev(w), group)
    codes_gpu = h.aq_unpack_w4(packed, N, K).cpu().numpy()
    codes, sc = oracle.quantize_weights(w, group)
    assert np.array_equal(codes_gpu, codes)
    assert np.array_equal(scales_to_oracle_layout(scales, N).view(np.uint16), sc.view(np.uint16))


# -------------------------------------------------------------------------- activations
@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("M,K", [(1, 128), (16, 768), (37, 1152), (300, 4096)])
def test_quantize_act_dynamic(bits, M, K):
    x = inputs.activations(M, K, seed=M + bits, outlier_frac=0.01, outlier_mult=20.0)
    for clip in (0, 3):
        q, e = handle().aq_quantize_act(dev(x), bits, binding.AQ_SCALE_DYNAMIC, clip)
        e_ref = oracle.layer_exponent(x, bits) - clip
        assert int(e.item()) == e_ref
        assert np.array_equal(q.cpu().numpy(), oracle.quantize_act(x, bits, e_ref))


@pytest.mark.parametrize("bits", [8, 4])
def test_quantize_act_small_dynamic_ties_over_the_exponent_range(bits):
    """The one-launch kernel for small activations: exact ties (x = (j + 1/2) * 2^e), clamped values and
    NaN, with the layer exponent swept over both of its code routes (half2 arithmetic while 2^-e is a
    normal half, fp32 otherwise)."""
    M, K = 8, 256
    qmax = (1 << (bits - 1)) - 1
    j = (np.arange(M * K) % (2 * qmax)) - qmax
    base = (j + 0.5).astype(np.float64).reshape(M, K)          # ties; the largest magnitude sets the exponent
    base[0, 0] = qmax
    h = handle()
    for s in range(-20, 9):
        x = np.ldexp(base, s).astype(np.float16)
        x[1, 1] = np.nan
        q, e = h.aq_quantize_act(dev(x), bits, binding.AQ_SCALE_DYNAMIC, 0)
        e_ref = oracle.layer_exponent(x, bits)
        assert int(e.item()) == e_ref, s
        assert np.array_equal(q.cpu().numpy(), oracle.quantize_act(x, bits, e_ref)), s
        q, e = h.aq_quantize_act(dev(x), bits, binding.AQ_SCALE_DYNAMIC, 2)     # lower exponent: values clamp
        assert np.array_equal(q.cpu().numpy(), oracle.quantize_act(x, bits, e_ref - 2)), s


def test_quantize_act_static_rowidx_and_nonfinite():
    M, K = 40, 256
    x = inputs.activations(M, K, seed=5, outlier_frac=0.01, outlier_mult=20.0)
    x[3, 5] = np.nan
    x[7, 9] = np.inf
    x[8, 1] = -np.inf
    x[0, 0] = 30000.0                     # dropped by row_idx below
    rows = np.array([1, 3, 7, 8, 20, 39, 2], np.int32)
    h = handle()
    for bits in (8, 4):
        q, e = h.aq_quantize_act(dev(x), bits, binding.AQ_SCALE_STATIC, -2, row_idx=dev(rows))
        assert int(e.item()) == -2
        assert np.array_equal(q.cpu().numpy(), oracle.quantize_act(x, bits, -2, rows))
        q, e = h.aq_quantize_act(dev(x), bits, binding.AQ_SCALE_DYNAMIC, 0, row_idx=dev(rows))
        e_ref = oracle.layer_exponent(x, bits, rows)
        assert int(e.item()) == e_ref == (10 if bits == 8 else 14)      # +Inf counts as 65504
        assert np.array_equal(q.cpu().numpy(), oracle.quantize_act(x, bits, e_ref, rows))
    fin = np.array([2, 20, 39], np.int32)
    q, e = h.aq_quantize_act(dev(x), 8, binding.AQ_SCALE_DYNAMIC, 0, row_idx=dev(fin))
    assert int(e.item()) == oracle.layer_exponent(x, 8, fin)
    z = np.zeros((4, 128), np.float16)
    q, e = h.aq_quantize_act(dev(z), 8)
    assert int(e.item()) == 0 and not q.any().item()


@pytest.mark.parametrize("bits", [8, 4])
def test_quantize_act_one_pass_kernel_edges(bits):
    # sizes above the small-activation limit take the cooperative one-pass kernel: ragged split over
    # the CTAs, exact ties, non-finite values, gathered (repeated, permuted) rows, and exponents on
    # both sides of the half-precision fast path
    M, K = 701, 1152
    g = np.random.Generator(np.random.Philox(key=77 + bits))
    h = handle()
    # (a) multiples of 1/2 with max 127: e = 0 for 8 bits, every second value is an exact tie
    x = (g.integers(-254, 255, size=(M, K)) * 0.5).astype(np.float16)
    x[5, 7] = 127.0
    for clip in (0, 2):
        q, e = h.aq_quantize_act(dev(x), bits, binding.AQ_SCALE_DYNAMIC, clip)
        e_ref = oracle.layer_exponent(x, bits) - clip
        assert int(e.item()) == e_ref
        assert np.array_equal(q.cpu().numpy(), oracle.quantize_act(x, bits, e_ref))
    # (b) NaN / Inf inside, rows gathered with repeats and out of order
    x2 = inputs.activations(M, K, seed=9, outlier_frac=0.01, outlier_mult=20.0)
    x2[3, 5] = np.nan
    x2[700, 1151] = np.nan
    x2[17, 9] = np.inf
    x2[18, 1] = -np.inf
    rows = g.integers(0, M, size=650).astype(np.int32)
    rows[:4] = [700, 3, 17, 18]
    q, e = h.aq_quantize_act(dev(x2), bits, binding.AQ_SCALE_DYNAMIC, 0, row_idx=dev(rows))
    e_ref = oracle.layer_exponent(x2, bits, rows)
    assert int(e.item()) == e_ref == (10 if bits == 8 else 14)
    assert np.array_equal(q.cpu().numpy(), oracle.quantize_act(x2, bits, e_ref, rows))
    # (c) tiny and large magnitudes: exponents far below / near the top of what fp16 inputs can give
    for scale in (2.0 ** -20, 2.0 ** -12, 300.0):
        x3 = (inputs.activations(M, K, seed=11).astype(np.float32) * np.float32(scale)).astype(np.float16)
        q, e = h.aq_quantize_act(dev(x3), bits)
        e_ref = oracle.layer_exponent(x3, bits)
        assert int(e.item()) == e_ref
        assert np.array_equal(q.cpu().numpy(), oracle.quantize_act(x3, bits, e_ref))


def test_quantize_act_all_fp16_magnitudes_exponent():
    # one value at a time through the absmax -> exponent path: every binade and mantissa edge
    h = handle()
    vals = [6e-8, 1e-4, 0.0078125, 0.99, 0.9921875, 1.0, 7.0, 7.5, 127.0, 127.06, 128.0, 254.0, 255.0,
            1000.0, 32512.0, 65024.0, 65504.0]
    for v in vals:
        x = np.zeros((2, 128), np.float16)
        x[1, 77] = -v
        for bits in (8, 4):
            _, e = h.aq_quantize_act(dev(x), bits)
            assert int(e.item()) == oracle.layer_exponent(x, bits), (v, bits)


# ---------------------------------------------------------------------------- the layer
SHAPES = [
    # M, K, N, group
    (16, 768, 768, 0),         # OPT-125M-like single layer
    (1, 256, 128, 0),
    (3, 384, 200, 128),        # ragged N
    (17, 512, 136, 0),
    (129, 384, 200, 128),      # spans token tiles with a ragged tail
    (300, 1024, 384, 0),
    (260, 1152, 520, 128),
    (130, 256, 203, 128),      # N not a multiple of 8: outputs take direct stores instead of TMA stores
    (70, 256, 77, 0),
    (950, 256, 2556, 128),     # 192-token tiles (5 x 20 tiles in one round), ragged last tile, direct stores
    (950, 384, 2560, 128),     # the same tiles with TMA stores
]


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("M,K,N,group", SHAPES)
def test_linear_w4a8_matches_checker(kernel, M, K, N, group):
    x = inputs.activations(M, K, seed=M + N, outlier_frac=0.01, outlier_mult=20.0)
    w = inputs.weights(N, K, seed=K + N)
    gpu, ref = run_layer_both(x, w, 8, group, kernel)
    assert gpu["e"] == ref["e"]
    assert np.array_equal(gpu["q"], ref["q"])
    assert np.array_equal(gpu["acc"], ref["acc"])
    assert_y_close(gpu["y"], ref["y"])


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("M,K,N", [(1, 160, 136), (5, 96, 200), (16, 4224, 128), (140, 160, 264), (300, 4224, 384),
                                   (70, 32, 77), (1, 32, 8), (200, 1120, 130)])
def test_k_a_multiple_of_32_with_one_scale_per_channel(kernel, M, K, N):
    """K % 128 != 0 (one scale per channel): the last 128-k block of the packed weights is padded with zero
    codes, so the activation codes beyond K never count, in every product kernel."""
    x = inputs.activations(M, K, seed=M + N + 3, outlier_frac=0.02, outlier_mult=20.0)
    w = inputs.weights(N, K, seed=K + N + 3)
    gpu, ref = run_layer_both(x, w, 8, 0, kernel)
    assert gpu["e"] == ref["e"]
    assert np.array_equal(gpu["q"], ref["q"])
    assert np.array_equal(gpu["acc"], ref["acc"])
    assert_y_close(gpu["y"], ref["y"])
    # extreme codes over a ragged K: a slip in the padding would show as a wrong count of terms
    xe = np.full((M, K), -128.0, np.float16)
    we = np.full((N, K), -0.01, np.float16)
    gpu, ref = run_layer_both(xe, we, 8, 0, kernel, scale_mode=1, clip=0)
    assert np.array_equal(gpu["acc"], ref["acc"]) and ref["acc"].max() == 128 * 7 * K
    if K % 128:
        with pytest.raises(binding.AgileqError) as ei:      # per-group scales keep K % 128 == 0
            handle().aq_pack_w4(dev(w), 128)
        assert ei.value.status == binding.AQ_ERR_SHAPE


@pytest.mark.parametrize("group", [0, 128])
@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 8, 11, 16])
def test_decode_rows_1_to_16(M, group):
    """The M <= 16 path (dp4a up to 4 rows, warp MMA above) over several k splits and a ragged N."""
    for K, N in [(1280, 392), (5120, 128)]:
        x = inputs.activations(M, K, seed=M + K, outlier_frac=0.01, outlier_mult=20.0)
        w = inputs.weights(N, K, seed=N + K)
        gpu, ref = run_layer_both(x, w, 8, group, binding.AQ_KERNEL_AUTO)
        assert gpu["e"] == ref["e"] and np.array_equal(gpu["q"], ref["q"])
        assert np.array_equal(gpu["acc"], ref["acc"])
        assert_y_close(gpu["y"], ref["y"])
    # extreme codes: the largest sums the 16x-widened weights can produce
    K, N = 13824, 128
    x = np.full((M, K), -128.0, np.float16)
    w = np.full((N, K), -0.01, np.float16)
    gpu, ref = run_layer_both(x, w, 8, group, binding.AQ_KERNEL_AUTO, scale_mode=1, clip=0)
    assert np.array_equal(gpu["acc"], ref["acc"])
    assert_y_close(gpu["y"], ref["y"])


@pytest.mark.parametrize("M,K,N", [(2, 12288, 4096), (16, 13824, 5120), (5, 7680, 6400), (9, 9216, 5700),
                                   (16, 13824, 4000)])
def test_decode_clusters_of_five_to_eight(M, K, N):
    """Long k ranges with 2..16 rows take clusters of 8, 7, 5, 6 and 8 CTAs per channel tile (uneven channel
    slices for 5 to 7; a ragged N twice): integer sums exact, outputs within tolerance, and the chained call,
    which keeps clusters of at most 4, gives the codes of the quantizer applied to these outputs."""
    x = inputs.activations(M, K, seed=M + K, outlier_frac=0.01, outlier_mult=20.0)
    w = inputs.weights(N, K, seed=N + K)
    gpu, ref = run_layer_both(x, w, 8, 0, binding.AQ_KERNEL_AUTO)
    assert gpu["e"] == ref["e"] and np.array_equal(gpu["q"], ref["q"])
    assert np.array_equal(gpu["acc"], ref["acc"])
    assert_y_close(gpu["y"], ref["y"])
    h = handle()
    packed, scales = h.aq_pack_w4(dev(w), 0)
    y = h.aq_linear_w4a8(dev(x), packed, scales, N, 0)            # without the dump of the sums: the plain-output loop
    assert np.array_equal(y.cpu().numpy().view(np.uint16), gpu["y"].view(np.uint16))
    if N % 32 == 0:
        e_next = oracle.layer_exponent(gpu["y"], 8) - 1
        q_next = h.aq_linear_chain(8, dev(x), packed, scales, N, 0, 8, e_next)
        assert np.array_equal(q_next.cpu().numpy(), oracle.quantize_act(gpu["y"], 8, e_next))


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("M,K,N,group", [(16, 768, 768, 0), (129, 384, 200, 128), (260, 1152, 520, 128)])
def test_linear_w4a4_matches_checker(kernel, M, K, N, group):
    x = inputs.activations(M, K, seed=M + N + 1, outlier_frac=0.005, outlier_mult=30.0)
    w = inputs.weights(N, K, seed=K + N + 1)
    gpu, ref = run_layer_both(x, w, 4, group, kernel, clip=4)
    assert gpu["e"] == ref["e"]
    assert gpu["q"].min() == -8 and gpu["q"].max() == 7
    assert np.array_equal(gpu["q"], ref["q"])
    assert np.array_equal(gpu["acc"], ref["acc"])
    assert_y_close(gpu["y"], ref["y"])


@pytest.mark.parametrize("kernel", KERNELS)
def test_linear_extreme_codes_and_patterns(kernel):
    """Largest-magnitude sums and an identity-like weight matrix: catches layout slips
    (a swapped nibble, a transposed tile, a wrong swizzle) that random data could blur."""
    h = handle()
    M, K, N = 130, 512, 256
    x = np.full((M, K), -128.0, np.float16)
    w = np.full((N, K), -0.01, np.float16)                 # every code is -7
    gpu, ref = run_layer_both(x, w, 8, 0, kernel, scale_mode=1, clip=0)
    assert np.array_equal(gpu["acc"], ref["acc"]) and ref["acc"].max() == 128 * 7 * K
    assert_y_close(gpu["y"], ref["y"])
    # x[m,k] = small integers depending on (m,k); w picks single k per channel
    xm = ((np.arange(M)[:, None] * 7 + np.arange(K)[None, :] * 3) % 255 - 127).astype(np.float16)
    wm = np.zeros((N, K), np.float16)
    wm[np.arange(N), (np.arange(N) * 5 + 3) % K] = 1.0
    wm[np.arange(N), (np.arange(N) * 11 + 130) % K] = -0.5
    for group in (0, 128):
        gpu, ref = run_layer_both(xm, wm, 8, group, kernel, scale_mode=1, clip=0)
        assert np.array_equal(gpu["q"], ref["q"])
        assert np.array_equal(gpu["acc"], ref["acc"])
        assert_y_close(gpu["y"], ref["y"])


@pytest.mark.parametrize("kernel", KERNELS)
def test_linear_with_row_idx_equals_compacted_input(kernel):
    M_in, K, N = 200, 512, 256
    x = inputs.activations(M_in, K, seed=77, outlier_frac=0.01, outlier_mult=25.0)
    w = inputs.weights(N, K, seed=78)
    scores = inputs.token_scores(M_in, 77)
    n_keep = int(math.ceil(0.6 * M_in))
    idx = oracle.token_select(scores, n_keep)
    gpu, ref = run_layer_both(x, w, 8, 0, kernel, row_idx=idx)
    assert gpu["e"] == ref["e"] and np.array_equal(gpu["q"], ref["q"])
    assert np.array_equal(gpu["acc"], ref["acc"])
    assert_y_close(gpu["y"], ref["y"])


@pytest.mark.parametrize("M,K,N", [(300, 1024, 512), (257, 384, 250), (129, 4224, 256), (1000, 256, 5120), (1400, 640, 6400),
                                   (700, 2048, 1024), (193, 160, 1536)])
def test_one_scale_per_channel_on_tiles_of_two_channel_blocks(M, K, N):
    """More than 128 tokens and an even number of 128-channel blocks: the tensor-core kernel whose tile is two
    channel blocks sharing an activation tile of 128 or 192 tokens. Ragged token and channel edges, K not a
    multiple of 128, more tiles than SMs (several tiles per CTA), both tile heights, with the zero-point term
    and with chaining."""
    x = inputs.activations(M, K, seed=M + N + 9, outlier_frac=0.01, outlier_mult=20.0)
    w = inputs.weights(N, K, seed=K + N + 9)
    for bits, clip in ((8, 0), (4, 4)):
        gpu, ref = run_layer_both(x, w, bits, 0, TENSOR, clip=clip)
        assert gpu["e"] == ref["e"] and np.array_equal(gpu["q"], ref["q"])
        assert np.array_equal(gpu["acc"], ref["acc"])
        assert_y_close(gpu["y"], ref["y"])
    gpu2, _ = run_layer_both(x, w, 8, 0, TENSOR, want_acc=False)          # as the benchmark calls it
    gpu1, _ = run_layer_both(x, w, 8, 0, TENSOR)
    assert np.array_equal(gpu1["y"].view(np.uint16), gpu2["y"].view(np.uint16))
    # extreme codes: the largest sums
    xe = np.full((M, K), -128.0, np.float16)
    we = np.full((N, K), -0.01, np.float16)
    gpu, ref = run_layer_both(xe, we, 8, 0, TENSOR, scale_mode=1, clip=0)
    assert np.array_equal(gpu["acc"], ref["acc"]) and ref["acc"].max() == 128 * 7 * K


@pytest.mark.parametrize("group", [0, 128])
def test_several_tiles_per_cta_and_deep_k(group):
    """More tiles than SMs and more k blocks than any ring is deep: every ring and every
    accumulator stage wraps many times inside one persistent CTA."""
    M, K, N = 1100, 2048, 4992          # 39 channel tiles x 9 (or 5) token tiles, 16 k blocks
    x = inputs.activations(M, K, seed=123, outlier_frac=0.005, outlier_mult=30.0)
    w = inputs.weights(N, K, seed=124)
    gpu, ref = run_layer_both(x, w, 8, group, TENSOR)
    assert gpu["e"] == ref["e"] and np.array_equal(gpu["q"], ref["q"])
    assert np.array_equal(gpu["acc"], ref["acc"])
    assert_y_close(gpu["y"], ref["y"])


@pytest.mark.parametrize("M,N,K", [(200, 520, 8192), (200, 520, 11008), (380, 12800, 4096), (380, 12800, 8192)])
def test_shared_tiles_of_a_partial_last_round(M, N, K):
    """A last round that fills less than half of the SMs: those tiles are shared by two CTAs (half of K
    each, partial sums exchanged). 200 x 520: ten 128-token tiles, every tile is shared; 380 x 12800: two
    hundred 192-token tiles, one whole round and then 52 shared tiles, at the smallest depth that shares
    such tiles (32 k blocks) and at 64."""
    x = inputs.activations(M, K, seed=125, outlier_frac=0.005, outlier_mult=30.0)
    w = inputs.weights(N, K, seed=126)
    assert binding.aq_workspace_bytes(M, K, N, 128) > binding.aq_workspace_bytes(M, K, N, 0)   # room for the partial sums
    gpu, ref = run_layer_both(x, w, 8, 128, TENSOR)
    assert gpu["e"] == ref["e"] and np.array_equal(gpu["q"], ref["q"])
    assert np.array_equal(gpu["acc"], ref["acc"])
    assert_y_close(gpu["y"], ref["y"])
    gpu2, _ = run_layer_both(x, w, 8, 128, TENSOR, want_acc=False)
    assert np.array_equal(gpu["y"].view(np.uint16), gpu2["y"].view(np.uint16))     # whichever half arrives second


@pytest.mark.parametrize("seed", range(10))
def test_seeded_random_shapes_per_group_scales(seed):
    """Shapes drawn from a seeded generator: token counts that leave ragged 128- and 192-token tiles,
    channel counts that are not multiples of 128 (some not of 8), 1 to 12 k blocks; with and without
    int4 activations."""
    rng = np.random.default_rng(1000 + seed)
    M = int(rng.integers(129, 1400))
    K = 128 * int(rng.integers(1, 13))
    N = int(rng.integers(1, 700)) * (4 if seed % 3 == 0 else 8)
    bits = 4 if seed % 2 else 8
    x = inputs.activations(M, K, seed=seed, outlier_frac=0.01, outlier_mult=25.0)
    w = inputs.weights(N, K, seed=seed + 50)
    gpu, ref = run_layer_both(x, w, bits, 128, TENSOR, clip=4 if bits == 4 else 0)
    assert gpu["e"] == ref["e"] and np.array_equal(gpu["q"], ref["q"])
    assert np.array_equal(gpu["acc"], ref["acc"])
    assert_y_close(gpu["y"], ref["y"])
    gpu2, _ = run_layer_both(x, w, bits, 128, TENSOR, clip=4 if bits == 4 else 0, want_acc=False)
    assert np.array_equal(gpu["y"].view(np.uint16), gpu2["y"].view(np.uint16))


def test_results_are_deterministic_run_to_run():
    M, K, N = 260, 1152, 520
    x = inputs.activations(M, K, seed=9, outlier_frac=0.01, outlier_mult=20.0)
    w = inputs.weights(N, K, seed=10)
    h = handle()
    packed, scales = h.aq_pack_w4(dev(w), 128)
    xd = dev(x)
    ws = h.alloc_workspace(M, K, N, 128)
    first = None
    for _ in range(10):
        y = h.aq_linear_w4a8(xd, packed, scales, N, 128, workspace=ws).cpu().numpy().view(np.uint16)
        first = y if first is None else first
        assert np.array_equal(y, first)


# ------------------------------------------------------------------------ token pruning
@pytest.mark.parametrize("M,ratio", [(1, 1.0), (7, 0.5), (257, 0.6), (4096, 0.6), (1000, 0.0), (4097, 1.0), (8192, 0.3),
                                     (10000, 0.6), (65536, 0.41)])
def test_token_select_and_compact(M, ratio):
    h = handle()
    scores = inputs.token_scores(M, seed=M)
    if M > 100:
        scores[::3] = scores[1]           # many equal scores around the cut
    n_keep = int(math.ceil(ratio * M))
    idx = h.aq_token_select(dev(scores), n_keep).cpu().numpy()
    ref = oracle.token_select(scores, n_keep)
    assert np.array_equal(idx, ref)
    if n_keep:
        x = inputs.activations(M, 128, seed=M + 1)
        xp = h.aq_token_compact(dev(x), dev(ref)).cpu().numpy()
        assert np.array_equal(xp.view(np.uint16), oracle.token_compact(x, ref).view(np.uint16))


@pytest.mark.parametrize("M", [64, 5000, 9001])
def test_token_select_on_signed_scores_zeros_and_infinities(M):
    """Scores of both signs with -0 and +0 (equal in a float comparison, so they tie by index), infinities,
    subnormals and long runs of equal values; every n_keep that cuts inside a run of ties."""
    h = handle()
    rng = np.random.default_rng(M)
    scores = rng.standard_normal(M).astype(np.float32)
    scores[rng.integers(0, M, M // 4)] = 0.0
    scores[rng.integers(0, M, M // 4)] = -0.0
    scores[rng.integers(0, M, M // 8)] = np.float32(1e-42)
    scores[rng.integers(0, M, M // 8)] = np.float32(-1e-42)
    scores[rng.integers(0, M, 3)] = np.inf
    scores[rng.integers(0, M, 3)] = -np.inf
    scores[rng.integers(0, M, M // 8)] = scores[0]
    sd = dev(scores)
    n_zero_or_more = int((scores >= 0).sum())
    for n_keep in sorted({1, 2, 3, M // 2, n_zero_or_more - 1, n_zero_or_more, int((scores > 0).sum()) + 1, M - 1, M}):
        if 0 < n_keep <= M:
            idx = h.aq_token_select(sd, n_keep).cpu().numpy()
            assert np.array_equal(idx, oracle.token_select(scores, n_keep)), n_keep


# ------------------------------------------------------------------------ device status
def test_a_status_word_left_in_the_control_block_is_reported():
    """Every wait inside the kernels is bounded; a wait that gives up leaves a non-zero status word in the
    workspace's control block, which aq_check_workspace turns into AQ_ERR_DEVICE_TIMEOUT. No kernel is made
    to wait here: the word is written from the host side, as a kernel would have left it."""
    h = handle()
    M, K, N = 4, 256, 128
    ws = h.alloc_workspace(M, K, N, 0)
    ws.zero_()
    assert h.aq_check_workspace(ws) == binding.AQ_OK
    status = ws[8:12].view(torch.int32)              # Control::status
    for code in (1, 7, 10):
        status.fill_(code)
        assert h.aq_check_workspace(ws) == binding.AQ_ERR_DEVICE_TIMEOUT
        assert "bounded wait" in binding.status_string(binding.AQ_ERR_DEVICE_TIMEOUT)
    status.fill_(11)                                  # the attention kernel's "negative code" report
    assert h.aq_check_workspace(ws) == binding.AQ_ERR_INVALID_ARG
    # the next call on the workspace starts from a clean record
    x = dev(inputs.activations(M, K, seed=1))
    packed, scales = h.aq_pack_w4(dev(inputs.weights(N, K, seed=2)), 0)
    for kernel in (DECODE, TENSOR):
        status.fill_(5)
        h.aq_set_kernel(kernel)
        try:
            h.aq_linear_w4a8(x, packed, scales, N, 0, workspace=ws)
            assert h.aq_check_workspace(ws) == binding.AQ_OK
        finally:
            h.aq_set_kernel(binding.AQ_KERNEL_AUTO)


# --------------------------------------------------------------------- argument checking
def test_bad_arguments_are_refused():
    h = handle()
    x = torch.zeros((4, 256), dtype=torch.float16, device="cuda")
    w = torch.zeros((128, 256), dtype=torch.float16, device="cuda")
    packed, scales = h.aq_pack_w4(w, 0)
    with pytest.raises(binding.AgileqError) as ei:
        h.aq_linear_w4a8(x, packed, scales, 128, 64)
    assert ei.value.status == binding.AQ_ERR_SHAPE
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.AgileqError) as ei:
        h.aq_linear_w4a8(x, packed, scales, 128, 0, workspace=small)
    assert ei.value.status == binding.AQ_ERR_WORKSPACE
    ws = torch.empty(h.alloc_workspace(4, 256, 128, 0).numel() + 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.AgileqError) as ei:
        h.aq_linear_w4a8(x, packed, scales, 128, 0, workspace=ws[1:])
    assert ei.value.status == binding.AQ_ERR_ALIGNMENT
    with pytest.raises(binding.AgileqError) as ei:
        h.aq_quantize_act(x, 5)
    assert ei.value.status == binding.AQ_ERR_INVALID_ARG
    with pytest.raises(binding.AgileqError) as ei:
        h.aq_token_select(torch.zeros(8, device="cuda"), 9)
    assert ei.value.status == binding.AQ_ERR_SHAPE
