"""aq_linear_w4a8_noalloc: the layer for callers that cannot allocate device memory (code
living inside a memory pool that owns the whole GPU, hosts that forbid cudaMalloc once they
are serving, real-time loops). Its scratch is a fixed buffer inside the library, shared by
all calls and never cleared between them, so the check is: two calls in a row, on different
inputs and shapes, each give what aq_linear_w4a8 gives with a workspace of its own and what
the CPU checker gives, and the amount of free device memory does not move across a call.

This file is named to be collected last: a run that stops at the first failure has then
already run every other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2312_05693_b200 import binding, inputs
from gpu_util import assert_y_close, dev, handle

pytestmark = pytest.mark.gpu


def _both(h, M, K, N, group, seed, check_memory=False):
    x_np = inputs.activations(M, K, seed=seed, outlier_frac=0.01, outlier_mult=20.0)
    w_np = inputs.weights(N, K, seed=seed + 1)
    x, w = dev(x_np), dev(w_np)
    packed, scales = h.aq_pack_w4(w, group)
    y_ref = h.aq_linear_w4a8(x, packed, scales, N, group)
    y = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    if check_memory:
        # a first call has done the one-time set-up; from here on the call must leave the device's free
        # memory exactly as it found it (the output tensor above is the caller's)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
    h.aq_linear_w4a8_noalloc(x, packed, scales, N, group, y)
    assert h.aq_check_noalloc() == binding.AQ_OK           # synchronizes; no bounded wait gave up
    if check_memory:
        assert torch.cuda.mem_get_info()[0] == free_before
    codes, sc = oracle.quantize_weights(w_np, group)
    y_cpu = oracle.linear(x_np, codes, sc, 8, group, 0, 0)["y"]
    return y.cpu().numpy(), y_ref.cpu().numpy(), y_cpu


def test_two_calls_in_a_row_match_the_workspace_entry_point_and_the_checker():
    h = handle()
    # second call is smaller and differently shaped: stale contents of the shared buffer
    # (codes and control block of the first call) must not leak into it
    for i, (M, K, N, group, seed) in enumerate([(300, 1024, 384, 128, 40), (9, 512, 200, 0, 41),
                                                (300, 1024, 384, 128, 42)]):
        y, y_ref, y_cpu = _both(h, M, K, N, group, seed, check_memory=i > 0)
        assert np.all(np.isfinite(y))
        assert_y_close(y, y_cpu)
        assert_y_close(y, y_ref)
        assert np.array_equal(y.view(np.uint16), y_ref.view(np.uint16))


def test_a_prefill_shape_with_per_group_scales_fits_and_matches_the_checker():
    """M = 2048, K = N = 4096 with group-128 scales: 8 Mi codes. The workspace entry point would also
    like room for the partial sums of shared tiles; the built-in buffer serves what it has left for that
    (or none), which may move an output by the last fp32 rounding but never beyond the layer's tolerance."""
    h = handle()
    M, K, N, group = 2048, 4096, 4096, 128
    assert binding.aq_workspace_min_bytes(M, K, N, group) <= binding.AQ_NOALLOC_SCRATCH_BYTES
    rows = 96                                           # the checker runs on a slice of the tokens
    x_np = inputs.activations(M, K, seed=50, outlier_frac=0.005, outlier_mult=30.0)
    w_np = inputs.weights(N, K, seed=51)
    x = dev(x_np)
    packed, scales = h.aq_pack_w4(dev(w_np), group)
    y = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    codes, sc = oracle.quantize_weights(w_np, group)
    e = oracle.layer_exponent(x_np, 8)
    sel = np.r_[0:rows // 2, M - rows // 2:M]
    ref = oracle.linear(x_np[sel], codes, sc, 8, group, 1, e)["y"]          # same exponent as the whole layer
    for _ in range(2):
        y.fill_(float("nan"))
        h.aq_linear_w4a8_noalloc(x, packed, scales, N, group, y)
        assert h.aq_check_noalloc() == binding.AQ_OK
        y_ref = h.aq_linear_w4a8(x, packed, scales, N, group)
        yn, yr = y.cpu().numpy(), y_ref.cpu().numpy()
        assert np.all(np.isfinite(yn))
        assert_y_close(yn, yr)
        a, b = yn[sel].astype(np.float64), ref.astype(np.float64)
        assert np.abs(a - b).max() <= 1e-3 * np.abs(yr.astype(np.float64)).max()


def test_sizes_beyond_the_built_in_buffer_are_refused():
    h = handle()
    M, K, N = 4200, 4096, 128                      # M*K = 17.2 M codes, over the 16 Mi limit
    assert binding.aq_workspace_min_bytes(M, K, N, 0) > binding.AQ_NOALLOC_SCRATCH_BYTES
    x = torch.zeros((M, K), dtype=torch.float16, device="cuda")
    w = torch.zeros((N, K), dtype=torch.float16, device="cuda")
    packed, scales = h.aq_pack_w4(w, 0)
    y = torch.zeros((M, N), dtype=torch.float16, device="cuda")
    with pytest.raises(binding.AgileqError) as ei:
        h.aq_linear_w4a8_noalloc(x, packed, scales, N, 0, y)
    assert ei.value.status == binding.AQ_ERR_TOO_LARGE
    assert "built-in" in binding.status_string(binding.AQ_ERR_TOO_LARGE)
