"""aq_linear_w4a8_noalloc: the layer for callers that cannot allocate device memory (code
living inside a memory pool that owns the whole GPU, hosts that forbid cudaMalloc once they
are serving, real-time loops). Its scratch is a fixed buffer inside the library, shared by
all calls and never cleared between them, so the check is: two calls in a row, on different
inputs and shapes, each give what aq_linear_w4a8 gives with a workspace of its own.

This file is named to be collected last: a run that stops at the first failure has then
already run every other test."""
import numpy as np
import pytest
import torch

from paper_2312_05693_b200 import binding, inputs
from gpu_util import assert_y_close, dev, handle

pytestmark = pytest.mark.gpu


def _both(h, M, K, N, group, seed):
    x = dev(inputs.activations(M, K, seed=seed, outlier_frac=0.01, outlier_mult=20.0))
    w = dev(inputs.weights(N, K, seed=seed + 1))
    packed, scales = h.aq_pack_w4(w, group)
    y_ref = h.aq_linear_w4a8(x, packed, scales, N, group)
    y = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    h.aq_linear_w4a8_noalloc(x, packed, scales, N, group, y)
    torch.cuda.synchronize()
    return y.cpu().numpy(), y_ref.cpu().numpy()


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    h = handle()
    # second call is smaller and differently shaped: stale contents of the shared buffer
    # (codes and control block of the first call) must not leak into it
    for (M, K, N, group, seed) in [(300, 1024, 384, 128, 40), (9, 512, 200, 0, 41), (300, 1024, 384, 128, 42)]:
        y, y_ref = _both(h, M, K, N, group, seed)
        assert np.all(np.isfinite(y))
        assert_y_close(y, y_ref)
        assert np.array_equal(y.view(np.uint16), y_ref.view(np.uint16))


def test_sizes_beyond_the_built_in_buffer_are_refused():
    h = handle()
    M, K, N = 4200, 4096, 128                      # M*K = 17.2 M codes, over the 16 Mi limit
    assert binding.aq_workspace_bytes(M, K, N, 0) > binding.AQ_NOALLOC_SCRATCH_BYTES
    x = torch.zeros((M, K), dtype=torch.float16, device="cuda")
    w = torch.zeros((N, K), dtype=torch.float16, device="cuda")
    packed, scales = h.aq_pack_w4(w, 0)
    y = torch.zeros((M, N), dtype=torch.float16, device="cuda")
    with pytest.raises(binding.AgileqError) as ei:
        h.aq_linear_w4a8_noalloc(x, packed, scales, N, 0, y)
    assert ei.value.status == binding.AQ_ERR_TOO_LARGE
    assert "built-in" in binding.status_string(binding.AQ_ERR_TOO_LARGE)
