"""The C-ABI library builds, loads and exports every function the header declares.
No kernel runs here (no GPU needed)."""
import ctypes as C

import pytest

from paper_2312_05693_b200 import binding, build


def test_build_and_exports():
    path = build.build()
    lib = C.CDLL(path)
    names = binding.declared_symbols()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), n


def test_size_functions_and_status_strings():
    L = binding.load()
    assert L.aq_version() >= 100
    assert binding.aq_packed_w4_bytes(768, 768) == 768 * 768 // 2
    assert binding.aq_packed_w4_bytes(200, 256) == 256 * 256 // 2          # rows padded to 128
    assert binding.aq_packed_w4_bytes(128, 100) == 0                        # K must be a multiple of 128
    assert binding.aq_scales_bytes(768, 768, 0) == 768 * 2
    assert binding.aq_scales_bytes(200, 512, 128) == 4 * 256 * 2
    assert binding.aq_scales_bytes(200, 512, 64) == 0
    ws = binding.aq_workspace_bytes(16, 768, 768, 0)
    assert ws % 256 == 0 and ws >= 256 + 16 * 768
    assert binding.aq_workspace_bytes(0, 768, 768, 0) == 0
    assert L.aq_act4_bytes(16, 768) == 16 * 768 // 2 and L.aq_act4_bytes(16, 48) == 0   # K % 32 == 0
    assert binding.aq_workspace_bytes(16, 768 + 64, 768, 0) == 0
    assert binding.aq_linear_host_scratch_bytes(16, 768, 768, 0) >= ws + 16 * 768 * 2 * 2
    seen = {binding.status_string(s) for s in range(0, -8, -1)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert binding.status_string(-99) == "unknown status"


def test_null_handle_is_rejected_without_touching_a_device():
    L = binding.load()
    assert L.aq_set_kernel(None, 0) == binding.AQ_ERR_INVALID_ARG
    assert L.aq_pack_w4(None, None, 128, 128, 0, None, None, None) == binding.AQ_ERR_INVALID_ARG
    assert L.aq_create(None, 0) == binding.AQ_ERR_INVALID_ARG


def test_prune_schedule_host_function():
    # Eq. 9 (host only: runs without a GPU). After m layers about (1 - beta) of the tokens are left.
    import oracle
    keep, gamma = binding.aq_prune_schedule(4096, 0.4, 4)
    assert abs(gamma - oracle.progressive_ratio(0.4, 4)) < 1e-15
    assert len(keep) == 4 and all(a >= b for a, b in zip([4096] + keep, keep))
    assert abs(keep[-1] - 4096 * 0.6) <= 4                     # ceil at every layer adds at most one token each
    assert binding.aq_prune_schedule(4096, 0.75, 2)[0] == [2048, 1024]       # gamma = 1/2 exactly
    assert binding.aq_prune_schedule(100, 0.0, 3)[0] == [100, 100, 100]
    assert binding.aq_prune_schedule(3, 0.99, 5)[0][-1] >= 1
    for bad in [(0, 0.5, 2), (10, 1.0, 2), (10, -0.1, 2), (10, 0.5, 0)]:
        with pytest.raises(binding.AgileqError):
            binding.aq_prune_schedule(*bad)
