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
    assert binding.aq_packed_w4_layout_version() == 2
    assert binding.aq_packed_w4_bytes(768, 768) == 768 * 768 // 2
    assert binding.aq_packed_w4_bytes(200, 256) == 256 * 256 // 2          # rows padded to 128
    assert binding.aq_packed_w4_bytes(128, 100) == 0                        # K must be a multiple of 32
    assert binding.aq_packed_w4_bytes(128, 160) == 128 * 256 // 2          # ... and is padded to 128
    assert binding.aq_scales_bytes(128, 160, 0) == 128 * 2
    assert binding.aq_scales_bytes(128, 160, 128) == 0                      # per-group scales need K % 128 == 0
    assert binding.aq_workspace_bytes(16, 160, 128, 0) >= 256 + 16 * 160
    assert binding.aq_workspace_bytes(16, 160, 128, 128) == 0
    assert binding.aq_scales_bytes(768, 768, 0) == 768 * 2
    assert binding.aq_scales_bytes(200, 512, 128) == 4 * 256 * 2
    assert binding.aq_scales_bytes(200, 512, 64) == 0
    ws = binding.aq_workspace_bytes(16, 768, 768, 0)
    assert ws % 256 == 0 and ws >= 256 + 16 * 768
    assert binding.aq_workspace_bytes(0, 768, 768, 0) == 0
    assert L.aq_act4_bytes(16, 768) == 16 * 768 // 2 and L.aq_act4_bytes(16, 48) == 0   # K % 32 == 0
    assert binding.aq_workspace_bytes(16, 768 + 16, 768, 0) == 0
    assert binding.aq_linear_host_scratch_bytes(16, 768, 768, 0) >= ws + 16 * 768 * 2 * 2
    seen = {binding.status_string(s) for s in range(0, -8, -1)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert binding.status_string(-99) == "unknown status"


def test_which_shapes_fit_the_built_in_scratch_buffer():
    # aq_linear_w4a8_noalloc accepts a shape when the part of the workspace no call can do without fits
    # its array; the optional area of the per-group kernel does not count
    cap = binding.AQ_NOALLOC_SCRATCH_BYTES

    def up(v):
        return (v + 255) // 256 * 256

    for (M, K, N, g) in [(2048, 4096, 4096, 128), (2048, 4096, 11008, 128), (2048, 8192, 4096, 128),
                         (4096, 4096, 4096, 0), (2048, 8192, 15360, 0), (16, 13824, 5120, 0)]:
        need = binding.aq_workspace_min_bytes(M, K, N, g)
        assert need == 256 + up(M * K) + up(M) + up(4 * N)
        assert need <= cap, (M, K, N, g)
        assert binding.aq_workspace_bytes(M, K, N, g) >= need
    # the LLaMA-7B down projection at 2048 tokens has 22.5 Mi codes: over the limit, as is 16 Mi codes with a
    # very wide output
    for (M, K, N, g) in [(2048, 11008, 4096, 128), (4200, 4096, 128, 0), (2048, 8192, 16384, 0)]:
        assert binding.aq_workspace_min_bytes(M, K, N, g) > cap, (M, K, N, g)
    # the per-group kernel's optional area is what separates the two size functions
    assert binding.aq_workspace_bytes(2048, 4096, 4096, 128) > binding.aq_workspace_min_bytes(2048, 4096, 4096, 128)
    assert binding.aq_workspace_bytes(2048, 4096, 4096, 0) == binding.aq_workspace_min_bytes(2048, 4096, 4096, 0)


def test_null_handle_is_rejected_without_touching_a_device():
    L = binding.load()
    assert L.aq_set_kernel(None, 0) == binding.AQ_ERR_INVALID_ARG
    assert L.aq_set_weights_stable(None, 1) == binding.AQ_ERR_INVALID_ARG
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
