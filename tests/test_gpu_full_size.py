"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (kernel
choice left to the library). Everything that is cheap on the CPU is compared in full (weight
codes and scales, the layer exponent, activation codes, decode outputs); the int32 sums
of the prefill products are compared on seeded sample positions that always include the corners and
the ragged last tile; the fp16 outputs of the LLaMA-7B prefill shapes are compared in full against
the CPU layer, those of the largest (token-pruned) shapes on the sample positions."""
import numpy as np
import pytest
import torch

import oracle
from paper_2312_05693_b200 import binding, inputs
from gpu_util import assert_y_close, dev, handle, scales_to_oracle_layout

pytestmark = pytest.mark.gpu

N_SAMPLES = 3000


def _check_prefill_shape(wl, M_in, shape, sub, row_idx=None, full_y=False):
    h = handle()
    K, N, group, bits = shape.K, shape.N, wl.group_size, wl.act_bits
    x = inputs.activations(M_in, K, wl.seed, wl.outlier_frac, wl.outlier_mult, sub=sub)
    w = inputs.weights(N, K, wl.seed, sub=sub)
    M = M_in if row_idx is None else len(row_idx)
    G = K // 128 if group else 1
    # weights: full comparison of codes and scale bit patterns
    packed, scales = h.aq_pack_w4(dev(w), group)
    codes, sc = oracle.quantize_weights(w, group)
    assert np.array_equal(h.aq_unpack_w4(packed, N, K).cpu().numpy(), codes)
    assert np.array_equal(scales_to_oracle_layout(scales, N).view(np.uint16), sc.view(np.uint16))
    # the layer, once with the integer sums dumped and once exactly as the benchmark calls it
    fn = h.aq_linear_w4a8 if bits == 8 else h.aq_linear_w4a4
    xd = dev(x)
    ri = None if row_idx is None else dev(row_idx)
    ws = h.alloc_workspace(M, K, N, group)
    acc = torch.empty((M, N, G), dtype=torch.int32, device="cuda")
    y_dump = fn(xd, packed, scales, N, group, binding.AQ_SCALE_DYNAMIC, wl.clip_shift, row_idx=ri,
                acc_dump=acc, workspace=ws)
    y = fn(xd, packed, scales, N, group, binding.AQ_SCALE_DYNAMIC, wl.clip_shift, row_idx=ri, workspace=ws)
    assert h.aq_check_workspace(ws) == binding.AQ_OK
    assert torch.equal(y, y_dump)
    assert torch.isfinite(y).all().item()
    # exponent and activation codes: full comparison
    e_ref = oracle.layer_exponent(x, bits, row_idx) - wl.clip_shift
    q_ref = oracle.quantize_act(x, bits, e_ref, row_idx)
    assert int(ws[4:8].view(torch.int32).item()) == e_ref
    assert np.array_equal(ws[256:256 + M * K].view(torch.int8).reshape(M, K).cpu().numpy(), q_ref)
    # sampled outputs
    rows, cols = inputs.sample_coords(M, N, N_SAMPLES, wl.seed + sub)
    rows[4:8] = [M - 1, M - 2, 0, M - 1]                   # last (ragged) token tile x last channel tile
    cols[4:8] = [N - 1, N - 2, N - 129, N - 129]
    acc_ref, y_ref = oracle.linear_sampled(q_ref, codes, sc, e_ref, group, rows, cols)
    rt, ct = torch.from_numpy(rows.astype(np.int64)).cuda(), torch.from_numpy(cols.astype(np.int64)).cuda()
    assert np.array_equal(acc[rt, ct].cpu().numpy(), acc_ref)
    y_s = y[rt, ct].cpu().numpy()
    scale = float(np.abs(y_ref.astype(np.float64)).max())
    assert np.abs(y_s.astype(np.float64) - y_ref.astype(np.float64)).max() <= 1e-3 * scale
    del acc
    if full_y:
        # every output element against the whole layer on the CPU (a few seconds per shape on the machine's cores):
        # covers the interior of every tile, every shared tile and the ragged last token tile
        ref = oracle.linear(x, codes, sc, bits, group, binding.AQ_SCALE_DYNAMIC, wl.clip_shift, row_idx=row_idx)
        assert ref["e"] == e_ref
        assert_y_close(y.cpu().numpy(), ref["y"])


@pytest.mark.parametrize("name", ["llama7b_prefill_w4a8", "llama7b_prefill_w4a4"])
def test_llama7b_prefill_full_size(name):
    wl = inputs.WORKLOADS[name]
    for sub, shape in enumerate(wl.shapes):
        _check_prefill_shape(wl, wl.Ms[0], shape, sub, full_y=True)


def test_opt125m_single_layer_full():
    wl = inputs.WORKLOADS["opt125m_w4a8"]
    h = handle()
    s = wl.shapes[0]
    M = wl.Ms[0]
    x = inputs.activations(M, s.K, wl.seed, wl.outlier_frac, wl.outlier_mult)
    w = inputs.weights(s.N, s.K, wl.seed)
    packed, scales = h.aq_pack_w4(dev(w), 0)
    acc = torch.empty((M, s.N, 1), dtype=torch.int32, device="cuda")
    y = h.aq_linear_w4a8(dev(x), packed, scales, s.N, 0, acc_dump=acc)
    codes, sc = oracle.quantize_weights(w, 0)
    ref = oracle.linear(x, codes, sc, 8, 0, want_acc=True)
    assert np.array_equal(acc.cpu().numpy(), ref["acc"])
    assert_y_close(y.cpu().numpy(), ref["y"])


def test_llama13b_decode_full():
    wl = inputs.WORKLOADS["llama13b_decode_w4a8"]
    h = handle()
    for sub, s in enumerate(wl.shapes):
        w = inputs.weights(s.N, s.K, wl.seed, sub=sub)
        packed, scales = h.aq_pack_w4(dev(w), 0)
        codes, sc = oracle.quantize_weights(w, 0)
        assert np.array_equal(h.aq_unpack_w4(packed, s.N, s.K).cpu().numpy(), codes)
        for M in wl.Ms:
            x = inputs.activations(M, s.K, wl.seed, wl.outlier_frac, wl.outlier_mult, sub=sub)
            acc = torch.empty((M, s.N, 1), dtype=torch.int32, device="cuda")
            y_dump = h.aq_linear_w4a8(dev(x), packed, scales, s.N, 0, acc_dump=acc)
            y = h.aq_linear_w4a8(dev(x), packed, scales, s.N, 0)
            ref = oracle.linear(x, codes, sc, 8, 0, want_acc=True)
            assert np.array_equal(acc.cpu().numpy(), ref["acc"])
            assert torch.equal(y, y_dump)
            assert_y_close(y.cpu().numpy(), ref["y"])


def test_opt30b_pruned_prefill_full_size():
    wl = inputs.WORKLOADS["opt30b_pruned_prefill_w4a8"]
    h = handle()
    M_in = wl.Ms[0]
    n_keep = wl.n_keep(M_in)
    assert n_keep == 2458
    scores = inputs.token_scores(M_in, wl.seed)
    idx = h.aq_token_select(dev(scores), n_keep).cpu().numpy()
    assert np.array_equal(idx, oracle.token_select(scores, n_keep))
    for sub, shape in enumerate(wl.shapes):
        _check_prefill_shape(wl, M_in, shape, sub, row_idx=idx)
    # gather + plain layer gives the same bits as the fused row_idx path
    s = wl.shapes[0]
    x = inputs.activations(M_in, s.K, wl.seed, wl.outlier_frac, wl.outlier_mult, sub=0)
    w = inputs.weights(s.N, s.K, wl.seed, sub=0)
    packed, scales = h.aq_pack_w4(dev(w), 0)
    xd, idxd = dev(x), dev(idx)
    xp = h.aq_token_compact(xd, idxd)
    assert np.array_equal(xp.cpu().numpy().view(np.uint16), x[idx].view(np.uint16))
    y_fused = h.aq_linear_w4a8(xd, packed, scales, s.N, 0, row_idx=idxd)
    y_plain = h.aq_linear_w4a8(xp, packed, scales, s.N, 0)
    assert torch.equal(y_fused, y_plain)


def test_widened_entry_points_at_a_benchmark_shape():
    """TRIP factors, the zero-point variant and the chained call on the LLaMA-7B (4096 -> 11008) layer at
    M = 2048, through the tensor kernel as the benchmark runs them: codes and exponents in full, integer
    sums and outputs on sampled positions."""
    wl = inputs.WORKLOADS["llama7b_prefill_w4a4"]
    h = handle()
    M, shape, group = wl.Ms[0], wl.shapes[1], wl.group_size
    K, N, G = shape.K, shape.N, shape.K // 128
    x = inputs.activations(M, K, wl.seed, wl.outlier_frac, wl.outlier_mult, sub=1)
    w = inputs.weights(N, K, wl.seed, sub=1)
    xd = dev(x)
    packed, scales = h.aq_pack_w4(dev(w), group)
    codes, sc = oracle.quantize_weights(w, group)
    rows, cols = inputs.sample_coords(M, N, N_SAMPLES, 77)
    rt, ct = torch.from_numpy(rows.astype(np.int64)).cuda(), torch.from_numpy(cols.astype(np.int64)).cuda()
    ws = h.alloc_workspace(M, K, N, group)
    acc = torch.empty((M, N, G), dtype=torch.int32, device="cuda")

    def close(y_s, y_ref):
        scale = float(np.abs(y_ref.astype(np.float64)).max())
        assert np.abs(y_s.astype(np.float64) - y_ref.astype(np.float64)).max() <= 1e-3 * scale

    # ---- TRIP factors (Eq. 5-8), 4-bit codes, k_max = 4
    k_max = 4
    alpha_t, e_t = h.aq_trip_calibrate(xd, k_max)
    e_ref = oracle.trip_base_exponent(x, 4, k_max)
    alpha = oracle.trip_calibrate(x, 4, e_ref, k_max)
    assert int(e_t.item()) == e_ref and np.array_equal(alpha_t.cpu().numpy(), alpha)
    y = h.aq_linear_w4a4_trip(xd, packed, scales, N, group, alpha_t, k_max, acc_dump=acc, workspace=ws)
    assert h.aq_check_workspace(ws) == binding.AQ_OK
    v_ref = oracle.quantize_act_trip(x, 4, e_ref, alpha)
    assert np.array_equal(ws[256:256 + M * K].view(torch.int8).reshape(M, K).cpu().numpy(), v_ref)
    acc_ref, y_ref = oracle.linear_sampled(v_ref, codes, sc, e_ref, group, rows, cols)
    assert np.array_equal(acc[rt, ct].cpu().numpy(), acc_ref)
    close(y[rt, ct].cpu().numpy(), y_ref)

    # ---- zero point (Eq. 2, Eq. 5-7), 8-bit codes, on shifted activations
    xs = (x.astype(np.float32) + np.float32(2.0)).astype(np.float16)
    r = h.aq_weight_offsets(packed, scales, N, K, group)
    y = h.aq_linear_asym(8, dev(xs), packed, scales, r, N, group, acc_dump=acc, workspace=ws)
    assert h.aq_check_workspace(ws) == binding.AQ_OK
    e_a, zp = oracle.asym_params(xs, 8)
    q_u = oracle.quantize_act_asym(xs, 8, e_a, zp)
    q_s = (q_u.astype(np.int16) - 128).astype(np.int8)
    assert np.array_equal(ws[256:256 + M * K].view(torch.int8).reshape(M, K).cpu().numpy(), q_s)
    acc_raw, _ = oracle.linear_sampled(q_s, codes, sc, e_a, group, rows, cols)
    assert np.array_equal(acc[rt, ct].cpu().numpy(), acc_raw)
    colsum = codes.astype(np.int64).reshape(N, G, 128).sum(axis=2)
    true_acc = acc_raw.astype(np.int64) - (zp - 128) * colsum[cols]
    y_ref = ((true_acc.astype(np.float64) * sc.astype(np.float64)[cols]).sum(axis=1) * 2.0 ** e_a).astype(np.float16)
    close(y[rt, ct].cpu().numpy(), y_ref)

    # ---- chained call: the next layer's codes equal the quantizer applied to the plain call's fp16 output
    y_plain = h.aq_linear_w4a8(xd, packed, scales, N, group, workspace=ws)
    e_next = oracle.layer_exponent(y_plain[rt, ct].cpu().numpy().reshape(1, -1)[:, :N_SAMPLES // 128 * 128], 8)
    q_next = h.aq_linear_chain(8, xd, packed, scales, N, group, 8, e_next, workspace=ws)
    ref = oracle.quantize_act(y_plain.cpu().numpy(), 8, e_next)
    assert np.array_equal(q_next.cpu().numpy(), ref)
    del acc
