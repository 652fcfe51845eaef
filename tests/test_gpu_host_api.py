"""The host-buffer entry points (copy in, layer, copy out) and the layer calls under CUDA graph
capture: same results as the device-buffer calls and as the CPU checker."""
import numpy as np
import pytest
import torch

import oracle
from paper_2312_05693_b200 import binding, inputs
from gpu_util import assert_y_close, dev, handle

pytestmark = pytest.mark.gpu


def _reference(x, w, group, bits, clip):
    c, sc = oracle.quantize_weights(w, group)
    e = oracle.layer_exponent(x, bits) - clip
    q = oracle.quantize_act(x, bits, e)
    M, K = x.shape
    acc = oracle.int_gemm(q, c, group)
    return oracle.dequant(acc.reshape(M, w.shape[0], K // 128 if group else 1), sc, e)


@pytest.mark.parametrize("bits,clip", [(8, 0), (4, 2)])
@pytest.mark.parametrize("M,K,N,group", [(1, 256, 384, 0), (16, 768, 768, 0), (300, 1024, 520, 128)])
def test_host_call_matches_checker(bits, clip, M, K, N, group):
    x = inputs.activations(M, K, seed=71, outlier_frac=0.01, outlier_mult=20.0)
    w = inputs.weights(N, K, 71)
    h = handle()
    packed, scales = h.aq_pack_w4(dev(w), group)
    x_host = torch.from_numpy(x).pin_memory()
    y_host = torch.empty((M, N), dtype=torch.float16).pin_memory()
    scratch = torch.empty(binding.aq_linear_host_scratch_bytes(M, K, N, group), dtype=torch.uint8, device="cuda")
    h.aq_linear_host(bits, x_host, packed, scales, N, group, y_host, scratch, clip_shift_or_exp=clip)
    assert_y_close(y_host.numpy(), _reference(x, w, group, bits, clip))


def test_asynchronous_host_calls_on_two_streams():
    shapes = [(300, 1024, 520, 128, 72), (129, 768, 384, 0, 73)]
    h = handle()
    jobs = []
    for M, K, N, group, seed in shapes:
        x = inputs.activations(M, K, seed=seed, outlier_frac=0.01, outlier_mult=20.0)
        w = inputs.weights(N, K, seed)
        packed, scales = h.aq_pack_w4(dev(w), group)
        jobs.append(dict(x=x, w=w, group=group, N=N, packed=packed, scales=scales,
                         x_host=torch.from_numpy(x).pin_memory(),
                         y_host=torch.zeros((M, N), dtype=torch.float16).pin_memory(),
                         scratch=torch.empty(binding.aq_linear_host_scratch_bytes(M, K, N, group), dtype=torch.uint8,
                                             device="cuda"),
                         stream=torch.cuda.Stream()))
    torch.cuda.synchronize()
    for _ in range(3):                                        # the same buffers again behind the first use
        for j in jobs:
            with torch.cuda.stream(j["stream"]):
                h.aq_linear_host_async(8, j["x_host"], j["packed"], j["scales"], j["N"], j["group"], j["y_host"],
                                       j["scratch"])
    for j in jobs:
        j["stream"].synchronize()
        assert_y_close(j["y_host"].numpy(), _reference(j["x"], j["w"], j["group"], 8, 0))


@pytest.mark.parametrize("M,K,N,group", [(1, 1024, 640, 0), (4, 768, 768, 0), (16, 512, 384, 128), (300, 1024, 520, 128)])
def test_layer_call_replayed_from_a_cuda_graph(M, K, N, group):
    # the product launch overlaps the call's own quantize kernel; captured and replayed it must give the same result
    x = inputs.activations(M, K, seed=74, outlier_frac=0.01, outlier_mult=20.0)
    w = inputs.weights(N, K, 74)
    h = handle()
    packed, scales = h.aq_pack_w4(dev(w), group)
    xd = dev(x)
    ws = h.alloc_workspace(M, K, N, group)
    y = torch.empty((M, N), dtype=torch.float16, device="cuda")
    h.aq_linear_w4a8(xd, packed, scales, N, group, y=y, workspace=ws)
    torch.cuda.synchronize()
    eager = y.clone()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        h.aq_linear_w4a8(xd, packed, scales, N, group, y=y, workspace=ws)
        h.aq_linear_w4a8(xd, packed, scales, N, group, y=y, workspace=ws)
    for _ in range(3):
        y.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(y, eager)
    assert h.aq_check_workspace(ws) == binding.AQ_OK
    assert_y_close(eager.cpu().numpy(), _reference(x, w, group, 8, 0))
