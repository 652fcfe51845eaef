"""Seeded synthetic inputs for the quantized linear layer.

This module only draws random tensors. It holds none of the method's arithmetic
(no quantizer, no scale, no matmul) so that the CUDA path and the CPU checker can
both be fed from it without sharing any computation.

Recipe (shapes follow LLaMA / OPT layers; structure follows the paper's finding in
Sec. 3.2 / Fig. 1 that activation outliers sit in a few fixed channels across
tokens):

* activations  X[M, K] ~ N(0, 1) drawn in fp32, a seeded choice of
  ceil(outlier_frac * K) channels multiplied by ``outlier_mult``, rounded to fp16;
* weights      W[N, K] ~ N(0, 0.02) drawn in fp32, rounded to fp16;
* token scores s[M]    ~ Uniform(0, 1) in fp32.

Every tensor gets its own Philox stream keyed by (seed, tensor tag), so a tensor
does not change when another one is added to a configuration.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np

_TAGS = {"x": 1, "w": 2, "scores": 3, "outlier_channels": 4, "rows": 5, "cols": 6}


def _rng(seed: int, tag: str, sub: int = 0) -> np.random.Generator:
    key = (int(seed) & 0xFFFFFFFF) | (_TAGS[tag] << 32) | ((int(sub) & 0xFFFFFF) << 40)
    return np.random.Generator(np.random.Philox(key=key))


def outlier_channels(K: int, frac: float, seed: int) -> np.ndarray:
    """Sorted indices of the ceil(frac*K) channels that carry outliers."""
    n = int(math.ceil(frac * K)) if frac > 0 else 0
    if n == 0:
        return np.zeros((0,), dtype=np.int64)
    return np.sort(_rng(seed, "outlier_channels").choice(K, size=n, replace=False))


def activations(M: int, K: int, seed: int, outlier_frac: float = 0.0,
                outlier_mult: float = 1.0, sub: int = 0) -> np.ndarray:
    """fp16 [M, K]; N(0,1) body, fixed outlier channels scaled by outlier_mult."""
    g = _rng(seed, "x", sub)
    x = g.standard_normal(size=(M, K), dtype=np.float32)
    ch = outlier_channels(K, outlier_frac, seed)
    if ch.size:
        x[:, ch] *= np.float32(outlier_mult)
    return x.astype(np.float16)


def weights(N: int, K: int, seed: int, std: float = 0.02, sub: int = 0) -> np.ndarray:
    """fp16 [N, K] ~ N(0, std)."""
    g = _rng(seed, "w", sub)
    out = np.empty((N, K), dtype=np.float16)
    step = max(1, (1 << 24) // max(K, 1))          # bound the fp32 temporary
    for n0 in range(0, N, step):
        n1 = min(N, n0 + step)
        blk = g.standard_normal(size=(n1 - n0, K), dtype=np.float32)
        blk *= np.float32(std)
        out[n0:n1] = blk.astype(np.float16)
    return out


def token_scores(M: int, seed: int) -> np.ndarray:
    """fp32 [M] ~ U(0,1): stands in for the attention paid to the start token."""
    return _rng(seed, "scores").random(size=(M,), dtype=np.float32)


def sample_coords(M: int, N: int, count: int, seed: int) -> Tuple[np.ndarray, np.ndarray]:
    """Seeded (row, col) pairs used to spot-check full-size outputs."""
    r = _rng(seed, "rows").integers(0, M, size=count, dtype=np.int64)
    c = _rng(seed, "cols").integers(0, N, size=count, dtype=np.int64)
    # always include the corners and the last (possibly ragged) tile
    r[:4] = [0, 0, M - 1, M - 1]
    c[:4] = [0, N - 1, 0, N - 1]
    return r.astype(np.int32), c.astype(np.int32)


@dataclass(frozen=True)
class LayerShape:
    K: int
    N: int


@dataclass(frozen=True)
class Workload:
    """One of the benchmark configurations."""
    name: str
    seed: int
    Ms: Tuple[int, ...]
    shapes: Tuple[LayerShape, ...]
    act_bits: int
    group_size: int            # 0 = one scale per output channel, 128 = per 128-K group
    clip_shift: int
    outlier_frac: float
    outlier_mult: float
    keep_ratio: float = 1.0    # < 1: tokens are pruned before the layer
    note: str = ""

    def n_keep(self, M: int) -> int:
        return M if self.keep_ratio >= 1.0 else int(math.ceil(self.keep_ratio * M))


WORKLOADS = {
    "opt125m_w4a8": Workload(
        "opt125m_w4a8", 0, (16,), (LayerShape(768, 768),), 8, 0, 0, 0.01, 20.0,
        note="single OPT-125M-like layer, per-output-channel weight scales"),
    "llama7b_prefill_w4a8": Workload(
        "llama7b_prefill_w4a8", 1, (2048,),
        (LayerShape(4096, 4096), LayerShape(4096, 11008), LayerShape(11008, 4096)),
        8, 128, 0, 0.005, 30.0,
        note="LLaMA-7B attention projection, MLP up/gate, MLP down; group-128 scales"),
    "llama7b_prefill_w4a4": Workload(
        "llama7b_prefill_w4a4", 2, (2048,),
        (LayerShape(4096, 4096), LayerShape(4096, 11008), LayerShape(11008, 4096)),
        4, 128, 4, 0.005, 30.0,
        note="same shapes, int4 activations; clip_shift lets outlier channels saturate"),
    "llama13b_decode_w4a8": Workload(
        "llama13b_decode_w4a8", 3, (1, 4, 16),
        (LayerShape(5120, 5120), LayerShape(5120, 13824), LayerShape(13824, 5120)),
        8, 0, 0, 0.005, 30.0,
        note="memory-bound decode, per-output-channel scales"),
    "opt30b_pruned_prefill_w4a8": Workload(
        "opt30b_pruned_prefill_w4a8", 4, (4096,),
        (LayerShape(7168, 7168), LayerShape(7168, 28672)),
        8, 0, 0, 0.01, 25.0, keep_ratio=0.6,
        note="keep the top 60% tokens by score, then W4A8"),
}
