"""Seeded synthetic layers shaped like the pointwise (1x1) convolutions of MobileNetV1 and
ResNet-50, pruned with the SIMD-structured block pattern (blocks of g consecutive output
channels that share one input-channel index).

The tensors stand in for the ImageNet networks the paper prunes: same layer shapes, synthetic
values.  Only inputs are produced here (weights, block masks, activations, bias); nothing in
this module multiplies or packs anything.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import List

import numpy as np

from . import rng

BASE_SEED = 2109_00170


@dataclass(frozen=True)
class LayerSpec:
    """One sparse pointwise convolution problem: Y[n,cout,h*w] = W[cout,cin] X[n,cin,h*w] + b."""
    name: str
    cin: int
    cout: int
    h: int
    w: int
    n: int = 1
    g: int = 4
    dtype: str = "f32"            # "f32": fp32 everywhere; "f16": fp16 W/X/Y, fp32 accumulate
    sparsity: float = 0.8         # fraction of blocks dropped (exact count) for mask_kind="uniform"
    mask_kind: str = "uniform"    # "uniform" | "zipf"
    x_dist: str = "uniform"       # "uniform" U[0,1) | "halfnormal" |N(0,1)|
    relu: bool = True
    bias: bool = True
    seed: int = BASE_SEED

    @property
    def hw(self) -> int:
        return self.h * self.w

    @property
    def rows(self) -> int:
        """Number of block rows R = ceil(cout / g)."""
        return (self.cout + self.g - 1) // self.g

    @property
    def np_dtype(self):
        return np.float32 if self.dtype == "f32" else np.float16


# stream ids inside one layer seed
_S_W, _S_MASK, _S_X, _S_BIAS, _S_ZIPF_N, _S_ZIPF_PERM = 1, 2, 3, 4, 5, 1000


def make_weights(spec: LayerSpec) -> np.ndarray:
    """W[cout, cin] ~ N(0, 1/cin) (variance), rounded to the layer dtype."""
    w = rng.normal(spec.seed, _S_W, spec.cout * spec.cin, sigma=spec.cin ** -0.5)
    return w.reshape(spec.cout, spec.cin).astype(spec.np_dtype)


def make_bias(spec: LayerSpec) -> np.ndarray | None:
    """bias[cout] ~ N(0, 0.01) (variance, sigma = 0.1), always fp32."""
    if not spec.bias:
        return None
    return rng.normal(spec.seed, _S_BIAS, spec.cout, sigma=0.1).astype(np.float32)


def make_x(spec: LayerSpec) -> np.ndarray:
    """X[n, cin, h*w], contiguous NCHW, U[0,1) or |N(0,1)|, rounded to the layer dtype."""
    cnt = spec.n * spec.cin * spec.hw
    if spec.x_dist == "uniform":
        x = rng.uniform01(spec.seed, _S_X, cnt)
    elif spec.x_dist == "halfnormal":
        x = np.abs(rng.normal(spec.seed, _S_X, cnt)).astype(np.float32)
    else:
        raise ValueError(spec.x_dist)
    return x.reshape(spec.n, spec.cin, spec.hw).astype(spec.np_dtype)


def uniform_block_mask(rows: int, cin: int, sparsity: float, seed: int) -> np.ndarray:
    """Exactly round(sparsity * rows * cin) blocks dropped, chosen by a seeded shuffle."""
    total = rows * cin
    drop = int(round(sparsity * total))
    drop = min(max(drop, 0), total)
    perm = rng.permutation(seed, _S_MASK, total)
    m = np.ones(total, dtype=np.uint8)
    m[perm[:drop]] = 0
    return m.reshape(rows, cin)


def zipf_block_mask(rows: int, cin: int, seed: int, a: float = 1.2) -> np.ndarray:
    """Skewed rows: the kept-block count of each block row follows a Zipf(a) law truncated
    to {1..cin} (pmf ~ k^-a, seeded inverse CDF); its columns are the first n_r entries of a
    seeded permutation of the input channels."""
    k = np.arange(1, cin + 1, dtype=np.float64)
    cdf = np.cumsum(k ** (-a))
    cdf /= cdf[-1]
    u = rng.uniform01_f64(seed, _S_ZIPF_N, rows)
    counts = np.minimum(np.searchsorted(cdf, u, side="left") + 1, cin)
    m = np.zeros((rows, cin), dtype=np.uint8)
    for r in range(rows):
        perm = rng.permutation(seed, _S_ZIPF_PERM + r, cin)
        m[r, perm[: counts[r]]] = 1
    return m


def make_mask(spec: LayerSpec) -> np.ndarray:
    """Block mask [rows, cin], 1 = block kept."""
    if spec.mask_kind == "uniform":
        return uniform_block_mask(spec.rows, spec.cin, spec.sparsity, spec.seed)
    if spec.mask_kind == "zipf":
        return zipf_block_mask(spec.rows, spec.cin, spec.seed)
    raise ValueError(spec.mask_kind)


# ----------------------------------------------------------------------------------------
# The five workload families.

MOBILENET_V1_PW = [  # (cin, cout, h=w) of the 13 pointwise convolutions at 224x224 input
    (32, 64, 112), (64, 128, 56), (128, 128, 56), (128, 256, 28), (256, 256, 28),
    (256, 512, 14), (512, 512, 14), (512, 512, 14), (512, 512, 14), (512, 512, 14),
    (512, 512, 14), (512, 1024, 7), (1024, 1024, 7),
]

RESNET50_BOTTLENECK_PW = [
    (256, 64, 56), (64, 256, 56), (512, 128, 28), (128, 512, 28),
    (1024, 256, 14), (256, 1024, 14), (2048, 512, 7), (512, 2048, 7),
]

SWEEP_SPARSITY = (0.50, 0.70, 0.80, 0.90, 0.95)
SWEEP_G = (1, 4, 8, 16)


def _seed(config: int, layer: int) -> int:
    return BASE_SEED + 1000 * config + layer


def single_layer() -> List[LayerSpec]:
    """One 64->128 conv at 56x56, batch 1, fp32, g=4, 70 % of blocks dropped."""
    return [LayerSpec("c1_64x128@56", 64, 128, 56, 56, n=1, g=4, sparsity=0.70, seed=_seed(1, 0))]


def mobilenet_stack(batch: int, config: int, sparsity=0.8) -> List[LayerSpec]:
    """MobileNetV1-224 pointwise stack.  sparsity: a float, or "draw" for a per-layer seeded
    draw from U[0.6, 0.9]."""
    out = []
    if sparsity == "draw":
        u = rng.uniform01_f64(_seed(config, 999), 7, len(MOBILENET_V1_PW))
        sp = [float(np.round(0.6 + 0.3 * x, 4)) for x in u]
    else:
        sp = [float(sparsity)] * len(MOBILENET_V1_PW)
    for i, (ci, co, s) in enumerate(MOBILENET_V1_PW):
        out.append(LayerSpec(f"mbv1_pw{i + 1:02d}_{ci}x{co}@{s}", ci, co, s, s, n=batch, g=4,
                             sparsity=sp[i], seed=_seed(config, i)))
    return out


def resnet50_stack(batch: int = 32) -> List[LayerSpec]:
    """ResNet-50 bottleneck 1x1 convs, g=8, fp16 in / fp32 accumulate, 75 % of blocks dropped."""
    return [LayerSpec(f"rn50_pw{i + 1}_{ci}x{co}@{s}", ci, co, s, s, n=batch, g=8, dtype="f16",
                      sparsity=0.75, x_dist="halfnormal", seed=_seed(4, i))
            for i, (ci, co, s) in enumerate(RESNET50_BOTTLENECK_PW)]


def sweep(batch: int = 256) -> List[LayerSpec]:
    """512->512 at 14x14: block sparsity x group size grid, plus Zipf-skewed rows at g=4."""
    out, i = [], 0
    for g in SWEEP_G:
        for s in SWEEP_SPARSITY:
            out.append(LayerSpec(f"sweep_g{g}_s{int(round(s * 100))}", 512, 512, 14, 14, n=batch,
                                 g=g, sparsity=s, seed=_seed(5, i)))
            i += 1
    out.append(LayerSpec("sweep_g4_zipf1.2", 512, 512, 14, 14, n=batch, g=4, mask_kind="zipf",
                         sparsity=float("nan"), seed=_seed(5, i)))
    return out


def config_layers(idx: int) -> List[LayerSpec]:
    """Layer lists of the five benchmark configurations, 0-based."""
    if idx == 0:
        return single_layer()
    if idx == 1:
        return mobilenet_stack(1, 2, 0.8)
    if idx == 2:
        return mobilenet_stack(64, 3, "draw")
    if idx == 3:
        return resnet50_stack(32)
    if idx == 4:
        return sweep(256)
    raise IndexError(idx)


def with_batch(spec: LayerSpec, n: int) -> LayerSpec:
    """Same layer (same weights, mask, bias seed) at another batch size."""
    return replace(spec, n=n)
