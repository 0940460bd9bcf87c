"""Seeded synthetic k x k layers shaped like the 3x3 convolutions of ResNet-18 (one of the
networks the paper prunes), with the SIMD-structured block pattern over the flattened-filter
columns (c, r, s).  Inputs only: nothing here multiplies or packs anything.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import numpy as np

from . import rng
from .layers import BASE_SEED, uniform_block_mask


@dataclass(frozen=True)
class Conv2dSpec:
    """Y[n,cout,oh,ow] = conv(W[cout,cin,kh,kw], X[n,cin,h,w]; stride, zero padding) + bias."""
    name: str
    cin: int
    cout: int
    h: int
    w: int
    kh: int = 3
    kw: int = 3
    stride: int = 1
    pad: int = 1
    n: int = 1
    g: int = 4
    sparsity: float = 0.7
    relu: bool = True
    bias: bool = True
    seed: int = BASE_SEED

    @property
    def k(self) -> int:
        """Columns of the flattened-filter matrix."""
        return self.cin * self.kh * self.kw

    @property
    def rows(self) -> int:
        return (self.cout + self.g - 1) // self.g

    @property
    def oh(self) -> int:
        return (self.h + 2 * self.pad - self.kh) // self.stride + 1

    @property
    def ow(self) -> int:
        return (self.w + 2 * self.pad - self.kw) // self.stride + 1


def make_weights2d(s: Conv2dSpec) -> np.ndarray:
    """W[cout,cin,kh,kw] ~ N(0, 1/(cin*kh*kw)) (variance), fp32."""
    w = rng.normal(s.seed, 1, s.cout * s.k, sigma=s.k ** -0.5)
    return w.reshape(s.cout, s.cin, s.kh, s.kw).astype(np.float32)


def make_mask2d(s: Conv2dSpec) -> np.ndarray:
    """Block mask [rows, cin*kh*kw]: exactly round(sparsity * blocks) blocks dropped, seeded shuffle."""
    return uniform_block_mask(s.rows, s.k, s.sparsity, s.seed)


def make_x2d(s: Conv2dSpec) -> np.ndarray:
    """X[n,cin,h,w] ~ U[0,1), fp32."""
    return rng.uniform01(s.seed, 3, s.n * s.cin * s.h * s.w).reshape(s.n, s.cin, s.h, s.w)


def make_bias2d(s: Conv2dSpec):
    if not s.bias:
        return None
    return rng.normal(s.seed, 4, s.cout, sigma=0.1).astype(np.float32)


# (cin, cout, input h=w, stride) of the distinct 3x3 convolutions of ResNet-18 at 224x224 input
RESNET18_3X3 = [(64, 64, 56, 1), (64, 128, 56, 2), (128, 128, 28, 1), (128, 256, 28, 2),
                (256, 256, 14, 1), (256, 512, 14, 2), (512, 512, 7, 1)]


def resnet18_3x3_stack(batch: int = 32, sparsity: float = 0.7, g: int = 4) -> List[Conv2dSpec]:
    """ResNet-18's 3x3 convolutions (pad 1), fp32, g = 4, 70 % of the blocks dropped: the paper's
    pruned ResNet-18 keeps 548M of 1.8G FLOPs, about 30 %."""
    return [Conv2dSpec(f"rn18_3x3_{i + 1}_{ci}x{co}@{s}s{st}", ci, co, s, s, stride=st, n=batch, g=g,
                       sparsity=sparsity, seed=BASE_SEED + 6000 + i)
            for i, (ci, co, s, st) in enumerate(RESNET18_3X3)]
