"""Seeded synthetic inputs for the HBMM path.

This module only draws random tensors and names workload shapes; it holds none of
the method's arithmetic (no binarization, no scales, no packing), so both the CUDA
path's callers and the CPU checker can be fed from it.  Everything comes from
``numpy.random.Generator(PCG64(seed))`` in float32.

The shapes stand in for the workloads the paper evaluates on (its datasets and
trained weights are not needed by a data-independent kernel): standard-normal
matrices, post-ReLU activations, He-normal weights, ResNet-18 3x3 convolution
shapes at batch 64 and an AlexNet-style fully connected stack.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import numpy as np


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def normal(shape, seed: int) -> np.ndarray:
    """N(0,1), float32."""
    return _rng(seed).standard_normal(shape, dtype=np.float32)


def relu_normal(shape, seed: int) -> np.ndarray:
    """max(0, N(0,1)): a post-ReLU activation map (every element >= 0)."""
    return np.maximum(_rng(seed).standard_normal(shape, dtype=np.float32), np.float32(0))


def he_normal(n_out: int, fan_in: int, seed: int) -> np.ndarray:
    """N(0, 2/fan_in) weight matrix [n_out, fan_in], float32."""
    w = _rng(seed).standard_normal((n_out, fan_in), dtype=np.float32)
    return (w * np.float32(np.sqrt(2.0 / fan_in))).astype(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Nearest-even bfloat16 encoding (uint16) of finite float32 data."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return u.astype(np.uint16)


def bf16_values(bits: np.ndarray) -> np.ndarray:
    """float32 values of bfloat16 encodings."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def as_bf16(x: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """(uint16 encodings, the same values widened back to float32)."""
    b = bf16_bits(x)
    return b, bf16_values(b)


@dataclass(frozen=True)
class ConvShape:
    name: str
    B: int
    C: int
    H: int
    W: int
    N: int  # filters
    kh: int = 3
    kw: int = 3
    stride: int = 1
    pad: int = 1

    @property
    def M(self) -> int:
        ho = (self.H + 2 * self.pad - self.kh) // self.stride + 1
        wo = (self.W + 2 * self.pad - self.kw) // self.stride + 1
        return self.B * ho * wo

    @property
    def K(self) -> int:
        return self.C * self.kh * self.kw


def resnet18_convs(batch: int = 64) -> List[ConvShape]:
    """The four 3x3 stride-1 pad-1 convolution shapes of ResNet-18's stages conv2_x..conv5_x."""
    return [
        ConvShape("conv2_x", batch, 64, 56, 56, 64),
        ConvShape("conv3_x", batch, 128, 28, 28, 128),
        ConvShape("conv4_x", batch, 256, 14, 14, 256),
        ConvShape("conv5_x", batch, 512, 7, 7, 512),
    ]


# (K, N) of the AlexNet-style fully connected stack.
ALEXNET_FC = [(9216, 4096), (4096, 4096), (4096, 1000)]

# Seeds per workload family (activation seed, weight seed); a layer index is added.
SEEDS = {
    "square256": (19051, 19052),
    "square_sweep": (19053, 19073),
    "resnet_hbmm": (19100, 19110),
    "resnet_hbwn": (19120, 19130),
    "alexnet_fc": (19140, 19150),
}


def conv_activation(s: ConvShape, seed: int, signed: bool = False) -> np.ndarray:
    """NCHW activation tensor for a convolution shape: post-ReLU by default, N(0,1)
    (a batch-norm output) when ``signed``."""
    shape = (s.B, s.C, s.H, s.W)
    return normal(shape, seed) if signed else relu_normal(shape, seed)
