"""Seeded synthetic inputs for the convolution-forward workloads.

This module holds input *generation* only: a counter-based random generator and the tensor
shapes / value distributions of the benchmark configurations.  It contains none of the
convolution arithmetic and imports neither the CUDA binding nor the CPU oracle, so both sides of
a parity test can be fed from it.

Generator: SplitMix64 (a 64-bit counter hashed by two multiply-xorshift rounds) gives uniform
doubles in [0, 1) from the top 53 bits; normals come from the Box-Muller transform of two such
streams.  No library RNG is used, so a (seed, shape) pair always yields the same fp32 array.

The configurations stand in for the paper's benchmark set (the unique convolutions of AlexNet,
NiN and GoogLeNet-v1 at batch sizes 1, 5 and 20, Section 5), whose item list the paper does not
print: shapes are the ones named by the build's baseline description, values are synthetic.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

BASE_SEED = 0x160600094
_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(counter: np.ndarray) -> np.ndarray:
    """SplitMix64 output function applied to an array of uint64 counters (wrapping arithmetic)."""
    with np.errstate(over="ignore"):
        z = counter + np.uint64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    return z


def uniform01(seed: int, n: int, stream: int = 0) -> np.ndarray:
    """n doubles in [0, 1): element i is SplitMix64(seed*2^32-ish + stream, i) >> 11 scaled by 2^-53."""
    with np.errstate(over="ignore"):
        base = _splitmix64(np.array([np.uint64(seed & 0xFFFFFFFFFFFFFFFF)], dtype=np.uint64))[0]
        base = base ^ (np.uint64(stream) * np.uint64(0xD1342543DE82EF95))
        idx = np.arange(n, dtype=np.uint64) * np.uint64(0x9E3779B97F4A7C15) + base
    bits = _splitmix64(idx)
    return (bits >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def uniform(seed: int, shape, lo: float, hi: float) -> np.ndarray:
    n = int(np.prod(shape))
    return (lo + (hi - lo) * uniform01(seed, n)).astype(np.float32).reshape(shape)


def normal(seed: int, shape, mean: float = 0.0, std: float = 1.0) -> np.ndarray:
    """Box-Muller on two independent SplitMix64 streams."""
    n = int(np.prod(shape))
    u1 = 1.0 - uniform01(seed, n, stream=1)          # (0, 1]
    u2 = uniform01(seed, n, stream=2)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)
    return (mean + std * z).astype(np.float32).reshape(shape)


def half_normal(seed: int, shape) -> np.ndarray:
    """|N(0,1)|: the value distribution of a post-ReLU activation."""
    return np.abs(normal(seed, shape))


def integers(seed: int, shape, lo: int = -8, hi: int = 8) -> np.ndarray:
    """Integer-valued fp32 in [lo, hi]: exactly representable in TF32, used by bit-exact tests."""
    n = int(np.prod(shape))
    v = np.floor(uniform01(seed, n) * (hi - lo + 1)) + lo
    return np.clip(v, lo, hi).astype(np.float32).reshape(shape)


@dataclass(frozen=True)
class ConvShape:
    N: int
    C: int
    H: int
    W: int
    K: int
    R: int
    S: int
    stride: int = 1
    pad: int = 0
    relu: bool = True

    @property
    def P(self) -> int:
        return (self.H + 2 * self.pad - self.R) // self.stride + 1

    @property
    def Q(self) -> int:
        return (self.W + 2 * self.pad - self.S) // self.stride + 1

    @property
    def flops(self) -> int:
        return 2 * self.N * self.K * self.P * self.Q * self.C * self.R * self.S

    @property
    def min_bytes(self) -> int:
        return 4 * (self.N * self.C * self.H * self.W + self.K * self.C * self.R * self.S + self.K
                    + self.N * self.K * self.P * self.Q)

    def as_tuple(self) -> Tuple[int, ...]:
        return (self.N, self.C, self.H, self.W, self.K, self.R, self.S, self.stride, self.pad,
                int(self.relu))


@dataclass(frozen=True)
class LayerConfig:
    """One single-layer benchmark configuration: a shape and the distributions of its tensors."""
    cfg_id: int
    name: str
    shape: ConvShape
    in_dist: str            # "uniform[-1,1]" | "uniform[0,1]" | "half_normal"
    w_dist: str             # "normal(0.1)" | "he_normal"

    def tensors(self, layer: int = 0):
        s = self.shape
        seed = BASE_SEED ^ (self.cfg_id << 8) ^ (layer << 4)
        if self.in_dist == "uniform[-1,1]":
            x = uniform(seed ^ 0, (s.N, s.C, s.H, s.W), -1.0, 1.0)
        elif self.in_dist == "uniform[0,1]":
            x = uniform(seed ^ 0, (s.N, s.C, s.H, s.W), 0.0, 1.0)
        elif self.in_dist == "half_normal":
            x = half_normal(seed ^ 0, (s.N, s.C, s.H, s.W))
        else:
            raise ValueError(self.in_dist)
        if self.w_dist == "normal(0.1)":
            w = normal(seed ^ 1, (s.K, s.C, s.R, s.S), 0.0, 0.1)
        elif self.w_dist == "he_normal":
            w = normal(seed ^ 1, (s.K, s.C, s.R, s.S), 0.0, math.sqrt(2.0 / (s.C * s.R * s.S)))
        else:
            raise ValueError(self.w_dist)
        b = normal(seed ^ 2, (s.K,), 0.0, 0.01)
        return x, w, b


# The four single-layer configurations (ids 1..4) and the layers of the stack (id 5).
CONFIGS = {
    1: LayerConfig(1, "small3x3", ConvShape(1, 3, 32, 32, 16, 3, 3, 1, 1), "uniform[-1,1]", "normal(0.1)"),
    2: LayerConfig(2, "alexnet_conv1_b1", ConvShape(1, 3, 227, 227, 96, 11, 11, 4, 0), "uniform[0,1]", "he_normal"),
    3: LayerConfig(3, "inception_1x1_b5", ConvShape(5, 480, 14, 14, 192, 1, 1, 1, 0), "half_normal", "he_normal"),
    4: LayerConfig(4, "alexnet_conv3_b20", ConvShape(20, 256, 13, 13, 384, 3, 3, 1, 1), "half_normal", "he_normal"),
}


@dataclass(frozen=True)
class StackOp:
    kind: str                         # "conv" | "pool"
    shape: Optional[ConvShape] = None  # conv only
    ksz: int = 3                      # pool only
    stride: int = 2                   # pool only


def alexnet_stack(N: int = 20) -> List[StackOp]:
    """AlexNet-shaped, ungrouped conv stack: conv1 pool conv2 pool conv3 conv4 conv5 pool."""
    return [
        StackOp("conv", ConvShape(N, 3, 227, 227, 96, 11, 11, 4, 0)),
        StackOp("pool"),
        StackOp("conv", ConvShape(N, 96, 27, 27, 256, 5, 5, 1, 2)),
        StackOp("pool"),
        StackOp("conv", ConvShape(N, 256, 13, 13, 384, 3, 3, 1, 1)),
        StackOp("conv", ConvShape(N, 384, 13, 13, 384, 3, 3, 1, 1)),
        StackOp("conv", ConvShape(N, 384, 13, 13, 256, 3, 3, 1, 1)),
        StackOp("pool"),
    ]


def stack_tensors(N: int = 20, cfg_id: int = 5):
    """Input image batch U[0,1] and, per conv layer, He-normal filters and N(0, 0.01) biases."""
    ops = alexnet_stack(N)
    first = ops[0].shape
    x = uniform(BASE_SEED ^ (cfg_id << 8), (first.N, first.C, first.H, first.W), 0.0, 1.0)
    params = []
    layer = 0
    for op in ops:
        if op.kind != "conv":
            continue
        layer += 1
        s = op.shape
        seed = BASE_SEED ^ (cfg_id << 8) ^ (layer << 4)
        w = normal(seed ^ 1, (s.K, s.C, s.R, s.S), 0.0, math.sqrt(2.0 / (s.C * s.R * s.S)))
        b = normal(seed ^ 2, (s.K,), 0.0, 0.01)
        params.append((w, b))
    return x, params


def stack_flops(N: int = 20) -> int:
    return sum(op.shape.flops for op in alexnet_stack(N) if op.kind == "conv")
