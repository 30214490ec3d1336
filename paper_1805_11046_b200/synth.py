"""Seeded synthetic inputs shaped like the paper's CNN workloads.

The paper trains ResNet-18/50 on ImageNet (Section 6); no dataset is used here.
These generators produce tensors with the same shapes, layouts and value
structure (ReLU'd activations with half zeros, Kaiming-initialised filters,
small-variance gradients, per-channel shifted and scaled Gaussians) from fixed
seeds, on the host, with numpy only.  This module holds none of the method's
arithmetic: it is the one module that both the CPU oracle's tests and the CUDA
path's tests and benchmark draw their inputs from.

Layouts: activations NHWC, filters KRSC, matrices row-major; dtype float32.
"""
from __future__ import annotations

import numpy as np


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def normal(shape, seed: int, std: float = 1.0, mean: float = 0.0) -> np.ndarray:
    x = _rng(seed).standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    if mean != 0.0:
        x += np.float32(mean)
    return x


def uniform(shape, seed: int, bound: float) -> np.ndarray:
    x = _rng(seed).random(size=shape, dtype=np.float32)
    return (x * np.float32(2.0 * bound) - np.float32(bound)).astype(np.float32)


def relu_normal(shape, seed: int) -> np.ndarray:
    x = normal(shape, seed)
    np.maximum(x, 0.0, out=x)
    return x


def kaiming_normal(shape_krsc, seed: int) -> np.ndarray:
    """Filter [K,R,S,C]; std = sqrt(2 / fan_in), fan_in = R*S*C."""
    fan_in = int(np.prod(shape_krsc[1:]))
    return normal(shape_krsc, seed, std=float(np.sqrt(2.0 / fan_in)))


def kaiming_uniform_linear(k_in: int, n_out: int, seed: int) -> np.ndarray:
    """Weight [k_in, n_out] of y = x w; bound = sqrt(6 / fan_in), fan_in = k_in."""
    return uniform((k_in, n_out), seed, float(np.sqrt(6.0 / k_in)))


def channel_gaussian(shape_nhwc, seed_stats: int, seed_x: int) -> np.ndarray:
    """x[..., c] ~ N(mu_c, sigma_c^2) with mu_c ~ U(-1, 1), sigma_c ~ U(0.5, 2)."""
    C = shape_nhwc[-1]
    g = _rng(seed_stats)
    mu = (g.random(C, dtype=np.float32) * 2.0 - 1.0).astype(np.float32)
    sigma = (g.random(C, dtype=np.float32) * 1.5 + 0.5).astype(np.float32)
    x = normal(shape_nhwc, seed_x)
    x *= sigma
    x += mu
    return x


# ---- the five workloads -----------------------------------------------------

def linear_layer(batch: int = 64, k_in: int = 256, n_out: int = 128):
    """Single quantised linear layer + Range BN: X ~ N(0,1), W Kaiming-uniform,
    upstream gradient ~ N(0, variance 1e-2)."""
    return dict(x=normal((batch, k_in), 1),
                w=kaiming_uniform_linear(k_in, n_out, 2),
                dy=normal((batch, n_out), 3, std=0.1),
                seed=0, id8=1, id16=1)      # one tensor id for the gradient: both copies draw from its stream


def conv3x3_layer(batch: int = 256, hw: int = 56, c_in: int = 64, k_out: int = 64):
    """ResNet-18 conv2_x 3x3 layer, stride 1, pad 1: ReLU'd N(0,1) input (half
    zeros), Kaiming-normal filter, upstream gradient ~ N(0, std 0.1)."""
    return dict(x=relu_normal((batch, hw, hw, c_in), 10),
                w=kaiming_normal((k_out, 3, 3, c_in), 11),
                dy=normal((batch, hw, hw, k_out), 12, std=0.1),
                conv=dict(N=batch, H=hw, W=hw, C=c_in, K=k_out, R=3, S=3, stride=1, pad=1),
                seed=0, id8=1, id16=1)


RANGEBN_SWEEP = ((56, 64), (28, 128), (14, 256), (7, 512), (7, 2048))


def rangebn_case(batch: int, hw: int, channels: int):
    """Range BN / quantiser sweep tensor: per-channel shifted, scaled Gaussian; dY ~ N(0,1)."""
    shape = (batch, hw, hw, channels)
    return dict(x=channel_gaussian(shape, 20, 21), dy=normal(shape, 22))


def bottleneck_stack(batch: int = 256, hw: int = 28):
    """ResNet-50 conv3_x bottleneck: 1x1 256->128, 3x3 128->128, 1x1 128->512,
    each followed by Range BN + ReLU; no residual branch."""
    convs = [dict(N=batch, H=hw, W=hw, C=256, K=128, R=1, S=1, stride=1, pad=0),
             dict(N=batch, H=hw, W=hw, C=128, K=128, R=3, S=3, stride=1, pad=1),
             dict(N=batch, H=hw, W=hw, C=128, K=512, R=1, S=1, stride=1, pad=0)]
    return dict(x=normal((batch, hw, hw, 256), 30),
                w=[kaiming_normal((128, 1, 1, 256), 31),
                   kaiming_normal((128, 3, 3, 128), 32),
                   kaiming_normal((512, 1, 1, 128), 33)],
                dy=normal((batch, hw, hw, 512), 34, std=0.1),
                convs=convs, seed=0)


def dense_gemm(M: int, N: int, K: int, parts=("a", "b", "x", "g")):
    """Dense sweep operands: A [M,K], B [K,N] ~ N(0,1); for the weight-gradient
    product X [M,K] (8-bit side) and G [M,N] (16-bit side), reduced over M.
    parts: which of the four to generate (each is up to 1 GB at 16384^2)."""
    shapes = dict(a=((M, K), 40), b=((K, N), 41), x=((M, K), 42), g=((M, N), 43))
    return {k: normal(*shapes[k]) for k in parts}
