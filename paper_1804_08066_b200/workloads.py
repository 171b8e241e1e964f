"""Seeded synthetic inputs shaped like the gradients MQGrad quantizes.

This module only draws numbers.  It contains none of the codec's arithmetic and is
the one piece shared by the CUDA path's tests, the CPU checker's tests and the
benchmark, so that both sides always see identical input bits.

The paper trains a CIFAR-10 network (Section 4.1); the hot path only ever sees flat
fp32 (or bf16) gradient vectors, so seeded vectors with the sizes and value
distributions of such gradients stand in for them.
"""
from __future__ import annotations

import numpy as np

DATA_SEED_BASE = 1804080660  # + config number + 1000 * worker

ALEXNET_SHAPES = [
    (96, 3, 11, 11), (96,),
    (256, 48, 5, 5), (256,),
    (384, 256, 3, 3), (384,),
    (384, 192, 3, 3), (384,),
    (256, 192, 3, 3), (256,),
    (4096, 9216), (4096,),
    (4096, 4096), (4096,),
    (1000, 4096), (1000,),
]


def _rng(config: int, worker: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([DATA_SEED_BASE + config, worker, stream]))


def normal(n: int, sigma: float, config: int = 1, worker: int = 0) -> np.ndarray:
    """iid N(0, sigma) as float32."""
    return _rng(config, worker).standard_normal(n, dtype=np.float32) * np.float32(sigma)


def laplace(n: int, scale: float, config: int = 2, worker: int = 0) -> np.ndarray:
    """iid Laplace(0, scale) as float32, by the inverse CDF of a uniform."""
    u = _rng(config, worker).random(n, dtype=np.float32) - np.float32(0.5)
    a = np.minimum(2.0 * np.abs(u).astype(np.float64), 1.0 - 2.0 ** -24)   # keep the log finite
    mag = (-np.log1p(-a)).astype(np.float32)
    return (np.sign(u) * mag * np.float32(scale)).astype(np.float32)


def params(n: int, sigma: float = 0.05, config: int = 1) -> np.ndarray:
    """Initial shared parameters, N(0, sigma)."""
    return _rng(config, 0, stream=7).standard_normal(n, dtype=np.float32) * np.float32(sigma)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16, returned as uint16 bit patterns."""
    b = np.ascontiguousarray(x, np.float32).view(np.uint32).astype(np.uint64)
    b = (b + 0x7FFF + ((b >> 16) & 1)) >> 16
    return b.astype(np.uint16)


def student_t_bf16(n: int, scale: float = 1e-4, nu: float = 3.0, zero_frac: float = 1e-3,
                   config: int = 5, worker: int = 0) -> np.ndarray:
    """Heavy-tailed Student-t(nu) * scale with a fraction of exact zeros, as bf16 bits."""
    g = _rng(config, worker)
    x = g.standard_t(nu, n).astype(np.float32) * np.float32(scale)
    x[g.random(n) < zero_frac] = 0.0
    return f32_to_bf16_bits(x)


# The CNN of the paper's evaluation (Section 4.1): two 5x5 convolutions, two large fully connected
# layers and the softmax layer.  Only the two large weight matrices are quantized (99 % of the
# parameters); they come first in the flat layout used here so that they form two adjacent
# segments, and everything else follows uncompressed.
PAPER_CNN_QUANTIZED = [(3136, 2304), (2304, 3840)]
PAPER_CNN_UNCOMPRESSED = [(5, 5, 3, 64), (64,), (5, 5, 64, 64), (64,), (2304,), (3840,), (3840, 10), (10,)]


def paper_cnn_layout():
    """(seg_off of the two quantized matrices, total elements of the flat gradient)."""
    sizes = [int(np.prod(s)) for s in PAPER_CNN_QUANTIZED]
    seg_off = np.zeros(len(sizes) + 1, np.uint64)
    seg_off[1:] = np.cumsum(sizes)
    total = int(seg_off[-1]) + sum(int(np.prod(s)) for s in PAPER_CNN_UNCOMPRESSED)
    return seg_off, total


def paper_cnn_gradient(config: int = 6, worker: int = 0) -> np.ndarray:
    """Flat synthetic gradient of that model: every tensor N(0, sigma_l), sigma_l log-uniform."""
    sizes = [int(np.prod(s)) for s in PAPER_CNN_QUANTIZED + PAPER_CNN_UNCOMPRESSED]
    return layered(sizes, config=config, worker=worker)


def alexnet_segments():
    """(seg_off, sizes) of the AlexNet-shaped layered gradient, weights and biases in order."""
    sizes = [int(np.prod(s)) for s in ALEXNET_SHAPES]
    seg_off = np.zeros(len(sizes) + 1, np.uint64)
    seg_off[1:] = np.cumsum(sizes)
    return seg_off, sizes


def layered(sizes, config: int = 3, worker: int = 0, sigma_lo: float = 1e-5,
            sigma_hi: float = 1e-2) -> np.ndarray:
    """One flat gradient; layer l is N(0, sigma_l), sigma_l log-uniform in [lo, hi].

    The per-layer sigmas depend on the config only, so all workers share them."""
    sig = 10.0 ** _rng(config, 0, stream=3).uniform(np.log10(sigma_lo), np.log10(sigma_hi),
                                                    len(sizes))
    g = _rng(config, worker)
    parts = [g.standard_normal(s, dtype=np.float32) * np.float32(sg)
             for s, sg in zip(sizes, sig)]
    return np.concatenate(parts) if parts else np.zeros(0, np.float32)
