"""Seeded synthetic inputs shaped like the linear layers of the Llama models the paper evaluates.

This module holds no arithmetic of the W4A8 method: it draws Gaussian tensors, plants outlier
channels and converts fp32 to BF16 bit patterns (a storage cast).  The CPU oracle and the CUDA
library are both fed from here so that they see identical buffers.
"""
from __future__ import annotations

import math

import numpy as np

# name -> list of (M, K, N) problems plus the generation recipe.
CONFIGS = {
    # single small linear: smoke / latency case
    "c1": dict(shapes=[(16, 1024, 1024)], sigma=0.02, outlier_frac=0.0, outlier_mult=1.0),
    # decode sweep on the Llama-3-8B MLP up-projection shape
    "c2": dict(shapes=[(1, 4096, 14336), (4, 4096, 14336), (16, 4096, 14336)], sigma=0.02,
               outlier_frac=0.01, outlier_mult=20.0),
    # prefill on the attention output-projection shape
    "c3": dict(shapes=[(2048, 4096, 4096)], sigma=0.02, outlier_frac=0.01, outlier_mult=20.0),
    # large prefill on the Llama-3-70B gate+up shape
    "c4": dict(shapes=[(8192, 8192, 28672)], sigma=0.015, outlier_frac=0.005, outlier_mult=30.0),
    # the four linears of a Llama-3-8B decoder block, for M in {1,8,32,128,512,4096}
    "c5": dict(shapes=[(m, k, n) for m in (1, 8, 32, 128, 512, 4096)
                       for (k, n) in ((4096, 6144), (4096, 4096), (4096, 28672), (14336, 4096))],
               sigma=0.02, outlier_frac=0.01, outlier_mult=20.0),
}

GROUP = 128


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Storage cast fp32 -> BF16 bit patterns (uint16), round-to-nearest-even, finite inputs."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def make_weight(N: int, K: int, sigma: float, seed: int) -> np.ndarray:
    """fp32 [N, K] drawn from N(0, sigma^2)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    w = rng.standard_normal((N, K), dtype=np.float32)
    w *= np.float32(sigma)
    return w


def outlier_columns(K: int, frac: float, seed: int) -> np.ndarray:
    """Indices of the ceil(frac*K) input features that carry outliers (same for every token)."""
    n = int(math.ceil(frac * K)) if frac > 0 else 0
    rng = np.random.Generator(np.random.PCG64(seed + 7919))
    return np.sort(rng.choice(K, size=n, replace=False)) if n else np.zeros(0, dtype=np.int64)


def make_activation(M: int, K: int, seed: int, outlier_frac: float = 0.0,
                    outlier_mult: float = 1.0) -> np.ndarray:
    """BF16 bit patterns [M, K]: N(0,1) with a fixed set of outlier channels scaled by outlier_mult."""
    rng = np.random.Generator(np.random.PCG64(seed + 104729))
    x = rng.standard_normal((M, K), dtype=np.float32)
    cols = outlier_columns(K, outlier_frac, seed)
    if cols.size:
        x[:, cols] *= np.float32(outlier_mult)
    return f32_to_bf16_bits(x)


def make_small_int_activation(M: int, K: int, seed: int, lo: int = -4, hi: int = 4) -> np.ndarray:
    """BF16 bit patterns of small integers: makes fp32 accumulation exact (layout tests)."""
    rng = np.random.Generator(np.random.PCG64(seed + 15485863))
    x = rng.integers(lo, hi + 1, size=(M, K)).astype(np.float32)
    return f32_to_bf16_bits(x)


def random_codes(N: int, K: int, seed: int, group: int = GROUP, asymmetric: bool = False,
                 scale_bits=None):
    """Random packed INT4 codes with random BF16 group scales (and zero-points): exercises every
    nibble value independently of any quantizer.  Returns (codes, gscale_bits, gzero or None)."""
    rng = np.random.Generator(np.random.PCG64(seed + 32452843))
    codes = rng.integers(0, 256, size=(N, K // 2), dtype=np.uint8)
    G = K // group
    if scale_bits is None:
        s = np.exp2(rng.uniform(-6.0, 5.5, size=(N, G))).astype(np.float32)
        gscale = f32_to_bf16_bits(s)
    else:
        gscale = np.full((N, G), scale_bits, dtype=np.uint16)
    gzero = rng.integers(0, 16, size=(N, G), dtype=np.uint8) if asymmetric else None
    return codes, gscale, gzero
