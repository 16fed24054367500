"""Seeded synthetic inputs and bit-layout marshalling.

This module serves both the CUDA library's callers and the CPU oracle's tests, so it
holds none of the method's arithmetic: it only draws random tensors and converts
between one-int8-per-element +-1 tensors and the packed sign-bit layout
(bit 1 = +1, bit 0 = -1; channel c of a pixel lives in byte c // 8, bit c % 8, which
is ``numpy.packbits(..., bitorder="little")`` along the channel axis, so 32- and
64-bit little-endian words see the same memory).

The tensors stand in for the ImageNet-scale activations of the paper's network
(Section 5.1 trains on 224x224 crops with zero-mean unit-variance normalisation):
same shapes, no dataset items.
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 20100704


def seed_for(config: int, layer: int = 0) -> int:
    """One seed per (workload, layer)."""
    return BASE_SEED + 1000 * int(config) + int(layer)


def rng_for(config: int, layer: int = 0) -> np.random.Generator:
    return np.random.default_rng(seed_for(config, layer))


def pm1(rng: np.random.Generator, shape) -> np.ndarray:
    """i.i.d. Bernoulli(0.5) values in {-1, +1}, int8."""
    return (rng.integers(0, 2, size=shape, dtype=np.int8) * 2 - 1).astype(np.int8)


def random_bits(rng: np.random.Generator, shape_bytes) -> np.ndarray:
    """i.i.d. Bernoulli(0.5) sign bits already packed: uint8 array of the given byte shape."""
    return rng.integers(0, 256, size=shape_bytes, dtype=np.uint8)


def real_input(rng: np.random.Generator, shape) -> np.ndarray:
    """Zero-mean unit-variance real activations, fp32."""
    return rng.standard_normal(size=shape, dtype=np.float32)


def thresholds(rng: np.random.Generator, K: int, N: int) -> np.ndarray:
    """Integer thresholds uniform on [-K//4, K//4], both ends included, int32."""
    return rng.integers(-(K // 4), K // 4 + 1, size=N, dtype=np.int64).astype(np.int32)


def pack_bits(v: np.ndarray) -> np.ndarray:
    """+-1 (or 0/1) tensor -> packed sign bits along the last axis (length % 8 == 0), uint8."""
    v = np.asarray(v)
    assert v.shape[-1] % 8 == 0
    return np.packbits(v > 0, axis=-1, bitorder="little")


def unpack_bits(bits: np.ndarray, n: int | None = None) -> np.ndarray:
    """Packed sign bits along the last axis -> int8 +-1 tensor (first n entries of that axis)."""
    bits = np.ascontiguousarray(bits).view(np.uint8)
    u = np.unpackbits(bits, axis=-1, bitorder="little")
    if n is not None:
        u = u[..., :n]
    return (u.astype(np.int8) * 2 - 1).astype(np.int8)
