"""Seeded synthetic tensors for the grouped-convolution workloads.

A counter-based generator: element ``i`` of tensor ``tensor_id`` under ``seed`` is a pure function
of (seed, tensor_id, i), so any slice can be regenerated anywhere and nothing depends on a library
RNG's version.  This module holds no convolution arithmetic; it is the one module that both the
CUDA path's callers and the oracle's callers may import.
"""
from __future__ import annotations

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(z: np.ndarray) -> np.ndarray:
    z = (z + np.uint64(0x9E3779B97F4A7C15)) & _M64
    z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
    z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
    return z ^ (z >> np.uint64(31))


def _bits(seed: int, tensor_id: int, stream: int, n: int, start: int = 0) -> np.ndarray:
    with np.errstate(over="ignore"):
        key = _splitmix64(np.array([(seed * 0x100000001B3 + tensor_id * 7919 + stream * 104729) & 0xFFFFFFFFFFFFFFFF],
                                   dtype=np.uint64))[0]
        idx = np.arange(start, start + n, dtype=np.uint64)
        return _splitmix64(idx ^ key)


def uniform(shape, seed: int, tensor_id: int = 0, lo: float = -1.0, hi: float = 1.0) -> np.ndarray:
    """float32 tensor, i.i.d. uniform on [lo, hi) with 24-bit resolution."""
    n = int(np.prod(shape))
    u = (_bits(seed, tensor_id, 0, n) >> np.uint64(40)).astype(np.float64) * (1.0 / (1 << 24))
    return (lo + (hi - lo) * u).astype(np.float32).reshape(shape)


def normal(shape, seed: int, tensor_id: int = 0, std: float = 1.0) -> np.ndarray:
    """float32 tensor, i.i.d. N(0, std^2) by Box-Muller on two independent 24-bit uniforms."""
    n = int(np.prod(shape))
    u1 = ((_bits(seed, tensor_id, 1, n) >> np.uint64(40)).astype(np.float64) + 1.0) * (1.0 / (1 << 24))
    u2 = (_bits(seed, tensor_id, 2, n) >> np.uint64(40)).astype(np.float64) * (1.0 / (1 << 24))
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return (std * z).astype(np.float32).reshape(shape)


def layer_seed(*ints: int) -> int:
    """Mix a tuple of small integers (config id, shape id, groups, N, ...) into one 63-bit seed."""
    h = 0x9E3779B9
    for v in ints:
        h = int(_splitmix64(np.array([(h ^ (int(v) & 0xFFFFFFFF)) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))[0])
    return h & 0x7FFFFFFFFFFFFFFF


def make_layer_tensors(N, C_in, H, W, C_out, KH, KW, groups, seed, x_dist="uniform"):
    """Inputs of one layer: x ~ U[-1,1) or N(0,1); w ~ N(0, 2/(Cg*KH*KW)) (He-normal on the per-group fan-in)."""
    Cg = C_in // groups
    if x_dist == "uniform":
        x = uniform((N, C_in, H, W), seed, 0)
    elif x_dist == "normal":
        x = normal((N, C_in, H, W), seed, 0)
    else:
        raise ValueError(x_dist)
    w = normal((C_out, Cg, KH, KW), seed, 1, std=float(np.sqrt(2.0 / (Cg * KH * KW))))
    return x, w
