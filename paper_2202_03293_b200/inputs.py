"""Seeded synthetic input generators (NumPy, host side).

This module only *produces* tensors; it contains none of the ops' arithmetic
and is the one piece shared by the CUDA path's callers and the CPU oracle's
callers, so that both sides see bit-identical inputs.

Generator: counter based, independent of any library RNG state.
    h(i) = splitmix64(seed ^ (tensor_id << 56) ^ i)          (i = linear index)
    uniform[-1,1):  u = (h >> 40) * 2**-23 - 1                (24 bits, exact in f32)
    normal(0,1):    Box-Muller in f64 on two such hashes, rounded to f32
bf16 tensors are the f32 sample rounded to nearest-even to 8 significant bits;
they are returned both as the uint16 bit pattern (what the GPU reads) and as
the same values widened to f32 (what the oracle reads).
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 220203293

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def splitmix64(x: np.ndarray) -> np.ndarray:
    """Vectorised splitmix64 finaliser on uint64 (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        z = (x + np.uint64(0x9E3779B97F4A7C15)) & _M64
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        return z ^ (z >> np.uint64(31))


def _hash(seed: int, tensor_id: int, count: int, stream: int = 0) -> np.ndarray:
    key = (int(seed) ^ (int(tensor_id) << 56) ^ (int(stream) << 48)) & 0xFFFFFFFFFFFFFFFF
    idx = np.arange(count, dtype=np.uint64)
    return splitmix64(idx ^ np.uint64(key))


def uniform(shape, seed: int, tensor_id: int) -> np.ndarray:
    """f32 tensor, values uniform on the 2**-23 grid in [-1, 1)."""
    count = int(np.prod(shape)) if len(shape) else 1
    h = _hash(seed, tensor_id, count)
    u = (h >> np.uint64(40)).astype(np.float64) * (2.0 ** -23) - 1.0
    return u.astype(np.float32).reshape(shape)


def normal(shape, seed: int, tensor_id: int) -> np.ndarray:
    """f32 tensor, standard normal via Box-Muller on two hashed uniforms."""
    count = int(np.prod(shape)) if len(shape) else 1
    h1 = _hash(seed, tensor_id, count, stream=1)
    h2 = _hash(seed, tensor_id, count, stream=2)
    u1 = ((h1 >> np.uint64(11)).astype(np.float64) + 1.0) * (2.0 ** -53)   # (0, 1]
    u2 = (h2 >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)           # [0, 1)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return z.astype(np.float32).reshape(shape)


def small_ints(shape, seed: int, tensor_id: int, lo: int = -2, hi: int = 2) -> np.ndarray:
    """f32 tensor of integers in [lo, hi]: products and short sums are exact in every path."""
    count = int(np.prod(shape)) if len(shape) else 1
    h = _hash(seed, tensor_id, count, stream=3)
    span = np.uint64(hi - lo + 1)
    return ((h >> np.uint64(33)) % span).astype(np.float32).reshape(shape) + np.float32(lo)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round f32 to bf16 (nearest, ties to even); returns the uint16 patterns."""
    b = np.ascontiguousarray(x, np.float32).view(np.uint32)
    rounded = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def as_bf16(x: np.ndarray):
    """(bits_uint16, values_f32) of the bf16 rounding of ``x``."""
    bits = to_bf16_bits(x)
    return bits, bf16_bits_to_f32(bits).reshape(x.shape)


def make(shape, seed: int, tensor_id: int, dist: str = "uniform", dtype: str = "f32"):
    """One operand: returns (device_payload, oracle_f32).

    ``device_payload`` is the f32 array itself for ``dtype='f32'`` and the
    uint16 bf16 bit patterns for ``dtype='bf16'``; ``oracle_f32`` always holds
    exactly the values the device payload encodes.
    """
    if dist == "uniform":
        x = uniform(shape, seed, tensor_id)
    elif dist == "normal":
        x = normal(shape, seed, tensor_id)
    elif dist == "ints":
        x = small_ints(shape, seed, tensor_id)
    else:
        raise ValueError(dist)
    if dtype == "f32":
        return x, x
    if dtype == "bf16":
        bits, vals = as_bf16(x)
        return bits.reshape(shape), vals
    raise ValueError(dtype)
