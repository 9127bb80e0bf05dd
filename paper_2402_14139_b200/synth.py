"""Seeded synthetic inputs: counter-based, host-side, numpy only.

This module holds no arithmetic of the training method.  It only turns
(seed, tensor id, element index) into reproducible numbers, so that the CUDA
path and the CPU checker can be handed identical arrays.

Generator: element ``idx`` of tensor ``tensor_id`` draws the 64-bit word
``splitmix64(seed ^ (tensor_id << 40) + idx)`` (the SplitMix64 finaliser of
Steele, Lea and Flood).  Normal deviates use Box-Muller in float64 on two
words drawn from the even/odd counters ``2*idx`` and ``2*idx + 1``.
"""
from __future__ import annotations

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def splitmix64(z: np.ndarray) -> np.ndarray:
    """SplitMix64 output function applied to every element of a uint64 array."""
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = z + np.uint64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    return z


def _words(seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    base = np.uint64((seed ^ (tensor_id << 40)) & 0xFFFFFFFFFFFFFFFF)
    idx = np.arange(start, start + count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return splitmix64(base + idx)


def uniform01(seed: int, tensor_id: int, count: int, start: int = 0) -> np.ndarray:
    """``count`` float64 values in (0, 1): the top 53 bits of each word, offset by half an ulp."""
    w = _words(seed, tensor_id, start, count)
    return ((w >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, tensor_id: int, shape, std: float = 1.0, chunk: int = 1 << 22) -> np.ndarray:
    """float64 N(0, std^2) array of the given shape (row-major element index = counter)."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float64)
    for s in range(0, n, chunk):
        c = min(chunk, n - s)
        u = uniform01(seed, tensor_id, 2 * c, start=2 * s)
        u1, u2 = u[0::2], u[1::2]
        out[s:s + c] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return (out * std).reshape(shape)


def labels(seed: int, tensor_id: int, count: int, classes: int) -> np.ndarray:
    """int32 labels uniform on [0, classes)."""
    w = _words(seed, tensor_id, 0, count)
    return (w % np.uint64(classes)).astype(np.int32)


def permutation(seed: int, tensor_id: int, n: int) -> np.ndarray:
    """Fisher-Yates shuffle of arange(n) driven by the counter generator (int32)."""
    w = _words(seed, tensor_id, 0, n)
    p = np.arange(n, dtype=np.int32)
    for i in range(n - 1, 0, -1):
        j = int(w[i] % np.uint64(i + 1))
        p[i], p[j] = p[j], p[i]
    return p


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round a float array to the nearest bfloat16 (ties to even); returns float32 holding bf16 values."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = ((u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)) << np.uint64(16)
    return (r & np.uint64(0xFFFFFFFF)).astype(np.uint32).view(np.float32).reshape(f.shape)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) of a float array, round to nearest even."""
    return (round_bf16(a).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """float32 values of bfloat16 bit patterns."""
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)
