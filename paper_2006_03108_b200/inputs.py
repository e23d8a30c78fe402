"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds no arithmetic of the operators: it only draws numbers from
numpy's counter-based Philox generator and converts fp32 to bfloat16 bit
patterns.  A tensor is always drawn as the *global* array and cut into shards
afterwards, so a value depends only on (seed, global index).
"""

import numpy as np


def _rng(seed):
    return np.random.Generator(np.random.Philox(int(seed)))


def uniform_pm1(shape, seed):
    """fp32 values uniform in [-1, 1)."""
    r = _rng(seed).random(size=shape, dtype=np.float32)
    return (r * np.float32(2.0) - np.float32(1.0)).astype(np.float32)


def normal(shape, seed, std=1.0):
    """fp32 values normal(0, std)."""
    r = _rng(seed).standard_normal(size=shape, dtype=np.float32)
    return (r * np.float32(std)).astype(np.float32)


def integers(shape, seed, lo=-4, hi=5):
    """Small integer-valued fp32 values (sums of these are exact in any order)."""
    return _rng(seed).integers(lo, hi, size=shape).astype(np.float32)


def f32_to_bf16_bits(a):
    """Round fp32 to bfloat16 (round to nearest even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits):
    """Widen bfloat16 bit patterns exactly to fp32."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32)
