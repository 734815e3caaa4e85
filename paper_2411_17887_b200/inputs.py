"""Seeded synthetic inputs for the scan library's tests and benchmark.

This module holds no scan arithmetic: it only draws random numbers with NumPy's
``Generator(PCG64(seed))`` and encodes them in the library's input types.  It is
the one module that both the CPU oracle's tests and the GPU path's tests use.

The paper reports no experiments and names no dataset, so every workload here
is synthetic; the shapes, value ranges and distributions are those of the five
build configurations (int8 uniform integers, fp16 uniform reals, bf16 normal
reals).

Encodings: int8 -> ``np.int8``; fp16 -> ``np.float16`` (fp32 draws rounded to
nearest even); bf16 -> ``np.uint16`` bit patterns (fp32 draws rounded to nearest
even on the upper 16 bits), since NumPy has no bfloat16 type.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Tuple

import numpy as np

BASE_SEED = 2411_17887


def rng(seed_offset: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(BASE_SEED + int(seed_offset)))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to bfloat16 (nearest, ties to even); return the uint16 bit patterns.

    Only finite inputs are expected (the generators below produce no NaN/Inf).
    """
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((b >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((b + bias) >> np.uint32(16)).astype(np.uint16)


def int8_uniform(n, lo: int, hi: int, seed_offset: int) -> np.ndarray:
    """i.i.d. integers uniform on the closed range [lo, hi]."""
    return rng(seed_offset).integers(lo, hi + 1, size=n, dtype=np.int8)


def f16_uniform(n, lo: float, hi: float, seed_offset: int) -> np.ndarray:
    """i.i.d. fp32 uniform on [lo, hi), rounded to fp16."""
    g = rng(seed_offset)
    out = np.empty(n, dtype=np.float16)
    flat = out.reshape(-1)
    step = 1 << 24
    for i in range(0, flat.size, step):           # chunked: keeps the fp32 temporary small
        m = min(step, flat.size - i)
        u = g.random(m, dtype=np.float32)
        flat[i:i + m] = (lo + (hi - lo) * u).astype(np.float16)
    return out


def bf16_normal(shape, seed_offset: int) -> np.ndarray:
    """i.i.d. standard normal fp32 draws rounded to bf16; uint16 bit patterns."""
    g = rng(seed_offset)
    out = np.empty(shape, dtype=np.uint16)
    flat = out.reshape(-1)
    step = 1 << 24
    for i in range(0, flat.size, step):
        m = min(step, flat.size - i)
        flat[i:i + m] = f32_to_bf16_bits(g.standard_normal(m, dtype=np.float32))
    return out


@dataclass(frozen=True)
class Config:
    """One build configuration: what is scanned and how."""
    name: str
    dtype: str              # "i8", "f16", "bf16"
    shape: Tuple[int, ...]  # (n,) or (rows, cols)
    s: Tuple[int, ...]      # tile sizes exercised
    exclusive: Tuple[bool, ...]
    index: int              # seed offset


CONFIGS = {
    "C1": Config("C1", "i8", (1 << 16,), (16,), (False,), 1),
    "C2": Config("C2", "f16", (1 << 24,), (16,), (False, True), 2),
    "C3": Config("C3", "i8", (1 << 28,), (16,), (False,), 3),
    "C4": Config("C4", "bf16", (4096, 65536), (16,), (False,), 4),
    "C5": Config("C5", "f16", (1 << 26,), (16, 64, 128), (False,), 5),
    # single-array 16-bit run of the headline size (the fp16 counterpart of C3)
    "C3h": Config("C3h", "f16", (1 << 28,), (16,), (False,), 6),
}


def make(cfg: Config, shape=None) -> np.ndarray:
    """Draw the input of a configuration (optionally at a reduced shape, same distribution)."""
    shape = cfg.shape if shape is None else tuple(shape)
    if cfg.name == "C1":
        return int8_uniform(shape, -8, 8, cfg.index)
    if cfg.name == "C2" or cfg.name == "C3h":
        return f16_uniform(shape, -1.0, 1.0, cfg.index)
    if cfg.name == "C3":
        return int8_uniform(shape, -127, 127, cfg.index)
    if cfg.name == "C4":
        return bf16_normal(shape, cfg.index)
    if cfg.name == "C5":
        return f16_uniform(shape, 0.0, 1.0, cfg.index)
    raise KeyError(cfg.name)
