"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke entry.

This module only draws random matrices; it contains none of the method's
arithmetic and imports neither the CUDA binding nor the CPU oracle.
All arrays are returned indexed [row, col] (C order); callers that need
column-major storage transpose on their side.
"""
from __future__ import annotations

import numpy as np


def lognormal_matrix(rows: int, cols: int, phi: float, seed: int) -> np.ndarray:
    """Entries (U - 0.5) * exp(phi * Z), U uniform on [0,1), Z standard normal:
    draw the whole U array first, then the whole Z array, from
    numpy.random.default_rng(seed).  FP64."""
    rng = np.random.default_rng(seed)
    U = rng.random((rows, cols))
    Z = rng.standard_normal((rows, cols))
    return (U - 0.5) * np.exp(phi * Z)


def exponent_spread_matrix(rows: int, cols: int, phi: int, seed: int) -> np.ndarray:
    """Entries +-(1 + u) * 2^e, u uniform on [0,1), e a uniform integer in
    {0..phi}: the test-matrix law of the paper's accuracy evaluation."""
    rng = np.random.default_rng(seed)
    u = rng.random((rows, cols))
    e = rng.integers(0, phi + 1, size=(rows, cols))
    sign = np.where(rng.random((rows, cols)) < 0.5, -1.0, 1.0)
    return sign * np.ldexp(1.0 + u, e.astype(np.int32))


def small_integer_matrix(rows: int, cols: int, bound: int, seed: int) -> np.ndarray:
    """FP64 matrix of uniform integers in [-bound, bound]."""
    rng = np.random.default_rng(seed)
    return rng.integers(-bound, bound + 1, size=(rows, cols)).astype(np.float64)


def int8_matrix(rows: int, cols: int, seed: int) -> np.ndarray:
    """int8 entries uniform on [-128, 127]."""
    rng = np.random.default_rng(seed)
    return rng.integers(-128, 128, size=(rows, cols), dtype=np.int8)
