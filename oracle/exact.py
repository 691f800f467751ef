"""Section 1 of the paper: the ideal output fl(AB), every inner product formed
exactly and rounded once to nearest (ties to even), and the normwise error
metric of Section 7.1.

Oracle code (test infrastructure): exact big-integer arithmetic.
"""
from __future__ import annotations

from fractions import Fraction

import numpy as np


def decompose(X: np.ndarray) -> tuple[np.ndarray, int]:
    """X = I * 2^e elementwise with I an object array of Python integers and e
    one common exponent."""
    X = np.asarray(X, dtype=np.float64)
    if not np.all(np.isfinite(X)):
        raise ValueError("non-finite input")
    mant, exp = np.frexp(X)                              # X = mant * 2^exp
    imant = np.ldexp(mant, 53).astype(np.int64)          # exact 53-bit integers
    e = exp.astype(np.int64) - 53
    nz = imant != 0
    emin = int(e[nz].min()) if nz.any() else 0
    up = np.where(nz, e - emin, 0)
    I = np.empty(X.shape, dtype=object)
    fi, fm, fu = I.reshape(-1), imant.reshape(-1), up.reshape(-1)
    for idx in range(fi.size):
        fi[idx] = int(fm[idx]) << int(fu[idx])
    return I, emin


def exact_products(A: np.ndarray, B: np.ndarray) -> tuple[np.ndarray, int]:
    """(AB)_ij = N_ij * 2^e exactly; N is an object array of Python integers."""
    IA, ea = decompose(A)
    IB, eb = decompose(B)
    return np.dot(IA, IB), ea + eb


def round_int_scaled(n: int, e: int) -> float:
    """RN_even(n * 2^e) as a double (single rounding; int/int and int -> float
    are correctly rounded in Python)."""
    n = int(n)
    if n == 0:
        return 0.0
    return float(n << e) if e >= 0 else n / (1 << (-e))


def fl_matmul(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """fl(AB): each element of the exact product rounded once."""
    N, e = exact_products(A, B)
    C = np.empty(N.shape, dtype=np.float64)
    fc, fn = C.reshape(-1), N.reshape(-1)
    for idx in range(fc.size):
        fc[idx] = round_int_scaled(fn[idx], e)
    return C


def normwise_error(C: np.ndarray, A: np.ndarray, B: np.ndarray,
                   against_rounded: bool = False) -> float:
    """Section 7.1: max_ij |C_ij - (AB)_ij| / sum_k |A_ik||B_kj|, the reference
    being the exact product (or its single rounding fl(AB) if asked)."""
    N, e = exact_products(A, B)
    D, _ = exact_products(np.abs(A), np.abs(B))
    worst = Fraction(0)
    for idx in np.ndindex(*N.shape):
        den = int(D[idx])
        if den == 0:
            continue
        ref = Fraction(int(N[idx])) * Fraction(2) ** e
        if against_rounded:
            ref = Fraction(round_int_scaled(N[idx], e))
        err = abs(Fraction(float(C[idx])) - ref) / (Fraction(den) * Fraction(2) ** e)
        if err > worst:
            worst = err
    return float(worst)
