"""Ozaki scheme I on base-13 E2M1 limbs (Section 4 of the paper).

Oracle code (test infrastructure).  Steps in the paper's order: shared-exponent integer
conversion with c = floor(log2 min(X_p, 2^53)) (Section 4.2), greedy decomposition into p limbs
(Lemma 1), the p x q limb products grouped along anti-diagonals i + j = g (Eq. 1, Fig. 2), the
weighted sum over the p + q - 1 groups, inverse scaling and one rounding.
"""
from __future__ import annotations

import math

import numpy as np

from .base13 import BASE, gap_free_range, greedy_limb_planes
from .ozaki2 import round_scaled_to_double, shared_shifts, to_integers


def capacity_bits_oz1(p: int) -> int:
    """Section 4.2: c = floor(log2 min(X_p, 2^53))."""
    return int(math.floor(math.log2(min(gap_free_range(p), 2 ** 53))))


def dgemm(A: np.ndarray, B: np.ndarray, p: int = 15, q: int = 15):
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    M, K = A.shape
    N = B.shape[1]
    c = min(capacity_bits_oz1(p), capacity_bits_oz1(q))
    s = shared_shifts(A, axis=1, c=c)
    t = shared_shifts(B, axis=0, c=c)
    At = to_integers(A, s, axis=1)
    Bt = to_integers(B, t, axis=0)
    a = [pl.astype(np.float64) for pl in greedy_limb_planes(At, p)]
    b = [pl.astype(np.float64) for pl in greedy_limb_planes(Bt, q)]
    # group sums G_g = sum_{i+j=g} a_i b_j; float64 matmuls are exact here: every partial sum is an
    # integer below min(p,q) * 64 * K << 2^53
    X = np.zeros((M, N), dtype=object)
    for g in range(p + q - 1):
        G = np.zeros((M, N), dtype=np.float64)
        for i in range(max(0, g - q + 1), min(p, g + 1)):
            G += a[i] @ b[g - i]
        X = X + np.rint(G).astype(np.int64).astype(object) * (BASE ** g)
    C = np.empty((M, N), dtype=np.float64)
    for i in range(M):
        for j in range(N):
            C[i, j] = round_scaled_to_double(int(X[i, j]), int(s[i] + t[j]))
    return C, X, At, Bt
