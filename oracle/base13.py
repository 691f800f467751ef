"""Section 3 of the paper: base-13 limbs over the doubled E2M1 value set.

Oracle code (test infrastructure): plain Python integers, no blocking.
"""
from __future__ import annotations

import numpy as np

# Section 3: the eight non-negative E2M1 magnitudes, in code order 0..7
# (1 sign bit, 2 exponent bits, 1 mantissa bit).
E2M1_MAGNITUDES = (0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0)

# Section 3: doubling every E2M1 value gives the integer set S.
S_POSITIVE = tuple(int(2 * v) for v in E2M1_MAGNITUDES)          # 0,1,2,3,4,6,8,12
S = tuple(sorted(set(S_POSITIVE) | {-v for v in S_POSITIVE}))

BASE = 13


def gap_free_range(p: int) -> int:
    """Lemma 1: p limbs represent every |N| <= X_p = (13^p - 1)/3 without gaps."""
    return (BASE ** p - 1) // 3


def greedy_digit(n: int) -> int:
    """Lemma 1 / Lemma 2: the representative of n mod 13 of smallest magnitude
    (|c| <= 6), with +-5 (not in S) replaced by -+8 of the same class."""
    r = n % BASE                      # Python: 0..12
    if r > 6:
        r -= BASE                     # -6..6
    if r == 5:
        r = -8
    elif r == -5:
        r = 8
    return r


def greedy_limbs(n: int, p: int) -> list[int]:
    """Lemma 1: n = sum_i 13^i c_i with c_i in S by the greedy recursion
    (take the digit, recurse on the exact quotient).  Raises if p limbs do not
    suffice."""
    limbs = []
    q = int(n)
    for _ in range(p):
        c = greedy_digit(q)
        limbs.append(c)
        q = (q - c) // BASE           # exact: q - c is a multiple of 13
    if q != 0:
        raise OverflowError(f"{n} does not fit {p} greedy limbs")
    return limbs


def limbs_value(limbs) -> int:
    """Positional value sum_i 13^i c_i."""
    return sum(int(c) * BASE ** i for i, c in enumerate(limbs))


def e2m1_code(c: int) -> int:
    """4-bit E2M1 code storing the limb c as the value c/2 (Section 3):
    bit 3 = sign, bits 2..0 = index into E2M1_MAGNITUDES."""
    mag = S_POSITIVE.index(abs(int(c)))
    return (8 if c < 0 else 0) | mag


def e2m1_decode_doubled(code: int) -> int:
    """Inverse of e2m1_code: twice the E2M1 value of a 4-bit code."""
    v = S_POSITIVE[code & 7]
    return -v if code & 8 else v


def greedy_limb_planes(X: np.ndarray, p: int) -> list[np.ndarray]:
    """Elementwise greedy decomposition of an int64 array into p limb planes
    (the recursion of greedy_limbs, written on whole arrays)."""
    q = np.asarray(X, dtype=np.int64).copy()
    planes = []
    for _ in range(p):
        r = np.mod(q, BASE)                       # 0..12
        r = np.where(r > 6, r - BASE, r)          # -6..6
        r = np.where(r == 5, -8, np.where(r == -5, 8, r))
        planes.append(r.astype(np.int64))
        q = (q - r) // BASE
    if np.any(q != 0):
        raise OverflowError(f"values do not fit {p} greedy limbs")
    return planes


def igemm_i8_by_limbs(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """Section 3 (last paragraph) with Eq. 1: INT8 x INT8 -> INT32 GEMM from
    p = q = 3 greedy limbs and 9 limb products weighted by 13^(i+j).

    Each limb product is an integer matrix product of values |c| <= 8; it is
    evaluated with a float64 matmul, which is exact here because every partial
    sum is an integer below 64*K << 2^53.
    """
    A = np.asarray(A, dtype=np.int64)
    B = np.asarray(B, dtype=np.int64)
    a = [pl.astype(np.float64) for pl in greedy_limb_planes(A, 3)]
    b = [pl.astype(np.float64) for pl in greedy_limb_planes(B, 3)]
    C = np.zeros((A.shape[0], B.shape[1]), dtype=np.int64)
    for i in range(3):
        for j in range(3):
            G = a[i] @ b[j]
            C += BASE ** (i + j) * np.rint(G).astype(np.int64)
    # INT32 output: exact while K * 2^14 < 2^31.
    return C.astype(np.int32)


def igemm_i8_definition(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """The plain definition C_ij = sum_k A_ik B_kj in 64-bit integers."""
    return (np.asarray(A, dtype=np.int64) @ np.asarray(B, dtype=np.int64))
