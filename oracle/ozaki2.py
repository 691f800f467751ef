"""Ozaki scheme II on base-13 E2M1 limbs, integer pipeline (Sections 4.2, 5.1, 5.2).

Oracle code (test infrastructure).  Matrices are numpy arrays indexed [row, col];
memory order is irrelevant here.  Steps follow the paper's order:

  1. shared-exponent integer conversion of the rows of A and columns of B (Sec. 4.2)
  2. residues mod each m_l, two limbs each, four limb partial products,
     residue composition (Sec. 5.1)
  3. single-pass direct CRT in integers, symmetric representative (Sec. 5.2)
  4. inverse scaling and one rounding to FP64 (Sec. 4.2)
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

from .base13 import BASE, S
from .moduli import capacity_bits, crt_weights, limb_pair_table, limb_pair_table_karatsuba, select_moduli


# ----------------------------------------------------------------------------
# Step 1 (Section 4.2): shared exponents and integer conversion
# ----------------------------------------------------------------------------
def floor_log2_abs(x: float) -> int:
    """e with 2^e <= |x| < 2^(e+1) for finite non-zero x (subnormals included)."""
    m, e = math.frexp(abs(x))          # |x| = m * 2^e, 0.5 <= m < 1
    return e - 1


def shared_shifts(A: np.ndarray, axis: int, c: int) -> np.ndarray:
    """Section 4.2: s_i = c - 1 - e_i with 2^e_i <= max|.| < 2^(e_i+1) taken over
    `axis` (axis=1: one shift per row; axis=0: one per column); an all-zero
    row or column gets 0."""
    amax = np.max(np.abs(A), axis=axis) if A.shape[axis] else np.zeros(A.shape[1 - axis])
    out = np.zeros(amax.shape, dtype=np.int64)
    for i, v in enumerate(amax):
        if not math.isfinite(v):
            raise ValueError("non-finite input")
        out[i] = 0 if v == 0.0 else c - 1 - floor_log2_abs(float(v))
    return out


def round_half_even_scaled(x: float, s: int) -> int:
    """round(x * 2^s) to the nearest integer, ties to even, computed exactly on
    the integer significand (the scaling is an exponent shift; only the rounding
    to an integer loses anything)."""
    if x == 0.0:
        return 0
    m, e = math.frexp(x)               # x = m * 2^e exactly
    mant = int(m * (1 << 53))          # exact 53-bit signed integer
    sh = e - 53 + s                    # x * 2^s = mant * 2^sh
    if sh >= 0:
        return mant << sh
    sh = -sh
    sign = -1 if mant < 0 else 1
    mant = abs(mant)
    q, r = mant >> sh, mant & ((1 << sh) - 1)
    half = 1 << (sh - 1)
    if r > half or (r == half and (q & 1)):
        q += 1
    return sign * q


def to_integers(A: np.ndarray, shifts: np.ndarray, axis: int) -> np.ndarray:
    """Section 4.2: A~ = round(A * 2^s) with one shift per row (axis=1) or per
    column (axis=0), as int64.  np.ldexp is an exact exponent shift here
    (|A * 2^s| <= 2^53, or < 2^62 in the extended-capacity mode of dgemm, both
    far inside the FP64 range; a result too small to be normal rounds to 0
    either way); np.rint rounds half to even and leaves values of 2^52 and
    above, which are integers already, unchanged."""
    sh = shifts.astype(np.int64)
    sh = sh[:, None] if axis == 1 else sh[None, :]
    scaled = np.ldexp(A, sh.astype(np.int32) if np.all(np.abs(sh) < 2 ** 31) else sh)
    return np.rint(scaled).astype(np.int64)


# ----------------------------------------------------------------------------
# Step 2 (Section 5.1): residues, limbs, partial products, composition
# ----------------------------------------------------------------------------
def residue_limb_planes(X: np.ndarray, m: int) -> tuple[np.ndarray, np.ndarray]:
    """rho = X mod m in [0, m), then rho = x0 + 13 x1 (mod m) with x0, x1 in S."""
    rho = np.mod(X, m)                                  # numpy: sign of divisor
    table = np.array(limb_pair_table(m), dtype=np.int64)
    return table[rho, 0], table[rho, 1]


def residue_product(At: np.ndarray, Bt: np.ndarray, m: int) -> np.ndarray:
    """r = (A~ B~) mod m in [0, m) composed from the four limb partial products
    ab = a0 b0 + 13 (a0 b1 + a1 b0) + 13^2 a1 b1 (mod m)   (Section 5.1).

    Each partial product is a matrix product of limbs with |c| <= 12.  It is
    evaluated with a float64 matmul, exact because every partial sum is an
    integer below 288*K << 2^53."""
    a0, a1 = (p.astype(np.float64) for p in residue_limb_planes(At, m))
    b0, b1 = (p.astype(np.float64) for p in residue_limb_planes(Bt, m))
    D0 = np.rint(a0 @ b0).astype(np.int64)
    D1 = np.rint(a0 @ b1 + a1 @ b0).astype(np.int64)
    D2 = np.rint(a1 @ b1).astype(np.int64)
    return np.mod(D0 + BASE * D1 + BASE * BASE * D2, m).astype(np.int64)


def residue_product_karatsuba(At: np.ndarray, Bt: np.ndarray, m: int) -> np.ndarray:
    """The same residue from three limb products (Section 5.1, last paragraph): with limb pairs whose sums
    a_s = a0 + a1, b_s = b0 + b1 are doubled E2M1 values again,
        a0 b1 + a1 b0 = a_s b_s - a0 b0 - a1 b1,
    so r = (D0 + 13 (Ds - D0 - D2) + 169 D2) mod m with D0 = a0 b0, D2 = a1 b1, Ds = a_s b_s summed over k.
    Only for the moduli moduli.karatsuba_moduli admits."""
    table = limb_pair_table_karatsuba(m)
    if table is None:
        raise ValueError(f"modulus {m} has residue classes without a Karatsuba limb pair")
    table = np.array(table, dtype=np.int64)
    ra, rb = np.mod(At, m), np.mod(Bt, m)
    a0, a1, b0, b1 = table[ra, 0], table[ra, 1], table[rb, 0], table[rb, 1]
    a_s, b_s = a0 + a1, b0 + b1
    assert np.isin(a_s, S).all() and np.isin(b_s, S).all()
    D0 = a0 @ b0                                            # int64 matrix products: |sum| <= 144 K
    D2 = a1 @ b1
    Ds = a_s @ b_s
    return np.mod(D0 + BASE * (Ds - D0 - D2) + BASE * BASE * D2, m).astype(np.int64)


# ----------------------------------------------------------------------------
# Step 3 (Section 5.2): direct CRT, and Garner's algorithm as a cross-check
# ----------------------------------------------------------------------------
def crt_direct(residues: list[np.ndarray], moduli: list[int]) -> np.ndarray:
    """x = (sum_l r_l w_l) mod P mapped to the symmetric range (x - P if x > P/2).
    Returns an object array of Python integers."""
    P, w = crt_weights(moduli)
    S = np.zeros(residues[0].shape, dtype=object)
    for r, wl in zip(residues, w):
        S = S + r.astype(object) * wl
    x = S % P
    flat = x.reshape(-1)
    for i in range(flat.size):
        if 2 * flat[i] > P:
            flat[i] -= P
    return x


def crt_quotients(residues: list[np.ndarray], moduli: list[int]) -> np.ndarray:
    """floor(S / P) for S = sum r_l w_l (the footnote of Section 5.2)."""
    P, w = crt_weights(moduli)
    S = np.zeros(residues[0].shape, dtype=object)
    for r, wl in zip(residues, w):
        S = S + r.astype(object) * wl
    return S // P


def garner_scalar(residues: list[int], moduli: list[int]) -> int:
    """Garner's mixed-radix reconstruction (Section 5.2, first paragraph),
    returning the symmetric representative.  Independent of crt_weights."""
    digits = []
    for i, (r, m) in enumerate(zip(residues, moduli)):
        # value so far: sum_j digits[j] * prod_{t<j} m_t ; solve for digit i mod m
        acc, rad = 0, 1
        for j in range(i):
            acc = (acc + digits[j] * rad) % m
            rad = (rad * moduli[j]) % m
        d = ((r - acc) * pow(rad, -1, m)) % m
        digits.append(d)
    x, rad = 0, 1
    for d, m in zip(digits, moduli):
        x += d * rad
        rad *= m
    return x - rad if 2 * x > rad else x


# ----------------------------------------------------------------------------
# Step 4 (Section 4.2): inverse scaling, one rounding
# ----------------------------------------------------------------------------
def round_scaled_to_double(x: int, shift: int) -> float:
    """RN_even(x * 2^-shift) as a double.  Python's int/int true division and
    int -> float conversion are correctly rounded (ties to even), so this is a
    single rounding of the exact rational."""
    x = int(x)
    if x == 0:
        return 0.0
    if shift >= 0:
        return x / (1 << shift)
    try:
        return float(x << (-shift))
    except OverflowError:            # beyond the FP64 range: IEEE 754 round-to-nearest gives +-infinity
        return math.copysign(math.inf, x)


@dataclass
class Ozaki2Result:
    C: np.ndarray
    moduli: list[int]
    c_bits: int
    s: np.ndarray
    t: np.ndarray
    At: np.ndarray
    Bt: np.ndarray
    residues: list[np.ndarray] = field(repr=False, default_factory=list)
    x: np.ndarray = field(repr=False, default=None)


MAX_EXTENDED_BITS = 62


def dgemm(A: np.ndarray, B: np.ndarray, num_moduli: int = 19, max_bits: int = 53) -> Ozaki2Result:
    """Emulated C = fl(AB) by Ozaki scheme II on base-13 limbs.

    max_bits = 53 is the paper's method (Section 4.2 caps the integer width at
    53 bits).  A larger max_bits (up to 62) is an EXTENSION the paper does not
    have: the same steps with the cap of the width c lifted, so that with more
    than 19 moduli Eq. 3 admits wider integers; the row or column maximum then
    converts without rounding and smaller entries keep up to max_bits - 53 more
    bits below it."""
    if not 1 <= max_bits <= MAX_EXTENDED_BITS:
        raise ValueError("max_bits must lie in 1..62 (converted integers are held in int64)")
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    moduli = select_moduli(num_moduli)
    c = capacity_bits(max(K, 1), num_moduli, cap=max_bits)
    s = shared_shifts(A, axis=1, c=c)
    t = shared_shifts(B, axis=0, c=c)
    At = to_integers(A, s, axis=1)
    Bt = to_integers(B, t, axis=0)
    residues = [residue_product(At, Bt, m) for m in moduli]
    x = crt_direct(residues, moduli)
    C = np.empty((M, N), dtype=np.float64)
    for i in range(M):
        for j in range(N):
            C[i, j] = round_scaled_to_double(x[i, j], int(s[i] + t[j]))
    return Ozaki2Result(C=C, moduli=moduli, c_bits=c, s=s, t=t, At=At, Bt=Bt,
                        residues=residues, x=x)
