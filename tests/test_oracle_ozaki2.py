"""Pins for oracle.ozaki2 and oracle.exact: brute force on tiny shapes, special
cases with closed-form answers, an independent decimal route for fl(AB), and the
accuracy levels the paper prints (tests/golden/paper_constants.json)."""
import decimal
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import base13, exact, moduli, ozaki2
from paper_2608_06812_b200 import inputs

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.json")))


# ---- step 1: shared exponents and integer conversion --------------------------------------
def test_shared_shifts_definition():
    A = np.array([[1.0, -3.5, 0.25], [0.0, 0.0, 0.0], [2.0 ** -1060, 0.0, 0.0], [1.999, 1.0, -2.0]])
    s = ozaki2.shared_shifts(A, axis=1, c=53)
    assert list(s) == [53 - 1 - 1, 0, 53 - 1 + 1060, 53 - 1 - 1]
    for i in (0, 2, 3):
        amax = np.abs(A[i]).max()
        scaled = Fraction(float(amax)) * Fraction(2) ** int(s[i])
        assert 2 ** 52 <= scaled < 2 ** 53                  # the row maximum fills c bits
    t = ozaki2.shared_shifts(A, axis=0, c=40)
    assert list(t) == [40 - 1 - 0, 40 - 1 - 1, 40 - 1 - 1]
    with pytest.raises(ValueError):
        ozaki2.shared_shifts(np.array([[np.inf]]), 1, 53)


def test_integer_conversion_is_exact_rne():
    # ties, negative values, tiny and huge exponents: scalar integer route ...
    cases = [(0.5, 0, 0), (1.5, 0, 2), (2.5, 0, 2), (-0.5, 0, 0), (-1.5, 0, -2), (0.75, 1, 2),
             (1.25, 1, 2), (1.75, 1, 4), (3.0, -1, 2), (5.0, -1, 2), (7.0, -1, 4), (2.0 ** -1074, 1074, 1),
             (2.0 ** -1074, 1073, 0), (3 * 2.0 ** -1074, 1073, 2), (1.0, 52, 2 ** 52), (-(2.0 ** 52 + 1), 0, -(2 ** 52 + 1))]
    for x, s, want in cases:
        assert ozaki2.round_half_even_scaled(x, s) == want, (x, s)
    # ... against exact rationals on random data ...
    rng = np.random.default_rng(11)
    X = (rng.random((6, 40)) - 0.5) * np.exp(4 * rng.standard_normal((6, 40)))
    for c in (20, 42, 53):
        s = ozaki2.shared_shifts(X, 1, c)
        I = ozaki2.to_integers(X, s, 1)
        assert np.abs(I).max() <= 2 ** c
        for i, j in np.ndindex(*X.shape):
            exactv = Fraction(float(X[i, j])) * Fraction(2) ** int(s[i])
            n = int(I[i, j])
            assert abs(exactv - n) <= Fraction(1, 2)
            if abs(exactv - n) == Fraction(1, 2):
                assert n % 2 == 0
            assert n == ozaki2.round_half_even_scaled(float(X[i, j]), int(s[i]))
    # column direction is the transpose of the row direction
    t = ozaki2.shared_shifts(X.T.copy(), 0, 53)
    assert np.array_equal(ozaki2.to_integers(X.T.copy(), t, 0), ozaki2.to_integers(X, t, 1).T)


def test_row_maximum_can_round_up_to_two_pow_c():
    x = np.array([[2.0 - 2.0 ** -52, 1.0]])
    s = ozaki2.shared_shifts(x, 1, 40)
    assert int(ozaki2.to_integers(x, s, 1)[0, 0]) == 2 ** 40


# ---- step 2: residues through the four limb products ---------------------------------------
@pytest.mark.parametrize("m", [169, 115, 112, 53, 11])
def test_residue_product_equals_bigint_product_mod_m(m):
    rng = np.random.default_rng(m)
    At = rng.integers(-2 ** 53, 2 ** 53, size=(5, 37), dtype=np.int64)
    Bt = rng.integers(-2 ** 53, 2 ** 53, size=(37, 4), dtype=np.int64)
    At[0, 0], Bt[0, 0] = 2 ** 53, -2 ** 53
    r = ozaki2.residue_product(At, Bt, m)
    ref = np.dot(At.astype(object), Bt.astype(object))
    assert r.min() >= 0 and r.max() < m
    for idx in np.ndindex(*r.shape):
        assert int(r[idx]) == int(ref[idx]) % m
    a0, a1 = ozaki2.residue_limb_planes(At, m)
    assert np.all((a0 + 13 * a1 - At) % m == 0)
    if m == 169:                                           # 13^2 = 0 (mod 169): the a1 b1 term drops
        b0, b1 = ozaki2.residue_limb_planes(Bt, m)
        r3 = np.mod(a0 @ b0 + 13 * (a0 @ b1 + a1 @ b0), m)
        assert np.array_equal(r3, r)


# ---- step 3: CRT ---------------------------------------------------------------------------
@pytest.mark.parametrize("L", [2, 5, 14, 19, 27])
def test_crt_direct_identity_garner_and_range(L):
    mods = moduli.select_moduli(L)
    P = moduli.product(mods)
    rng = np.random.default_rng(L)
    xs = [0, 1, -1, P // 2 - 1, -(P // 2) + 1] + [int(rng.integers(-2 ** 62, 2 ** 62)) * (P // 2 ** 63 + 1) % (P // 2) for _ in range(20)]
    xs = [x for x in xs if 2 * abs(x) < P]
    res = [np.array([x % m for x in xs], dtype=np.int64) for m in mods]
    got = ozaki2.crt_direct(res, mods)
    for k, x in enumerate(xs):
        assert int(got[k]) == x
        assert all((int(got[k]) - int(r[k])) % m == 0 for r, m in zip(res, mods))
        assert ozaki2.garner_scalar([int(r[k]) for r in res], mods) == x
    q = ozaki2.crt_quotients(res, mods)
    assert all(0 <= int(v) <= sum(m - 1 for m in mods) for v in q)


def test_max_quotient_footnote():
    mods = moduli.select_moduli(19)
    res = [np.array([m - 1], dtype=np.int64) for m in mods]
    assert int(ozaki2.crt_quotients(res, mods)[0]) == GOLD["section5_2_max_quotient"]


# ---- step 4: one rounding ------------------------------------------------------------------
def _rne_by_bits(x: int, shift: int) -> float:
    """Test-side rounding of x * 2^-shift by explicit bit manipulation."""
    if x == 0:
        return 0.0
    sign, n = (-1.0 if x < 0 else 1.0), abs(x)
    e = n.bit_length() - 1 - shift                         # value in [2^e, 2^(e+1))
    lsb = max(e - 52, -1074)                               # exponent of the last kept bit
    drop = lsb + shift                                     # bits of n below the kept ones
    if drop <= 0:
        q = n << (-drop)
    else:
        q, r = n >> drop, n & ((1 << drop) - 1)
        half = 1 << (drop - 1)
        if r > half or (r == half and (q & 1)):
            q += 1
    return sign * math.ldexp(float(q), lsb)                # q <= 2^53: exact


def test_single_rounding_against_bit_level_rne():
    rng = np.random.default_rng(2)
    for _ in range(2000):
        bits = int(rng.integers(1, 125))
        x = int(rng.integers(0, 2 ** 62)) ** 2 % (2 ** bits) * (1 if rng.random() < 0.5 else -1)
        shift = int(rng.integers(-40, 1200))
        assert ozaki2.round_scaled_to_double(x, shift) == _rne_by_bits(x, shift)
    # ties to even at 53 bits, and in the subnormal range
    assert ozaki2.round_scaled_to_double(2 ** 53 + 1, 0) == 2.0 ** 53
    assert ozaki2.round_scaled_to_double(2 ** 53 + 3, 0) == 2.0 ** 53 + 4
    assert ozaki2.round_scaled_to_double(3, 1075) == 2 * 2.0 ** -1074
    assert ozaki2.round_scaled_to_double(1, 1075) == 0.0
    assert ozaki2.round_scaled_to_double(-5, 1) == -2.5
    # overflow follows IEEE 754 round-to-nearest: the largest finite double, then infinity
    assert ozaki2.round_scaled_to_double(2 ** 53 - 1, -(1023 - 52)) == float.fromhex("0x1.fffffffffffffp+1023")
    assert ozaki2.round_scaled_to_double(2 ** 54 - 1, -(1023 - 53)) == math.inf
    assert ozaki2.round_scaled_to_double(-3, -1100) == -math.inf


# ---- fl(AB) --------------------------------------------------------------------------------
def _fl_matmul_decimal(A, B):
    ctx = decimal.Context(prec=6000, Emax=decimal.MAX_EMAX, Emin=decimal.MIN_EMIN)
    C = np.empty((A.shape[0], B.shape[1]))
    for i in range(A.shape[0]):
        for j in range(B.shape[1]):
            acc = decimal.Decimal(0)
            for k in range(A.shape[1]):
                acc = ctx.add(acc, ctx.multiply(decimal.Decimal(float(A[i, k])), decimal.Decimal(float(B[k, j]))))
            C[i, j] = float(acc)                            # correctly rounded string -> double
    return C


def test_fl_matmul_against_decimal_route_and_cancellation():
    rng = np.random.default_rng(7)
    A = (rng.random((4, 23)) - 0.5) * np.exp(6 * rng.standard_normal((4, 23)))
    B = (rng.random((23, 3)) - 0.5) * np.exp(6 * rng.standard_normal((23, 3)))
    assert np.array_equal(exact.fl_matmul(A, B), _fl_matmul_decimal(A, B))
    # catastrophic cancellation that a plain double sum loses
    a = np.array([[1e200, 1.0, -1e200, 2.0 ** -60]])
    b = np.array([[1e100], [3.0], [1e100], [1.0]])
    assert exact.fl_matmul(a, b)[0, 0] == 3.0 + 2.0 ** -60 == _fl_matmul_decimal(a, b)[0, 0]
    # error metric: a result off by one ulp of 1.0 on a sum of magnitude 4
    A1, B1 = np.array([[1.0, 1.0]]), np.array([[1.0], [-3.0]])
    err = exact.normwise_error(np.array([[-2.0 + 2.0 ** -51]]), A1, B1)
    assert err == 2.0 ** -51 / 4


# ---- whole pipeline ------------------------------------------------------------------------
@pytest.mark.parametrize("L", [2, 3, 8, 14, 19, 20, 27])
def test_pipeline_brute_force_tiny(L):
    rng = np.random.default_rng(100 + L)
    for (M, N, K) in [(1, 1, 1), (3, 2, 5), (8, 8, 8)]:
        A = (rng.random((M, K)) - 0.5) * np.exp(rng.standard_normal((M, K)))
        B = (rng.random((K, N)) - 0.5) * np.exp(rng.standard_normal((K, N)))
        A[0, 0] = 0.0
        r = ozaki2.dgemm(A, B, L)
        assert r.c_bits == moduli.capacity_bits(K, L)
        for i in range(M):
            for j in range(N):
                tot = sum(int(r.At[i, k]) * int(r.Bt[k, j]) for k in range(K))
                assert int(r.x[i, j]) == tot
                want = float(Fraction(tot) / Fraction(2) ** int(r.s[i] + r.t[j]))
                assert r.C[i, j] == want and math.copysign(1, r.C[i, j]) == math.copysign(1, want)


def test_small_integer_inputs_reduce_to_integer_gemm():
    A = inputs.small_integer_matrix(6, 50, 1000, seed=1)
    B = inputs.small_integer_matrix(50, 5, 1000, seed=2)
    A[2, :] = 0.0                                          # zero row: s = 0, output row exactly 0
    r = ozaki2.dgemm(A, B, 19)
    ref = A.astype(np.int64) @ B.astype(np.int64)
    assert np.array_equal(r.C, ref.astype(np.float64))
    assert r.s[2] == 0 and np.all(r.C[2] == 0.0) and not np.any(np.signbit(r.C[2]))


def test_phi0_paper_law_is_exact_and_reaches_58_bits():
    """Section 7.1: at phi = 0 the conversion is error-free, so the result is the
    exact product rounded once: 3.1e-18, 58.2 bits at K = 8192."""
    K = 8192
    A = inputs.exponent_spread_matrix(32, K, 0, seed=0)
    B = inputs.exponent_spread_matrix(K, 32, 0, seed=1)
    r = ozaki2.dgemm(A, B, 19)
    assert np.array_equal(r.C, exact.fl_matmul(A, B))
    err = exact.normwise_error(r.C, A, B)
    assert abs(-math.log2(err) - GOLD["section7_1_bits_phi0"]) < 0.6
    assert 0.5 * GOLD["section7_1_error_phi0"] < err < 1.1 * GOLD["section7_1_error_phi0"] * 1.05


def test_phi32_paper_law_accuracy_level():
    """Section 7.1: about 52.3 bits at phi = 32 (statistical: other seed, smaller block)."""
    K = 8192
    A = inputs.exponent_spread_matrix(12, K, 32, seed=0)
    B = inputs.exponent_spread_matrix(K, 12, 32, seed=1)
    r = ozaki2.dgemm(A, B, 19)
    bits = -math.log2(exact.normwise_error(r.C, A, B))
    assert abs(bits - GOLD["section7_1_bits_phi32"]) < 1.5


def test_config1_law_error_levels():
    """256-long inner products, phi = 0.5 law: L = 19 stays below 1e-15 normwise,
    fewer moduli keep fewer bits (Eq. 3 read for general L)."""
    A = inputs.lognormal_matrix(24, 256, 0.5, seed=0)
    B = inputs.lognormal_matrix(256, 24, 0.5, seed=1)
    errs = {L: exact.normwise_error(ozaki2.dgemm(A, B, L).C, A, B, against_rounded=True) for L in (14, 17, 19)}
    assert errs[19] <= 1e-15 and errs[17] <= 1e-15
    assert errs[14] > errs[17] >= errs[19] * 0.999


# ---- extended capacity (not in the paper: the 53-bit cap of Section 4.2 lifted) -------------------
@pytest.mark.parametrize("L,max_bits", [(20, 56), (22, 62), (27, 62)])
def test_extended_capacity_brute_force_tiny(L, max_bits):
    """Same pins as the paper's mode: x is the exact integer product of the converted inputs, C its
    single rounding; the width follows Eq. 3 with the new cap; entries within 2^(c-53) of their row
    or column maximum convert without any rounding."""
    rng = np.random.default_rng(7 * L + max_bits)
    for (M, N, K) in [(1, 1, 1), (3, 2, 5), (8, 8, 8)]:
        A = (rng.random((M, K)) - 0.5) * np.exp(2.0 * rng.standard_normal((M, K)))
        B = (rng.random((K, N)) - 0.5) * np.exp(2.0 * rng.standard_normal((K, N)))
        r = ozaki2.dgemm(A, B, L, max_bits=max_bits)
        assert r.c_bits == moduli.capacity_bits(K, L, cap=max_bits) and 53 < r.c_bits <= max_bits
        assert np.max(np.abs(r.At)) < 2 ** r.c_bits and np.max(np.abs(r.Bt)) < 2 ** r.c_bits
        for i in range(M):
            for k in range(K):
                want = Fraction(float(A[i, k])) * Fraction(2) ** int(r.s[i])
                if abs(A[i, k]) * 2.0 ** (r.c_bits - 53) >= np.max(np.abs(A[i])):
                    assert Fraction(int(r.At[i, k])) == want          # no rounding near the maximum
                else:
                    assert abs(Fraction(int(r.At[i, k])) - want) <= Fraction(1, 2)
            for j in range(N):
                tot = sum(int(r.At[i, k]) * int(r.Bt[k, j]) for k in range(K))
                assert int(r.x[i, j]) == tot
                assert r.C[i, j] == float(Fraction(tot) / Fraction(2) ** int(r.s[i] + r.t[j]))


def test_extended_capacity_default_is_the_papers_mode_and_range_is_checked():
    A = inputs.lognormal_matrix(5, 40, 1.0, seed=3)
    B = inputs.lognormal_matrix(40, 4, 1.0, seed=4)
    assert np.array_equal(ozaki2.dgemm(A, B, 22).C, ozaki2.dgemm(A, B, 22, max_bits=53).C)
    assert moduli.capacity_bits(16384, 19, cap=62) == 54 and moduli.capacity_bits(16384, 22, cap=62) == 62   # Eq. 3 still limits c
    with pytest.raises(ValueError):
        ozaki2.dgemm(A, B, 22, max_bits=63)


def test_extended_capacity_recovers_bits_on_wide_exponent_ranges():
    """At phi = 4 the paper's mode saturates at L = 19 (53-bit cap); each further modulus of the
    extended mode keeps about three more bits of the small entries."""
    A = inputs.lognormal_matrix(16, 512, 4.0, seed=0)
    B = inputs.lognormal_matrix(512, 16, 4.0, seed=1)
    err = {(L, mb): exact.normwise_error(ozaki2.dgemm(A, B, L, max_bits=mb).C, A, B, against_rounded=True)
           for (L, mb) in [(19, 53), (22, 53), (20, 62), (21, 62), (22, 62)]}
    assert err[(22, 53)] == err[(19, 53)]
    assert err[(20, 62)] < err[(19, 53)] / 16 and err[(21, 62)] < err[(20, 62)] / 2   # c = 59, then 62
    assert err[(22, 62)] == err[(21, 62)]                                             # the int64 cap


# ---- scheme I (Section 4) ---------------------------------------------------------------------
def test_scheme1_equals_integer_product_and_scheme2_bit_for_bit():
    """Section 7.1: both schemes compute the exact product of the same converted integers and round
    once, so their outputs agree bit for bit; c = floor(log2 min(X_15, 2^53)) = 53."""
    from oracle import ozaki1
    assert ozaki1.capacity_bits_oz1(15) == 53 and ozaki1.capacity_bits_oz1(14) == 50
    rng = np.random.default_rng(21)
    A = (rng.random((9, 70)) - 0.5) * np.exp(2 * rng.standard_normal((9, 70)))
    B = (rng.random((70, 7)) - 0.5) * np.exp(2 * rng.standard_normal((70, 7)))
    A[3, :] = 0.0
    C1, X1, At, Bt = ozaki1.dgemm(A, B)
    ref = np.dot(At.astype(object), Bt.astype(object))
    assert all(int(X1[idx]) == int(ref[idx]) for idx in np.ndindex(*X1.shape))
    C2 = ozaki2.dgemm(A, B, 19).C
    assert np.array_equal(C1.view(np.uint64), C2.view(np.uint64))


def test_limb_products_through_float64_are_exact_at_the_headline_k():
    """The oracle forms the four limb products with float64 matrix products (magnitudes 288 K << 2^53, so exact).
    At K = 16384, with adversarial limbs of one sign as well as random ones, they equal Python big-integer sums."""
    K = 16384
    rng = np.random.default_rng(5)
    for m in (169, 115, 53):
        for kind in ("random", "extreme"):
            if kind == "random":
                At = rng.integers(-2 ** 52, 2 ** 52, size=(3, K), dtype=np.int64)
                Bt = rng.integers(-2 ** 52, 2 ** 52, size=(K, 2), dtype=np.int64)
            else:                                                  # every residue the same: limb sums of one sign
                At = np.full((3, K), 2 ** 52 - 1, dtype=np.int64)
                Bt = np.full((K, 2), 2 ** 52 - 3, dtype=np.int64)
            got = ozaki2.residue_product(At, Bt, m)
            want = np.array([[sum(int(At[i, k]) * int(Bt[k, j]) for k in range(K)) % m for j in range(2)] for i in range(3)])
            assert np.array_equal(np.asarray(got, dtype=np.int64), want), (m, kind)


def test_karatsuba_moduli_are_the_papers_seven():
    """Section 5.1, last paragraph: among the 19 moduli exactly 83, 73, 71, 67, 61, 59, 53 have, in every residue
    class, a limb pair whose sum is representable too (68 products instead of 75)."""
    mods = moduli.select_moduli(19)
    assert moduli.karatsuba_moduli(mods) == [83, 73, 71, 67, 61, 59, 53]
    assert 4 * 19 - 1 - len(moduli.karatsuba_moduli(mods)) == 68
    # the continuation of the list (47 ... 11) admits it as well; 79 and everything above 83 does not
    assert moduli.karatsuba_moduli(moduli.select_moduli(27)) == [83, 73, 71, 67, 61, 59, 53, 47, 43, 41, 31, 29, 19, 17, 11]
    for m in (83, 53, 11):
        for rho, (c0, c1) in enumerate(moduli.limb_pair_table_karatsuba(m)):
            assert c0 in base13.S and c1 in base13.S and c0 + c1 in base13.S and (c0 + 13 * c1 - rho) % m == 0
            assert max(abs(c0), abs(c1)) <= 8                          # sum limbs reach 12, the limbs themselves 8


def test_karatsuba_residue_product_equals_the_four_product_form():
    rng = np.random.default_rng(8)
    At = rng.integers(-2 ** 52, 2 ** 52, size=(5, 300), dtype=np.int64)
    Bt = rng.integers(-2 ** 52, 2 ** 52, size=(300, 4), dtype=np.int64)
    for m in (83, 73, 71, 67, 61, 59, 53, 11):
        got = ozaki2.residue_product_karatsuba(At, Bt, m)
        assert np.array_equal(got, ozaki2.residue_product(At, Bt, m))
        want = np.array([[sum(int(At[i, k]) * int(Bt[k, j]) for k in range(300)) % m for j in range(4)] for i in range(5)])
        assert np.array_equal(got, want)
    with pytest.raises(ValueError):
        ozaki2.residue_product_karatsuba(At, Bt, 79)
