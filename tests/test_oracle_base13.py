"""Pins for oracle.base13 and oracle.moduli against what the paper prints
(tests/golden/paper_constants.json) and brute force."""
import itertools
import json
import math
import os

import numpy as np
import pytest

from oracle import base13, moduli

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_constants.json")))


def test_value_sets_match_section3():
    assert list(base13.E2M1_MAGNITUDES) == GOLD["section3_e2m1_values"]
    assert list(base13.S_POSITIVE) == GOLD["section3_doubled_set_S"]
    assert len(base13.S) == 15 and all(-v in base13.S for v in base13.S)
    # every doubled E2M1 value is an integer
    assert all(float(2 * v).is_integer() for v in base13.E2M1_MAGNITUDES)


def test_lemma1_every_class_mod13_covered_and_redundancy():
    reps = {}
    for c in base13.S:
        reps.setdefault(c % 13, []).append(c)
    assert sorted(reps) == list(range(13))
    assert sorted(k for k, v in reps.items() if len(v) > 1) == GOLD["lemma1_redundant_classes_mod13"]
    assert sorted(reps[1]) == [-12, 1] and sorted(reps[12]) == [-1, 12]


@pytest.mark.parametrize("p", [1, 2, 3, 4, 5])
def test_lemma1_gap_free_range_by_brute_force(p):
    X = base13.gap_free_range(p)
    if str(p) in GOLD["lemma1_gap_free_X"]:
        assert X == GOLD["lemma1_gap_free_X"][str(p)]
    # brute force: the set of all p-limb values (any limbs in S), p <= 4
    if p <= 4:
        values = {0}
        for i in range(p):
            values = {v + 13 ** i * c for v in values for c in base13.S}
        assert all(n in values for n in range(-X, X + 1))
        assert (X + 1) not in values          # the first gap sits right after X_p
    # greedy succeeds on the whole range, round-trips, keeps |c| <= 8
    for n in range(-X, X + 1) if p <= 4 else range(-X, X + 1, 97):
        limbs = base13.greedy_limbs(n, p)
        assert base13.limbs_value(limbs) == n
        assert all(c in base13.S and abs(c) <= GOLD["lemma2_greedy_limb_abs_max"] for c in limbs)
    with pytest.raises(OverflowError):
        base13.greedy_limbs(X + 1, p)
    with pytest.raises(OverflowError):
        base13.greedy_limbs(-X - 1, p)


def test_limb_counts_section4_1():
    need = lambda bits: next(p for p in range(1, 40) if base13.gap_free_range(p) >= 2 ** bits - 1)
    # INT8 magnitudes up to 128, FP32 24-bit and FP64 53-bit significands
    assert next(p for p in range(1, 9) if base13.gap_free_range(p) >= 128) == 3
    assert [3, need(24), need(53)] == GOLD["section4_1_limbs_int8_fp32_fp64"]
    assert 15 * 15 == 225


def test_int8_round_trip_and_codes():
    for n in range(-128, 128):
        limbs = base13.greedy_limbs(n, 3)
        assert base13.limbs_value(limbs) == n
        for c in limbs:
            code = base13.e2m1_code(c)
            assert 0 <= code < 16 and base13.e2m1_decode_doubled(code) == c
    # code table: magnitude index in the E2M1 order, bit 3 the sign
    assert [base13.e2m1_code(c) for c in (0, 1, 2, 3, 4, 6, 8, 12)] == list(range(8))
    assert base13.e2m1_code(-8) == 8 + 6


def test_vector_planes_equal_scalar_greedy():
    rng = np.random.default_rng(3)
    X = rng.integers(-732, 733, size=(7, 11))
    planes = base13.greedy_limb_planes(X, 3)
    for idx in np.ndindex(*X.shape):
        assert [int(pl[idx]) for pl in planes] == base13.greedy_limbs(int(X[idx]), 3)


def test_int8_gemm_by_limbs_is_exact():
    rng = np.random.default_rng(5)
    A = rng.integers(-128, 128, size=(9, 200), dtype=np.int8)
    B = rng.integers(-128, 128, size=(200, 6), dtype=np.int8)
    A[0, :] = -128
    B[:, 0] = -128                                   # extreme corner
    ref = np.zeros((9, 6), dtype=np.int64)
    for i in range(9):
        for j in range(6):
            ref[i, j] = sum(int(A[i, k]) * int(B[k, j]) for k in range(200))
    assert np.array_equal(base13.igemm_i8_definition(A, B), ref)
    assert np.array_equal(base13.igemm_i8_by_limbs(A, B).astype(np.int64), ref)


def test_lemma2_and_lemma3_bounds():
    assert moduli.k_bound_partial_product() == GOLD["lemma2_K_bound_144"] == GOLD["lemma3_K_bounds"]["partial"]
    assert moduli.k_bound_cross_term() == GOLD["lemma3_K_bounds"]["cross"]
    assert moduli.k_bound_composition() == GOLD["lemma3_K_bounds"]["composition"]
    assert moduli.k_bound_crt(moduli.select_moduli(19)) == GOLD["lemma3_K_bounds"]["crt"]
    assert moduli.k_bound_grouped(15) == GOLD["lemma2_K_bound_deepest_group_ng15"]
    assert (1 + 2 * 13 + 169) * 144 == 28224


def test_representable_moduli_section5_1():
    rep = moduli.representable_moduli(400)
    small = GOLD["section5_1_all_below_or_equal"]
    assert [m for m in rep if m <= small] == list(range(2, small + 1))
    assert [m for m in rep if m > small] == GOLD["section5_1_exceptional_moduli"]
    # the printed example: class 57 of 115 needs -58 = 13*(-4) - 6
    ex = GOLD["section5_1_example_m115_class57"]
    assert 57 not in moduli.TWO_LIMB_PAIRS
    assert (ex["c0"], ex["c1"]) in moduli.TWO_LIMB_PAIRS[ex["representative"]]
    assert ex["representative"] % 115 == 57


def test_modulus_selection_matches_printed_list():
    sel = moduli.select_moduli(19)
    assert sel == GOLD["section5_1_moduli_L19"]
    for a, b in itertools.combinations(sel, 2):
        assert math.gcd(a, b) == 1
    P = moduli.product(sel)
    assert round(math.log2(P)) == GOLD["section5_1_log2_P_approx"]
    assert 2 * 16384 * 2 ** 106 < P                       # Eq. 3 at K = 16384
    assert 4 * len(sel) - 1 == GOLD["section5_1_gemm_count"]
    # prefixes and the continuation are deterministic and pairwise coprime
    full = moduli.select_moduli(moduli.MAX_MODULI)
    assert full[:19] == sel and len(set(full)) == moduli.MAX_MODULI
    for a, b in itertools.combinations(full, 2):
        assert math.gcd(a, b) == 1
    with pytest.raises(ValueError):
        moduli.select_moduli(moduli.MAX_MODULI + 1)


def test_best_18_subset_cannot_reach_2_pow_121():
    """Section 5.1: the best product of 18 pairwise-coprime representable moduli
    is 2^117.80, so L = 19 is minimal at K = 16384.  Branch and bound."""
    cands = sorted(moduli.representable_moduli(200), reverse=True)
    logs = {m: math.log2(m) for m in cands}
    best = [0.0]

    def dfs(start, chosen, acc):
        k = len(chosen)
        if k == 18:
            best[0] = max(best[0], acc)
            return
        # bound: the (18-k) largest remaining candidates coprime to the chosen set
        rest = [m for m in cands[start:] if all(math.gcd(m, c) == 1 for c in chosen)]
        if len(rest) < 18 - k:
            return
        if acc + sum(logs[m] for m in rest[:18 - k]) <= best[0] + 1e-12:
            return
        for m in rest:
            dfs(cands.index(m) + 1, chosen + [m], acc + logs[m])

    dfs(0, [], 0.0)
    assert abs(best[0] - GOLD["section5_1_best_18_log2"]) < 0.005
    assert best[0] < 121


def test_limb_pair_tables_cover_every_class_with_small_limbs():
    for m in moduli.select_moduli(moduli.MAX_MODULI):
        table = moduli.limb_pair_table(m)
        assert len(table) == m
        for rho, (c0, c1) in enumerate(table):
            assert c0 in base13.S and c1 in base13.S
            assert (c0 + 13 * c1 - rho) % m == 0
            # every class of every selected modulus has a pair with |c| <= 8,
            # which tightens the 144/288 products of Lemma 3 to 64/128
            assert max(abs(c0), abs(c1)) <= 8


def test_crt_weights_identity_and_footnote_constants():
    sel = moduli.select_moduli(19)
    P, w = moduli.crt_weights(sel)
    for i, (m, wi) in enumerate(zip(sel, w)):
        assert wi % m == 1
        assert all(wi % other == 0 for j, other in enumerate(sel) if j != i)
        assert wi < 2 ** 128
    assert sum(m - 1 for m in sel) == GOLD["section5_2_sum_m_minus_1"]
    Smax = sum((m - 1) * wi for m, wi in zip(sel, w))
    assert Smax // P == GOLD["section5_2_max_quotient"]
    assert Smax < 2 ** GOLD["section5_2_S_below_2_pow"]


def test_capacity_bits_eq3():
    assert moduli.capacity_bits(16384, 19) == 53
    assert moduli.capacity_bits(8192, 19) == 53
    # definition re-checked from the inequality for a sweep
    for K in (1, 256, 4096, 16384, 70000):
        for L in range(4, 24):
            P = moduli.product(moduli.select_moduli(L))
            c = moduli.capacity_bits(K, L, cap=10 ** 6)
            assert 2 * K * 4 ** c < P <= 2 * K * 4 ** (c + 1)
    assert moduli.capacity_bits(256, 14) == 42 and moduli.capacity_bits(16384, 18) == 51
