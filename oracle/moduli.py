"""Section 5.1 of the paper: two-limb representability, modulus selection,
CRT constants and the exactness bounds of Lemmas 2 and 3.

Oracle code (test infrastructure): exhaustive searches and Python integers.
"""
from __future__ import annotations

from math import gcd

from .base13 import BASE, S

# All values c0 + 13*c1 with c0, c1 in S, mapped to every limb pair giving them.
TWO_LIMB_PAIRS: dict[int, list[tuple[int, int]]] = {}
for _c1 in S:
    for _c0 in S:
        TWO_LIMB_PAIRS.setdefault(_c0 + BASE * _c1, []).append((_c0, _c1))


def is_two_limb_representable(m: int) -> bool:
    """Section 5.1: every residue class of m contains some c0 + 13*c1."""
    classes = {v % m for v in TWO_LIMB_PAIRS}
    return len(classes) == m


def representable_moduli(limit: int) -> list[int]:
    """All m in [2, limit] passing the representability condition."""
    return [m for m in range(2, limit + 1) if is_two_limb_representable(m)]


def select_moduli(count: int) -> list[int]:
    """Section 5.1: take 169 = 13^2 as the only multiple of 13, then choose
    greedily in descending order subject to pairwise coprimality."""
    chosen: list[int] = []
    for m in range(169, 1, -1):
        if len(chosen) == count:
            break
        if not is_two_limb_representable(m):
            continue
        if m != 169 and m % BASE == 0:
            continue
        if all(gcd(m, c) == 1 for c in chosen):
            chosen.append(m)
    if len(chosen) < count:
        raise ValueError(f"only {len(chosen)} moduli exist under the rule")
    return chosen


MAX_MODULI = 27          # the rule above is exhausted after 27 moduli


def limb_pair_table(m: int) -> list[tuple[int, int]]:
    """For each residue rho in [0, m) one limb pair (c0, c1) in S x S with
    c0 + 13*c1 = rho (mod m).  The paper fixes no choice among the valid pairs
    (it gives only 57 -> -58 = 13*(-4) - 6 for m = 115); this oracle takes the
    pair of smallest max(|c0|, |c1|), ties by |c0 + 13 c1|, then by (c1, c0)."""
    table = []
    for rho in range(m):
        best = None
        for v, pairs in TWO_LIMB_PAIRS.items():
            if (v - rho) % m:
                continue
            for (c0, c1) in pairs:
                key = (max(abs(c0), abs(c1)), abs(v), c1, c0)
                if best is None or key < best[0]:
                    best = (key, (c0, c1))
        if best is None:
            raise ValueError(f"class {rho} of {m} is not two-limb representable")
        table.append(best[1])
    return table


def limb_pair_table_karatsuba(m: int):
    """Section 5.1, last paragraph: a limb pair per residue class whose sum c0 + c1 is itself a doubled E2M1
    value, so that Karatsuba's third product (a0 + a1)(b0 + b1) can be formed from one more limb plane.  Returns
    None when some class of m has no such pair.  Among the valid pairs: smallest max(|c0|, |c1|), then |c0 + c1|,
    then (c1, c0)."""
    table = []
    for rho in range(m):
        best = None
        for v, pairs in TWO_LIMB_PAIRS.items():
            if (v - rho) % m:
                continue
            for (c0, c1) in pairs:
                if c0 + c1 not in S:
                    continue
                key = (max(abs(c0), abs(c1)), abs(c0 + c1), c1, c0)
                if best is None or key < best[0]:
                    best = (key, (c0, c1))
        if best is None:
            return None
        table.append(best[1])
    return table


def karatsuba_moduli(moduli) -> list[int]:
    """The moduli of the list that admit the Karatsuba form (the paper names 83, 73, 71, 67, 61, 59, 53 among its 19)."""
    return [m for m in moduli if limb_pair_table_karatsuba(m) is not None]


def product(moduli) -> int:
    P = 1
    for m in moduli:
        P *= int(m)
    return P


def crt_weights(moduli) -> tuple[int, list[int]]:
    """Section 5.2: P and w_i = M_i * (M_i^{-1} mod m_i), M_i = P / m_i."""
    P = product(moduli)
    weights = []
    for m in moduli:
        Mi = P // m
        weights.append(Mi * pow(Mi % m, -1, m))
    return P, weights


def capacity_bits(K: int, num_moduli: int, cap: int = 53) -> int:
    """Eq. 3 read for a general integer width c: the converted inputs satisfy
    |a| <= 2^c, so |sum| <= K * 2^(2c) and the signed reconstruction needs
    2K * 2^(2c) < P.  The width is additionally capped at 53 bits
    (Section 4.2: integers must be exact in FP64).  With the 19 printed moduli
    and K <= 16384 this gives the paper's 53."""
    P = product(select_moduli(num_moduli))
    c = 0
    while 2 * K * (1 << (2 * (c + 1))) < P:
        c += 1
    return min(cap, c)


# Lemma 2 and Lemma 3: closed-form limits on the inner-product length K.
def k_bound_partial_product(limb_max: int = 12) -> int:
    return (1 << 24) // (limb_max * limb_max)            # 144 K <= 2^24


def k_bound_cross_term(limb_max: int = 12) -> int:
    return (1 << 24) // (2 * limb_max * limb_max)        # 288 K <= 2^24


def k_bound_composition(limb_max: int = 12) -> int:
    return (1 << 31) // ((1 + 2 * BASE + BASE * BASE) * limb_max * limb_max)


def k_bound_crt(moduli, bits: int = 53) -> int:
    # 2 K 2^(2 bits) < P, strict.
    P = product(moduli)
    return (P - 1) // (2 << (2 * bits))


def k_bound_grouped(n_g: int, limb_max: int = 8) -> int:
    # Lemma 2, greedy limbs: n_g * 64 * K <= 2^24  <=>  K <= 2^18 / n_g.
    return (1 << 24) // (n_g * limb_max * limb_max)
