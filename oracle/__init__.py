"""CPU oracle for Ozaki scheme II on FP4 (base-13 E2M1 limbs).

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain restatement of the
paper's method that the CUDA library is checked against.  Only the tests, the
smoke entry and the benchmark's CPU-baseline leg may import it; the product
path never does, and nothing here imports the CUDA binding.

Modules
-------
base13   Section 3: the doubled E2M1 set S, Lemma 1, greedy limbs, INT8 emulation.
moduli   Section 5.1: two-limb representability, modulus selection, CRT weights,
         Lemma 2/3 bounds, Eq. 3 capacity.
ozaki2   Sections 4.2, 5.1, 5.2: shared-exponent conversion, residues through the
         four limb partial products, direct CRT, Garner cross-check, final rounding.
exact    Section 1: fl(AB), each inner product formed exactly and rounded once.

Parity pins: every function is pinned by tests run with -m "not gpu" against
values the paper prints, closed forms, brute force or an independent library
route; none is "parity unpinned" except the hardware byte formats (E2M1 nibble
codes and UE8M0 scale bytes), which only a GPU instruction can pin.
"""
