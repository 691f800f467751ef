"""Partial Karatsuba variant (Section 5.1, last paragraph; Section 6.4) switched on: sum-limb planes from the encoder,
three products per Karatsuba modulus in the CTA-pair limb GEMM, the same residues and the same C bit for bit."""
import numpy as np
import pytest
import torch

from oracle import base13, moduli, ozaki2
from paper_2608_06812_b200 import binding as ozk
from paper_2608_06812_b200 import inputs
from tests import gpu_util as gu
from tests.test_gpu_stages import read_plane, run_preprocess

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def karatsuba_on():
    ozk.check(ozk.ozk_stage_set_karatsuba(True), "ozk_stage_set_karatsuba")
    yield
    ozk.check(ozk.ozk_stage_set_karatsuba(False), "ozk_stage_set_karatsuba")


def test_workspace_grows_by_the_sum_limb_planes():
    on = ozk.ozk_dgemm_workspace_bytes(1024, 1024, 2048, 19)            # K beyond the two-accumulator form, which has planes of its own
    ozk.ozk_stage_set_karatsuba(False)
    off = ozk.ozk_dgemm_workspace_bytes(1024, 1024, 2048, 19)
    ozk.ozk_stage_set_karatsuba(True)
    assert on - off == 7 * 2 * 1024 * 1024                              # seven more planes of 1024 x 2048 nibbles per operand
    assert ozk.ozk_dgemm_workspace_bytes(64, 64, 64, 11) == (ozk.ozk_stage_set_karatsuba(False), ozk.ozk_dgemm_workspace_bytes(64, 64, 64, 11),
                                                             ozk.ozk_stage_set_karatsuba(True))[1]   # no Karatsuba modulus among the first 11


@pytest.mark.parametrize("shape,L", [((130, 70, 300), 19), ((33, 257, 65), 27)])
def test_planes_and_sum_limbs(shape, L):
    M, N, K = shape
    A = inputs.lognormal_matrix(M, K, 1.0, seed=0)
    B = inputs.lognormal_matrix(K, N, 1.0, seed=1)
    s, t, At, Bt = run_preprocess(A, B, L)
    mods = moduli.select_moduli(L)
    kara = moduli.karatsuba_moduli(mods)
    for l, m in enumerate(mods):
        if l not in (0, 10, 11, 12, 13, L - 1):
            continue
        for op, X in (("A", At), ("B", Bt.T)):
            c0 = read_plane(op, M, N, K, L, l, 0)
            c1 = read_plane(op, M, N, K, L, l, 1)
            assert np.isin(c0, base13.S).all() and np.isin(c1, base13.S).all()
            assert max(np.abs(c0).max(), np.abs(c1).max()) <= 8
            assert np.all((c0 + 13 * c1 - X) % m == 0)
            if m in kara:
                cs = read_plane(op, M, N, K, L, l, 2)
                assert np.array_equal(cs, c0 + c1) and np.isin(cs, base13.S).all()
            else:
                out = torch.zeros((K, X.shape[0]), dtype=torch.int8, device="cuda")
                assert ozk.ozk_stage_read_planes(op, M, N, K, L, l, 2, out.data_ptr(), gu.stream()) == ozk.OZK_ERR_INVALID_ARG


@pytest.mark.parametrize("shape,L,phi", [((256, 256, 256), 14, 0.5), ((384, 512, 1000), 19, 1.0), ((128, 256, 2048), 27, 0.5),
                                         ((130, 70, 300), 19, 4.0)])
def test_residues_match_the_oracle(shape, L, phi):
    M, N, K = shape
    A = inputs.lognormal_matrix(M, K, phi, seed=0)
    B = inputs.lognormal_matrix(K, N, phi, seed=1)
    ref = ozaki2.dgemm(A, B, L)
    run_preprocess(A, B, L)
    dR = torch.full((L, N, M), 255, dtype=torch.uint8, device="cuda")
    ozk.check(ozk.ozk_stage_residue_gemm(M, N, K, L, dR.data_ptr(), gu.stream()), "residue_gemm")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    R = dR.cpu().numpy()
    mods = moduli.select_moduli(L)
    for l in range(L):
        assert np.array_equal(R[l].T.astype(np.int64), ref.residues[l]), f"modulus index {l}"
    for l, m in enumerate(mods):
        if m in moduli.karatsuba_moduli(mods) and l in (11, 13, L - 1):
            assert np.array_equal(R[l].T.astype(np.int64), ozaki2.residue_product_karatsuba(ref.At, ref.Bt, m))


@pytest.mark.parametrize("shape,L", [((256, 256, 256), 19), ((200, 300, 520), 19), ((128, 512, 20000), 19), ((64, 256, 70000), 20),
                                     ((96, 40, 200), 27), ((1, 1, 1), 12)])
def test_dgemm_bit_exact_with_the_variant_on(shape, L):
    """Pair kernel with fast and integer recombination (K beyond 17152), two k ranges (K beyond 65536 with the variant
    on), and shapes that fall back to the single-CTA kernel (which forms four products from the same planes)."""
    M, N, K = shape
    A = inputs.lognormal_matrix(M, K, 0.5, seed=40)
    B = inputs.lognormal_matrix(K, N, 0.5, seed=41)
    if M > 1:
        A[0, :] = np.abs(A[0, :])                       # no cancellation in one row / column: the largest partial sums
        B[:, 0] = np.abs(B[:, 0])
    assert gu.bits_equal(gu.dgemm(A, B, L), ozaki2.dgemm(A, B, L).C)


def test_variant_off_again_gives_the_same_result():
    A = inputs.lognormal_matrix(256, 512, 1.0, seed=1)
    B = inputs.lognormal_matrix(512, 256, 1.0, seed=2)
    on = gu.dgemm(A, B, 19)
    ozk.ozk_stage_set_karatsuba(False)
    off = gu.dgemm(A, B, 19)
    assert gu.bits_equal(on, off)
