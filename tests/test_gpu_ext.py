"""ozk_dgemm_ext (extended capacity: the 53-bit cap of the converted integers lifted to at most 62 bits, an
extension the paper does not have) against the CPU oracle's max_bits mode, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import exact, moduli, ozaki2
from paper_2608_06812_b200 import binding as ozk
from paper_2608_06812_b200 import inputs
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("L,max_bits,phi", [(20, 56, 1.0), (20, 57, 1.0), (21, 60, 4.0), (22, 62, 4.0), (24, 62, 0.5),
                                            (27, 62, 4.0), (19, 62, 1.0), (22, 54, 2.0)])
def test_extended_capacity_bit_exact(L, max_bits, phi):
    """Widths on both sides of the 56-bit boundary where the encoder takes a fifth piece, several tiles, ragged edges."""
    M, N, K = 150, 300, 260
    A = inputs.lognormal_matrix(M, K, phi, seed=L)
    B = inputs.lognormal_matrix(K, N, phi, seed=max_bits)
    ref = ozaki2.dgemm(A, B, L, max_bits=max_bits)
    assert ref.c_bits == ozk.ozk_capacity_bits_ext(K, L, max_bits)
    assert gu.bits_equal(gu.dgemm(A, B, L, lda=M + 1, ldb=K + 3, ldc=M + 2, max_bits=max_bits), ref.C)


def test_extended_capacity_long_inner_product_and_extreme_exponents():
    """K beyond the fast recombination limit at the full 62 bits, with rows scaled across the FP64 exponent range."""
    M, N, K, L = 40, 128, 20000, 22
    A = inputs.lognormal_matrix(M, K, 1.0, seed=1)
    B = inputs.lognormal_matrix(K, N, 1.0, seed=2)
    A[3, :] *= 2.0 ** 300
    A[4, :] *= 2.0 ** -400
    B[:, 5] *= 2.0 ** -500
    ref = ozaki2.dgemm(A, B, L, max_bits=62)
    assert ref.c_bits == 62
    assert gu.bits_equal(gu.dgemm(A, B, L, max_bits=62), ref.C)


def test_max_bits_53_is_ozk_dgemm_and_bad_values_are_rejected():
    A = inputs.lognormal_matrix(70, 200, 2.0, seed=8)
    B = inputs.lognormal_matrix(200, 90, 2.0, seed=9)
    assert gu.bits_equal(gu.dgemm(A, B, 22, max_bits=53), gu.dgemm(A, B, 22))
    gu.register_small_workspace(8 << 20)
    for bad in (0, -1, 63, 64):
        assert ozk.ozk_dgemm_ext(8, 8, 8, None, 8, None, 8, None, 8, 22, bad, gu.stream()) == ozk.OZK_ERR_INVALID_ARG
    assert ozk.ozk_dgemm_ext(8, 8, 8, None, 8, None, 8, None, 8, 22, 62, gu.stream()) == ozk.OZK_ERR_INVALID_ARG   # null pointers


def test_extended_capacity_4096_phi4_samples_and_error():
    """M=N=K=4096 at phi = 4, where the paper's mode saturates near 1e-11: 22 moduli at 62 bits against the oracle on
    a 128 x 128 block plus scattered rows and columns, and the error against fl(AB) at least 100 times smaller."""
    n, L = 4096, 22
    A = inputs.lognormal_matrix(n, n, 4.0, seed=0)
    B = inputs.lognormal_matrix(n, n, 4.0, seed=1)
    dA = torch.from_numpy(np.ascontiguousarray(A.T)).cuda()
    dB = torch.from_numpy(np.ascontiguousarray(B.T)).cuda()
    gu.ensure_workspace(ozk.ozk_dgemm_workspace_bytes(n, n, n, L))
    rng = np.random.default_rng(4)
    rows = np.concatenate([np.arange(128), np.sort(rng.choice(np.arange(128, n), 24, replace=False))])
    cols = np.concatenate([np.arange(128), np.sort(rng.choice(np.arange(128, n), 24, replace=False))])
    got = {}
    for max_bits in (53, 62):
        dC = torch.empty((n, n), dtype=torch.float64, device="cuda")
        ozk.check(ozk.ozk_dgemm_ext(n, n, n, dA.data_ptr(), n, dB.data_ptr(), n, dC.data_ptr(), n, L, max_bits, gu.stream()), "ext")
        ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
        got[max_bits] = dC[torch.from_numpy(cols).cuda()][:, torch.from_numpy(rows).cuda()].cpu().numpy().T
        assert gu.bits_equal(got[max_bits], ozaki2.dgemm(A[rows], B[:, cols], L, max_bits=max_bits).C)
    assert moduli.capacity_bits(n, L, cap=62) == 62
    err = {mb: exact.normwise_error(got[mb][:16, :16], A[rows[:16]], B[:, cols[:16]], against_rounded=True) for mb in (53, 62)}
    assert err[62] < err[53] / 100


def test_extended_capacity_with_two_k_ranges():
    """K beyond one limb-GEMM range in the extended mode: residues of the two ranges are added modulo m."""
    M, N, K, L = 16, 64, 135000, 22
    A = inputs.lognormal_matrix(M, K, 2.0, seed=11)
    B = inputs.lognormal_matrix(K, N, 2.0, seed=12)
    ref = ozaki2.dgemm(A, B, L, max_bits=62)
    assert 53 < ref.c_bits < 62                                # Eq. 3 limits the width at this K
    assert gu.bits_equal(gu.dgemm(A, B, L, max_bits=62), ref.C)
