"""Ozaki scheme I on FP4 limbs (ozk_dgemm_oz1): bit-exact against the scheme-I oracle and, as the paper
states for its two schemes, against scheme II with 19 moduli."""
import numpy as np
import pytest
import torch

from oracle import ozaki1, ozaki2
from paper_2608_06812_b200 import binding as ozk
from paper_2608_06812_b200 import inputs
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def dgemm_oz1(A, B, lda=None, ldb=None, ldc=None):
    M, K = A.shape
    N = B.shape[1]
    lda, ldb, ldc = lda or max(M, 1), ldb or max(K, 1), ldc or max(M, 1)
    gu.ensure_workspace(ozk.ozk_dgemm_oz1_workspace_bytes(M, N, K))
    dA, dB = gu.to_dev_colmajor(A, lda), gu.to_dev_colmajor(B, ldb)
    dC = torch.full((max(N, 1), ldc), float("nan"), dtype=torch.float64, device="cuda")
    ozk.check(ozk.ozk_dgemm_oz1(M, N, K, dA.data_ptr(), lda, dB.data_ptr(), ldb, dC.data_ptr(), ldc, gu.stream()), "ozk_dgemm_oz1")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    return gu.from_dev_colmajor(dC, M, N)


@pytest.mark.parametrize("shape,phi", [((1, 1, 1), 0.5), ((3, 4, 0), 0.5), ((130, 70, 300), 4.0), ((81, 129, 257), 1.0),
                                       ((256, 256, 512), 0.5), ((200, 333, 1000), 2.0)])
def test_small_shapes_bit_exact(shape, phi):
    M, N, K = shape
    A = inputs.lognormal_matrix(M, K, phi, seed=0)
    B = inputs.lognormal_matrix(K, N, phi, seed=1)
    if M > 2:
        A[2, :] = 0.0
    C = dgemm_oz1(A, B, lda=M + 3, ldb=K + 1, ldc=M + 2)
    ref, _, _, _ = ozaki1.dgemm(A, B)
    assert gu.bits_equal(C, ref)
    assert gu.bits_equal(C, gu.dgemm(A, B, 19))              # scheme I == scheme II (Section 7.1)


def test_extreme_magnitudes_and_signs():
    A = inputs.lognormal_matrix(96, 640, 6.0, seed=3)
    B = inputs.lognormal_matrix(640, 80, 6.0, seed=4)
    A[0, :] = np.abs(A[0, :]).max()                           # every element at the row maximum: 53-bit integers everywhere
    B[:, 0] = -np.abs(B[:, 0]).max()
    A[1, :] *= 2.0 ** -700
    C = dgemm_oz1(A, B)
    assert gu.bits_equal(C, ozaki1.dgemm(A, B)[0])


def test_config3_8192_phi4_samples():
    """M=N=K=8192, phi=4: block and scattered samples against the oracles of both schemes."""
    n = 8192
    A = inputs.lognormal_matrix(n, n, 4.0, seed=0)
    B = inputs.lognormal_matrix(n, n, 4.0, seed=1)
    gu.ensure_workspace(ozk.ozk_dgemm_oz1_workspace_bytes(n, n, n))
    dA = torch.from_numpy(np.ascontiguousarray(A.T)).cuda()
    dB = torch.from_numpy(np.ascontiguousarray(B.T)).cuda()
    dC = torch.empty((n, n), dtype=torch.float64, device="cuda")
    ozk.check(ozk.ozk_dgemm_oz1(n, n, n, dA.data_ptr(), n, dB.data_ptr(), n, dC.data_ptr(), n, gu.stream()), "ozk_dgemm_oz1")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    rng = np.random.default_rng(3)
    rows = np.concatenate([np.arange(64), np.sort(rng.choice(np.arange(64, n), 24, replace=False))])
    cols = np.concatenate([np.arange(64), np.sort(rng.choice(np.arange(64, n), 24, replace=False))])
    got = dC[torch.from_numpy(cols).cuda()][:, torch.from_numpy(rows).cuda()].cpu().numpy().T
    assert gu.bits_equal(got, ozaki2.dgemm(A[rows], B[:, cols], 19).C)
    assert gu.bits_equal(got[:24, :24], ozaki1.dgemm(A[rows[:24]], B[:, cols[:24]])[0])


def test_argument_errors():
    gu.register_small_workspace(8 << 20)
    assert ozk.ozk_dgemm_oz1(8, 8, 100000, None, 8, None, 100000, None, 8, 0) == ozk.OZK_ERR_UNSUPPORTED
    assert ozk.ozk_dgemm_oz1(8, 8, 8, None, 8, None, 8, None, 8, 0) == ozk.OZK_ERR_INVALID_ARG
    assert ozk.ozk_dgemm_oz1(4096, 4096, 4096, None, 4096, None, 4096, None, 4096, 0) == ozk.OZK_ERR_WORKSPACE
