"""ozk_dgemm_host: operands in (pinned) host memory, copies overlapped with the stages, C produced in
blocks of 4096 columns.  The result must equal the CPU oracle, hence ozk_dgemm, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import ozaki2
from paper_2608_06812_b200 import binding as ozk
from paper_2608_06812_b200 import inputs
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def dgemm_host(A, B, L, lda=None, ldb=None, ldc=None):
    M, K = A.shape
    N = B.shape[1]
    lda, ldb, ldc = lda or max(M, 1), ldb or max(K, 1), ldc or max(M, 1)
    gu.ensure_workspace(ozk.ozk_dgemm_host_workspace_bytes(M, N, K, L))
    hA = torch.zeros((max(K, 1), lda), dtype=torch.float64).pin_memory()
    hB = torch.zeros((max(N, 1), ldb), dtype=torch.float64).pin_memory()
    hC = torch.full((max(N, 1), ldc), float("nan"), dtype=torch.float64).pin_memory()
    hA[:K, :M] = torch.from_numpy(np.ascontiguousarray(A.T))
    hB[:N, :K] = torch.from_numpy(np.ascontiguousarray(B.T))
    ozk.check(ozk.ozk_dgemm_host(M, N, K, hA.data_ptr(), lda, hB.data_ptr(), ldb, hC.data_ptr(), ldc, L, gu.stream()), "ozk_dgemm_host")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    out = hC.numpy()
    assert np.isnan(out[:N, M:]).all()                      # the padding between M and ldc is not touched
    return out[:N, :M].T.copy()


@pytest.mark.parametrize("shape,L", [((130, 70, 300), 19), ((300, 5000, 700), 19), ((64, 9000, 512), 14), ((257, 12288, 256), 20),
                                     ((1, 1, 1), 19), ((5, 4097, 0), 19)])
def test_host_pipeline_bit_exact(shape, L):
    M, N, K = shape
    A = inputs.lognormal_matrix(M, K, 1.0, seed=30)
    B = inputs.lognormal_matrix(K, N, 1.0, seed=31)
    C = dgemm_host(A, B, L, lda=M + 2, ldb=K + 3, ldc=M + 1)
    assert gu.bits_equal(C, ozaki2.dgemm(A, B, L).C)


def test_back_to_back_calls_and_device_path_agree():
    A = inputs.lognormal_matrix(200, 600, 0.5, seed=1)
    B1 = inputs.lognormal_matrix(600, 8200, 0.5, seed=2)
    B2 = inputs.lognormal_matrix(600, 8200, 4.0, seed=3)
    C1 = dgemm_host(A, B1, 19)
    C2 = dgemm_host(A, B2, 19)
    assert gu.bits_equal(C1, gu.dgemm(A, B1, 19)) and gu.bits_equal(C2, gu.dgemm(A, B2, 19))


def test_row_and_column_blocks_agree_with_the_device_path():
    """More than one block in both directions (4096-row blocks of A, 4096-column blocks of B), with ragged
    last blocks: the device-resident path, itself checked against the oracle, must give the same bits."""
    for (M, N, K, L) in [(4100, 4200, 96, 19), (8200, 300, 160, 14), (9000, 8500, 64, 19)]:
        A = inputs.lognormal_matrix(M, K, 2.0, seed=40)
        B = inputs.lognormal_matrix(K, N, 2.0, seed=41)
        A[4097 % M, :] = 0.0
        C = dgemm_host(A, B, L, lda=M + 2, ldb=K + 3, ldc=M + 1)
        assert gu.bits_equal(C, gu.dgemm(A, B, L)), (M, N, K, L)
    # and one ragged multi-block case straight against the oracle on sampled rows / columns
    M, N, K, L = 4100, 4200, 96, 19
    A = inputs.lognormal_matrix(M, K, 2.0, seed=40)
    B = inputs.lognormal_matrix(K, N, 2.0, seed=41)
    C = dgemm_host(A, B, L)
    rows = np.array([0, 1, 4095, 4096, 4099]); cols = np.array([0, 255, 4095, 4096, 4199])
    assert gu.bits_equal(C[np.ix_(rows, cols)], ozaki2.dgemm(A[rows], B[:, cols], L).C)


def test_argument_errors():
    gu.register_small_workspace(8 << 20)
    assert ozk.ozk_dgemm_host(4096, 4096, 4096, None, 4096, None, 4096, None, 4096, 19, 0) == ozk.OZK_ERR_WORKSPACE
    assert ozk.ozk_dgemm_host(8, 8, 8, None, 8, None, 8, None, 8, 19, 0) == ozk.OZK_ERR_INVALID_ARG     # null pointers
    assert ozk.ozk_dgemm_host(-1, 8, 8, None, 8, None, 8, None, 8, 19, 0) == ozk.OZK_ERR_INVALID_ARG
    assert ozk.ozk_dgemm_host_workspace_bytes(4096, 16384, 4096, 19) > ozk.ozk_dgemm_workspace_bytes(4096, 4096, 4096, 19)
