"""Bit-exact INT8 x INT8 -> INT32 GEMM on FP4 limbs (ozk_igemm_i8) against the int64 definition."""
import numpy as np
import pytest
import torch

from oracle import base13
from paper_2608_06812_b200 import binding as ozk
from paper_2608_06812_b200 import inputs
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def igemm(A, B, lda=None, ldb=None, ldc=None):
    M, K = A.shape
    N = B.shape[1]
    lda, ldb, ldc = lda or max(M, 1), ldb or max(K, 1), ldc or max(M, 1)
    gu.ensure_workspace(ozk.ozk_igemm_i8_workspace_bytes(M, N, K))
    dA, dB = gu.to_dev_colmajor(A, lda), gu.to_dev_colmajor(B, ldb)
    dC = torch.full((max(N, 1), ldc), -7, dtype=torch.int32, device="cuda")
    ozk.check(ozk.ozk_igemm_i8(M, N, K, dA.data_ptr(), lda, dB.data_ptr(), ldb, dC.data_ptr(), ldc, gu.stream()), "ozk_igemm_i8")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    return gu.from_dev_colmajor(dC, M, N), dC


@pytest.mark.parametrize("shape", [(1, 1, 1), (3, 5, 0), (130, 70, 300), (81, 129, 257), (256, 256, 512), (400, 333, 1000)])
def test_small_shapes_exact(shape):
    M, N, K = shape
    A, B = inputs.int8_matrix(M, K, seed=0), inputs.int8_matrix(K, N, seed=1)
    C, dC = igemm(A, B, lda=M + 3, ldb=K + 1, ldc=M + 2)
    assert np.array_equal(C.astype(np.int64), base13.igemm_i8_definition(A, B))
    assert np.array_equal(C, base13.igemm_i8_by_limbs(A, B))
    # the padding rows of C between M and ldc are not written
    assert (dC.cpu().numpy()[:N, M:] == -7).all()


def test_extreme_values_exact():
    M, N, K = 160, 96, 4096
    A = np.full((M, K), -128, dtype=np.int8)
    B = np.full((K, N), -128, dtype=np.int8)
    A[1::2, :] = 127
    B[:, 1::3] = 127
    C, _ = igemm(A, B)
    assert np.array_equal(C.astype(np.int64), base13.igemm_i8_definition(A, B))
    assert C.max() == 128 * 128 * K


def test_config4_8192_cubed_block_samples_and_freivalds():
    """M=N=K=8192, int8 uniform on [-128,127], seeds 0/1: a 128x128 block and scattered rows/columns
    against the int64 definition, and the whole matrix by a Freivalds check in exact int64."""
    n = 8192
    A, B = inputs.int8_matrix(n, n, seed=0), inputs.int8_matrix(n, n, seed=1)
    C, _ = igemm(A, B)
    rng = np.random.default_rng(7)
    rows = np.concatenate([np.arange(128), rng.choice(n, 48, replace=False)])
    cols = np.concatenate([np.arange(128), rng.choice(n, 48, replace=False)])
    ref = A[rows].astype(np.int64) @ B[:, cols].astype(np.int64)
    assert np.array_equal(C[np.ix_(rows, cols)].astype(np.int64), ref)
    for trial in range(2):
        v = rng.integers(0, 1 << 20, size=n).astype(np.int64)
        left = C.astype(np.int64) @ v                       # |C| <= 2^27, sums < 2^60
        right = A.astype(np.int64) @ (B.astype(np.int64) @ v)
        assert np.array_equal(left, right)


def test_argument_errors():
    gu.register_small_workspace(8 << 20)          # every call below must be rejected before anything is launched
    assert ozk.ozk_igemm_i8(8, 8, 100000, None, 8, None, 100000, None, 8, 0) == ozk.OZK_ERR_UNSUPPORTED
    assert ozk.ozk_igemm_i8(8, 8, 8, None, 8, None, 8, None, 8, 0) == ozk.OZK_ERR_INVALID_ARG
    assert ozk.ozk_igemm_i8(4096, 4096, 4096, None, 4096, None, 4096, None, 4096, 0) == ozk.OZK_ERR_WORKSPACE
    assert ozk.ozk_igemm_i8_workspace_bytes(8192, 8192, 8192) >= 2 * 3 * 8192 * 8192 // 2
