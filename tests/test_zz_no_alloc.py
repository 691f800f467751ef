"""ozk_row_shifts_noalloc, the entry point for callers that cannot allocate device memory (its
scratch is a fixed array inside the library): its output must equal the shifts the regular,
workspace-based stage 1 produces, and the oracle's, on two calls in a row that reuse the same scratch."""
import numpy as np
import pytest
import torch

from oracle import moduli, ozaki2
from paper_2608_06812_b200 import binding as ozk
from paper_2608_06812_b200 import inputs
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def shifts_by_workspace_path(A, B, L):
    M, K = A.shape
    N = B.shape[1]
    gu.ensure_workspace(ozk.ozk_dgemm_workspace_bytes(M, N, K, L))
    dA, dB = gu.to_dev_colmajor(A), gu.to_dev_colmajor(B)
    ds = torch.zeros(M, dtype=torch.int32, device="cuda")
    ozk.check(ozk.ozk_stage_preprocess(M, N, K, dA.data_ptr(), M, dB.data_ptr(), K, L, ds.data_ptr(), None, None, None,
                                       gu.stream()), "ozk_stage_preprocess")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    return ds.cpu().numpy()


def shifts_by_noalloc_path(A, L, lda=None):
    M, K = A.shape
    lda = lda or M
    dA = gu.to_dev_colmajor(A, lda)
    ds = torch.full((M,), 12345, dtype=torch.int32, device="cuda")
    ozk.check(ozk.ozk_row_shifts_noalloc(M, K, dA.data_ptr(), lda, L, ds.data_ptr(), gu.stream()), "ozk_row_shifts_noalloc")
    torch.cuda.synchronize()
    return ds.cpu().numpy()


def test_two_calls_in_a_row_match_the_workspace_path():
    L = 19
    # first call: large magnitudes; second call: fewer rows of much smaller magnitude and a zero row,
    # so any maximum left over from the first call would show up as a wrong shift
    A1 = inputs.lognormal_matrix(700, 333, 4.0, seed=0) * 2.0 ** 40
    A2 = inputs.lognormal_matrix(300, 200, 0.5, seed=2) * 2.0 ** -30
    A2[5, :] = 0.0
    B1 = inputs.lognormal_matrix(333, 8, 0.5, seed=1)
    B2 = inputs.lognormal_matrix(200, 8, 0.5, seed=3)
    got1 = shifts_by_noalloc_path(A1, L, lda=705)
    got2 = shifts_by_noalloc_path(A2, L)
    assert np.array_equal(got1, shifts_by_workspace_path(A1, B1, L))
    assert np.array_equal(got2, shifts_by_workspace_path(A2, B2, L))
    assert np.array_equal(got1, ozaki2.shared_shifts(A1, 1, moduli.capacity_bits(333, L)))
    assert np.array_equal(got2, ozaki2.shared_shifts(A2, 1, moduli.capacity_bits(200, L)))
    assert got2[5] == 0
    # and a third call on the first input again gives the first answer again
    assert np.array_equal(shifts_by_noalloc_path(A1, L), got1)


def test_subnormal_row_maximum_and_empty_inner_dimension():
    L = 19
    A = inputs.lognormal_matrix(40, 12, 0.5, seed=7)
    A[3, :] = [k * 2.0 ** -1074 for k in range(12)]          # the row maximum is subnormal
    A[4, :] = 0.0
    A[4, 2] = -(2.0 ** -1074)                                  # the smallest magnitude there is
    B = inputs.lognormal_matrix(12, 8, 0.5, seed=8)
    got = shifts_by_noalloc_path(A, L)
    assert np.array_equal(got, shifts_by_workspace_path(A, B, L))
    assert np.array_equal(got, ozaki2.shared_shifts(A, 1, moduli.capacity_bits(12, L)))
    # K = 0: every row is empty, every shift 0, and nothing is read from A
    ds = torch.full((9,), 777, dtype=torch.int32, device="cuda")
    ozk.check(ozk.ozk_row_shifts_noalloc(9, 0, None, 9, L, ds.data_ptr(), gu.stream()), "ozk_row_shifts_noalloc")
    torch.cuda.synchronize()
    assert np.array_equal(ds.cpu().numpy(), np.zeros(9, dtype=np.int32))
    # the same array serves the next call
    assert np.array_equal(shifts_by_noalloc_path(A, L), got)


def test_limits_and_flags():
    d = torch.zeros(16, dtype=torch.float64, device="cuda")
    s = torch.zeros(16, dtype=torch.int32, device="cuda")
    too_many = 65536 + 1
    assert ozk.ozk_row_shifts_noalloc(too_many, 1, d.data_ptr(), too_many, 19, s.data_ptr(), gu.stream()) == ozk.OZK_ERR_UNSUPPORTED
    assert ozk.ozk_row_shifts_noalloc(4, 4, d.data_ptr(), 3, 19, s.data_ptr(), gu.stream()) == ozk.OZK_ERR_INVALID_ARG
    assert ozk.ozk_row_shifts_noalloc(0, 4, None, 1, 19, None, gu.stream()) == ozk.OZK_OK
    A = np.ones((4, 4))
    A[2, 1] = np.inf
    got = shifts_by_noalloc_path(A, 19)
    assert got[2] == np.iinfo(np.int32).min and got[0] == ozk.ozk_capacity_bits(4, 19) - 1
