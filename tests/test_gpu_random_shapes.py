"""Randomised shapes, modulus counts and leading dimensions: ozk_dgemm against the CPU oracle bit for bit, and
many calls enqueued back to back on one stream before any synchronisation."""
import numpy as np
import pytest
import torch

from oracle import ozaki2
from paper_2608_06812_b200 import binding as ozk
from paper_2608_06812_b200 import inputs
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def test_random_shapes_bit_exact():
    rng = np.random.default_rng(2024)
    for trial in range(24):
        M = int(rng.integers(1, 300))
        N = int(rng.integers(1, 600))
        K = int(rng.integers(0, 700))
        L = int(rng.integers(2, 28))
        phi = float(rng.choice([0.5, 1.0, 4.0]))
        A = inputs.lognormal_matrix(M, K, phi, seed=1000 + trial)
        B = inputs.lognormal_matrix(K, N, phi, seed=2000 + trial)
        C = gu.dgemm(A, B, L, lda=M + int(rng.integers(0, 5)), ldb=max(K, 1) + int(rng.integers(0, 5)), ldc=M + int(rng.integers(0, 5)))
        assert gu.bits_equal(C, ozaki2.dgemm(A, B, L).C), (M, N, K, L, phi)


def test_back_to_back_calls_without_synchronisation():
    """Calls that share the workspace are ordered by the stream alone: results of a mixed sequence (both limb-GEMM
    kernels, different modulus counts) must not depend on host synchronisation between them."""
    cases = [(256, 256, 512, 19), (130, 70, 300, 14), (384, 512, 256, 20), (64, 768, 1024, 12), (200, 130, 64, 27)]
    gu.ensure_workspace(max(ozk.ozk_dgemm_workspace_bytes(M, N, K, L) for M, N, K, L in cases))
    work = []
    for rep in range(3):
        for (M, N, K, L) in cases:
            A = inputs.lognormal_matrix(M, K, 1.0, seed=rep * 10 + L)
            B = inputs.lognormal_matrix(K, N, 1.0, seed=rep * 10 + L + 1)
            dA, dB = gu.to_dev_colmajor(A), gu.to_dev_colmajor(B)
            dC = torch.empty((N, M), dtype=torch.float64, device="cuda")
            work.append((A, B, L, dA, dB, dC))
    for (A, B, L, dA, dB, dC) in work:                       # enqueue everything, synchronise once
        M, K = A.shape
        N = B.shape[1]
        ozk.check(ozk.ozk_dgemm(M, N, K, dA.data_ptr(), M, dB.data_ptr(), K, dC.data_ptr(), M, L, gu.stream()), "ozk_dgemm")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    for (A, B, L, dA, dB, dC) in work:
        M, N = A.shape[0], B.shape[1]
        assert gu.bits_equal(gu.from_dev_colmajor(dC, M, N), ozaki2.dgemm(A, B, L).C)


def test_operands_at_odd_addresses():
    """A, B and C start 8 bytes past a 16-byte boundary and have odd leading dimensions: every vectorised load and
    store in the O(N^2) kernels has to fall back to its scalar form and give the same bits."""
    M, N, K, L = 203, 331, 517, 19
    A = inputs.lognormal_matrix(M, K, 1.0, seed=77)
    B = inputs.lognormal_matrix(K, N, 1.0, seed=78)
    lda, ldb, ldc = M + 2, K + 4, M + 4                      # odd leading dimensions: columns alternate in alignment
    bufA = torch.zeros(K * lda + 1, dtype=torch.float64, device="cuda")
    bufB = torch.zeros(N * ldb + 1, dtype=torch.float64, device="cuda")
    bufC = torch.full((N * ldc + 1,), float("nan"), dtype=torch.float64, device="cuda")
    bufA[1:].view(K, lda)[:, :M] = torch.from_numpy(np.ascontiguousarray(A.T)).cuda()
    bufB[1:].view(N, ldb)[:, :K] = torch.from_numpy(np.ascontiguousarray(B.T)).cuda()
    assert bufA[1:].data_ptr() % 16 == 8
    gu.ensure_workspace(ozk.ozk_dgemm_workspace_bytes(M, N, K, L))
    ozk.check(ozk.ozk_dgemm(M, N, K, bufA[1:].data_ptr(), lda, bufB[1:].data_ptr(), ldb, bufC[1:].data_ptr(), ldc, L, gu.stream()),
              "ozk_dgemm")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    C = bufC[1:].view(N, ldc).cpu().numpy()
    assert gu.bits_equal(C[:, :M].T.copy(), ozaki2.dgemm(A, B, L).C)
    assert np.isnan(C[:, M:]).all() and np.isnan(bufC[0].item())   # nothing outside C was written


def test_cuda_graph_capture_and_replay():
    """ozk_dgemm only enqueues work on its stream (kernels, memsets, one cooperative launch), so a call can be
    captured into a CUDA graph and replayed on new data in the same buffers."""
    M, N, K, L = 384, 512, 640, 19
    A1 = inputs.lognormal_matrix(M, K, 1.0, seed=5)
    B1 = inputs.lognormal_matrix(K, N, 1.0, seed=6)
    A2 = inputs.lognormal_matrix(M, K, 2.0, seed=7)
    B2 = inputs.lognormal_matrix(K, N, 2.0, seed=8)
    gu.ensure_workspace(ozk.ozk_dgemm_workspace_bytes(M, N, K, L))
    dA, dB = gu.to_dev_colmajor(A1), gu.to_dev_colmajor(B1)
    dC = torch.zeros((N, M), dtype=torch.float64, device="cuda")
    ozk.check(ozk.ozk_dgemm(M, N, K, dA.data_ptr(), M, dB.data_ptr(), K, dC.data_ptr(), M, L, gu.stream()), "warm-up")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ozk.check(ozk.ozk_dgemm(M, N, K, dA.data_ptr(), M, dB.data_ptr(), K, dC.data_ptr(), M, L, gu.stream()), "capture")
    dC.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert gu.bits_equal(gu.from_dev_colmajor(dC, M, N), ozaki2.dgemm(A1, B1, L).C)
    dA.copy_(gu.to_dev_colmajor(A2))
    dB.copy_(gu.to_dev_colmajor(B2))
    graph.replay()
    torch.cuda.synchronize()
    assert gu.bits_equal(gu.from_dev_colmajor(dC, M, N), ozaki2.dgemm(A2, B2, L).C)
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")


@pytest.mark.parametrize("M,N,K", [(70000, 40, 96), (40, 60000, 96), (66000, 300, 20)])
def test_very_tall_and_very_wide_outputs(M, N, K):
    """Grid dimensions beyond 65535 blocks in either direction; sampled rows and columns against the oracle
    (shifts are per row / per column, so sub-matrices reproduce the same elements)."""
    L = 19
    A = inputs.lognormal_matrix(M, K, 1.0, seed=M % 97)
    B = inputs.lognormal_matrix(K, N, 1.0, seed=N % 89)
    C = gu.dgemm(A, B, L)
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([[0, 1, M - 2, M - 1], rng.integers(0, M, 60)]))
    cols = np.unique(np.concatenate([[0, 1, N - 2, N - 1], rng.integers(0, N, 60)]))
    assert gu.bits_equal(C[np.ix_(rows, cols)], ozaki2.dgemm(A[rows], B[:, cols], L).C)
    assert np.isfinite(C).all()


def test_random_shapes_with_special_inputs():
    """Random shapes combined with zero rows / columns, global scalings across the FP64 exponent range, rows and
    columns in the subnormal range, integer data, single huge columns, and (for L >= 19) widths beyond 53 bits."""
    from oracle import moduli
    rng = np.random.default_rng(77)
    done = 0
    while done < 40:
        M, N, K = int(rng.integers(1, 400)), int(rng.integers(1, 500)), int(rng.integers(1, 1500))
        L = int(rng.integers(2, 28))
        if moduli.capacity_bits(K, L) < 1:
            continue
        phi = float(rng.choice([0.5, 1.0, 4.0, 8.0]))
        A = inputs.lognormal_matrix(M, K, phi, seed=int(rng.integers(1 << 30)))
        B = inputs.lognormal_matrix(K, N, phi, seed=int(rng.integers(1 << 30)))
        kind = done % 6
        if kind == 1:
            A[rng.integers(0, M), :] = 0.0
            B[:, rng.integers(0, N)] = 0.0
        elif kind == 2:
            A *= 2.0 ** int(rng.integers(-900, 900))
        elif kind == 3:
            A[rng.integers(0, M), :] *= 2.0 ** -1040
            B[:, rng.integers(0, N)] *= 2.0 ** -1030
        elif kind == 4:
            A, B = np.rint(A * 1000), np.rint(B * 1000)
        elif kind == 5:
            A[:, rng.integers(0, K)] *= 2.0 ** 60
        max_bits = int(rng.integers(54, 63)) if (L >= 19 and rng.random() < 0.3) else None
        with np.errstate(all="ignore"):
            ref = ozaki2.dgemm(A, B, L, max_bits=max_bits or 53).C
        C = gu.dgemm(A, B, L, lda=M + int(rng.integers(0, 4)), ldb=K + int(rng.integers(0, 4)), ldc=M + int(rng.integers(0, 4)),
                     max_bits=max_bits)
        assert gu.bits_equal(C, ref), (M, N, K, L, phi, kind, max_bits)
        done += 1
