"""Parity at the full configured sizes, in the launch configuration bench.py times (ozk_dgemm on
column-major device buffers): a 128x128 output block (the paper's own evaluation protocol) plus
scattered rows and columns against the CPU oracle bit for bit, the error against exact fl(AB) on
a sub-block, every reconstructed integer by a Freivalds check modulo two primes (4096 and 8192 on
the host, 16384 with the reconstructed integers left on the device), and C against the oracle's
rounding of its own reconstructed integer on a million elements."""
import numpy as np
import pytest
import torch

from oracle import exact, moduli, ozaki2
from paper_2608_06812_b200 import binding as ozk
from paper_2608_06812_b200 import inputs
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def upload(n, phi):
    A = inputs.lognormal_matrix(n, n, phi, seed=0)
    B = inputs.lognormal_matrix(n, n, phi, seed=1)
    dA = torch.from_numpy(np.ascontiguousarray(A.T)).cuda()
    dB = torch.from_numpy(np.ascontiguousarray(B.T)).cuda()
    return A, B, dA, dB


def run(n, dA, dB, L):
    gu.ensure_workspace(ozk.ozk_dgemm_workspace_bytes(n, n, n, L))
    dC = torch.empty((n, n), dtype=torch.float64, device="cuda")
    ozk.check(ozk.ozk_dgemm(n, n, n, dA.data_ptr(), n, dB.data_ptr(), n, dC.data_ptr(), n, L, gu.stream()), "ozk_dgemm")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    return dC


def sample_sets(n, seed, extra=40):
    rng = np.random.default_rng(seed)
    rows = np.concatenate([np.arange(128), np.sort(rng.choice(np.arange(128, n), extra, replace=False))])
    cols = np.concatenate([np.arange(128), np.sort(rng.choice(np.arange(128, n), extra, replace=False))])
    return rows, cols


def check_samples(A, B, dC, L, rows, cols):
    ref = ozaki2.dgemm(A[rows], B[:, cols], L)              # shifts are per row / per column: sub-matrices give the same elements
    got = dC[torch.from_numpy(cols).cuda()][:, torch.from_numpy(rows).cuda()].cpu().numpy().T
    assert gu.bits_equal(got, ref.C)
    return got


def freivalds(n, L, A, B, x_words):
    """x_words[j, i, 6] (two's complement, 32-bit words) must equal sum_k At[i,k] Bt[k,j] for every i, j:
    compare x v with At (Bt v) modulo two 31-bit primes for random v."""
    c = moduli.capacity_bits(n, L)
    At = ozaki2.to_integers(A, ozaki2.shared_shifts(A, 1, c), 1)
    Bt = ozaki2.to_integers(B, ozaki2.shared_shifts(B, 0, c), 0)
    W = x_words.astype(np.int64) & 0xFFFFFFFF
    negative = W[:, :, 5] >> 31
    rng = np.random.default_rng(99)
    for q in (2147483647, 2147483629):
        pw = [pow(2, 32 * k, q) for k in range(6)]
        xm = np.zeros(W.shape[:2], dtype=np.int64)
        for k in range(6):
            xm = (xm + (W[:, :, k] % q) * pw[k]) % q
        xm = (xm - negative * pow(2, 192, q)) % q             # xm[j, i] = x_ij mod q
        v = rng.integers(0, q, size=n).astype(np.int64)
        Bv = np.zeros(n, dtype=np.int64)
        Btm = np.mod(Bt, q)
        for j0 in range(0, n, 1024):                          # products < 2^62, reduced before summing
            Bv = (Bv + ((Btm[:, j0:j0 + 1024] * v[None, j0:j0 + 1024]) % q).sum(axis=1)) % q
        Atm = np.mod(At, q)
        right = np.zeros(n, dtype=np.int64)
        for k0 in range(0, n, 1024):
            right = (right + ((Atm[:, k0:k0 + 1024] * Bv[None, k0:k0 + 1024]) % q).sum(axis=1)) % q
        left = np.zeros(n, dtype=np.int64)
        for j0 in range(0, n, 1024):
            left = (left + ((xm[j0:j0 + 1024, :] * v[j0:j0 + 1024, None]) % q).sum(axis=0)) % q
        assert np.array_equal(left, right)


def x_words_by_stages(n, L, dA, dB):
    """The three stages called one by one (they keep their data in the workspace between calls): the
    reconstructed integers x_ij as 192-bit words, and C."""
    gu.ensure_workspace(ozk.ozk_dgemm_workspace_bytes(n, n, n, L))
    dX = torch.empty((n, n, 6), dtype=torch.int32, device="cuda")
    dC2 = torch.empty((n, n), dtype=torch.float64, device="cuda")
    ozk.check(ozk.ozk_stage_preprocess(n, n, n, dA.data_ptr(), n, dB.data_ptr(), n, L, None, None, None, None, gu.stream()),
              "ozk_stage_preprocess")
    ozk.check(ozk.ozk_stage_residue_gemm(n, n, n, L, None, gu.stream()), "ozk_stage_residue_gemm")
    ozk.check(ozk.ozk_stage_crt(n, n, n, L, None, None, None, dC2.data_ptr(), n, dX.data_ptr(), gu.stream()), "ozk_stage_crt")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    return dX.cpu().numpy(), dC2


def freivalds_on_device(n, L, A, B, dX):
    """The same identity with the 192-bit words left on the device (dX[j, i, 6], int32): x v = At (Bt v) modulo two
    31-bit primes.  At, Bt come from the CPU oracle; torch int64 arithmetic on the GPU is test infrastructure.
    A is M x K, B is K x N (n is the square size of the callers above and is not used for the extents)."""
    (M, K), N = A.shape, B.shape[1]
    c = moduli.capacity_bits(K, L)
    dAt = torch.from_numpy(ozaki2.to_integers(A, ozaki2.shared_shifts(A, 1, c), 1)).cuda()     # [i, k]
    dBt = torch.from_numpy(ozaki2.to_integers(B, ozaki2.shared_shifts(B, 0, c), 0)).cuda()     # [k, j]
    gen = torch.Generator(device="cuda")
    gen.manual_seed(99)
    step = 512
    for q in (2147483647, 2147483629):
        v = torch.randint(0, q, (N,), dtype=torch.int64, device="cuda", generator=gen)
        Bv = torch.zeros(K, dtype=torch.int64, device="cuda")
        for j0 in range(0, N, step):                          # every product is reduced (< 2^31) before the sum
            Bv = (Bv + ((dBt[:, j0:j0 + step] % q) * v[None, j0:j0 + step] % q).sum(dim=1)) % q
        right = torch.zeros(M, dtype=torch.int64, device="cuda")
        for k0 in range(0, K, step):
            right = (right + ((dAt[:, k0:k0 + step] % q) * Bv[None, k0:k0 + step] % q).sum(dim=1)) % q
        pw = [pow(2, 32 * k, q) for k in range(6)]
        left = torch.zeros(M, dtype=torch.int64, device="cuda")
        for j0 in range(0, N, step):
            W = dX[j0:j0 + step].to(torch.int64) & 0xFFFFFFFF                                   # [j, i, 6]
            xm = torch.zeros(W.shape[:2], dtype=torch.int64, device="cuda")
            for k in range(6):
                xm = (xm + (W[:, :, k] % q) * pw[k]) % q
            xm = (xm - (W[:, :, 5] >> 31) * pow(2, 192, q)) % q                                 # two's complement sign
            left = (left + (xm * v[j0:j0 + step, None] % q).sum(dim=0)) % q
        assert torch.equal(left, right)


def words_to_int(w) -> int:
    v = sum((int(x) & 0xFFFFFFFF) << (32 * k) for k, x in enumerate(w))
    return v - (1 << 192) if v >> 191 else v


def test_config2_4096_moduli_sweep():
    """M=N=K=4096, phi=0.5, moduli count 12..20: bit-exact samples for every count; the error bound
    1e-15 against fl(AB) from 17 moduli on; Freivalds over the whole matrix at 19 moduli."""
    n = 4096
    A, B, dA, dB = upload(n, 0.5)
    rows, cols = sample_sets(n, seed=2, extra=24)
    errs = {}
    for L in range(12, 21):
        dC = run(n, dA, dB, L)
        got = check_samples(A, B, dC, L, rows, cols)
        errs[L] = exact.normwise_error(got[:32, :32], A[rows[:32]], B[:, cols[:32]], against_rounded=True)
        if L == 19:
            X, dC2 = x_words_by_stages(n, L, dA, dB)
            assert torch.equal(dC2.view(torch.int64), dC.view(torch.int64))
            freivalds(n, L, A, B, X)
            # C is the oracle's single rounding of the reconstructed integer, scaled by the oracle's shifts:
            # a million random elements plus the first column
            c = moduli.capacity_bits(n, L)
            s_ref, t_ref = ozaki2.shared_shifts(A, 1, c), ozaki2.shared_shifts(B, 0, c)
            C = dC.cpu().numpy()                              # [j, i]
            rng = np.random.default_rng(7)
            ii = np.concatenate([rng.integers(0, n, 1_000_000), np.arange(n)])
            jj = np.concatenate([rng.integers(0, n, 1_000_000), np.zeros(n, dtype=np.int64)])
            want = np.array([ozaki2.round_scaled_to_double(words_to_int(X[j, i]), int(s_ref[i]) + int(t_ref[j]))
                             for i, j in zip(ii, jj)])
            assert gu.bits_equal(C[jj, ii], want)
    assert all(errs[L] <= 1e-15 for L in range(17, 21)), errs
    assert errs[12] > errs[15] > errs[18]                     # fewer moduli keep fewer bits


def test_config3_8192_phi4_wide_exponent_range():
    """M=N=K=8192, phi=4: bit-exact against the oracle; the method saturates at 19 moduli (53-bit cap,
    one exponent per row/column), so the error against fl(AB) is reported, not bounded by 1e-15."""
    n = 8192
    A, B, dA, dB = upload(n, 4.0)
    rows, cols = sample_sets(n, seed=3, extra=24)
    got = {}
    for L in (19, 20):
        dC = run(n, dA, dB, L)
        got[L] = check_samples(A, B, dC, L, rows, cols)
    assert gu.bits_equal(got[19], got[20])                    # capacity is capped at 53 bits: more moduli change nothing
    err = exact.normwise_error(got[19][:16, :16], A[rows[:16]], B[:, cols[:16]], against_rounded=True)
    assert 1e-15 < err < 1e-8
    X, dC2 = x_words_by_stages(n, 20, dA, dB)
    assert torch.equal(dC2.view(torch.int64), dC.view(torch.int64))   # staged calls and ozk_dgemm agree on every element
    freivalds(n, 20, A, B, X)


def test_config5_16384_headline_configuration():
    """M=N=K=16384, phi=1, 19 moduli (the benchmark's workload): bit-exact samples, 1e-15 bound."""
    n = 16384
    A, B, dA, dB = upload(n, 1.0)
    rows, cols = sample_sets(n, seed=5, extra=40)
    dC = run(n, dA, dB, 19)
    got = check_samples(A, B, dC, 19, rows, cols)
    err = exact.normwise_error(got[:16, :16], A[rows[:16]], B[:, cols[:16]], against_rounded=True)
    assert err <= 1e-15
    assert torch.isfinite(dC).all()
    # every element: the reconstructed integers of the staged run (left on the device) satisfy the Freivalds
    # identity against the oracle's converted integers, and the staged run's C equals ozk_dgemm's bit for bit
    gu.ensure_workspace(ozk.ozk_dgemm_workspace_bytes(n, n, n, 19))
    dX = torch.empty((n, n, 6), dtype=torch.int32, device="cuda")
    dC2 = torch.empty((n, n), dtype=torch.float64, device="cuda")
    ozk.check(ozk.ozk_stage_preprocess(n, n, n, dA.data_ptr(), n, dB.data_ptr(), n, 19, None, None, None, None, gu.stream()),
              "ozk_stage_preprocess")
    ozk.check(ozk.ozk_stage_residue_gemm(n, n, n, 19, None, gu.stream()), "ozk_stage_residue_gemm")
    ozk.check(ozk.ozk_stage_crt(n, n, n, 19, None, None, None, dC2.data_ptr(), n, dX.data_ptr(), gu.stream()), "ozk_stage_crt")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    assert torch.equal(dC2.view(torch.int64), dC.view(torch.int64))
    del dC2
    freivalds_on_device(n, 19, A, B, dX)
    # and C against the oracle's rounding of x on scattered elements
    c = moduli.capacity_bits(n, 19)
    s_ref, t_ref = ozaki2.shared_shifts(A, 1, c), ozaki2.shared_shifts(B, 0, c)
    rng = np.random.default_rng(11)
    ii, jj = rng.integers(0, n, 20000), rng.integers(0, n, 20000)
    Xs = dX[torch.from_numpy(jj).cuda(), torch.from_numpy(ii).cuda()].cpu().numpy()
    Cs = dC[torch.from_numpy(jj).cuda(), torch.from_numpy(ii).cuda()].cpu().numpy()
    want = np.array([ozaki2.round_scaled_to_double(words_to_int(Xs[k]), int(s_ref[ii[k]]) + int(t_ref[jj[k]])) for k in range(ii.size)])
    assert gu.bits_equal(Cs, want)


@pytest.mark.parametrize("M,N,K", [(8192, 8192, 1024), (16384, 4096, 512)])
def test_short_k_whole_matrix(M, N, K):
    """Short K at full width (the two-accumulator limb GEMM: row tiles of 120 with a ragged last one, many more tiles
    than CTA pairs, residues staged through shared memory): every reconstructed integer by the Freivalds identity,
    a 128 x 128 block plus scattered rows and columns of C against the oracle bit for bit, staged calls = ozk_dgemm."""
    L = 19
    A = inputs.lognormal_matrix(M, K, 1.0, seed=0)
    B = inputs.lognormal_matrix(K, N, 1.0, seed=1)
    dA = torch.from_numpy(np.ascontiguousarray(A.T)).cuda()
    dB = torch.from_numpy(np.ascontiguousarray(B.T)).cuda()
    gu.ensure_workspace(ozk.ozk_dgemm_workspace_bytes(M, N, K, L))
    dC = torch.empty((N, M), dtype=torch.float64, device="cuda")
    ozk.check(ozk.ozk_dgemm(M, N, K, dA.data_ptr(), M, dB.data_ptr(), K, dC.data_ptr(), M, L, gu.stream()), "ozk_dgemm")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    rng = np.random.default_rng(8)
    rows = np.concatenate([np.arange(128), np.sort(rng.choice(np.arange(128, M), 40, replace=False)), np.arange(M - 24, M)])
    cols = np.concatenate([np.arange(128), np.sort(rng.choice(np.arange(128, N), 40, replace=False)), np.arange(N - 24, N)])
    check_samples(A, B, dC, L, rows, cols)
    dX = torch.empty((N, M, 6), dtype=torch.int32, device="cuda")
    dC2 = torch.empty((N, M), dtype=torch.float64, device="cuda")
    ozk.check(ozk.ozk_stage_preprocess(M, N, K, dA.data_ptr(), M, dB.data_ptr(), K, L, None, None, None, None, gu.stream()),
              "ozk_stage_preprocess")
    ozk.check(ozk.ozk_stage_residue_gemm(M, N, K, L, None, gu.stream()), "ozk_stage_residue_gemm")
    ozk.check(ozk.ozk_stage_crt(M, N, K, L, None, None, None, dC2.data_ptr(), M, dX.data_ptr(), gu.stream()), "ozk_stage_crt")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    assert torch.equal(dC2.view(torch.int64), dC.view(torch.int64))
    freivalds_on_device(0, L, A, B, dX)
