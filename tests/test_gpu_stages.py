"""Stage-by-stage parity of the CUDA kernels with the CPU oracle, through the C ABI:
shifts and converted integers (bit-exact), limb planes (property: values in S, |c| <= 8,
c0 + 13 c1 = a (mod m)), residues (bit-exact), CRT + rounding (bit-exact)."""
import numpy as np
import pytest
import torch

from oracle import base13, moduli, ozaki2
from paper_2608_06812_b200 import binding as ozk
from paper_2608_06812_b200 import inputs
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def run_preprocess(A, B, L, lda=None, ldb=None):
    M, K = A.shape
    N = B.shape[1]
    lda, ldb = lda or max(M, 1), ldb or max(K, 1)
    gu.ensure_workspace(ozk.ozk_dgemm_workspace_bytes(M, N, K, L))
    dA, dB = gu.to_dev_colmajor(A, lda), gu.to_dev_colmajor(B, ldb)
    ds = torch.zeros(M, dtype=torch.int32, device="cuda")
    dt = torch.zeros(N, dtype=torch.int32, device="cuda")
    dAt = torch.zeros((K, M), dtype=torch.int64, device="cuda")
    dBt = torch.zeros((N, K), dtype=torch.int64, device="cuda")
    ozk.check(ozk.ozk_stage_preprocess(M, N, K, dA.data_ptr(), lda, dB.data_ptr(), ldb, L, ds.data_ptr(), dt.data_ptr(),
                                       dAt.data_ptr(), dBt.data_ptr(), gu.stream()), "preprocess")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    return ds.cpu().numpy(), dt.cpu().numpy(), dAt.cpu().numpy().T.copy(), dBt.cpu().numpy().T.copy()


def read_plane(op, M, N, K, L, l, limb):
    rows = M if op == "A" else N
    out = torch.zeros((K, rows), dtype=torch.int8, device="cuda")
    ozk.check(ozk.ozk_stage_read_planes(op, M, N, K, L, l, limb, out.data_ptr(), gu.stream()), "read_planes")
    torch.cuda.synchronize()
    return out.cpu().numpy().T.astype(np.int64)          # [row, k]


@pytest.mark.parametrize("shape,L,phi", [((256, 256, 256), 14, 0.5), ((130, 70, 300), 19, 4.0), ((33, 257, 65), 27, 1.0),
                                         ((1, 1, 1), 2, 0.5), ((128, 128, 513), 12, 0.5)])
def test_preprocess_matches_oracle(shape, L, phi):
    M, N, K = shape
    A = inputs.lognormal_matrix(M, K, phi, seed=0)
    B = inputs.lognormal_matrix(K, N, phi, seed=1)
    if M > 2:
        A[2, :] = 0.0                                     # zero row: shift 0, zero limbs
        A[1, 0] = 2.0 ** -1060                            # element far below its row maximum
    s, t, At, Bt = run_preprocess(A, B, L, lda=M + 3, ldb=K + 5)
    c = moduli.capacity_bits(K, L)
    assert c == ozk.ozk_capacity_bits(K, L)
    s_ref, t_ref = ozaki2.shared_shifts(A, 1, c), ozaki2.shared_shifts(B, 0, c)
    assert np.array_equal(s, s_ref) and np.array_equal(t, t_ref)
    assert np.array_equal(At, ozaki2.to_integers(A, s_ref, 1))
    assert np.array_equal(Bt, ozaki2.to_integers(B, t_ref, 0))
    mods = moduli.select_moduli(L)
    for l in sorted({0, 1, L // 2, L - 1}):
        for op, X, rows in (("A", At, M), ("B", Bt.T, N)):
            c0 = read_plane(op, M, N, K, L, l, 0)
            c1 = read_plane(op, M, N, K, L, l, 1)
            assert np.isin(c0, base13.S).all() and np.isin(c1, base13.S).all()
            assert max(np.abs(c0).max(), np.abs(c1).max()) <= 8
            assert np.all((c0 + 13 * c1 - X) % mods[l] == 0)


def test_gamma_planes_of_the_two_accumulator_form():
    """Short K on CTA pairs (column count a multiple of 256): the A side also carries the limb planes of 13 a mod m
    (planes 3 and 4 of ozk_stage_read_planes), with which a b = a0 beta + a1 gamma needs two accumulators only."""
    M, N, K, L = 130, 256, 300, 19
    A = inputs.lognormal_matrix(M, K, 1.0, seed=0)
    B = inputs.lognormal_matrix(K, N, 1.0, seed=1)
    s, t, At, Bt = run_preprocess(A, B, L)
    mods = moduli.select_moduli(L)
    for l in (0, 1, 7, 18):
        g0 = read_plane("A", M, N, K, L, l, 3)
        g1 = read_plane("A", M, N, K, L, l, 4)
        assert np.isin(g0, base13.S).all() and np.isin(g1, base13.S).all()
        assert max(np.abs(g0).max(), np.abs(g1).max()) <= 8
        assert np.all((g0 + 13 * g1 - 13 * At) % mods[l] == 0)
    out = torch.zeros((K, N), dtype=torch.int8, device="cuda")
    assert ozk.ozk_stage_read_planes("B", M, N, K, L, 0, 3, out.data_ptr(), gu.stream()) == ozk.OZK_ERR_INVALID_ARG


def test_subnormal_and_extreme_rows():
    A = np.array([[2.0 ** -1074, 3 * 2.0 ** -1074, 0.0, -(2.0 ** -1070)],
                  [1.7e308, -1e300, 1e-300, 5e307],
                  [2.0 - 2.0 ** -52, 1.0, 0.5, 0.25]])
    B = inputs.lognormal_matrix(4, 3, 0.5, seed=4)
    for L in (14, 19):
        s, t, At, Bt = run_preprocess(A, B, L)
        c = moduli.capacity_bits(4, L)
        s_ref = ozaki2.shared_shifts(A, 1, c)
        assert np.array_equal(s, s_ref)
        assert np.array_equal(At, ozaki2.to_integers(A, s_ref, 1))
        assert np.abs(At).max() <= 2 ** c


def test_nonfinite_input_is_flagged():
    A = inputs.lognormal_matrix(8, 8, 0.5, seed=0)
    B = inputs.lognormal_matrix(8, 8, 0.5, seed=1)
    B[3, 4] = np.nan
    M = N = K = 8
    gu.ensure_workspace(ozk.ozk_dgemm_workspace_bytes(M, N, K, 19))
    dA, dB = gu.to_dev_colmajor(A), gu.to_dev_colmajor(B)
    ozk.check(ozk.ozk_stage_preprocess(M, N, K, dA.data_ptr(), M, dB.data_ptr(), K, 19, None, None, None, None, gu.stream()), "pre")
    assert ozk.ozk_get_async_status(gu.stream()) == ozk.OZK_ERR_NONFINITE
    assert ozk.ozk_get_async_status(gu.stream()) == ozk.OZK_OK          # reading clears it


@pytest.mark.parametrize("shape,L,phi", [((256, 256, 256), 14, 0.5), ((130, 70, 300), 19, 4.0), ((384, 129, 1000), 20, 1.0),
                                         ((5, 3, 2), 2, 0.5), ((128, 256, 2048), 27, 0.5)])
def test_residue_gemm_matches_oracle(shape, L, phi):
    M, N, K = shape
    A = inputs.lognormal_matrix(M, K, phi, seed=0)
    B = inputs.lognormal_matrix(K, N, phi, seed=1)
    ref = ozaki2.dgemm(A, B, L)
    run_preprocess(A, B, L)
    dR = torch.full((L, N, M), 255, dtype=torch.uint8, device="cuda")
    ozk.check(ozk.ozk_stage_residue_gemm(M, N, K, L, dR.data_ptr(), gu.stream()), "residue_gemm")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    R = dR.cpu().numpy()
    for l in range(L):
        assert np.array_equal(R[l].T.astype(np.int64), ref.residues[l]), f"modulus index {l}"


def words_to_int(words: np.ndarray) -> int:
    v = sum(int(w) << (32 * i) for i, w in enumerate(words))
    return v - (1 << 192) if v >> 191 else v


@pytest.mark.parametrize("fast", [False, True])
@pytest.mark.parametrize("L", [2, 9, 12, 13, 14, 15, 16, 17, 18, 19, 20, 21, 22, 23, 24, 27])
def test_crt_stage_matches_oracle_on_arbitrary_residues(L, fast):
    """fast=False: one element per thread, with the reconstructed integers exported; fast=True: the
    tensor-core kernel the full pipeline uses (row count a multiple of 16: one full block of 128 rows and a
    ragged one; no export)."""
    M, N, K = (144, 9, 16) if fast else (37, 29, 16)
    mods = moduli.select_moduli(L)
    P = moduli.product(mods)
    rng = np.random.default_rng(L)
    # integers spread over the whole symmetric range, plus the extremes
    xs = np.empty((M, N), dtype=object)
    for idx in np.ndindex(M, N):
        xs[idx] = int(rng.integers(0, 2 ** 62)) * int(rng.integers(0, 2 ** 62)) * int(rng.integers(1, 2 ** 40)) % P - P // 2
        if 2 * abs(xs[idx]) >= P:
            xs[idx] = 0
    xs[0, 0], xs[1, 0], xs[2, 0], xs[3, 0] = 0, (P - 1) // 2, -((P - 1) // 2), 1
    xs[4, 0], xs[5, 0] = 2 ** 53 + 1, -(2 ** 54 + 2 ** 0 + 2)             # ties and near-ties of the final rounding
    # every residue m_l - 1 (the largest weighted sum and quotient), and the neighbours of the range's ends
    xs[6, 0], xs[7, 0], xs[12, 0], xs[13, 0] = -1, 1 - P // 2, P // 2 - 1, -2
    xs[M - 1, N - 1], xs[M - 2, N - 1] = -1, (P - 1) // 2
    for idx in np.ndindex(M, N):
        if 2 * abs(xs[idx]) >= P:
            xs[idx] = 0
    res = np.stack([np.array([[int(xs[i, j]) % m for j in range(N)] for i in range(M)], dtype=np.uint8) for m in mods])
    s = rng.integers(-60, 1200, size=M).astype(np.int32)
    t = rng.integers(-60, 1200, size=N).astype(np.int32)
    s[:8], t[:4] = 0, 0
    s[8:12], t[4:6] = -600, -500                                            # huge results, up to overflow
    gu.ensure_workspace(ozk.ozk_dgemm_workspace_bytes(M, N, K, L))
    dR = torch.from_numpy(np.ascontiguousarray(res.transpose(0, 2, 1))).cuda()     # [l][j][i]
    ds, dt = torch.from_numpy(s).cuda(), torch.from_numpy(t).cuda()
    dC = torch.zeros((N, M + 2), dtype=torch.float64, device="cuda")
    dX = torch.zeros((N, M, 6), dtype=torch.int64, device="cuda").to(torch.int32)
    ozk.check(ozk.ozk_stage_crt(M, N, K, L, dR.data_ptr(), ds.data_ptr(), dt.data_ptr(), dC.data_ptr(), M + 2,
                                None if fast else dX.data_ptr(), gu.stream()), "crt")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    C = gu.from_dev_colmajor(dC, M, N)
    X = dX.cpu().numpy().view(np.uint32)
    for i in range(M):
        for j in range(N):
            if not fast:
                assert words_to_int(X[j, i]) == int(xs[i, j]), (i, j)
            want = ozaki2.round_scaled_to_double(int(xs[i, j]), int(s[i]) + int(t[j]))
            assert np.float64(C[i, j]).view(np.uint64) == np.float64(want).view(np.uint64), (i, j, xs[i, j], s[i] + t[j])


def test_stage_timing_averages_over_the_calls_since_the_last_read():
    """Measurement aid: four events per ozk_dgemm call kept in a ring; one read after several calls returns
    positive per-stage averages and empties the ring."""
    A = inputs.lognormal_matrix(256, 512, 1.0, seed=1)
    B = inputs.lognormal_matrix(512, 256, 1.0, seed=2)
    ozk.check(ozk.ozk_stage_timing_enable(True), "enable")
    try:
        with pytest.raises(ozk.OzkError):
            ozk.ozk_stage_timing_read()                      # nothing recorded yet
        ref = gu.dgemm(A, B, 19)
        for _ in range(3):
            assert gu.bits_equal(gu.dgemm(A, B, 19), ref)
        ms = ozk.ozk_stage_timing_read()
        assert all(0.0 < v < 1000.0 for v in ms)
        with pytest.raises(ozk.OzkError):
            ozk.ozk_stage_timing_read()                      # the read emptied the ring
    finally:
        ozk.check(ozk.ozk_stage_timing_enable(False), "disable")
