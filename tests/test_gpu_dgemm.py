"""End-to-end parity of ozk_dgemm with the CPU oracle (bit for bit) and accuracy against fl(AB)."""
import numpy as np
import pytest

from oracle import exact, ozaki2
from paper_2608_06812_b200 import binding as ozk
from paper_2608_06812_b200 import inputs
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def test_config1_256_cubed_L14_bit_exact_and_error_levels():
    """M=N=K=256, phi=0.5, seeds 0/1: bit-exact against the oracle at 14 moduli; against the exact
    fl(AB) the bound 1e-15 holds from 17 moduli on (14 moduli keep only 42 bits, Eq. 3)."""
    A = inputs.lognormal_matrix(256, 256, 0.5, seed=0)
    B = inputs.lognormal_matrix(256, 256, 0.5, seed=1)
    F = exact.fl_matmul(A[:64], B[:, :64])
    for L in (14, 17, 19):
        C = gu.dgemm(A, B, L)
        ref = ozaki2.dgemm(A, B, L)
        assert gu.bits_equal(C, ref.C), f"L={L}"
        err = exact.normwise_error(C[:64, :64], A[:64], B[:, :64], against_rounded=True)
        if L >= 17:
            assert err <= 1e-15
    assert np.mean(gu.dgemm(A, B, 19)[:64, :64] == F) > 0.05   # many elements are the correctly rounded value itself


@pytest.mark.parametrize("shape", [(1, 1, 1), (2, 3, 0), (130, 70, 300), (257, 129, 255), (128, 384, 1025), (640, 512, 768)])
@pytest.mark.parametrize("L", [12, 19, 20])
def test_ragged_shapes_bit_exact(shape, L):
    M, N, K = shape
    A = inputs.lognormal_matrix(M, K, 1.0, seed=10)
    B = inputs.lognormal_matrix(K, N, 1.0, seed=11)
    C = gu.dgemm(A, B, L, lda=M + 1, ldb=K + 7, ldc=M + 5)
    assert gu.bits_equal(C, ozaki2.dgemm(A, B, L).C)


@pytest.mark.parametrize("L", [2, 13, 15, 16, 18, 24, 27])
def test_every_modulus_count_bit_exact(L):
    A = inputs.lognormal_matrix(96, 200, 0.5, seed=0)
    B = inputs.lognormal_matrix(200, 40, 0.5, seed=1)
    assert gu.bits_equal(gu.dgemm(A, B, L), ozaki2.dgemm(A, B, L).C)


@pytest.mark.parametrize("shape,L", [((64, 128, 20000), 19), ((40, 256, 65536), 19), ((128, 128, 131072), 20)])
def test_long_inner_products_bit_exact(shape, L):
    """K beyond 17476 takes the integer recombination before the TMEM release; K up to 131072 keeps every
    FP32 partial sum an exact integer (128 K <= 2^24 with limbs |c| <= 8)."""
    M, N, K = shape
    A = inputs.lognormal_matrix(M, K, 0.5, seed=20)
    B = inputs.lognormal_matrix(K, N, 0.5, seed=21)
    A[0, :] = np.abs(A[0, :])                         # a row of one sign against a column of one sign: no cancellation
    B[:, 0] = np.abs(B[:, 0])
    assert gu.bits_equal(gu.dgemm(A, B, L), ozaki2.dgemm(A, B, L).C)


@pytest.mark.parametrize("shape", [(16, 64, 140000), (16, 130, 290000)])
def test_k_beyond_one_limb_gemm_range_bit_exact(shape):
    """K above 131072 runs one limb GEMM per range of 131072 and adds the residues modulo each modulus (this build's
    extension: Lemma 3 only bounds K, the paper never splits it): a short last range (fast recombination) and
    three ranges with a long last one."""
    M, N, K = shape
    A = inputs.lognormal_matrix(M, K, 0.5, seed=30)
    B = inputs.lognormal_matrix(K, N, 0.5, seed=31)
    A[0, :] = np.abs(A[0, :])
    B[:, 0] = np.abs(B[:, 0])
    assert gu.bits_equal(gu.dgemm(A, B, 19), ozaki2.dgemm(A, B, 19).C)


@pytest.mark.parametrize("shape,L", [((384, 512, 700), 19), ((1000, 256, 64), 19), ((130, 768, 768), 27), ((2048, 1024, 512), 19),
                                     ((121, 256, 1), 12), ((600, 512, 1024), 19), ((250, 256, 1792), 19), ((250, 256, 1793), 19),
                                     ((9000, 512, 300), 16)])
def test_short_k_two_accumulator_form_bit_exact(shape, L):
    """K up to 1792 with a column count that pads to a multiple of 256 runs the two-accumulator limb GEMM (row tiles of
    120, the last one ragged, gamma planes on the A side, residues staged through shared memory, more tiles than CTA
    pairs in the 9000-row case); K = 1793 is the first size on the three-accumulator kernel."""
    M, N, K = shape
    A = inputs.lognormal_matrix(M, K, 1.0, seed=50)
    B = inputs.lognormal_matrix(K, N, 1.0, seed=51)
    A[0, :] = np.abs(A[0, :])
    B[:, 0] = np.abs(B[:, 0])
    assert gu.bits_equal(gu.dgemm(A, B, L), ozaki2.dgemm(A, B, L).C)


@pytest.mark.parametrize("L", list(range(2, 28)))
def test_every_moduli_count_on_cta_pairs(L):
    """256 columns put the product on CTA pairs: K = 200 on the two-accumulator kernel, K = 1900 on the three-accumulator
    one, for every moduli count the library accepts (the small shapes elsewhere run the single-CTA kernel)."""
    for K, seed in ((200, 60), (1900, 62)):
        A = inputs.lognormal_matrix(136, K, 0.5, seed=seed)
        B = inputs.lognormal_matrix(K, 256, 0.5, seed=seed + 1)
        assert gu.bits_equal(gu.dgemm(A, B, L), ozaki2.dgemm(A, B, L).C), f"K = {K}"


def test_more_than_65535_columns():
    """N beyond the y-dimension limit of a CUDA grid: the O(N^2) kernels loop over the columns.  Small integers
    make C the exact integer product, so the whole matrix is checked against an int64 product."""
    M, N, K = 20, 66000, 24
    A = inputs.small_integer_matrix(M, K, 1000, seed=5)
    B = inputs.small_integer_matrix(K, N, 1000, seed=6)
    C = gu.dgemm(A, B, 19)
    assert gu.bits_equal(C, (A.astype(np.int64) @ B.astype(np.int64)).astype(np.float64))
    j = np.array([0, 1, 65534, 65535, 65536, 65999])            # a few columns also against the oracle
    assert gu.bits_equal(C[:, j], ozaki2.dgemm(A, B[:, j], 19).C)


def test_k_ranges_small_integers_exact_over_several_tiles():
    """Two ranges over a 3 x 3 grid of tiles: integer inputs make C the exact integer product, which an FP64
    matrix product of these magnitudes (|sum| < 2^53) delivers without rounding."""
    M, N, K = 384, 300, 200000
    A = inputs.small_integer_matrix(M, K, 1000, seed=3)
    B = inputs.small_integer_matrix(K, N, 1000, seed=4)
    C = gu.dgemm(A, B, 19)
    assert gu.bits_equal(C, A @ B)


def test_small_integers_give_the_exact_integer_product():
    A = inputs.small_integer_matrix(200, 333, 1000, seed=1)
    B = inputs.small_integer_matrix(333, 150, 1000, seed=2)
    A[7, :] = 0.0
    C = gu.dgemm(A, B, 19)
    ref = (A.astype(np.int64) @ B.astype(np.int64)).astype(np.float64)
    assert gu.bits_equal(C, ref)


def test_paper_law_phi0_equals_fl_of_exact_product():
    """Section 7.1: with one exponent per row/column the conversion is exact, so the output is
    the exact product rounded once."""
    A = inputs.exponent_spread_matrix(64, 2048, 0, seed=0)
    B = inputs.exponent_spread_matrix(2048, 48, 0, seed=1)
    assert gu.bits_equal(gu.dgemm(A, B, 19), exact.fl_matmul(A, B))


def test_wide_exponent_range_and_extremes_bit_exact():
    A = inputs.lognormal_matrix(64, 128, 4.0, seed=0)
    B = inputs.lognormal_matrix(128, 64, 4.0, seed=1)
    A[0, :] *= 2.0 ** 500
    A[1, :] *= 2.0 ** -500
    B[:, 0] *= 2.0 ** 400
    B[:, 1] *= 2.0 ** -520                       # products reach the subnormal range
    A[2, :] = 0.0
    C = gu.dgemm(A, B, 19)
    assert gu.bits_equal(C, ozaki2.dgemm(A, B, 19).C)


def test_invalid_arguments():
    gu.register_small_workspace(8 << 20)          # every call below must be rejected before anything is launched
    assert ozk.ozk_dgemm(8, 8, 8, None, 8, None, 8, None, 8, 19, 0) == ozk.OZK_ERR_INVALID_ARG      # null pointers
    assert ozk.ozk_dgemm(4096, 4096, 4096, None, 4096, None, 4096, None, 4096, 19, 0) == ozk.OZK_ERR_WORKSPACE
    assert ozk.ozk_dgemm(0, 8, 8, None, 1, None, 8, None, 1, 19, 0) == ozk.OZK_OK                   # empty result


def test_single_cta_kernel_bit_exact_in_a_subprocess():
    """Shapes whose padded column count is a multiple of 256 run the CTA-pair kernel by default; with
    OZK_GEMM_PAIR=0 the same shapes run the single-CTA kernel and must give the same bits as the oracle."""
    import os
    import subprocess
    import sys
    code = (
        "import numpy as np\n"
        "from oracle import ozaki2\n"
        "from paper_2608_06812_b200 import inputs\n"
        "from tests import gpu_util as gu\n"
        "for (M, N, K, L) in [(256, 256, 256, 14), (384, 512, 1280, 19), (130, 768, 4096, 20), (200, 256, 20000, 19)]:\n"
        "    A = inputs.lognormal_matrix(M, K, 1.0, seed=0); B = inputs.lognormal_matrix(K, N, 1.0, seed=1)\n"
        "    assert gu.bits_equal(gu.dgemm(A, B, L), ozaki2.dgemm(A, B, L).C), (M, N, K, L)\n"
        "print('pair ok')\n")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", code], cwd=root, env=dict(os.environ, OZK_GEMM_PAIR="0"),
                         capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "pair ok" in out.stdout, out.stdout + out.stderr
