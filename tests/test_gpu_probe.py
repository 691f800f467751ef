"""Pins of the hardware formats with single tcgen05.mma sequences: E2M1 nibble codes, nibble order
inside a byte, UE8M0 scale byte, and exactness of the FP32 accumulation of integer limb products
(the assumption of Lemma 2 / Lemma 3) on this GPU."""
import numpy as np
import pytest
import torch

from oracle import base13
from paper_2608_06812_b200 import binding as ozk
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def pack(codes: np.ndarray) -> np.ndarray:
    """codes[r, k] in 0..15 -> bytes [r, k/2], the lower-k element in the low nibble."""
    return (codes[:, 0::2] | (codes[:, 1::2] << 4)).astype(np.uint8)


def doubled(codes: np.ndarray) -> np.ndarray:
    table = np.array([base13.e2m1_decode_doubled(c) for c in range(16)], dtype=np.int64)
    return table[codes]


def run_probe(Pc: np.ndarray, Qc: np.ndarray, scale_byte: int) -> np.ndarray:
    K = Pc.shape[1]
    gu.ensure_workspace(1 << 20)
    dP, dQ = torch.from_numpy(pack(Pc)).cuda(), torch.from_numpy(pack(Qc)).cuda()
    dD = torch.full((128, 128), float("nan"), dtype=torch.float32, device="cuda")
    ozk.check(ozk.ozk_stage_mma_probe(dP.data_ptr(), dQ.data_ptr(), K, scale_byte, dD.data_ptr(), gu.stream()), "probe")
    ozk.check(ozk.ozk_get_async_status(gu.stream()), "status")
    return dD.cpu().numpy().astype(np.float64)


def reference(Pc, Qc, scale_byte):
    scale = 2.0 ** (scale_byte - 127)
    return (doubled(Pc) @ doubled(Qc).T).astype(np.float64) / 4.0 * scale * scale


def test_every_code_pair_and_nibble_order():
    K = 256
    Pc = np.zeros((128, K), dtype=np.int64)
    Qc = np.zeros((128, K), dtype=np.int64)
    for r in range(128):                      # row r: code r % 16 at an odd or even k that depends on r
        Pc[r, (3 * r + 1) % K] = r % 16
        Qc[r, :] = (r // 8) % 16              # column c meets it with code c // 8
    for sb in (0x7F, 0x80):
        assert np.array_equal(run_probe(Pc, Qc, sb), reference(Pc, Qc, sb))


def test_scale_byte_is_a_power_of_two_exponent():
    rng = np.random.default_rng(0)
    Pc = rng.integers(0, 16, size=(128, 256))
    Qc = rng.integers(0, 16, size=(128, 256))
    base = run_probe(Pc, Qc, 0x7F)
    assert np.array_equal(base, reference(Pc, Qc, 0x7F))
    assert np.array_equal(run_probe(Pc, Qc, 0x80), 4.0 * base)
    assert np.array_equal(run_probe(Pc, Qc, 0x7E), 0.25 * base)


@pytest.mark.parametrize("K", [256, 1024, 16384, 65536])
def test_random_limbs_accumulate_exactly(K):
    rng = np.random.default_rng(K)
    Pc = rng.integers(0, 16, size=(128, K))
    Qc = rng.integers(0, 16, size=(128, K))
    assert np.array_equal(run_probe(Pc, Qc, 0x80), reference(Pc, Qc, 0x80))


@pytest.mark.parametrize("K", [16384, 65536, 131072])
def test_adversarial_accumulation_is_exact(K):
    """Same-sign +-8 limbs drive the running sum to 64*K (2^23 at K = 131072); rows that then add
    +-1 products must not lose them, and alternating signs must cancel exactly."""
    c8, cm8, c1, cm1 = base13.e2m1_code(8), base13.e2m1_code(-8), base13.e2m1_code(1), base13.e2m1_code(-1)
    Pc = np.full((128, K), c8, dtype=np.int64)
    Qc = np.full((128, K), c8, dtype=np.int64)
    Pc[1, K // 2:] = c1                         # large running sum, then +1 addends
    Pc[2, K // 2:] = cm1                        # ... and -1 addends
    Pc[3, 1::2] = cm8                           # alternating +64 / -64
    Pc[4, :K // 2] = c1                         # small addends first, large afterwards
    Qc[5, :] = cm8                              # all-negative column
    Qc[6, 0::2] = c1
    got = run_probe(Pc, Qc, 0x80)
    want = reference(Pc, Qc, 0x80)
    assert np.abs(want).max() == 64 * K
    assert np.array_equal(got, want)


def test_bounded_wait_expires_cleanly():
    """A barrier that expects 16 bytes nobody sends: the kernel's wait gives up after its time limit, the status word
    reads OZK_ERR_DEVICE_TIMEOUT exactly once, tensor memory is released and the next calls work as before."""
    import time
    from oracle import ozaki2
    from paper_2608_06812_b200 import inputs
    gu.ensure_workspace(1 << 20)
    t0 = time.perf_counter()
    ozk.check(ozk.ozk_stage_wait_probe(gu.stream()), "ozk_stage_wait_probe")
    assert ozk.ozk_get_async_status(gu.stream()) == ozk.OZK_ERR_DEVICE_TIMEOUT
    assert 1.0 < time.perf_counter() - t0 < 10.0             # the limit is two seconds
    assert ozk.ozk_get_async_status(gu.stream()) == ozk.OZK_OK   # reading the status cleared it
    A = inputs.lognormal_matrix(130, 300, 1.0, seed=1)
    B = inputs.lognormal_matrix(300, 260, 1.0, seed=2)
    assert gu.bits_equal(gu.dgemm(A, B, 19), ozaki2.dgemm(A, B, 19).C)
