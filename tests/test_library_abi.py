"""CPU-side checks of the C-ABI library: it builds, loads, exports every symbol the header
declares, and its host-side constants agree with the paper's printed values and the oracle."""
import json
import os
import re

import pytest

from oracle import moduli
from paper_2608_06812_b200 import binding as ozk
from paper_2608_06812_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLD = json.load(open(os.path.join(ROOT, "tests", "golden", "paper_constants.json")))


@pytest.fixture(scope="module", autouse=True)
def built():
    build.build()


def test_every_declared_symbol_is_exported_and_bound():
    header = open(os.path.join(ROOT, "include", "ozk.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(ozk_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    handle = ozk.lib()
    for name in sorted(declared):
        assert hasattr(handle, name), f"{name} is declared but not exported"
    assert declared == set(ozk.SIGNATURES), declared ^ set(ozk.SIGNATURES)


def test_moduli_match_the_printed_list_and_the_oracle():
    assert ozk.ozk_get_moduli(19) == GOLD["section5_1_moduli_L19"]
    assert ozk.ozk_get_moduli(27) == moduli.select_moduli(27)
    with pytest.raises(ozk.OzkError):
        ozk.ozk_get_moduli(28)


def test_capacity_and_crt_constants_match_the_oracle():
    for K in (1, 256, 4096, 8192, 16384, 131072, 300000, ozk.OZK_MAX_K):
        for L in range(4, 28):
            assert ozk.ozk_capacity_bits(K, L) == moduli.capacity_bits(K, L)
    for K in (40, 4096, 16384, 300000):
        for L in (19, 20, 21, 22, 27):
            for cap in (40, 53, 56, 57, 62):
                assert ozk.ozk_capacity_bits_ext(K, L, cap) == moduli.capacity_bits(K, L, cap=cap)
    assert ozk.ozk_capacity_bits_ext(16384, 22, 63) == ozk.OZK_ERR_INVALID_ARG
    assert ozk.ozk_capacity_bits(16384, 19) == 53
    assert ozk.ozk_capacity_bits(1 << 20, 2) == ozk.OZK_ERR_UNSUPPORTED
    for L in (2, 14, 19, 27):
        P, w = ozk.ozk_get_crt_constants(L)
        Pw, ww = moduli.crt_weights(moduli.select_moduli(L))
        assert P == Pw and w == ww


def test_argument_errors_need_no_gpu():
    assert ozk.ozk_dgemm_workspace_bytes(-1, 1, 1, 19) == 0
    assert ozk.ozk_dgemm_workspace_bytes(1, 1, 1, 1) == 0
    small, big = ozk.ozk_dgemm_workspace_bytes(256, 256, 256, 14), ozk.ozk_dgemm_workspace_bytes(4096, 4096, 4096, 19)
    assert 0 < small < big
    # planes: 2 limbs x L x (M + N) x K / 2 bytes, residues: L x M x N bytes
    assert big >= 19 * (2 * 2 * 4096 * 4096 // 2 + 4096 * 4096)
    # K beyond one limb-GEMM range: a second set of residue matrices for the ranges after the first
    one_range = ozk.ozk_dgemm_workspace_bytes(128, 128, ozk.OZK_CHUNK_K, 19)
    two_ranges = ozk.ozk_dgemm_workspace_bytes(128, 128, ozk.OZK_CHUNK_K + 256, 19)
    assert two_ranges - one_range >= 19 * 128 * 128 + 19 * 2 * 2 * 128 * 256 // 2
    ozk.ozk_set_workspace(None, 0)
    assert ozk.ozk_dgemm(8, 8, 8, None, 8, None, 8, None, 8, 19, None) == ozk.OZK_ERR_WORKSPACE
    assert ozk.ozk_dgemm(8, 8, ozk.OZK_MAX_K + 1, None, 8, None, ozk.OZK_MAX_K + 1, None, 8, 19, None) == ozk.OZK_ERR_UNSUPPORTED
    assert ozk.ozk_dgemm(8, 8, 8, None, 8, None, 8, None, 8, 1, None) == ozk.OZK_ERR_INVALID_ARG
    assert ozk.ozk_dgemm(-8, 8, 8, None, 8, None, 8, None, 8, 19, None) == ozk.OZK_ERR_INVALID_ARG
    assert ozk.ozk_set_workspace(12345, 1 << 20) == ozk.OZK_ERR_INVALID_ARG       # not 256-byte aligned
    assert "workspace" in ozk.ozk_status_string(ozk.OZK_ERR_WORKSPACE)
    assert "sm_100a" in ozk.ozk_version()
