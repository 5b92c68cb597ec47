"""Host-side logic of the C-ABI library, no GPU: the library loads, exports every symbol the
header declares, and its pure host functions agree with the independent oracle."""
import ctypes
import re
from pathlib import Path

import numpy as np
import pytest

import oracle
import paper_2605_02905_b200 as eosq

ROOT = Path(__file__).resolve().parents[1]


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2605_02905_b200 import build
    build.build()


def test_every_declared_symbol_is_exported():
    header = (ROOT / "include" / "eosq.h").read_text()
    declared = set(re.findall(r"^(?:int|size_t|double|int64_t|const char \*)\s*\*?\s*(eosq_[a-z_0-9]+)\s*\(", header, re.M))
    declared -= {"eosq_status"}
    assert declared == set(eosq.EXPORTS)
    L = ctypes.CDLL(str(eosq.LIB_PATH))
    for name in declared:
        assert hasattr(L, name), name


def test_pilot_k_matches_paper(golden):
    assert eosq.eosq_pilot_k(128) == golden["pilot_k_d128"]
    assert eosq.eosq_pilot_k(64) == golden["pilot_k_d64"]
    assert eosq.eosq_pilot_k(2) == -1


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_codebook_matches_oracle(bits):
    for d in (64, 128):
        c, t = eosq.eosq_codebook(bits, d)
        co, to = oracle.codebook(bits, d)
        assert np.abs(c - co).max() < 1e-12
        assert np.abs(t - to).max() < 1e-12
        assert t[len(t) // 2] == 0.0


def test_codebook_rejects_bad_arguments():
    L = eosq.lib()
    buf = np.zeros(512)
    assert L.eosq_codebook(0, 128, buf.ctypes.data, None) == eosq.EOSQ_ERR_INVALID_ARG
    assert L.eosq_codebook(9, 128, buf.ctypes.data, None) == eosq.EOSQ_ERR_INVALID_ARG
    assert L.eosq_codebook(2, 0, buf.ctypes.data, None) == eosq.EOSQ_ERR_INVALID_ARG
    assert L.eosq_codebook(2, 128, None, None) == eosq.EOSQ_ERR_INVALID_ARG


@pytest.mark.parametrize("d,seed", [(128, 0), (128, 2**63 + 5), (64, 9)])
def test_rotation_matches_oracle(d, seed):
    pi = eosq.eosq_rotation(d, seed)
    po = oracle.rotation(d, seed)
    assert np.abs(pi - po).max() < 1e-12
    assert np.abs(pi.T @ pi - np.eye(d)).max() < 1e-13


def test_layout_and_bit_accounting(golden):
    lay = eosq.eosq_layout(1024, 128, 2)
    assert lay["k"] == 11 and lay["rmax"] == 16 and lay["row_bytes"] == 32
    assert lay["codes_bytes"] == 1024 * 32 and lay["norms_bytes"] == 2048
    assert lay["P_bytes"] == 16 * 1024 * 2 and lay["V_bytes"] == 16 * 128 * 2
    for bad in ((64, 128, 2), (1024, 64, 2), (1024, 128, 5), (8192, 128, 2), (1028, 128, 2)):
        s = eosq._LayoutStruct()
        assert eosq.lib().eosq_layout(*bad, ctypes.addressof(s)) == eosq.EOSQ_ERR_UNSUPPORTED
    assert abs(eosq.eosq_bits_per_entry(0, 1, 128, 128, 4) - golden["svd1_overhead_bits_n128_d128_bs4"]) < 0.005
    assert abs(eosq.eosq_bits_per_entry(2, 5.6, 128, 128, 4) - 2 - golden["eoptshrinkq_overhead_bits_rbar5p6"]) < 0.005
    assert eosq.eosq_bits_per_entry(2, 3, 128, 128, 4, True) == oracle.bits_per_entry(2, 3, 128, 128, 4, prod=True)


def test_workspace_size_saturates():
    one = eosq.eosq_workspace_bytes(1, 1024, 128)
    assert one >= 128 * 128 * 8
    assert eosq.eosq_workspace_bytes(10**6, 1024, 128) == eosq.eosq_workspace_bytes(10**5, 1024, 128)
    assert eosq.eosq_workspace_bytes(0, 1024, 128) == 0
