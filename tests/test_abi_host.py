"""CPU-only checks of the boundary: the library loads, exports every symbol the header declares,
validates arguments before touching the device, and its host-side generators agree with the oracle."""
import ctypes
import math
import pathlib
import re

import numpy as np
import pytest
import torch

import __graft_entry__ as entry
import paper_2502_02617_b200 as pq
from paper_2502_02617_b200 import api
from oracle import polarquant_oracle as orc

ROOT = pathlib.Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def test_library_exports_every_declared_symbol():
    header = (ROOT / "include" / "polarquant.h").read_text()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(pq_[a-z0-9_]+)\s*\(", header))
    assert {"pq_make_rotation", "pq_fit_codebooks", "pq_encode_kv", "pq_append_kv", "pq_decode_attention"} <= declared
    handle = ctypes.CDLL(api.LIB_PATH)
    for name in declared:
        assert hasattr(handle, name), name
    assert declared == set(api._SIGNATURES), "python binding and header disagree"


def test_status_strings_and_constants():
    assert pq.status_string(0) == "ok"
    for code in range(-9, 0):
        assert pq.status_string(code) not in ("ok", "unknown status")
    assert pq.status_string(-99) == "unknown status"
    assert pq.token_block() % 8 == 0


@pytest.mark.parametrize("d", [16, 128])
def test_rotation_is_orthogonal_seeded_and_gaussianising(d):
    S = pq.pq_make_rotation(d, 5).double().numpy()
    assert np.max(np.abs(S.T @ S - np.eye(d))) < 1e-6  # float32 storage
    assert np.array_equal(pq.pq_make_rotation(d, 5).numpy().astype(np.float64), S)
    assert not np.allclose(pq.pq_make_rotation(d, 6).double().numpy(), S)
    # a Haar rotation of a fixed unit vector has coordinates ~ N(0, 1/d): check the second moment spread
    row = S[0] * math.sqrt(d)
    assert 0.5 < np.mean(row ** 2) < 1.5 and np.max(np.abs(row)) < 6.0


def test_rotation_rejects_bad_arguments():
    assert pq.lib().pq_make_rotation(0, 1, None) == pq.ERR_INVALID_ARG
    assert pq.lib().pq_make_rotation(16, 1, None) == pq.ERR_INVALID_ARG


def test_codebooks_match_the_oracle_and_reject_other_bit_widths():
    cen, bnd = pq.pq_fit_codebooks()
    cb = orc.fit_codebooks()
    assert np.max(np.abs(cen.numpy() - cb.flat_centroids())) < 1e-12
    assert np.max(np.abs(bnd.numpy() - cb.flat_boundaries())) < 1e-12
    with pytest.raises(pq.PolarQuantError) as e:
        pq.pq_fit_codebooks((3, 3, 3, 3))
    assert e.value.status == pq.ERR_UNSUPPORTED


def test_tables_reject_unsorted_or_out_of_range_codebooks():
    cen, bnd = pq.pq_fit_codebooks()
    assert pq.pq_build_tables(cen, bnd).numel() == pq.lib().pq_tables_bytes()
    bad = cen.clone()
    bad[3], bad[4] = cen[4], cen[3]
    with pytest.raises(pq.PolarQuantError):
        pq.pq_build_tables(bad, bnd)
    bad = bnd.clone()
    bad[20] = 2.0  # level-3 boundary outside (0, pi/2)
    with pytest.raises(pq.PolarQuantError):
        pq.pq_build_tables(cen, bad)


def test_cache_costs_62_bytes_per_token_at_d128():
    T = pq.token_block()
    assert pq.pq_cache_bytes(128, 1, 8, 32768) == 2 * 8 * 32768 * 62
    assert pq.pq_cache_bytes(128, 3, 2, T + 1) == 3 * 2 * 2 * (2 * T) * 62  # rounded up to token-blocks
    assert pq.pq_cache_bytes(64, 1, 1, T) == 2 * T * 31
    for bad in ((100, 1, 1, 64), (128, 0, 1, 64), (128, 1, 1, 0)):
        with pytest.raises(pq.PolarQuantError):
            pq.pq_cache_bytes(*bad)
    assert pq.pq_workspace_bytes(128, 8, 32, 8, 32768) > 8 * 32 * 128 * 4
    with pytest.raises(pq.PolarQuantError):
        pq.pq_workspace_bytes(128, 8, 30, 8, 1024)  # heads not divisible


def test_device_entry_points_validate_before_launching():
    L = pq.lib()
    nul = None
    assert L.pq_encode_kv(128, 8, nul, nul, nul, nul, 1, 1024, 128, nul, 1, 4, nul, nul, 64, nul, nul) == pq.ERR_INVALID_ARG
    assert L.pq_encode_kv(100, 8, 16, 16, 16, 16, 1, 1024, 128, 16, 1, 4, 16, 16, 64, 16, nul) == pq.ERR_UNSUPPORTED
    assert L.pq_encode_kv(128, 8, 24, 16, 16, 16, 1, 1024, 128, 16, 1, 4, 16, 16, 64, 16, nul) == pq.ERR_ALIGNMENT
    assert L.pq_encode_kv(128, 8, 16, 16, 16, 16, 7, 1024, 128, 16, 1, 4, 16, 16, 64, 16, nul) == pq.ERR_UNSUPPORTED
    assert L.pq_append_kv(128, 8, 16, 16, nul, 16, 1, 4, 16, 16, 64, 16, nul) == pq.ERR_INVALID_ARG
    assert L.pq_decode_attention(128, 32, 8, 16, 16, 16, 1, 16, 16, 0, 64, 64, 0.1, 16, 16, 16, nul) == pq.ERR_INVALID_ARG
    assert L.pq_decode_attention(128, 30, 8, 16, 16, 16, 1, 16, 16, 1, 64, 64, 0.1, 16, 16, 16, nul) == pq.ERR_INVALID_ARG
    assert L.pq_decode_attention(128, 32, 8, 16, 16, 8, 1, 16, 16, 1, 64, 64, 0.1, 16, 16, 16, nul) == pq.ERR_ALIGNMENT
    assert L.pq_unpack_codes(128, 8, 16, 1, 64, 65, 16, 16, nul) == pq.ERR_INVALID_ARG
    assert L.pq_dequant_kv(128, 8, 16, 16, 16, 1, 64, 0, 16, nul) == pq.ERR_INVALID_ARG


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "LIB_PATH", str(ROOT / "no_such_library.so"))
    with pytest.raises(ImportError):
        pq.pq_fit_codebooks()
