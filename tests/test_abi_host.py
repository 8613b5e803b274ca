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


@pytest.mark.parametrize("d", [16, 64, 128, 256])
def test_structured_preconditioners_equal_the_oracle(d):
    """Identity and sign-flipped Sylvester-Hadamard (Section 3.2's fast transforms; Section 5's rows without R): the
    library's closed form against the oracle's recursion, entry by entry after rounding to float32."""
    signs = np.random.default_rng(d).choice([-1, 1], size=d).astype(np.int8)
    S = pq.pq_make_structured_rotation(d, pq.ROTATION_HADAMARD, signs).numpy()
    want = orc.make_structured_rotation(d, "hadamard", signs.astype(np.float64))
    assert np.array_equal(S, want.astype(np.float32))
    assert np.max(np.abs(S.astype(np.float64).T @ S.astype(np.float64) - np.eye(d))) < 1e-6
    assert np.array_equal(pq.pq_make_structured_rotation(d, pq.ROTATION_IDENTITY).numpy(), np.eye(d, dtype=np.float32))
    bad = signs.copy()
    bad[3] = 0
    out = np.empty((d, d), dtype=np.float32)
    f = pq.lib().pq_make_structured_rotation
    assert f(d, pq.ROTATION_HADAMARD, bad.ctypes.data, out.ctypes.data) == pq.ERR_INVALID_ARG
    assert f(d, pq.ROTATION_HADAMARD, None, out.ctypes.data) == pq.ERR_INVALID_ARG
    assert f(d, 7, signs.ctypes.data, out.ctypes.data) == pq.ERR_INVALID_ARG
    assert f(d, pq.ROTATION_IDENTITY, None, None) == pq.ERR_INVALID_ARG
    assert f(48, pq.ROTATION_HADAMARD, signs.ctypes.data, out.ctypes.data) == pq.ERR_UNSUPPORTED


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


def test_level1_decision_table_is_built_for_any_ascending_codebook():
    """pq_build_tables checks its level-1 cell table against the boundaries it was built from (both guarantees of
    every cell) and would refuse a codebook whose table fails: random ascending level-1 codebooks, the uniform one
    turned by small and large angles, boundaries packed closely."""
    cen, bnd = pq.pq_fit_codebooks()
    rng = np.random.default_rng(0)
    cases = [np.sort(rng.uniform(0, 2 * math.pi, 16)) for _ in range(40)]
    cases += [((np.arange(16) + 0.5) * math.pi / 8 + s) % (2 * math.pi) for s in (1e-9, 1e-4, 0.01, 0.19, 0.2, math.pi / 16)]
    cases += [np.linspace(1.0, 1.0 + 15e-4, 16), np.linspace(0.0, 2 * math.pi - 1e-7, 16)]
    for theta in cases:
        c = cen.clone()
        c[:16] = torch.from_numpy(np.sort(theta))
        b = bnd.clone()
        b[:15] = 0.5 * (c[:15] + c[1:16])
        assert pq.pq_build_tables(c, b).numel() == pq.lib().pq_tables_bytes()


def test_histogram_clustering_matches_the_oracle():
    """pq_fit_codebooks_from_histograms against the oracle's k-means on the same binned sample: Gaussian and
    anisotropic rows, 1024 and 256 bins, a level without counts, and a start other than the analytic codebook."""
    rng = np.random.default_rng(3)
    S = orc.make_rotation(16, 5)
    off = orc.fit_codebooks()
    for n_bins, x in ((1024, rng.normal(size=(3000, 16))), (256, rng.normal(size=(2000, 16)) * np.linspace(0.1, 4, 16))):
        hist = orc.angle_histograms(x, S, 4, n_bins)
        cen, bnd = pq.pq_fit_codebooks_from_histograms(torch.from_numpy(hist))
        for level in range(1, 5):
            want, want_b = orc.kmeans_on_histogram(hist[level - 1], level, off.centroids[level - 1])
            o, n = (0, 16) if level == 1 else (16 + 4 * (level - 2), 4)
            ob = 0 if level == 1 else 15 + 3 * (level - 2)
            assert np.max(np.abs(cen.numpy()[o:o + n] - want)) < 1e-12
            assert np.max(np.abs(bnd.numpy()[ob:ob + n - 1] - want_b)) < 1e-12
        pq.pq_build_tables(cen, bnd)  # a valid codebook
    hist[2] = 0
    init = torch.from_numpy(off.flat_centroids() + 0.01)
    cen, _ = pq.pq_fit_codebooks_from_histograms(torch.from_numpy(hist), init)
    assert np.array_equal(cen.numpy()[20:24], init.numpy()[20:24])  # nothing observed at level 3
    want, _ = orc.kmeans_on_histogram(hist[3], 4, init.numpy()[24:28])
    assert np.max(np.abs(cen.numpy()[24:28] - want)) < 1e-12
    L = pq.lib()
    assert L.pq_fit_codebooks_from_histograms(None, 1024, None, cen.data_ptr(), cen.data_ptr()) == pq.ERR_INVALID_ARG
    assert L.pq_fit_codebooks_from_histograms(cen.data_ptr(), 4096, None, cen.data_ptr(), cen.data_ptr()) == pq.ERR_INVALID_ARG


def test_general_configurations_sizes_and_codebooks():
    """pq_general_*: the row of (4,2,2,2) at d = 128 is the 62 bytes of Section 4.1; the full recursion with 3 bits
    is Section 4's b_FPN + (d - 1) b bits (padded to bytes per level); codebooks equal the oracle's Lloyd-Max ones."""
    assert pq.GeneralConfig.of(128, (4, 2, 2, 2)).sizes() == (28, 24, 120, 8, 62)
    n_cen, n_bnd, n_codes, n_radii, row = pq.GeneralConfig.of(128, (3,) * 7).sizes()
    assert (n_cen, n_bnd, n_codes, n_radii) == (56, 49, 127, 1)
    code_bytes = sum(-(-(128 >> (l + 1)) * 3 // 8) for l in range(7))      # 24 + 12 + 6 + 3 + 2 + 1 + 1
    assert code_bytes == 49 and row == code_bytes + 1 + 2 and row * 8 >= 16 + 127 * 3   # radii start at an even offset
    for d, bits in ((64, (4, 3, 2)), (256, (2,) * 8), (16, (2, 2, 2, 2))):
        cen, bnd = pq.pq_general_fit_codebooks(pq.GeneralConfig.of(d, bits))
        cb = orc.fit_codebooks(bits)
        assert np.max(np.abs(cen.numpy() - cb.flat_centroids())) < 1e-10 and np.max(np.abs(bnd.numpy() - cb.flat_boundaries())) < 1e-10
    for d, bits in ((48, (2, 2)), (16, (2,) * 5), (64, (7, 2)), (512, (2, 2)), (64, ()), (64, (0, 2))):
        with pytest.raises(pq.PolarQuantError):
            pq.GeneralConfig.of(d, bits).sizes()
    cfg = pq.GeneralConfig.of(64, (4, 2))
    L = pq.lib()
    assert L.pq_general_cache_bytes(ctypes.addressof(cfg), 2, 3, 10) == 2 * 3 * 2 * 10 * cfg.sizes()[4]
    assert L.pq_general_encode_kv(ctypes.addressof(cfg), 2, None, 16, 16, 16, 1, 128, 64, 16, 1, 4, 16, 16, 8, 16, None) == pq.ERR_INVALID_ARG
    assert L.pq_general_decode_attention(ctypes.addressof(cfg), 18, 2, 16, 16, 16, 1, 16, 16, 1, 8, 0.1, 16, 16, None) == pq.ERR_UNSUPPORTED


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
    assert L.pq_angle_histograms(128, 8, 16, 16, 16, 1, 1024, 128, 4, 1024, nul, 16, nul) == pq.ERR_INVALID_ARG
    assert L.pq_angle_histograms(128, 8, 16, 16, 16, 1, 1024, 128, 4, 2048, 16, 16, nul) == pq.ERR_INVALID_ARG
    assert L.pq_angle_histograms(48, 8, 16, 16, 16, 1, 1024, 128, 4, 1024, 16, 16, nul) == pq.ERR_UNSUPPORTED
    assert L.pq_angle_histograms(128, 8, 16, 16, 16, 1, 1024, 128, 4, 1024, 20, 16, nul) == pq.ERR_ALIGNMENT
    assert L.pq_unpack_codes(128, 8, 16, 1, 64, 65, 16, 16, nul) == pq.ERR_INVALID_ARG
    good = api.Paging(16, 256, 4, 10)
    for bad in (api.Paging(0, 256, 4, 10), api.Paging(16, 0, 4, 10), api.Paging(16, 192, 4, 10), api.Paging(16, 256, 4, 0)):
        assert L.pq_decode_attention_paged(128, 32, 8, 16, 16, 16, 1, 16, 16, 1, ctypes.addressof(bad), 64, 0.1, 16, 16, 16,
                                           nul) == pq.ERR_INVALID_ARG
        assert L.pq_append_kv_paged(128, 8, 16, 16, 16, 16, 1, 4, 16, 16, ctypes.addressof(bad), 16, nul) == pq.ERR_INVALID_ARG
    assert L.pq_decode_attention_paged(128, 32, 8, 16, 16, 16, 1, 16, 16, 1, None, 64, 0.1, 16, 16, 16, nul) == pq.ERR_INVALID_ARG
    assert L.pq_encode_kv_paged(128, 8, 16, 16, 16, 16, 1, 1024, 128, nul, 1, 4, 16, 16, ctypes.addressof(good), 16,
                                nul) == pq.ERR_INVALID_ARG  # no cu_seqlens
    assert pq.pq_paged_cache_bytes(128, 8, 256, 10) == 10 * 8 * 256 * 2 * 62
    assert pq.pq_paged_cache_bytes(64, 2, 64, 3) == 3 * 2 * 64 * 2 * 31
    with pytest.raises(pq.PolarQuantError):
        pq.pq_paged_cache_bytes(128, 8, 192, 10)
    assert L.pq_dequant_kv(128, 8, 16, 16, 16, 1, 64, 0, 16, nul) == pq.ERR_INVALID_ARG


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "LIB_PATH", str(ROOT / "no_such_library.so"))
    with pytest.raises(ImportError):
        pq.pq_fit_codebooks()
