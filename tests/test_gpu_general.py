"""The general recursion depth / bit table entry points (pq_general_*) against the oracle, which is written for any
number of levels and any bits per level: codes, radii, DeQuant and attention for the full log2 d recursion with
3 bits everywhere (the count of Section 4), shallower recursions, other head dims, and the (4,2,2,2) case, whose
codes must equal those of the tuned path."""
import numpy as np
import pytest
import torch

import paper_2502_02617_b200 as pq
from paper_2502_02617_b200 import synthetic
from oracle import polarquant_oracle as orc
from parity_utils import (TOL_ATTENTION, TOL_DECODED, assert_codes_match, assert_radii_match, code_mismatch_report, radii_ulp_report,
                          rel_l2, to_f64)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
CASES = [(128, (3,) * 7, 8, 2), (64, (4, 3, 2), 4, 2), (256, (4, 2, 2, 2, 2), 2, 1), (16, (2, 2, 2, 2), 2, 1),
         (128, (4, 2, 2, 2), 8, 2), (32, (5,), 3, 3), (128, (6, 5, 4, 3, 2, 1, 1), 4, 1)]


@pytest.mark.parametrize("d,bits,Hq,Hkv", CASES)
def test_general_levels_and_bits_against_the_oracle(d, bits, Hq, Hkv):
    lens = [70, 1, 33]
    B, cap = len(lens), 80
    cache = pq.GeneralPolarQuantCache(B, Hq, Hkv, d, bits, cap, seed=4, device=DEV)
    n_angles = d - d // 2 ** len(bits)
    assert cache.n_codes == n_angles and cache.n_radii == d // 2 ** len(bits)
    code_bytes = sum(-(-(d >> (l + 1)) * b // 8) for l, b in enumerate(bits))
    assert cache.row_bytes == code_bytes + code_bytes % 2 + 2 * cache.n_radii
    dtype = torch.bfloat16 if d >= 64 else torch.float32
    K, V = synthetic.kv_like(50 + d, sum(lens), Hkv, d, dtype, DEV, n_outliers=4 if d >= 64 else 0)
    K[3] *= 1e-3
    V[5] = 0           # a zero vector: every angle is atan2(0, 0) = 0
    cache.encode(K[:40], V[:40], torch.tensor([0, 30, 31, 40], dtype=torch.int32, device=DEV))       # two chunks
    cache.encode(K[40:], V[40:], torch.tensor([0, 40, 40, 64], dtype=torch.int32, device=DEV))
    torch.cuda.synchronize()
    cache.check_status()
    assert cache.lens.cpu().tolist() == lens
    cb = orc.codebooks_from_arrays(bits, cache.centroids.numpy(), cache.boundaries.numpy())
    own = orc.fit_codebooks(bits)
    assert np.max(np.abs(cache.centroids.numpy() - own.flat_centroids())) < 1e-10
    S = cache.S_host.double().numpy()
    codes, radii = cache.unpack(max(lens))
    codes, radii = codes.cpu().numpy(), radii.cpu().numpy()
    xh = to_f64(cache.dequant(max(lens)))
    rows = {0: list(range(0, 30)) + list(range(40, 80)), 1: [30], 2: list(range(31, 40)) + list(range(80, 104))}
    total = dict(total=0, inside=0, outside=0)
    off = cnt = 0
    ref = orc.OracleCache(B, Hkv, cap, d, cb, S)
    for b, n in enumerate(lens):
        Kb, Vb = to_f64(K[rows[b]]), to_f64(V[rows[b]])
        ref.encode_chunk(b, Kb, Vb)
        for kv, X in ((0, Kb), (1, Vb)):
            for h in range(Hkv):
                rep = code_mismatch_report(codes[b, h, kv, :n], X[:, h], S, cb)
                o, c = radii_ulp_report(radii[b, h, kv, :n], rep["radii16"])
                off, cnt = off + o, cnt + c
                for key in total:
                    total[key] += rep[key]
                want = orc.dequant(rep["codes"], rep["radii16"], cb, S)
                assert rel_l2(xh[b, h, kv, :n], want) < TOL_DECODED
    assert total["total"] == 2 * Hkv * sum(lens) * n_angles
    assert_codes_match(total)
    assert_radii_match(counts=(off, cnt))
    for io in (torch.float32, torch.bfloat16):
        q = synthetic.queries(9, B, Hq, d, io, DEV)
        out = cache.attend(q)
        torch.cuda.synchronize()
        cache.check_status()
        want = ref.attend(to_f64(q), d ** -0.5)
        if io == torch.float32:
            for b in range(B):
                assert rel_l2(to_f64(out[b]), want[b]) < 1e-4, b    # float32 arithmetic throughout
        elif out.numel() >= 1024:
            assert rel_l2(to_f64(out), want) < TOL_ATTENTION


def test_general_path_with_4_2_2_2_bits_gives_the_codes_of_the_tuned_path():
    d, Hq, Hkv, n = 128, 8, 2, 300
    gen = pq.GeneralPolarQuantCache(1, Hq, Hkv, d, (4, 2, 2, 2), n, seed=7, device=DEV)
    fast = pq.PolarQuantCache(1, Hq, Hkv, d, capacity=n, seed=7, device=DEV,
                              codebooks=(gen.centroids, gen.boundaries))
    K, V = synthetic.kv_like(12, n, Hkv, d, torch.bfloat16, DEV)
    cu = torch.tensor([0, n], dtype=torch.int32, device=DEV)
    gen.encode(K, V, cu)
    fast.encode(K, V, cu)
    torch.cuda.synchronize()
    (gc, gr), (fc, fr) = gen.unpack(n), fast.unpack(n)
    assert gc.shape == fc.shape and int((gc != fc).sum()) <= 2      # both are float64 decisions: only exact ties may differ
    assert int((gr.view(torch.int16).int() - fr.view(torch.int16).int()).abs().max()) <= 1
    q = synthetic.queries(2, 1, Hq, d, torch.float32, DEV)
    assert rel_l2(to_f64(gen.attend(q)), to_f64(fast.attend(q))) < 1e-3
    assert gen.row_bytes == 62


def test_general_path_reports_capacity_empty_and_bad_configurations():
    cache = pq.GeneralPolarQuantCache(2, 2, 1, 32, (3, 3), 16, seed=1, device=DEV)
    K, V = synthetic.kv_like(1, 20, 1, 32, torch.float32, DEV, n_outliers=0)
    cache.encode(K, V, torch.tensor([0, 17, 20], dtype=torch.int32, device=DEV))   # sequence 0 does not fit
    torch.cuda.synchronize()
    assert cache.status.cpu().tolist()[0] == pq.ERR_CAPACITY and cache.lens.cpu().tolist() == [0, 3]
    cache.status.zero_()
    out = cache.attend(synthetic.queries(1, 2, 2, 32, torch.float32, DEV))
    torch.cuda.synchronize()
    assert cache.status.cpu().tolist()[0] == pq.ERR_EMPTY and bool((out[0] == 0).all()) and bool(torch.isfinite(out).all())
    for d, bits in ((48, (2, 2)), (16, (2,) * 5), (64, (7, 2)), (512, (2, 2)), (64, ())):
        with pytest.raises(pq.PolarQuantError):
            pq.GeneralConfig.of(d, bits).sizes()
