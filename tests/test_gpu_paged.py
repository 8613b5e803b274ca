"""The paged cache (a pool of pages behind a block table) against the contiguous cache holding the same tokens: the
codes, radii, decoded vectors and attention outputs must be the same bits, whatever the page order; the contiguous
path is itself checked against the oracle elsewhere, and once more here through the paged entry points."""
import numpy as np
import pytest
import torch

import paper_2502_02617_b200 as pq
from paper_2502_02617_b200 import synthetic
from parity_utils import assert_codes_match, assert_radii_match, code_mismatch_report, oracle_codebooks, radii_ulp_report, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _caches(B, Hq, Hkv, d, page_tokens, pages_per_seq, seed, extra_pages=3):
    n_pages = B * pages_per_seq + extra_pages
    rng = np.random.default_rng(seed)
    table = torch.from_numpy(rng.permutation(n_pages)[:B * pages_per_seq].reshape(B, pages_per_seq).astype(np.int32))
    paged = pq.PagedPolarQuantCache(B, Hq, Hkv, d, page_tokens, n_pages, table, seed=seed, device=DEV)
    flat = pq.PolarQuantCache(B, Hq, Hkv, d, capacity=page_tokens * pages_per_seq, seed=seed, device=DEV)
    return paged, flat


@pytest.mark.parametrize("d,Hq,Hkv,page_tokens", [(128, 8, 2, 128), (128, 16, 2, 256), (128, 4, 4, 1024), (64, 4, 2, 64), (16, 2, 1, 128)])
def test_paged_cache_equals_the_contiguous_one(d, Hq, Hkv, page_tokens):
    """Ragged prefill in two chunks, then appends that cross a page edge; every observable is compared after each
    phase: codes and radii, DeQuant, decode attention, multi-query attention (both of its kernels at d = 128)."""
    B = 3
    lens_a, lens_b = [300, 1, 700], [90, 126, 0]
    pages_per_seq = -(-(max(a + b for a, b in zip(lens_a, lens_b)) + 40) // page_tokens)
    paged, flat = _caches(B, Hq, Hkv, d, page_tokens, pages_per_seq, seed=5)
    dtype = torch.bfloat16 if d >= 64 else torch.float32
    for i, lens in enumerate((lens_a, lens_b)):
        K, V = synthetic.kv_like(40 + i, sum(lens), Hkv, d, dtype, DEV, n_outliers=4 if d >= 64 else 0)
        cu = torch.tensor(np.concatenate(([0], np.cumsum(lens))), dtype=torch.int32, device=DEV)
        for c in (paged, flat):
            c.encode(K, V, cu)
    for step in range(3):   # sequence 1 goes from 127 to 130 tokens: across the 128-token page edge
        k1, v1 = synthetic.kv_like(60 + step, B, Hkv, d, dtype, DEV, n_outliers=0)
        for c in (paged, flat):
            c.append(k1, v1)
    torch.cuda.synchronize()
    for c in (paged, flat):
        c.check_status()
    assert paged.lens.cpu().tolist() == flat.lens.cpu().tolist() == [a + b + 3 for a, b in zip(lens_a, lens_b)]
    n = int(flat.lens.max())
    lens = flat.lens.cpu().tolist()
    (pc, pr), (fc, fr) = paged.unpack(n), flat.unpack(n)
    pd, fd = paged.dequant(n), flat.dequant(n)
    for b in range(B):   # positions past a sequence's length hold whatever the memory held
        assert torch.equal(pc[b, :, :, :lens[b]], fc[b, :, :, :lens[b]])
        assert torch.equal(pr[b, :, :, :lens[b]], fr[b, :, :, :lens[b]])
        assert torch.equal(pd[b, :, :, :lens[b]], fd[b, :, :, :lens[b]])
    q = synthetic.queries(8, B, Hq, d, torch.bfloat16, DEV)
    assert torch.equal(paged.attend(q), flat.attend(q))
    g = torch.Generator(device=DEV)
    g.manual_seed(3)
    for n_q in (3, 70):
        qm = torch.randn((B, n_q, Hq, d), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
        for c in (paged, flat):
            c.status.zero_()          # a query that sees no token is reported (sequence 1 is short)
        om, of = paged.attend_multi(qm), flat.attend_multi(qm)
        assert torch.equal(om, of) and torch.isfinite(om.float()).all()
    torch.cuda.synchronize()


def test_paged_encode_against_the_oracle_and_pool_sharing():
    """Codes through the paged entry points against the oracle; two caches' worth of sequences share one pool
    without touching each other's pages (the pool's unused pages keep their fill)."""
    d, Hq, Hkv, P = 128, 8, 2, 128
    B, n = 2, 333
    n_pages = 9
    table = torch.tensor([[7, 2, 5], [0, 8, 3]], dtype=torch.int32)
    cache = pq.PagedPolarQuantCache(B, Hq, Hkv, d, P, n_pages, table, seed=2, device=DEV)
    cache.cache.fill_(0xAB)
    K, V = synthetic.kv_like(3, B * n, Hkv, d, torch.bfloat16, DEV)
    cache.encode(K, V, torch.tensor([0, n, 2 * n], dtype=torch.int32, device=DEV))
    torch.cuda.synchronize()
    cache.check_status()
    codes, radii = cache.unpack(n)
    cb, S = oracle_codebooks(cache), cache.S_host.double().numpy()
    total = dict(total=0, inside=0, outside=0)
    off = cnt = 0
    for b in range(B):
        for kv, X in ((0, K), (1, V)):
            for h in range(Hkv):
                rep = code_mismatch_report(codes[b, h, kv].cpu().numpy(), to_f64(X[b * n:(b + 1) * n, h]), S, cb)
                o, c = radii_ulp_report(radii[b, h, kv].cpu().numpy(), rep["radii16"])
                off, cnt = off + o, cnt + c
                for key in total:
                    total[key] += rep[key]
    assert_codes_match(total)
    assert_radii_match(counts=(off, cnt))
    page_bytes = cache.cache.numel() // n_pages
    pool = cache.cache.view(n_pages, page_bytes)
    for unused in (1, 4, 6):
        assert bool((pool[unused] == 0xAB).all())


def test_a_page_outside_the_pool_is_reported_and_nothing_is_written():
    d, Hq, Hkv, P = 128, 4, 1, 128
    table = torch.tensor([[1, 99], [0, 2]], dtype=torch.int32)   # sequence 0's second page does not exist
    cache = pq.PagedPolarQuantCache(2, Hq, Hkv, d, P, 3, table, seed=2, device=DEV)
    cache.cache.fill_(0xCD)
    before = cache.cache.clone()
    K, V = synthetic.kv_like(4, 400, Hkv, d, torch.bfloat16, DEV)
    cache.encode(K, V, torch.tensor([0, 200, 400], dtype=torch.int32, device=DEV))
    torch.cuda.synchronize()
    st = cache.status.cpu().tolist()
    assert st[0] == pq.ERR_INVALID_ARG
    page_bytes = cache.cache.numel() // 3
    pool, was = cache.cache.view(3, page_bytes), before.view(3, page_bytes)
    assert not torch.equal(pool[1], was[1]) and not torch.equal(pool[0], was[0]) and not torch.equal(pool[2], was[2])
    assert cache.lens.cpu().tolist() == [0, 200]   # the sequence that reaches the missing page does not grow
    # the reader reports the page too and stays inside the pool
    cache.lens.copy_(torch.tensor([200, 200], dtype=torch.int32))
    cache.status.zero_()
    out = cache.attend(synthetic.queries(1, 2, Hq, d, torch.bfloat16, DEV))
    torch.cuda.synchronize()
    assert cache.status.cpu().tolist()[0] == pq.ERR_INVALID_ARG and out.shape == (2, Hq, d)
    with pytest.raises(pq.PolarQuantError):
        pq.PagedPolarQuantCache(2, Hq, Hkv, d, 64, 3, table, seed=2, device=DEV)   # 64-token pages at d = 128
