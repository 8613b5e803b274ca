"""Partial attentions on the GPU against the oracle: decode attention with its log-sum-exp, the merge of partial
attentions (token shards as several GPUs would hold them, emulated here as several caches on one GPU), and the
compressed cache followed by an unquantised 16-bit window of recent tokens."""
import numpy as np
import pytest
import torch

import paper_2502_02617_b200 as pq
from paper_2502_02617_b200 import synthetic
from oracle import polarquant_oracle as orc
from parity_utils import TOL_ATTENTION, TOL_ATTENTION_F32_IO, oracle_codebooks, rel_l2, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _oracle_parts(cache, n):
    codes, radii = cache.unpack(max(n, 1))
    return codes.cpu().numpy(), radii.cpu().numpy()


@pytest.mark.parametrize("d,Hq,Hkv,paged", [(128, 8, 2, False), (128, 8, 2, True), (64, 4, 2, False), (16, 2, 1, False)])
def test_token_shards_merge_to_the_whole(d, Hq, Hkv, paged):
    """Three ranks' worth of token shards (position p on rank (p // 128) % 3): each shard's partial attention and
    log-sum-exp, merged, against the oracle over all tokens; a rank that holds nothing of a short sequence is no error."""
    W, lens = 3, [700, 130, 5]
    B, cap = len(lens), 768
    dtype = torch.bfloat16 if d >= 64 else torch.float32
    K, V = synthetic.kv_like(21, sum(lens), Hkv, d, dtype, DEV, n_outliers=4 if d >= 64 else 0)
    starts = np.concatenate(([0], np.cumsum(lens)))

    def make(b_lens):
        if paged:
            pages = -(-cap // 128)
            table = torch.from_numpy(np.random.default_rng(1).permutation(B * pages).reshape(B, pages).astype(np.int32))
            return pq.PagedPolarQuantCache(B, Hq, Hkv, d, 128, B * pages, table, seed=6, device=DEV)
        return pq.PolarQuantCache(B, Hq, Hkv, d, capacity=cap, seed=6, device=DEV)

    whole = make(lens)
    whole.encode(K, V, torch.tensor(starts, dtype=torch.int32, device=DEV))
    shards = []
    for r in range(W):
        pos = [pq.shard_positions(n, W, r) for n in lens]
        rows = torch.cat([p + int(s) for p, s in zip(pos, starts[:-1])]).to(DEV)
        c = make([len(p) for p in pos])
        cu = torch.tensor(np.concatenate(([0], np.cumsum([len(p) for p in pos]))), dtype=torch.int32, device=DEV)
        if rows.numel():
            c.encode(K[rows].contiguous(), V[rows].contiguous(), cu)
        shards.append(c)
    assert sum(int(c.lens.sum()) for c in shards) == sum(lens)
    q = synthetic.queries(4, B, Hq, d, torch.float32, DEV)
    parts = [c.attend_lse(q) for c in shards]
    torch.cuda.synchronize()
    for c in shards:
        assert c.check_status()[0] == 0
    assert torch.isinf(parts[1][1][2]).all() and torch.isinf(parts[2][1][2]).all()     # ranks 1, 2 hold none of the 5 tokens
    parts_out, parts_lse = torch.stack([p[0] for p in parts]), torch.stack([p[1] for p in parts])
    lse_out = torch.empty((B, Hq), dtype=torch.float32, device=DEV)
    out = pq.pq_merge_attention(parts_out, parts_lse, torch.empty_like(q), whole.status, lse_out=lse_out)
    out_bf16 = pq.pq_merge_attention(parts_out, parts_lse, torch.empty_like(q, dtype=torch.bfloat16), whole.status)
    torch.cuda.synchronize()
    whole.check_status()
    cb, S = oracle_codebooks(whole), whole.S_host.double().numpy()
    codes, radii = _oracle_parts(whole, max(lens))
    want = orc.decode_attention(to_f64(q), codes[:, :, 0], radii[:, :, 0], codes[:, :, 1], radii[:, :, 1], lens, cb, S, d ** -0.5)
    for b in range(B):
        assert rel_l2(to_f64(out[b]), want[b]) < TOL_ATTENTION_F32_IO, b
    assert torch.equal(out_bf16, out.to(torch.bfloat16))     # the same sum, rounded once
    if out.numel() >= 1024:                                   # fewer values: the rounding alone can exceed the bound
        assert rel_l2(to_f64(out_bf16), want) < TOL_ATTENTION
    # the merged log-sum-exp, and the unsharded kernel's own
    _, lse_whole = whole.attend_lse(q)
    g = Hq // Hkv
    for b in range(B):
        for h in range(Hq):
            Kh = orc.dequant(codes[b, h // g, 0, :lens[b]], radii[b, h // g, 0, :lens[b]], cb, S)
            ref = orc.log_sum_exp_scores(to_f64(q[b, h]), Kh, d ** -0.5)
            assert abs(float(lse_out[b, h]) - ref) < 2e-3 and abs(float(lse_whole[b, h]) - ref) < 2e-3
    # against the oracle's own merge of the GPU's parts: the merge kernel by itself
    mo, ml = orc.merge_attention(to_f64(parts_out), to_f64(parts_lse))
    assert np.max(np.abs(to_f64(out) - mo)) < 1e-5 and np.max(np.abs(to_f64(lse_out) - ml)) < 1e-5


def test_merge_reports_rows_without_any_token():
    B, Hq, d = 2, 3, 16
    parts_out = torch.randn((2, B, Hq, d), device=DEV)
    parts_lse = torch.tensor([[[0.5, -float("inf"), 1.0], [-float("inf")] * 3], [[1.5, -float("inf"), -2.0], [-float("inf")] * 3]],
                             device=DEV)
    status = torch.zeros(pq.STATUS_WORDS, dtype=torch.int32, device=DEV)
    lse = torch.empty((B, Hq), device=DEV)
    out = pq.pq_merge_attention(parts_out, parts_lse, torch.empty((B, Hq, d), device=DEV), status, lse_out=lse)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[0] == pq.ERR_EMPTY
    mo, ml = orc.merge_attention(to_f64(parts_out), to_f64(parts_lse))
    assert np.max(np.abs(to_f64(out) - mo)) < 1e-6
    assert np.array_equal(np.isinf(to_f64(lse)), np.isinf(ml)) and np.allclose(to_f64(lse)[0, [0, 2]], ml[0, [0, 2]], atol=1e-6)
    assert bool((out[1] == 0).all()) and bool((out[0, 1] == 0).all())


@pytest.mark.parametrize("d,Hq,Hkv,dtype", [(128, 8, 2, torch.bfloat16), (128, 32, 8, torch.bfloat16), (64, 4, 4, torch.bfloat16),
                                             (16, 2, 1, torch.float32),
                                             (128, 8, 1, torch.bfloat16), (128, 4, 2, torch.float32)])   # eight heads per kv head; float32 rows
def test_compressed_cache_followed_by_an_unquantised_window(d, Hq, Hkv, dtype):
    """Section 5.3's protocol: prompt tokens compressed, generated tokens kept in 16 bits.  Windows of 0, 3 and 600
    tokens (more than one step of the window kernel), one sequence with an empty compressed part."""
    lens, tails, T = [300, 0, 64], [0, 3, 600], 640
    B = len(lens)
    cache = pq.PolarQuantCache(B, Hq, Hkv, d, capacity=320, seed=8, device=DEV)
    K, V = synthetic.kv_like(31, sum(lens), Hkv, d, dtype, DEV, n_outliers=4 if d >= 64 else 0)
    cache.encode(K, V, torch.tensor(np.concatenate(([0], np.cumsum(lens))), dtype=torch.int32, device=DEV))
    kt, vt = synthetic.kv_like(32, B * T, Hkv, d, dtype, DEV, n_outliers=0)
    kt, vt = kt.view(B, T, Hkv, d).contiguous(), vt.view(B, T, Hkv, d).contiguous()
    tail_lens = torch.tensor(tails, dtype=torch.int32, device=DEV)
    cb, S = oracle_codebooks(cache), cache.S_host.double().numpy()
    codes, radii = _oracle_parts(cache, max(lens))
    for io in (torch.float32, torch.bfloat16):
        q = synthetic.queries(6, B, Hq, d, io, DEV)
        out = cache.attend_with_tail(q, kt, vt, tail_lens)
        torch.cuda.synchronize()
        assert cache.check_status()[0] == 0
        want, _ = orc.attention_with_tail(to_f64(q), codes[:, :, 0], radii[:, :, 0], codes[:, :, 1], radii[:, :, 1], lens, cb, S,
                                          d ** -0.5, to_f64(kt), to_f64(vt), tails)
        if io == torch.float32:
            for b in range(B):
                assert rel_l2(to_f64(out[b]), want[b]) < TOL_ATTENTION_F32_IO, b
        elif out.numel() >= 1024:
            assert rel_l2(to_f64(out), want) < TOL_ATTENTION
    # the window kernel by itself against exact attention, and its report of an empty window without an lse output
    q = synthetic.queries(7, B, Hq, d, torch.float32, DEV)
    out = torch.empty_like(q)
    lse = torch.empty((B, Hq), dtype=torch.float32, device=DEV)
    pq.pq_tail_attention(q, kt, vt, tail_lens, d ** -0.5, out, lse, cache.status)
    torch.cuda.synchronize()
    g = Hq // Hkv
    for b in (1, 2):
        for h in range(Hq):
            Kb, Vb = to_f64(kt[b, :tails[b], h // g]), to_f64(vt[b, :tails[b], h // g])
            assert np.allclose(to_f64(out[b, h]), orc.softmax_attention(to_f64(q[b, h]), Kb, Vb, d ** -0.5), atol=2e-5, rtol=1e-4)
            assert abs(float(lse[b, h]) - orc.log_sum_exp_scores(to_f64(q[b, h]), Kb, d ** -0.5)) < 1e-4
    assert torch.isinf(lse[0]).all() and bool((out[0] == 0).all()) and cache.check_status()[0] == 0
    pq.pq_tail_attention(q, kt, vt, tail_lens, d ** -0.5, out, None, cache.status)
    torch.cuda.synchronize()
    assert cache.status.cpu().tolist()[0] == pq.ERR_EMPTY
    # five splits of the window, merged, against the unsplit kernel
    cache.status.zero_()
    whole, whole_lse = torch.empty_like(q), torch.empty((B, Hq), dtype=torch.float32, device=DEV)
    pq.pq_tail_attention(q, kt, vt, tail_lens, d ** -0.5, whole, whole_lse, cache.status)
    parts, parts_lse = torch.empty((5,) + q.shape, device=DEV), torch.empty((5, B, Hq), device=DEV)
    pq.pq_tail_attention(q, kt, vt, tail_lens, d ** -0.5, parts, parts_lse, cache.status, n_splits=5)
    lse5 = torch.empty((B, Hq), device=DEV)
    merged = pq.pq_merge_attention(parts[:, 1:].contiguous(), parts_lse[:, 1:].contiguous(), torch.empty_like(q[1:]), cache.status, lse_out=lse5[1:])
    torch.cuda.synchronize()
    assert cache.check_status()[0] == 0
    assert torch.allclose(merged, whole[1:], atol=2e-6, rtol=1e-5) and torch.allclose(lse5[1:], whole_lse[1:], atol=1e-5)
    assert torch.isinf(parts_lse[:, 0]).all() and torch.isinf(parts_lse[3:, 1]).all()   # 3 tokens: splits 3 and 4 are empty
