"""Parity at the full sizes of the benchmark configurations, in the launch configuration bench.py
times, on sampled outputs the oracle can compute one by one: codes and radii of sampled vectors, and
attention outputs of sampled (sequence, kv head) units (the oracle dequantises the unit's codes as
the GPU stored them, after those codes have themselves been checked on samples)."""
import numpy as np
import pytest
import torch

import paper_2502_02617_b200 as pq
from paper_2502_02617_b200 import synthetic
from oracle import polarquant_oracle as orc
from parity_utils import (TOL_ATTENTION, assert_codes_match, assert_radii_match, code_mismatch_report, radii_ulp_report,
                          oracle_codebooks, rel_l2, to_f64)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
D, HQ, HKV = 128, 32, 8


def _check_sampled_codes(cache, b, K, V, start, rng, n_samples=384):
    """K, V: the [n, Hkv, d] rows that were encoded at positions start.. of sequence b."""
    cb, S = oracle_codebooks(cache), cache.S_host.double().numpy()
    n = K.shape[0]
    toks = np.sort(rng.choice(n, min(n, n_samples), replace=False))
    codes, radii = cache.unpack(start + n)
    idx = torch.as_tensor(toks, device=DEV)
    total = dict(total=0, inside=0, outside=0)
    radii_off = radii_n = 0
    for kv, X in ((0, K), (1, V)):
        for h in range(cache.n_kv_heads):
            rep = code_mismatch_report(codes[b, h, kv][idx + start].cpu().numpy(), to_f64(X[idx, h]), S, cb)
            off, cnt = radii_ulp_report(radii[b, h, kv][idx + start].cpu().numpy(), rep["radii16"])
            radii_off, radii_n = radii_off + off, radii_n + cnt
            for key in total:
                total[key] += rep[key]
    assert_codes_match(total)
    assert_radii_match(counts=(radii_off, radii_n))
    return codes, radii


def _check_attention_units(cache, codes, radii, q, out, units):
    """Outputs of the sampled (sequence, kv head) units against the oracle: the stated tolerance on the units
    together (a single unit of 512 bf16 values can reach it by its output rounding alone)."""
    cb, S = oracle_codebooks(cache), cache.S_host.double().numpy()
    lens = cache.lens.cpu().numpy()
    g = cache.n_q_heads // cache.n_kv_heads
    got, want = [], []
    for b, hk in units:
        n = int(lens[b])
        c, r = codes[b, hk, :, :n].cpu().numpy(), radii[b, hk, :, :n].cpu().numpy()
        want.append(orc.decode_attention(to_f64(q[b, hk * g:(hk + 1) * g])[None], c[0][None, None], r[0][None, None],
                                         c[1][None, None], r[1][None, None], [n], cb, S, cache.d ** -0.5)[0])
        got.append(to_f64(out[b, hk * g:(hk + 1) * g]))
    assert rel_l2(np.concatenate(got), np.concatenate(want)) < TOL_ATTENTION, units


def test_config2_and_config3_full_size():
    """Encode 8 kv heads x 32768 tokens (config 2) for each of 8 sequences, then decode attention with
    32 query heads over batch 8 x 32768 (config 3)."""
    B, n = 8, 32768
    rng = np.random.default_rng(2)
    cache = pq.PolarQuantCache(B, HQ, HKV, D, capacity=n, seed=1, device=DEV)
    codes = radii = None
    for b in range(B):
        K, V = synthetic.kv_like(10 + b, n, HKV, D, torch.bfloat16, DEV)
        cu = torch.zeros(B + 1, dtype=torch.int32, device=DEV)
        cu[b + 1:] = n
        cache.encode(K, V, cu)
        if b in (0, 5):
            codes, radii = _check_sampled_codes(cache, b, K, V, 0, rng)
    torch.cuda.synchronize()
    st = cache.check_status()
    assert cache.lens.cpu().tolist() == [n] * B
    assert 0 < st[3] < 2e-3 * B * n * HKV * 2 * 120  # a small fraction of decisions needed float64
    q = synthetic.queries(3, B, HQ, D, torch.bfloat16, DEV)
    out = cache.attend(q)
    torch.cuda.synchronize()
    cache.check_status()
    assert torch.isfinite(out).all()
    codes, radii = cache.unpack(n)
    _check_attention_units(cache, codes, radii, q, out, [(0, 0), (5, 7), (7, 3)])
    again = cache.attend(q)  # fixed merge order: bit-identical from run to run
    assert torch.equal(out, again)


def test_config2_every_code_against_the_oracle():
    """All 62.9 M codes and 4.2 M radii of one full config-2 encode (32768 tokens x 8 kv heads x K, V): none may
    differ outside the 1e-6 rad window around a boundary, fewer than 1e-5 of them inside it."""
    n = 32768
    cache = pq.PolarQuantCache(1, HQ, HKV, D, capacity=n, seed=1, device=DEV)
    K, V = synthetic.kv_like(1, n, HKV, D, torch.bfloat16, DEV)
    cache.encode(K, V, torch.tensor([0, n], dtype=torch.int32, device=DEV))
    torch.cuda.synchronize()
    cache.check_status()
    codes, radii = cache.unpack(n)
    cb, S = oracle_codebooks(cache), cache.S_host.double().numpy()
    total = dict(total=0, inside=0, outside=0)
    radii_off = radii_n = 0
    for kv, X in ((0, K), (1, V)):
        for h in range(HKV):
            rep = code_mismatch_report(codes[0, h, kv].cpu().numpy(), to_f64(X[:, h]), S, cb)
            off, cnt = radii_ulp_report(radii[0, h, kv].cpu().numpy(), rep["radii16"])
            radii_off, radii_n = radii_off + off, radii_n + cnt
            for key in total:
                total[key] += rep[key]
    print(f"config 2, all codes: {total}; radii one fp16 ulp off: {radii_off} of {radii_n}")
    assert total["total"] == 2 * HKV * n * 120
    assert total["outside"] == 0 and total["inside"] < 1e-5 * total["total"]
    assert_radii_match(counts=(radii_off, radii_n))


def test_chunk_of_64_queries_over_a_config3_cache():
    """Multi-query attention at full size: the last 64 positions of two 32768-token sequences (32 q / 8 kv heads)
    attend causally; all 64 queries of sampled (sequence, kv head) units against the oracle."""
    B, n, n_q = 2, 32768, 64
    cache = pq.PolarQuantCache(B, HQ, HKV, D, capacity=n, seed=1, device=DEV)
    for b in range(B):
        K, V = synthetic.kv_like(10 + b, n, HKV, D, torch.bfloat16, DEV)
        cu = torch.zeros(B + 1, dtype=torch.int32, device=DEV)
        cu[b + 1:] = n
        cache.encode(K, V, cu)
    g = torch.Generator(device=DEV)
    g.manual_seed(64)
    q = torch.randn((B, n_q, HQ, D), generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    out = cache.attend_multi(q)
    torch.cuda.synchronize()
    cache.check_status()
    assert torch.equal(out, cache.attend_multi(q))
    codes, radii = cache.unpack(n)
    cb, S = oracle_codebooks(cache), cache.S_host.double().numpy()
    grp = HQ // HKV
    for b, hk in ((0, 2), (1, 7)):
        c, r = codes[b, hk].cpu().numpy(), radii[b, hk].cpu().numpy()
        want = orc.multi_query_attention(to_f64(q[b:b + 1, :, hk * grp:(hk + 1) * grp]), c[0][None, None], r[0][None, None],
                                         c[1][None, None], r[1][None, None], [n], cb, S, D ** -0.5)[0]
        assert rel_l2(to_f64(out[b, :, hk * grp:(hk + 1) * grp]), want) < TOL_ATTENTION, (b, hk)


def test_config4_long_context_layers():
    """Three layers of the long-context shape (batch 1, 131072 tokens, 32 q / 8 kv heads), each from its own seed,
    sharing S and the codebooks as the layers of a model do; the benchmark runs 36 of them back to back."""
    n = 131072
    rng = np.random.default_rng(4)
    cache = pq.PolarQuantCache(1, HQ, HKV, D, capacity=n, seed=4, device=DEV)
    for layer in (0, 17, 35):
        cache.lens.zero_()
        K, V = synthetic.kv_like(4000 + layer, n, HKV, D, torch.bfloat16, DEV)
        cache.encode(K, V, torch.tensor([0, n], dtype=torch.int32, device=DEV))
        codes, radii = _check_sampled_codes(cache, 0, K, V, 0, rng)
        q = synthetic.queries(4500 + layer, 1, HQ, D, torch.bfloat16, DEV)
        out = cache.attend(q)
        torch.cuda.synchronize()
        cache.check_status()
        _check_attention_units(cache, codes, radii, q, out, [(0, int(rng.integers(HKV))), (0, int(rng.integers(HKV)))])
        del K, V, codes, radii


def test_config5_ragged_prefill_then_streaming_decode():
    """Batch 16, ragged contexts in [4096, 65536], prefill in 4096-token chunks, then 128 steps of
    (append one token per sequence, decode attention); parity on steps 1, 2, 64 and 128."""
    B, steps, chunk = 16, 128, 4096
    rng = np.random.default_rng(5)
    lens0 = synthetic.ragged_lengths(5, B, 4096, 65536)
    cap = max(lens0) + steps
    cache = pq.PolarQuantCache(B, HQ, HKV, D, capacity=cap, seed=5, device=DEV)
    done = [0] * B
    c_idx = 0
    while any(d < n for d, n in zip(done, lens0)):
        take = [min(chunk, n - d) for d, n in zip(done, lens0)]
        K, V = synthetic.kv_like(500 + c_idx, sum(take), HKV, D, torch.bfloat16, DEV)
        cu = torch.tensor(np.concatenate(([0], np.cumsum(take))), dtype=torch.int32, device=DEV)
        cache.encode(K, V, cu)
        if c_idx in (0, 7):  # sampled codes of one sequence's chunk (ragged chunk starts)
            b = int(np.argmax(take))
            row0 = int(np.sum(take[:b]))
            _check_sampled_codes(cache, b, K[row0:row0 + take[b]], V[row0:row0 + take[b]], done[b], rng, 128)
        done = [d + t for d, t in zip(done, take)]
        c_idx += 1
    torch.cuda.synchronize()
    cache.check_status()
    assert cache.lens.cpu().tolist() == lens0
    cb, S = oracle_codebooks(cache), cache.S_host.double().numpy()
    for step in range(1, steps + 1):
        k1, v1 = synthetic.kv_like(9000 + step, B, HKV, D, torch.bfloat16, DEV)
        q = synthetic.queries(9500 + step, B, HQ, D, torch.bfloat16, DEV)
        cache.append(k1, v1)
        out = cache.attend(q, max_len=cap)
        if step in (1, 2, 64, 128):
            torch.cuda.synchronize()
            cache.check_status()
            assert cache.lens.cpu().tolist() == [n + step for n in lens0]
            codes, radii = cache.unpack(cap)
            # the token just appended: codes against the oracle for every sequence and head
            for b in (0, B - 1, int(np.argmin(lens0))):
                pos = lens0[b] + step - 1
                for kv, X in ((0, k1), (1, v1)):
                    rep = code_mismatch_report(codes[b, :, kv, pos].cpu().numpy(), to_f64(X[b]), S, cb)
                    assert rep["outside"] == 0 and rep["inside"] <= 1
            units = [(int(np.argmin(lens0)), 1), (int(np.argmax(lens0)), 6), (int(rng.integers(B)), int(rng.integers(HKV)))]
            _check_attention_units(cache, codes, radii, q, out, units)
            del codes, radii
    torch.cuda.synchronize()
    cache.check_status()
