"""GPU parity: the CUDA path, called through the C ABI, against the float64 oracle on the same
seeded bytes.  Codes are compared bit for bit (mismatches are allowed only within 1e-6 rad of a
decision boundary and must stay below 1e-5 of all codes), decoded keys to 1e-3 and attention
outputs to 2e-3 relative L2."""
import numpy as np
import pytest
import torch

import paper_2502_02617_b200 as pq
from paper_2502_02617_b200 import synthetic
from oracle import polarquant_oracle as orc
from parity_utils import (TOL_ATTENTION, TOL_ATTENTION_F32_IO, TOL_DECODED, assert_codes_match, assert_radii_match, code_mismatch_report,
                          radii_ulp_report,
                          oracle_codebooks, rel_l2, to_f64)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _encode_and_compare(cache, K, V, lens_list, start=None):
    """Encode ragged K, V ([sum(lens), Hkv, d]) and compare codes / radii with the oracle."""
    cu = torch.tensor(np.concatenate(([0], np.cumsum(lens_list))), dtype=torch.int32, device=DEV)
    start = [0] * len(lens_list) if start is None else start
    cache.encode(K, V, cu)
    torch.cuda.synchronize()
    cache.check_status()
    cb = oracle_codebooks(cache)
    S = cache.S_host.double().numpy()
    n_max = max(s + n for s, n in zip(start, lens_list))
    codes, radii = cache.unpack(n_max)
    codes, radii = codes.cpu().numpy(), radii.cpu().numpy()
    Kc, Vc = to_f64(K), to_f64(V)
    total = dict(total=0, inside=0, outside=0)
    radii_off = radii_n = 0
    row = 0
    for b, n in enumerate(lens_list):
        for kv, X in ((0, Kc), (1, Vc)):
            for h in range(cache.n_kv_heads):
                rep = code_mismatch_report(codes[b, h, kv, start[b]:start[b] + n], X[row:row + n, h], S, cb)
                off, cnt = radii_ulp_report(radii[b, h, kv, start[b]:start[b] + n], rep["radii16"])
                radii_off, radii_n = radii_off + off, radii_n + cnt
                for key in total:
                    total[key] += rep[key]
        row += n
    assert_codes_match(total)
    assert_radii_match(counts=(radii_off, radii_n))
    return total


def _oracle_cache(cache, K, V, lens_list):
    cb = oracle_codebooks(cache)
    ref = orc.OracleCache(cache.batch, cache.n_kv_heads, cache.capacity, cache.d, cb, cache.S_host.double().numpy())
    Kc, Vc = to_f64(K), to_f64(V)
    row = 0
    for b, n in enumerate(lens_list):
        ref.encode_chunk(b, Kc[row:row + n], Vc[row:row + n])
        row += n
    return ref


def test_config1_tiny_reference_d16_fp32():
    """1 sequence, 1 kv head, 1 query head, d = 16, 256 tokens, fp32, full 4-level recursion."""
    d, n = 16, 256
    cache = pq.PolarQuantCache(1, 1, 1, d, capacity=n, seed=0, device=DEV)
    K, V = synthetic.kv_like(0, n, 1, d, torch.float32, DEV, n_outliers=0)
    rep = _encode_and_compare(cache, K, V, [n])
    assert rep["inside"] == 0  # the float64 path decides every angle here
    assert cache.lens.cpu().tolist() == [n]
    ref = _oracle_cache(cache, K, V, [n])
    xh = to_f64(cache.dequant(n))
    S = cache.S_host.double().numpy()
    assert rel_l2(xh[0, 0, 0], orc.dequant(ref.k_codes[0, 0], ref.k_radii[0, 0], ref.cb, S)) < TOL_DECODED
    assert rel_l2(xh[0, 0, 1], orc.dequant(ref.v_codes[0, 0], ref.v_radii[0, 0], ref.cb, S)) < TOL_DECODED
    q = synthetic.queries(0, 1, 1, d, torch.float32, DEV)
    out = cache.attend(q, scale=0.25)
    torch.cuda.synchronize()
    assert rel_l2(to_f64(out), ref.attend(to_f64(q), 0.25)) < TOL_ATTENTION


@pytest.mark.parametrize("d,Hq,Hkv", [(128, 8, 2), (128, 16, 2), (128, 6, 2), (64, 4, 4), (32, 2, 1), (16, 8, 1)])
def test_ragged_batch_encode_dequant_attention(d, Hq, Hkv):
    """Several token-blocks plus ragged tails; bf16 inputs with outlier key channels."""
    lens_list = [130, 1, 64, 257]
    B = len(lens_list)
    cache = pq.PolarQuantCache(B, Hq, Hkv, d, capacity=300, seed=3, device=DEV)
    K, V = synthetic.kv_like(7, sum(lens_list), Hkv, d, torch.bfloat16, DEV)
    _encode_and_compare(cache, K, V, lens_list)
    assert cache.lens.cpu().tolist() == lens_list
    ref = _oracle_cache(cache, K, V, lens_list)
    xh = to_f64(cache.dequant(max(lens_list)))
    S = cache.S_host.double().numpy()
    for b, n in enumerate(lens_list):
        for h in range(Hkv):
            assert rel_l2(xh[b, h, 0, :n], orc.dequant(ref.k_codes[b, h, :n], ref.k_radii[b, h, :n], ref.cb, S)) < TOL_DECODED
            assert rel_l2(xh[b, h, 1, :n], orc.dequant(ref.v_codes[b, h, :n], ref.v_radii[b, h, :n], ref.cb, S)) < TOL_DECODED
    q = synthetic.queries(9, B, Hq, d, torch.bfloat16, DEV)
    out = cache.attend(q)
    torch.cuda.synchronize()
    cache.check_status()
    want = ref.attend(to_f64(q), d ** -0.5)
    assert rel_l2(to_f64(out), want) < TOL_ATTENTION
    # per sequence too, so that a short sequence cannot hide behind a long one: with float32 I/O
    q32 = q.float()
    out32 = to_f64(cache.attend(q32))
    want32 = ref.attend(to_f64(q32), d ** -0.5)
    for b in range(B):
        assert rel_l2(out32[b], want32[b]) < TOL_ATTENTION_F32_IO


def test_chunked_prefill_and_append_equal_one_shot_and_oracle():
    d, Hq, Hkv = 128, 8, 2
    lens_list = [100, 37]
    B = len(lens_list)
    K, V = synthetic.kv_like(11, sum(lens_list), Hkv, d, torch.bfloat16, DEV)
    one = pq.PolarQuantCache(B, Hq, Hkv, d, capacity=160, seed=4, device=DEV)
    _encode_and_compare(one, K, V, lens_list)
    two = pq.PolarQuantCache(B, Hq, Hkv, d, capacity=160, seed=4, device=DEV)
    # chunk 1: first 60 / 20 tokens, chunk 2: the rest minus the last token, then append the last token
    first, rest = [60, 20], [39, 16]
    idx1 = torch.cat([torch.arange(0, 60), torch.arange(100, 120)]).to(DEV)
    idx2 = torch.cat([torch.arange(60, 99), torch.arange(120, 136)]).to(DEV)
    last = torch.tensor([99, 136], device=DEV)
    for idx, ls in ((idx1, first), (idx2, rest)):
        cu = torch.tensor(np.concatenate(([0], np.cumsum(ls))), dtype=torch.int32, device=DEV)
        two.encode(K[idx].contiguous(), V[idx].contiguous(), cu)
    two.append(K[last].contiguous(), V[last].contiguous())
    torch.cuda.synchronize()
    two.check_status()
    assert two.lens.cpu().tolist() == lens_list
    c1, r1 = one.unpack(100)
    c2, r2 = two.unpack(100)
    radii_off = radii_n = 0
    for b, n in enumerate(lens_list):
        assert torch.equal(c1[b, :, :, :n], c2[b, :, :, :n])  # codes do not depend on chunking or on the kernel used
        # radii come from float32-accurate norms whose last rounding may differ between the prefill and
        # the append kernel: equal, or one fp16 ulp apart on a small fraction
        off, cnt = radii_ulp_report(r1[b, :, :, :n].cpu().numpy(), r2[b, :, :, :n].cpu().numpy())
        radii_off, radii_n = radii_off + off, radii_n + cnt
    assert_radii_match(counts=(radii_off, radii_n))
    q = synthetic.queries(12, B, Hq, d, torch.bfloat16, DEV)
    assert rel_l2(to_f64(two.attend(q)), to_f64(one.attend(q))) < 1e-3


def test_streaming_decode_steps_follow_the_oracle():
    """Prefill, then append one token per sequence and attend, several steps; the partial last
    token-block is exercised because the lengths are not multiples of the block."""
    d, Hq, Hkv = 128, 8, 2
    lens_list = [63, 129]
    B = len(lens_list)
    cache = pq.PolarQuantCache(B, Hq, Hkv, d, capacity=140, seed=5, device=DEV)
    K, V = synthetic.kv_like(21, sum(lens_list), Hkv, d, torch.bfloat16, DEV)
    _encode_and_compare(cache, K, V, lens_list)
    ref = _oracle_cache(cache, K, V, lens_list)
    for step in range(4):
        k1, v1 = synthetic.kv_like(100 + step, B, Hkv, d, torch.bfloat16, DEV)
        q = synthetic.queries(200 + step, B, Hq, d, torch.bfloat16, DEV)
        cache.append(k1, v1)
        out = cache.attend(q)
        torch.cuda.synchronize()
        cache.check_status()
        ref.append(to_f64(k1), to_f64(v1))
        assert rel_l2(to_f64(out), ref.attend(to_f64(q), d ** -0.5)) < TOL_ATTENTION
    codes, _ = cache.unpack(133)
    codes = codes.cpu().numpy()
    for b, n in enumerate(lens_list):
        assert np.array_equal(codes[b, :, 0, :n + 4], ref.k_codes[b, :, :n + 4])
        assert np.array_equal(codes[b, :, 1, :n + 4], ref.v_codes[b, :, :n + 4])


def test_attention_special_cases_len1_and_identical_keys():
    d, Hq, Hkv = 128, 4, 1
    cache = pq.PolarQuantCache(2, Hq, Hkv, d, capacity=64, seed=6, device=DEV)
    K, V = synthetic.kv_like(31, 1 + 40, Hkv, d, torch.bfloat16, DEV)
    K[1:] = K[1]  # sequence 1: forty identical keys
    cu = torch.tensor([0, 1, 41], dtype=torch.int32, device=DEV)
    cache.encode(K, V, cu)
    q = synthetic.queries(32, 2, Hq, d, torch.float32, DEV)   # float32 I/O: single heads are looked at
    out = to_f64(cache.attend(q))
    xh = to_f64(cache.dequant(40))
    for h in range(Hq):
        assert rel_l2(out[0, h], xh[0, 0, 1, 0]) < TOL_ATTENTION_F32_IO          # len 1: the value itself
        assert rel_l2(out[1, h], xh[1, 0, 1, :40].mean(0)) < TOL_ATTENTION_F32_IO  # uniform weights: the mean


@pytest.mark.parametrize("d,Hq,Hkv,n_q", [(128, 8, 2, 5), (128, 8, 1, 3), (16, 4, 2, 4),            # one decode per query
                                           (128, 8, 1, 9), (128, 6, 2, 22), (128, 2, 2, 70),      # 64..127 rows, few units: still one decode per query
                                           (128, 8, 2, 32), (128, 8, 1, 16),                      # tcgen05 kernel, one query block: single CTAs
                                           (128, 8, 2, 40), (128, 8, 1, 20), (128, 6, 2, 50), (128, 2, 2, 150),   # two query blocks: a CTA pair
                                           (128, 10, 2, 70), (128, 8, 2, 140)])                   # odd block counts: a pair completed by an idle CTA
def test_multi_query_attention_is_causal_over_the_last_positions(d, Hq, Hkv, n_q):
    """The last n_q positions of every sequence attend at once; query j sees the tokens up to its own position.
    Float32 I/O against the oracle per query, and n_q = 1 equals decode attention bit for bit."""
    lens_list = [300, 70, 3]   # the last sequence is shorter than the chunk: its first queries see nothing
    B = len(lens_list)
    cache = pq.PolarQuantCache(B, Hq, Hkv, d, capacity=320, seed=21, device=DEV)
    K, V = synthetic.kv_like(22, sum(lens_list), Hkv, d, torch.bfloat16, DEV)
    _encode_and_compare(cache, K, V, lens_list)
    ref = _oracle_cache(cache, K, V, lens_list)
    g = torch.Generator(device=DEV)
    g.manual_seed(23)
    q = torch.randn((B, n_q, Hq, d), generator=g, device=DEV, dtype=torch.float32)
    out = cache.attend_multi(q)
    torch.cuda.synchronize()
    want = orc.multi_query_attention(to_f64(q), ref.k_codes, ref.k_radii, ref.v_codes, ref.v_radii, ref.lens, ref.cb,
                                     ref.S, d ** -0.5)
    got = to_f64(out)
    for b in range(B):
        for j in range(n_q):
            if lens_list[b] - (n_q - 1 - j) <= 0:
                assert np.all(got[b, j] == 0)
            else:
                assert rel_l2(got[b, j], want[b, j]) < TOL_ATTENTION_F32_IO, (b, j)
    assert cache.status.cpu().tolist()[0] in (pq.OK, pq.ERR_EMPTY)
    cache.status.zero_()
    one = cache.attend_multi(q[:, -1:].contiguous())
    assert torch.equal(one[:, 0], cache.attend(q[:, -1].contiguous()))
    qb = q.to(torch.bfloat16)
    assert rel_l2(to_f64(cache.attend_multi(qb))[:2], want_bf16(orc, ref, qb, d)[:2]) < TOL_ATTENTION
    if d == 128 and n_q * (Hq // Hkv) >= 64:
        # the same inputs through the register-fragment tensor-core kernel, which runs on request only
        pq.pq_debug_fail_next_wait(3)
        legacy = cache.attend_multi(q)
        torch.cuda.synchronize()
        assert rel_l2(to_f64(legacy), got) < 5e-4 and not torch.equal(legacy, out)   # different kernels, same answer


@pytest.mark.parametrize("n_q,B", [(32, 80), (16, 80), (16, 32), (8, 64)])
def test_multi_query_single_block_on_a_full_device(n_q, B):
    """One query block per (kv head, sequence).  With more units than half the SMs the tcgen05 kernel runs one CTA per
    unit, each decoding whole blocks; with fewer, a second CTA without rows shares the decoding.  Chunks of 32 to 127
    rows take the kernel when the batch is large enough for it to beat one decode attention per query (here: all four
    cases).  Against the oracle on the first and last sequence, against the register-fragment kernel everywhere."""
    d, Hq, Hkv, n = 128, 8, 2, 130
    lens_list = [n - (b % 3) for b in range(B)]
    cache = pq.PolarQuantCache(B, Hq, Hkv, d, capacity=n, seed=31, device=DEV)
    K, V = synthetic.kv_like(32, sum(lens_list), Hkv, d, torch.bfloat16, DEV)
    cu = torch.tensor(np.concatenate(([0], np.cumsum(lens_list))), dtype=torch.int32, device=DEV)
    cache.encode(K, V, cu)
    g = torch.Generator(device=DEV)
    g.manual_seed(33)
    q = torch.randn((B, n_q, Hq, d), generator=g, device=DEV, dtype=torch.float32)
    out = cache.attend_multi(q)
    torch.cuda.synchronize()
    cache.check_status()
    if n_q * (Hq // Hkv) >= 64:
        pq.pq_debug_fail_next_wait(3)
        legacy = cache.attend_multi(q)
        torch.cuda.synchronize()
        assert rel_l2(to_f64(legacy), to_f64(out)) < 5e-4 and not torch.equal(legacy, out)
    # one decode attention per query computes the same in another order: this chunk did not take that path
    last = cache.attend(q[:, -1].contiguous())
    assert not torch.equal(last, out[:, -1]) and rel_l2(to_f64(last), to_f64(out[:, -1])) < 5e-4
    cb = oracle_codebooks(cache)
    S = cache.S_host.double().numpy()
    Kc, Vc = to_f64(K), to_f64(V)
    for b in (0, B - 1):
        ref = orc.OracleCache(1, Hkv, n, d, cb, S)
        row = int(cu[b])
        ref.encode_chunk(0, Kc[row:row + lens_list[b]], Vc[row:row + lens_list[b]])
        want = orc.multi_query_attention(to_f64(q[b:b + 1]), ref.k_codes, ref.k_radii, ref.v_codes, ref.v_radii, ref.lens, ref.cb,
                                         ref.S, d ** -0.5)
        assert rel_l2(to_f64(out[b:b + 1]), want) < TOL_ATTENTION_F32_IO, b


def test_multi_query_random_shapes_agree_with_the_other_paths_and_repeat_bit_for_bit():
    """Seeded random (group size, kv heads, batch, capacity, chunk length, ragged lengths): whatever kernel the dispatch
    picks, the result repeats bit for bit and agrees with another path -- the register-fragment kernel for chunks of
    64 rows and more, one decode attention per query over the tokens that query sees for shorter ones."""
    rng = np.random.default_rng(5)
    for it in range(24):
        g, Hkv = int(rng.choice([1, 2, 3, 4, 5, 8])), int(rng.choice([1, 2, 4, 8]))
        B, cap = int(rng.choice([1, 2, 3, 8, 20, 40])), int(rng.choice([70, 200, 700, 2100]))
        n_q = max(1, min(int(rng.choice([32, 64, 100, 128, 160, 256, 300, 520])) // g, cap))
        lens = [cap] + [int(rng.integers(0, cap + 1)) for _ in range(B - 1)]
        cache = pq.PolarQuantCache(B, g * Hkv, Hkv, 128, capacity=cap, seed=it, device=DEV)
        K, V = synthetic.kv_like(it, sum(lens), Hkv, 128, torch.bfloat16, DEV)
        cache.encode(K, V, torch.tensor(np.concatenate(([0], np.cumsum(lens))), dtype=torch.int32, device=DEV))
        gen = torch.Generator(device=DEV)
        gen.manual_seed(it)
        q = torch.randn((B, n_q, g * Hkv, 128), generator=gen, device=DEV, dtype=torch.float32)
        out = cache.attend_multi(q).clone()
        again = cache.attend_multi(q)
        torch.cuda.synchronize()
        assert cache.status.cpu().tolist()[0] in (pq.OK, pq.ERR_EMPTY)
        assert torch.equal(out, again) and bool(torch.isfinite(out).all()), (it, g, Hkv, B, cap, n_q)
        cache.status.zero_()
        if n_q * g >= 64:
            pq.pq_debug_fail_next_wait(3)
            other = cache.attend_multi(q)
        else:
            held, parts = cache.lens.clone(), []
            for j in range(n_q):
                cache.lens.copy_((held - (n_q - 1 - j)).clamp(min=0))
                parts.append(cache.attend(q[:, j].contiguous()).clone())
            cache.lens.copy_(held)
            other = torch.stack(parts, dim=1)
        torch.cuda.synchronize()
        assert rel_l2(to_f64(out), to_f64(other)) < 6e-4, (it, g, Hkv, B, cap, n_q)
    pq.pq_debug_fail_next_wait(0)


def want_bf16(orc, ref, qb, d):
    return orc.multi_query_attention(to_f64(qb), ref.k_codes, ref.k_radii, ref.v_codes, ref.v_radii, ref.lens, ref.cb, ref.S,
                                     d ** -0.5)


@pytest.mark.parametrize("kind,d,dtype", [("hadamard", 128, torch.bfloat16), ("hadamard", 64, torch.float32),
                                           ("identity", 128, torch.bfloat16), ("identity", 16, torch.float32)])
def test_structured_preconditioners_encode_and_attend_like_the_oracle(kind, d, dtype):
    """S = sign-flipped Hadamard / sqrt(d) and S = I (the paper's rows without preconditioning) through the same entry
    points as a random S.  Without mixing, bf16 coordinates tie exactly (a = b puts a level-1 angle on a boundary of the
    uniform codebook): the float64 re-decision must break those ties like the oracle."""
    Hq, Hkv, lens_list = 8, 2, [300, 70]
    signs = np.random.default_rng(3).choice([-1, 1], size=d).astype(np.int8)
    S = pq.pq_make_structured_rotation(d, pq.ROTATION_HADAMARD if kind == "hadamard" else pq.ROTATION_IDENTITY, signs)
    cache = pq.PolarQuantCache(len(lens_list), Hq, Hkv, d, capacity=320, seed=0, device=DEV, S=S)
    K, V = synthetic.kv_like(41, sum(lens_list), Hkv, d, dtype, DEV, n_outliers=4 if d >= 64 else 0)
    _encode_and_compare(cache, K, V, lens_list)
    ref = _oracle_cache(cache, K, V, lens_list)
    q = synthetic.queries(42, len(lens_list), Hq, d, torch.float32, DEV)
    out = cache.attend(q)
    torch.cuda.synchronize()
    cache.check_status()
    want = ref.attend(to_f64(q), d ** -0.5)
    for b in range(len(lens_list)):
        assert rel_l2(to_f64(out[b]), want[b]) < TOL_ATTENTION_F32_IO, b
    if d == 128:
        n_q = 40   # 160 rows: the tcgen05 multi-query kernel rotates by the same S
        g = torch.Generator(device=DEV)
        g.manual_seed(43)
        qm = torch.randn((len(lens_list), n_q, Hq, d), generator=g, device=DEV, dtype=torch.float32)
        got = to_f64(cache.attend_multi(qm))
        torch.cuda.synchronize()
        wantm = orc.multi_query_attention(to_f64(qm), ref.k_codes, ref.k_radii, ref.v_codes, ref.v_radii, ref.lens, ref.cb,
                                          ref.S, d ** -0.5)
        for b in range(len(lens_list)):
            assert rel_l2(got[b], wantm[b]) < TOL_ATTENTION_F32_IO, b


def test_capacity_overflow_and_empty_sequence_are_reported_not_faulted():
    d, Hq, Hkv = 128, 4, 1
    cache = pq.PolarQuantCache(2, Hq, Hkv, d, capacity=64, seed=7, device=DEV)
    K, V = synthetic.kv_like(41, 70 + 10, Hkv, d, torch.bfloat16, DEV)
    cu = torch.tensor([0, 70, 80], dtype=torch.int32, device=DEV)
    cache.encode(K, V, cu)  # sequence 0 does not fit: nothing of it is written, lens stays 0
    torch.cuda.synchronize()
    assert cache.status.cpu().tolist()[0] == pq.ERR_CAPACITY
    assert cache.lens.cpu().tolist() == [0, 10]
    cache.status.zero_()
    q = synthetic.queries(42, 2, Hq, d, torch.bfloat16, DEV)
    out = cache.attend(q)
    torch.cuda.synchronize()
    assert cache.status.cpu().tolist()[0] == pq.ERR_EMPTY
    assert torch.all(out[0] == 0) and torch.isfinite(out).all()
    # append to a full sequence is refused the same way
    cache.lens.copy_(torch.tensor([64, 10], dtype=torch.int32))
    cache.status.zero_()
    cache.append(K[:2].contiguous(), V[:2].contiguous())
    torch.cuda.synchronize()
    assert cache.status.cpu().tolist()[0] == pq.ERR_CAPACITY and cache.lens.cpu().tolist() == [64, 11]


@pytest.mark.parametrize("n", [8, 40, 300])
def test_nonfinite_inputs_are_counted(n):
    """8 rows go through the per-vector kernel, 40 through the float32-FMA kernel, 300 through the tensor-core
    kernel: each records the error and counts the non-finite input elements; the other rows are encoded as usual."""
    d = 128
    cache = pq.PolarQuantCache(1, 2, 2, d, capacity=n, seed=8, device=DEV)
    K, V = synthetic.kv_like(51, n, 2, d, torch.bfloat16, DEV)
    K[3, 0, 5] = float("nan")
    V[n - 4, 1, 6] = float("inf")
    V[n - 4, 1, 7] = float("-inf")
    cache.encode(K, V, torch.tensor([0, n], dtype=torch.int32, device=DEV))
    torch.cuda.synchronize()
    st = cache.status.cpu().tolist()
    assert st[0] == pq.ERR_NONFINITE and st[1] == 3
    codes, _ = cache.unpack(n)
    cb, S = oracle_codebooks(cache), cache.S_host.double().numpy()
    keep = np.array([t for t in range(n) if t not in (3, n - 4)])
    for kv, X in ((0, K), (1, V)):
        for h in range(2):
            rep = code_mismatch_report(codes[0, h, kv].cpu().numpy()[keep], to_f64(X[:, h])[keep], S, cb)
            assert_codes_match(rep)


def test_wait_that_gives_up_in_the_encoder_is_reported_and_the_next_call_is_clean():
    """The armed launch treats the first bounded wait of its CTA 0 as failed (the copy it waited for did arrive):
    that CTA abandons its tiles, lets its copies land, releases tensor memory and records PQ_ERR_TIMEOUT.  Nothing
    is left waiting on the device, and the same call repeated afterwards encodes everything."""
    d, Hkv, n = 128, 2, 1024
    cache = pq.PolarQuantCache(1, 2, Hkv, d, capacity=n, seed=3, device=DEV)
    K, V = synthetic.kv_like(5, n, Hkv, d, torch.bfloat16, DEV)
    cu = torch.tensor([0, n], dtype=torch.int32, device=DEV)
    pq.pq_debug_fail_next_wait(1)
    cache.encode(K, V, cu)
    torch.cuda.synchronize()
    assert cache.status.cpu().tolist()[0] == pq.ERR_TIMEOUT
    cache.status.zero_()
    cache.lens.zero_()
    _encode_and_compare(cache, K, V, [n])   # the hook is disarmed: a normal call, checked against the oracle
    pq.pq_debug_fail_next_wait(0)


def test_wait_that_gives_up_in_decode_attention_is_reported_and_the_next_call_is_clean():
    d, Hq, Hkv, n = 128, 8, 2, 3000
    cache = pq.PolarQuantCache(1, Hq, Hkv, d, capacity=n, seed=4, device=DEV)
    K, V = synthetic.kv_like(6, n, Hkv, d, torch.bfloat16, DEV)
    cache.encode(K, V, torch.tensor([0, n], dtype=torch.int32, device=DEV))
    q = synthetic.queries(7, 1, Hq, d, torch.bfloat16, DEV)
    want = cache.attend(q)
    torch.cuda.synchronize()
    cache.check_status()
    pq.pq_debug_fail_next_wait(2)
    cache.attend(q)
    torch.cuda.synchronize()
    assert cache.status.cpu().tolist()[0] == pq.ERR_TIMEOUT
    cache.status.zero_()
    got = cache.attend(q)
    torch.cuda.synchronize()
    cache.check_status()
    assert torch.equal(got, want)
    pq.pq_debug_fail_next_wait(0)


def test_wait_that_gives_up_in_the_tcgen05_multi_query_kernel_is_reported_and_the_next_call_is_clean():
    """The MMA-issuing thread of one CTA gives up after two blocks: the decoder and row-owner warps of that CTA see the
    abort flag at their next waits, the CTA drains its copies and MMAs, frees tensor memory and reports PQ_ERR_TIMEOUT;
    the other CTAs finish, nothing stays behind and the next call is normal."""
    d, Hq, Hkv, n, n_q = 128, 8, 2, 1000, 70
    cache = pq.PolarQuantCache(2, Hq, Hkv, d, capacity=n, seed=4, device=DEV)
    K, V = synthetic.kv_like(6, 2 * n, Hkv, d, torch.bfloat16, DEV)
    cache.encode(K, V, torch.tensor([0, n, 2 * n], dtype=torch.int32, device=DEV))
    g = torch.Generator(device=DEV)
    g.manual_seed(5)
    q = torch.randn((2, n_q, Hq, d), generator=g, device=DEV, dtype=torch.float32)
    want = cache.attend_multi(q)
    torch.cuda.synchronize()
    cache.check_status()
    pq.pq_debug_fail_next_wait(4)
    got = cache.attend_multi(q)
    torch.cuda.synchronize()
    assert cache.status.cpu().tolist()[0] == pq.ERR_TIMEOUT
    assert torch.equal(got[1], want[1])          # the other sequence's CTAs are untouched
    cache.status.zero_()
    again = cache.attend_multi(q)
    torch.cuda.synchronize()
    cache.check_status()
    assert torch.equal(again, want)
    pq.pq_debug_fail_next_wait(0)


def test_mid_size_llama_shape_codes_with_window_accounting():
    """8 kv heads x 2048 tokens x d = 128 (the encode config's shape, shortened): ~3.9 M codes."""
    d, Hkv, n = 128, 8, 2048
    cache = pq.PolarQuantCache(1, 32, Hkv, d, capacity=n, seed=1, device=DEV)
    K, V = synthetic.kv_like(1, n, Hkv, d, torch.bfloat16, DEV)
    rep = _encode_and_compare(cache, K, V, [n])
    assert rep["total"] == 2 * Hkv * n * 120
    ref = _oracle_cache(cache, K, V, [n])
    q = synthetic.queries(2, 1, 32, d, torch.bfloat16, DEV)
    out = cache.attend(q)
    torch.cuda.synchronize()
    assert rel_l2(to_f64(out), ref.attend(to_f64(q), d ** -0.5)) < TOL_ATTENTION


def _perturbed_codebooks(seed):
    """A data-fitted-like codebook: the analytic centroids moved a little (still ascending), with
    midpoint boundaries.  Level 1 is no longer the uniform k*pi/8 grid."""
    cen, _ = pq.pq_fit_codebooks()
    rng = np.random.default_rng(seed)
    c = cen.numpy().copy()
    c[:16] += rng.uniform(-0.05, 0.05, 16)
    c[16:] += rng.uniform(-0.02, 0.02, 12)
    bnd = np.concatenate([0.5 * (c[o:o + n - 1] + c[o + 1:o + n]) for o, n in ((0, 16), (16, 4), (20, 4), (24, 4))])
    return torch.from_numpy(c), torch.from_numpy(bnd)


def _codebooks_with_level1(theta1, upper_shift=0.0):
    """The analytic codebooks with level 1 replaced by the ascending centroids `theta1` (midpoint boundaries) and
    the upper levels' centroids moved by `upper_shift` (no longer symmetric about pi/4)."""
    cen, _ = pq.pq_fit_codebooks()
    c = cen.numpy().copy()
    c[:16] = np.asarray(theta1, dtype=np.float64)
    c[16:] += upper_shift * np.array([1, -0.5, 0.7, -1] * 3)
    bnd = np.concatenate([0.5 * (c[o:o + n - 1] + c[o + 1:o + n]) for o, n in ((0, 16), (16, 4), (20, 4), (24, 4))])
    return torch.from_numpy(c), torch.from_numpy(bnd)


_UNIFORM16 = (np.arange(16) + 0.5) * np.pi / 8
_LEVEL1_CASES = {
    # every boundary a little off the uniform grid: what a fit on observed angles gives
    "fitted": _UNIFORM16 + np.random.default_rng(1).uniform(-0.06, 0.06, 16),
    # boundaries exactly on the axes and diagonals of the folding (the uniform grid turned by pi/8 has them all there)
    "on_axes": np.concatenate(([0.05], np.arange(1, 16) * np.pi / 8 + 1e-9 * np.arange(15))),
    # two boundaries 0.004 rad apart (one table cell holds both), a gap wider than two octants, centroids next to 0 and 2 pi
    "clustered": np.array([1e-4, 0.3, 0.304, 0.308, 0.9, 1.2, 1.5702, 1.5712, 1.6, 4.3, 4.6, 5.0, 5.4, 5.9, 6.2, 6.2831]),
    # boundaries 3e-4 rad on either side of a diagonal (the second lies past the octant's edge), and one 0.02 past the axis at pi
    "near_edges": np.concatenate(([np.pi / 4 - 6e-4, np.pi / 4, np.pi / 4 + 6e-4, np.pi - 1e-5 + 0.02, np.pi + 1e-5 + 0.02],
                                  np.linspace(3.5, 6.1, 11))),
}


@pytest.mark.parametrize("case", sorted(_LEVEL1_CASES))
@pytest.mark.parametrize("n", [40, 700])
def test_any_level1_codebook_is_decided_in_float32_by_the_table(case, n):
    """Codebooks other than the analytic ones (data-fitted, Section 4.1) take the table-driven level-1 test and the
    per-boundary upper-level test: codes equal the oracle's, and float64 decides only a small share of the angles
    unless the codebook is built to defeat the table (cells holding two boundaries)."""
    d, Hq, Hkv = 128, 8, 2
    cbk = _codebooks_with_level1(_LEVEL1_CASES[case], upper_shift=0.03 if case != "on_axes" else 0.0)
    cache = pq.PolarQuantCache(1, Hq, Hkv, d, capacity=n, seed=21, device=DEV, codebooks=cbk)
    K, V = synthetic.kv_like(300 + n, n, Hkv, d, torch.bfloat16, DEV)
    K[3] *= 1e-3   # small and large rows: the margins scale with the row
    V[5] *= 300.0
    K[7] = 0       # a zero row: every angle is atan2(0, 0) = 0
    rep = _encode_and_compare(cache, K, V, [n])
    st = cache.check_status()
    decisions = 2 * Hkv * n * 120
    assert rep["total"] == decisions
    if case in ("fitted", "on_axes"):
        assert st[3] < 0.01 * decisions + 200, st   # 120 of the zero row's angles alone
    ref = _oracle_cache(cache, K, V, [n])
    q = synthetic.queries(n, 1, Hq, d, torch.bfloat16, DEV)
    out = cache.attend(q)
    torch.cuda.synchronize()
    cache.check_status()
    assert rel_l2(to_f64(out), ref.attend(to_f64(q), d ** -0.5)) < TOL_ATTENTION


def _hist_close(got, want):
    """Histograms of the same angles binned in float32 and in float64: the totals agree exactly, an angle may sit in
    the neighbouring bin (about 1e-5 rad of error against bins of 1.5e-3 rad and more: under 1 % of the angles),
    and no more than a few angles cross any one bin edge."""
    assert got.shape == want.shape
    for level in range(got.shape[0]):
        n = int(want[level].sum())
        assert int(got[level].sum()) == n
        assert np.abs(got[level] - want[level]).sum() <= 0.03 * n + 4
        assert np.abs(np.cumsum(got[level] - want[level])).max() <= 5 + 3e-4 * n


@pytest.mark.parametrize("d,Hkv,n,dtype,n_bins", [(128, 2, 700, torch.bfloat16, 1024), (128, 3, 1000, torch.bfloat16, 256),
                                                   (128, 2, 40, torch.bfloat16, 1024), (128, 2, 300, torch.float32, 512),
                                                   (16, 1, 256, torch.float32, 1024), (64, 2, 100, torch.bfloat16, 64)])
def test_angle_histograms_against_the_oracle(d, Hkv, n, dtype, n_bins):
    """pq_angle_histograms (tensor-core kernel for long bf16 inputs at d = 128, the per-vector kernel otherwise)
    against the oracle's histogram of the same rows; a second call adds to the first; a row with a NaN is left out."""
    S_host = pq.pq_make_rotation(d, 31)
    S = S_host.to(DEV)
    status = torch.zeros(pq.STATUS_WORDS, dtype=torch.int32, device=DEV)
    big_k, big_v = synthetic.kv_like(900 + n, n, Hkv + 1, d + 64, dtype, DEV, n_outliers=4 if d >= 64 else 0)
    K, V = big_k[:, 1:, 32:32 + d], big_v[:, 1:, 32:32 + d]   # strided views
    big_k[n // 2, 1, 32 + 5] *= 1e-4
    hist = torch.zeros((4, n_bins), dtype=torch.int64, device=DEV)
    pq.pq_angle_histograms(S, K, V, hist, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist()[:2] == [0, 0]
    x = np.concatenate([to_f64(K).reshape(-1, d), to_f64(V).reshape(-1, d)])
    want = orc.angle_histograms(x, S_host.double().numpy(), 4, n_bins)
    assert want[0].sum() == 2 * n * Hkv * d // 2 and want[3].sum() == 2 * n * Hkv * d // 16
    _hist_close(hist.cpu().numpy(), want)
    pq.pq_angle_histograms(S, K, V, hist, status)
    _hist_close(hist.cpu().numpy(), 2 * want)
    # one key row with a NaN: its 16-blocks are skipped and reported
    bk2 = big_k.clone()
    bk2[n // 3, 1, 32 + 7] = float("nan")
    K2 = bk2[:, 1:, 32:32 + d]
    hist.zero_()
    pq.pq_angle_histograms(S, K2, V, hist, status)
    torch.cuda.synchronize()
    st = status.cpu().tolist()
    assert st[0] == pq.ERR_NONFINITE and st[1] == d // 16
    keep = np.ones(x.shape[0], dtype=bool)
    keep[(n // 3) * Hkv + 0] = False
    _hist_close(hist.cpu().numpy(), orc.angle_histograms(x[keep], S_host.double().numpy(), 4, n_bins))


@pytest.mark.parametrize("kind", ["outlier_channels", "anisotropic"])
def test_online_codebook_fit_then_encode_and_attend(kind):
    """Section 4.1's online variant end to end: histogram of the prompt's angles on the device, clustering, encode
    with the fitted codebook.  The codebook is compared with the oracle's own fit on the same rows (two fixed points
    of the discrete iteration reached from histograms that differ by a few moved angles: close, not equal); the codes
    are then compared exactly, with the library's codebook given to the oracle as data."""
    d, Hq, Hkv, n = 128, 8, 2, 1500
    cache = pq.PolarQuantCache(1, Hq, Hkv, d, capacity=n, seed=13, device=DEV)
    K, V = synthetic.kv_like(77, n, Hkv, d, torch.bfloat16, DEV)
    if kind == "anisotropic":   # rows whose rotated coordinates have unequal scales: the angle densities move
        scales = torch.linspace(0.7, 1.4, d, device=DEV) * torch.tensor([2.0, 0.5], device=DEV).repeat(d // 2)
        St = cache.S.t().contiguous()
        K = ((K.float() @ cache.S) * scales @ St).to(torch.bfloat16)
        V = ((V.float() @ cache.S) * scales.flip(0) @ St).to(torch.bfloat16)
    analytic = cache.centroids.clone()
    S = cache.S_host.double().numpy()
    x = np.concatenate([to_f64(K).reshape(-1, d), to_f64(V).reshape(-1, d)])
    err_before = None
    for fitted in (False, True):
        if fitted:
            cache.lens.zero_()
            hist = cache.fit_online_codebooks(K, V)
            _hist_close(hist.cpu().numpy(), orc.angle_histograms(x, S, 4, pq.HIST_MAX_BINS))
            want = orc.fit_codebooks_online(x, S, n_bins=pq.HIST_MAX_BINS)
            for level in range(4):
                o, k = (0, 16) if level == 0 else (16 + 4 * (level - 1), 4)
                assert np.max(np.abs(cache.centroids.numpy()[o:o + k] - want.centroids[level])) < (2e-2 if level == 0 else 2e-3)
            if kind == "anisotropic":
                assert np.max(np.abs(cache.centroids.numpy() - analytic.numpy())) > 0.02  # the codebook followed the data
        rep = _encode_and_compare(cache, K, V, [n])
        st = cache.check_status()
        assert st[3] < 0.02 * rep["total"], st
        xh = to_f64(cache.dequant(n))[0]                                   # [Hkv, 2, n, d]
        got = np.concatenate([xh[:, 0].transpose(1, 0, 2).reshape(-1, d), xh[:, 1].transpose(1, 0, 2).reshape(-1, d)])
        err = np.sum((got - x) ** 2) / np.sum(x ** 2)
        if fitted:
            assert err < err_before * (0.97 if kind == "anisotropic" else 1.0005), (err, err_before)
        err_before = err
    ref = _oracle_cache(cache, K, V, [n])
    q = synthetic.queries(5, 1, Hq, d, torch.bfloat16, DEV)
    out = cache.attend(q)
    torch.cuda.synchronize()
    cache.check_status()
    assert rel_l2(to_f64(out), ref.attend(to_f64(q), d ** -0.5)) < TOL_ATTENTION


@pytest.mark.parametrize("n", [5, 40, 300])
def test_other_codebooks_fp32_inputs_and_strided_views(n):
    """Paths beside the bf16 tensor-core encoder: a non-uniform level-1 codebook, float32 inputs (FMA rotation), strided K/V views, and chunks of every size class
    (per-vector kernel < 32 rows, FMA kernel < 128 rows, tensor-core kernel above)."""
    d, Hq, Hkv = 128, 8, 2
    for dtype, cbk in ((torch.bfloat16, _perturbed_codebooks(3)), (torch.float32, None), (torch.bfloat16, None)):
        cache = pq.PolarQuantCache(1, Hq, Hkv, d, capacity=n + 3, seed=9, device=DEV, codebooks=cbk)
        big_k, big_v = synthetic.kv_like(70 + n, n, Hkv + 1, d + 64, dtype, DEV)
        K, V = big_k[:, 1:, 32:32 + d], big_v[:, 1:, 32:32 + d]  # views: token stride 3*(d+64), head stride d+64
        assert not K.is_contiguous()
        _encode_and_compare(cache, K, V, [n])
        ref = _oracle_cache(cache, K, V, [n])
        q = synthetic.queries(n, 1, Hq, d, torch.bfloat16, DEV)
        out = cache.attend(q)
        torch.cuda.synchronize()
        cache.check_status()
        assert rel_l2(to_f64(out), ref.attend(to_f64(q), d ** -0.5)) < TOL_ATTENTION
