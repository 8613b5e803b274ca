"""Decode attention of the d = 128 path on randomly drawn shapes (seeded): group sizes 1..8, one to many
(sequence, kv head) units per CTA, lengths around the tile / stage / token-block sizes, empty sequences.
float32 I/O, so that the tolerance tests the kernel's arithmetic and schedule rather than bf16 output
rounding; the oracle dequantises the codes as the GPU stored them (codes have their own tests)."""
import numpy as np
import pytest
import torch

import paper_2502_02617_b200 as pq
from paper_2502_02617_b200 import synthetic
from oracle import polarquant_oracle as orc
from parity_utils import oracle_codebooks, rel_l2, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL_F32_IO = 1e-3  # fp16 value path + hi/lo key path: measured ~4e-4


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes_against_oracle(seed):
    rng = np.random.default_rng(seed)
    for trial in range(10):
        Hkv = int(rng.choice([1, 2, 3, 8]))
        g = int(rng.choice([1, 2, 3, 4, 5, 8]))
        Hq = Hkv * g
        B = int(rng.choice([1, 2, 5, 9, 40]))
        mode = int(rng.integers(4))
        if mode == 0:
            lens = rng.integers(1, 40, B)
        elif mode == 1:
            lens = rng.integers(1, 700, B)
        elif mode == 2:
            lens = rng.choice([15, 16, 17, 63, 64, 65, 127, 128, 129, 255, 256, 257], B)
        else:
            lens = rng.integers(0, 3000, B)
        lens = [int(x) for x in lens]
        if max(lens) == 0:
            lens[0] = 5
        cap = max(lens) + int(rng.integers(0, 70))
        cache = pq.PolarQuantCache(B, Hq, Hkv, 128, capacity=cap, seed=int(rng.integers(1000)), device=DEV)
        K, V = synthetic.kv_like(int(rng.integers(10000)), sum(lens), Hkv, 128, torch.bfloat16, DEV)
        cu = torch.tensor(np.concatenate(([0], np.cumsum(lens))), dtype=torch.int32, device=DEV)
        cache.encode(K, V, cu)
        q = synthetic.queries(int(rng.integers(10000)), B, Hq, 128, torch.float32, DEV)
        out = cache.attend(q)
        again = cache.attend(q)
        torch.cuda.synchronize()
        assert torch.equal(out, again)  # fixed merge order
        codes, radii = cache.unpack(max(lens))
        cb, S = oracle_codebooks(cache), cache.S_host.double().numpy()
        for _ in range(3):
            b, hk = int(rng.integers(B)), int(rng.integers(Hkv))
            n = lens[b]
            got = to_f64(out[b, hk * g:(hk + 1) * g])
            if n == 0:  # empty sequence: zeros (and PQ_ERR_EMPTY in the status word)
                assert np.all(got == 0)
                continue
            c, r = codes[b, hk, :, :n].cpu().numpy(), radii[b, hk, :, :n].cpu().numpy()
            want = orc.decode_attention(to_f64(q[b, hk * g:(hk + 1) * g])[None], c[0][None, None], r[0][None, None],
                                        c[1][None, None], r[1][None, None], [n], cb, S, 128 ** -0.5)[0]
            assert rel_l2(got, want) < TOL_F32_IO, (seed, trial, B, Hq, Hkv, b, hk, n)


def test_one_long_sequence_and_many_short_ones():
    """A ragged batch in which the equal-cost split hands single CTAs more (sequence, kv head) units than they list
    at a time: one sequence of 61 000 tokens and 255 of 100 tokens, 8 kv heads (2048 units; the CTAs that hold only
    short units take about 17 each).  Outputs of sampled short units, of the units next to the long sequence and
    of the long sequence itself are compared with the oracle."""
    B, Hkv, Hq, d, long_len, short_len = 256, 8, 8, 128, 61000, 100
    lens = [short_len] * B
    lens[37] = long_len
    cache = pq.PolarQuantCache(B, Hq, Hkv, d, capacity=long_len, seed=77, device=DEV)
    K, V = synthetic.kv_like(78, sum(lens), Hkv, d, torch.bfloat16, DEV)
    cu = torch.tensor(np.concatenate(([0], np.cumsum(lens))), dtype=torch.int32, device=DEV)
    cache.encode(K, V, cu)
    q = synthetic.queries(79, B, Hq, d, torch.float32, DEV)
    out = cache.attend(q)
    again = cache.attend(q)
    torch.cuda.synchronize()
    cache.check_status()
    assert torch.equal(out, again)
    cb, S = oracle_codebooks(cache), cache.S_host.double().numpy()
    rng = np.random.default_rng(5)
    units = [(37, 0), (37, 7), (36, 7), (38, 0), (0, 0), (255, 7)] + [(int(rng.integers(B)), int(rng.integers(Hkv))) for _ in range(40)]
    for b, hk in units:
        n = lens[b]
        codes, radii = pq.pq_unpack_codes(d, Hkv, cache.cache[b * (cache.cache.numel() // B):(b + 1) * (cache.cache.numel() // B)],
                                          1, cache.capacity, n)
        c, r = codes[0, hk].cpu().numpy(), radii[0, hk].cpu().numpy()
        want = orc.decode_attention(to_f64(q[b, hk:hk + 1])[None], c[0][None, None], r[0][None, None], c[1][None, None],
                                    r[1][None, None], [n], cb, S, d ** -0.5)[0]
        assert rel_l2(to_f64(out[b, hk:hk + 1]), want) < TOL_F32_IO, (b, hk)
    # every short unit was written: none of the outputs is left at the fill value
    assert torch.isfinite(out).all() and (out.abs().amax(dim=(1, 2)) > 0).all()


@pytest.mark.parametrize("seed", [21, 22])
def test_random_encode_chunks_against_oracle(seed):
    """Encoder on randomly drawn chunk patterns: every sequence receives 1-4 chunks whose row counts sit around
    the kernels' dispatch limits (per-vector kernel < 32 rows, float32-FMA kernel < 128 rows or float32 input or
    odd strides, tensor-core kernel otherwise), from strided views; codes and radii of every stored vector are
    compared with the oracle."""
    from parity_utils import assert_codes_match, assert_radii_match, code_mismatch_report, radii_ulp_report
    rng = np.random.default_rng(seed)
    total = dict(total=0, inside=0, outside=0)
    radii_off = radii_n = 0
    for trial in range(8):
        Hkv = int(rng.choice([1, 2, 3, 8]))
        B = int(rng.choice([1, 2, 4, 7]))
        dt = torch.bfloat16 if rng.integers(3) else torch.float32
        cap = int(rng.integers(200, 1500))
        cache = pq.PolarQuantCache(B, Hkv, Hkv, 128, capacity=cap, seed=int(rng.integers(1000)), device=DEV)
        S, cb = cache.S_host.double().numpy(), oracle_codebooks(cache)
        done = [0] * B
        hist = [[] for _ in range(B)]
        for _chunk in range(int(rng.integers(1, 5))):
            take = [int(min(cap - done[b], rng.choice([0, 1, 3, 31, 32, 33, 100, 127, 128, 129, 300]))) for b in range(B)]
            n = sum(take)
            if n == 0:
                continue
            pad_h, pad_d = int(rng.integers(0, 2)), int(rng.choice([0, 8, 64]))
            if dt == torch.float32 and rng.integers(2):
                pad_d = 3
            big_k, big_v = synthetic.kv_like(int(rng.integers(100000)), n, Hkv + pad_h, 128 + pad_d, dt, DEV)
            off = 8 if pad_d and pad_d % 8 == 0 and rng.integers(2) else 0
            K, V = big_k[:, pad_h:, off:off + 128], big_v[:, pad_h:, off:off + 128]
            cu = torch.tensor(np.concatenate(([0], np.cumsum(take))), dtype=torch.int32, device=DEV)
            cache.encode(K, V, cu)
            r0 = 0
            for b in range(B):
                if take[b]:
                    hist[b].append((K[r0:r0 + take[b]].clone(), V[r0:r0 + take[b]].clone()))
                r0 += take[b]
                done[b] += take[b]
        torch.cuda.synchronize()
        cache.check_status()
        assert cache.lens.cpu().tolist() == done
        if max(done) == 0:
            continue
        codes, radii = cache.unpack(max(done))
        for b in range(B):
            if not done[b]:
                continue
            for kv in (0, 1):
                X = torch.cat([h[kv] for h in hist[b]])
                for h in range(Hkv):
                    rep = code_mismatch_report(codes[b, h, kv, :done[b]].cpu().numpy(), to_f64(X[:, h]), S, cb)
                    off, cnt = radii_ulp_report(radii[b, h, kv, :done[b]].cpu().numpy(), rep["radii16"])
                    radii_off, radii_n = radii_off + off, radii_n + cnt
                    for key in total:
                        total[key] += rep[key]
    assert_codes_match(total)
    assert_radii_match(counts=(radii_off, radii_n))
