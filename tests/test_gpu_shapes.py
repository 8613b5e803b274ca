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
