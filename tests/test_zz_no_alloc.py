"""The allocation-free decode-attention entry point (built-in scratch buffer) against the regular
one.  Kept in a file that pytest collects last so that a failure here cannot hide another test.

Who needs it: callers that reach decode attention at a point where they may not allocate or own
no workspace to pass (a serving loop with a fixed memory plan, a plugin handed only its tensors).
"""
import pytest
import torch

import paper_2502_02617_b200 as pq
from paper_2502_02617_b200 import synthetic
from parity_utils import TOL_ATTENTION, rel_l2, to_f64

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _filled_cache(d, Hq, Hkv, lens_list, seed):
    cache = pq.PolarQuantCache(len(lens_list), Hq, Hkv, d, capacity=max(lens_list) + 8, seed=seed, device=DEV)
    K, V = synthetic.kv_like(seed + 1, sum(lens_list), Hkv, d, torch.bfloat16, DEV)
    cu = torch.tensor([0] + list(torch.tensor(lens_list).cumsum(0)), dtype=torch.int32, device=DEV)
    cache.encode(K, V, cu)
    return cache


@pytest.mark.parametrize("d,Hq,Hkv,lens_list", [(128, 8, 2, [700, 129, 64]), (16, 2, 1, [100, 37])])
def test_static_scratch_entry_matches_workspace_entry_twice_in_a_row(d, Hq, Hkv, lens_list):
    cache = _filled_cache(d, Hq, Hkv, lens_list, seed=61)
    for call in range(2):  # the second call reuses whatever the first left in the shared buffer
        q = synthetic.queries(70 + call, len(lens_list), Hq, d, torch.bfloat16, DEV)
        want = cache.attend(q)
        got = torch.full_like(q, float("nan"))
        pq.pq_decode_attention_static(cache.S, cache.tables, q, cache.cache, cache.lens, Hkv, cache.capacity,
                                      cache.capacity, d ** -0.5, got, cache.status)
        torch.cuda.synchronize()
        cache.check_status()
        assert torch.isfinite(got).all()
        assert rel_l2(to_f64(got), to_f64(want)) < TOL_ATTENTION
        assert torch.equal(got, want)  # same kernels, same split order: bit-identical


def test_static_scratch_entry_after_a_call_of_the_other_kernel_family():
    """The head_dim-16 path counts its splits with small integers in the shared array; the head_dim-128 path that
    runs next on the same bytes (units shared by several CTAs) must not take them for arrivals of its own call.  Device
    memory in use is the same before and after: the entry allocates nothing."""
    small = _filled_cache(16, 2, 1, [100, 37], seed=62)
    big = _filled_cache(128, 8, 2, [9000, 5000], seed=63)   # few units, many CTAs per unit
    q16 = synthetic.queries(80, 2, 2, 16, torch.bfloat16, DEV)
    q128 = synthetic.queries(81, 2, 8, 128, torch.bfloat16, DEV)
    want = big.attend(q128)
    got16, got = torch.empty_like(q16), torch.empty_like(q128)
    torch.cuda.synchronize()
    free_before, allocated_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    for _ in range(2):
        pq.pq_decode_attention_static(small.S, small.tables, q16, small.cache, small.lens, 1, small.capacity,
                                      small.capacity, 0.25, got16, small.status)
        pq.pq_decode_attention_static(big.S, big.tables, q128, big.cache, big.lens, 2, big.capacity, big.capacity,
                                      128 ** -0.5, got, big.status)
        torch.cuda.synchronize()
        big.check_status()
        small.check_status()
        assert torch.equal(got, want)
    assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == allocated_before


def test_static_scratch_entry_rejects_oversized_problems_without_launching():
    d, Hq, Hkv, B, ctx = 128, 64, 8, 256, 1 << 20
    assert pq.pq_workspace_bytes(d, B, Hq, Hkv, ctx) > pq.pq_static_scratch_bytes()
    dummy = torch.zeros(64, dtype=torch.int32, device=DEV)
    q = torch.zeros((B, Hq, d), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(pq.PolarQuantError) as e:
        pq.pq_decode_attention_static(dummy, dummy, q, dummy, dummy, Hkv, ctx, ctx, 0.1, torch.empty_like(q), dummy)
    assert e.value.status == pq.ERR_SCRATCH
