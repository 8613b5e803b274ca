"""The N > 1 path on CPU: two gloo ranks own disjoint sequences, run independently (no data-path
collective), and only timings (max over ranks) and results (gather for the check) cross ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2502_02617_b200 import sharding, synthetic
from oracle import polarquant_oracle as orc

B, HQ, HKV, D, N = 5, 4, 2, 16, 40


def _whole_batch():
    cb = orc.fit_codebooks()
    S = orc.make_rotation(D, 3)
    q = synthetic.queries(1, B, HQ, D, torch.float32, "cpu").double().numpy()
    caches = orc.OracleCache(B, HKV, N, D, cb, S)
    for b in range(B):
        K, V = synthetic.kv_like(100 + b, N - b, HKV, D, torch.float32, "cpu", n_outliers=2)
        caches.encode_chunk(b, K.double().numpy(), V.double().numpy())
    return caches, q


def _worker(rank, world, port, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        caches, q = _whole_batch()
        mine = sharding.shard_range(B, rank, world)
        out = np.zeros((len(mine), HQ, D))
        for i, b in enumerate(mine):  # each rank touches only its own sequences
            out[i] = orc.decode_attention(q[b:b + 1], caches.k_codes[b:b + 1], caches.k_radii[b:b + 1],
                                          caches.v_codes[b:b + 1], caches.v_radii[b:b + 1], caches.lens[b:b + 1],
                                          caches.cb, caches.S, D ** -0.5)[0]
        full = sharding.gather_shards(torch.from_numpy(out), B, dist)
        slowest = sharding.max_over_ranks([1.0 + rank, 5.0 - rank], dist)
        if rank == 0:
            results.put((full.numpy(), slowest))
    finally:
        dist.destroy_process_group()


def _fake_local(rank):
    """What bench.py measures on one rank, with made-up numbers (no CUDA on this machine): rank 1 is the slower one."""
    slow = 1.0 + 0.5 * rank
    head = {"inner": 3, "e2e_inner": 2, "total_ms": 60.0 * slow, "e2e_total_ms": 90.0 * slow,
            "seg_ms": [0.1 * slow, 0.02 * slow, 0.15 * slow], "seg_best_ms": [0.09, 0.02, 0.14],
            "e2e_seg_ms": [2.0 * slow, 0.03 * slow, 0.2 * slow], "seg_samples": 60,
            "clocks": {"sm_mhz": 1965.0, "sm_max_mhz": 1965.0, "reasons": [], "samples": 10, "samples_under_load": 10},
            "match": None, "h2d_decode_bytes": 98304, "h2d_encode_bytes": 134217728, "d2h_bytes": 65536}
    cfg4 = {"layers": 36, "ctx": 131072, "batch": 1, "decode_step_ms": 3.0 * slow, "decode_step_best_ms": 2.9,
            "launches_per_step": 36, "compressed_bytes_per_step": 4680843264, "encode_ms_per_layer": 0.4 * slow}
    cfg5 = {"batch": 16, "steps": 128, "context_lengths": [4096, 65536], "cached_tokens_at_start": 600000,
            "total_ms_128_steps": 40.0 * slow, "ms_per_step": 0.3, "append_ms": 0.02 * slow, "decode_ms": 0.3 * slow,
            "compressed_bytes_per_step": 600000000, "prefill_chunk_tokens": 4096, "prefill_tokens_per_s": 2.5e8}
    return {"batch": 8, "headline": head, "cfg4": cfg4, "cfg5": cfg5}


def _bench_worker(rank, world, port, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    d, r, w, _ = bench.dist_setup("gloo")
    try:
        line = bench.reduce_and_format(_fake_local(rank), steps=20, warmup=3, rank=r, world=w, dist=d, device="cpu")
        if rank == 0:
            results.put(line)
        else:
            assert line is None
    finally:
        d.destroy_process_group()


def test_bench_rank_logic_takes_the_slowest_rank_and_sums_the_job():
    """bench.py's own reduction and JSON line under two gloo ranks (the CUDA measurements are replaced by made-up
    numbers): every time is the maximum over ranks, `value` is the whole job's throughput."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    results = ctx.Queue()
    procs = [ctx.Process(target=_bench_worker, args=(r, 2, port, results)) for r in range(2)]
    for p in procs:
        p.start()
    line = results.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    comp = 8 * 8 * 32769 * 124
    assert line["n_gpus"] == 2 and line["scaling"] == "weak" and line["steps"] == 20
    assert abs(line["config"]["decode_ms"] - 0.15 * 1.5) < 1e-12           # the slower rank's time
    assert abs(line["value"] - 2 * comp / (0.15 * 1.5 * 1e-3) / 1e9) < 1e-6  # both ranks' bytes over that time
    assert abs(line["ms_per_step"] - 60.0 * 1.5 / 20) < 1e-9
    assert abs(line["e2e"]["region_ms"] - (0.03 + 0.2) * 1.5) < 1e-12
    assert line["e2e"]["h2d_bytes_per_step"] == 98304 and line["gpu_launches"] == 5 * 20 * 3
    assert abs(line["configs"]["cfg4"]["decode_step_ms"] - 4.5) < 1e-12 and abs(line["configs"]["cfg5"]["decode_ms"] - 0.45) < 1e-12
    assert line["roofline"]["bound"] == "hbm" and abs(line["roofline"]["frac"] * line["roofline"]["peak"] - line["roofline"]["achieved"]) < 1e-6


def test_two_ranks_shard_sequences_without_data_path_collectives():
    assert [list(sharding.shard_range(5, r, 2)) for r in range(2)] == [[0, 1, 2], [3, 4]]
    assert [len(sharding.shard_range(8, r, 3)) for r in range(3)] == [3, 3, 2]
    assert sharding.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    results = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, results)) for r in range(2)]
    for p in procs:
        p.start()
    full, slowest = results.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    caches, q = _whole_batch()
    want = caches.attend(q, D ** -0.5)
    assert np.allclose(full, want, atol=1e-13)
    assert slowest == [2.0, 5.0]


def _token_shard_worker(rank, world, port, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        caches, q = _whole_batch()
        out = np.zeros((B, HQ, D))
        lse = np.full((B, HQ), -np.inf)
        g = HQ // HKV
        for b in range(B):   # this rank's tokens of every sequence: positions p with (p // 16) % world == rank
            pos = sharding.shard_positions(int(caches.lens[b]), world, rank, granule=16).numpy()
            for hk in range(HKV):
                Kh = orc.dequant(caches.k_codes[b, hk, pos], caches.k_radii[b, hk, pos], caches.cb, caches.S)
                Vh = orc.dequant(caches.v_codes[b, hk, pos], caches.v_radii[b, hk, pos], caches.cb, caches.S)
                for h in range(hk * g, (hk + 1) * g):
                    if len(pos):
                        out[b, h] = orc.softmax_attention(q[b, h], Kh, Vh, D ** -0.5)
                        lse[b, h] = orc.log_sum_exp_scores(q[b, h], Kh, D ** -0.5)
        parts_out, parts_lse = sharding.gather_partials(torch.from_numpy(out), torch.from_numpy(lse), dist)
        if rank == 0:
            results.put((parts_out.numpy(), parts_lse.numpy()))
    finally:
        dist.destroy_process_group()


def test_token_shards_gathered_from_two_ranks_merge_to_the_whole():
    """Token-sharded decode on CPU: the sharding rule, the all-gather of (out, lse) in rank order, and the merge
    (here the oracle's; on the GPU pq_merge_attention, tested against it) give the attention over all tokens."""
    assert sharding.shard_positions(300, 2, 1).tolist() == list(range(128, 256))
    assert sharding.shard_positions(5, 3, 2).tolist() == []
    got = sorted(sum((sharding.shard_positions(1000, 3, r, 64).tolist() for r in range(3)), []))
    assert got == list(range(1000))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    results = ctx.Queue()
    procs = [ctx.Process(target=_token_shard_worker, args=(r, 2, port, results)) for r in range(2)]
    for p in procs:
        p.start()
    parts_out, parts_lse = results.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert parts_out.shape == (2, B, HQ, D) and parts_lse.shape == (2, B, HQ)
    caches, q = _whole_batch()
    merged, _ = orc.merge_attention(parts_out, parts_lse)
    assert np.allclose(merged, caches.attend(q, D ** -0.5), atol=1e-12)
