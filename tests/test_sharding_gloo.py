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
