#!/usr/bin/env python
"""Benchmark of the PolarQuant hot path on B200.

One pass = the whole path once on synthetic Llama-3.1-8B-shaped data:
  (1) pq_encode_kv   : a prefill chunk of 32768 tokens x 8 KV heads x d=128, bf16 K and V (config 2; it
                       re-encodes one sequence of a resident batch),
  (2) pq_append_kv   : one new token for each of the 8 sequences,
  (3) pq_decode_attention : 32 query heads / 8 KV heads over batch 8 x ~32769 cached tokens (config 3).
Two resident caches alternate: a pass writes (1), (2) into one and reads (3) from the other, so that the
decode never finds in L2 what the encoder of the same pass just wrote.  A step is `inner` consecutive
passes (chosen so that the timed region lasts about two seconds; see `config.inner`); times are per pass.
The headline `value` is the decode-attention throughput on compressed bytes (62 B per token per KV head
for K and again for V), from CUDA events around call (3); the encoder's tokens/s, the long-context step
(config 4: 36 layers x 131072 tokens) and the streaming loop (config 5: ragged batch 16, 128 steps) are
reported beside it.  With --gpus N every rank runs the same per-GPU workload on its own sequences (no
data-path collective; weak scaling) and the slowest rank's time counts.

`--impl reference` times the float64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

D, HQ, HKV, BATCH, CTX = 128, 32, 8, 8, 32768
BYTES_PER_TOKEN_HEAD = 124  # 62 B of K + 62 B of V
ENCODE_BYTES_PER_VECTOR = 256 + 62
METRIC = "decode_attention_compressed_kv_throughput"
UNIT = "GB/s"
WORKLOAD = ("decode attention: batch 8 x ctx 32768, 32 q / 8 kv heads, d=128 (config 3); encode chunk 32768 tokens x "
            "8 kv heads (config 2); append 1 token/sequence")
TARGET_REGION_S = 2.2
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "decode_attention_fast_kernel_batch4_ctx32768.json")


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (earlier pool measurement)"


def _decode_traffic(batch):
    """DRAM bytes of one decode-attention launch, from the ncu capture recorded beside the profile summary
    (taken at a smaller batch; the traffic is proportional to the batch)."""
    try:
        with open(TRAFFIC_FILE) as f:
            t = json.load(f)
        return (t["dram_bytes_read"] + t["dram_bytes_write"]) * batch / t["batch"]
    except (OSError, KeyError, ValueError):
        return None


_POLLER = r"""
import sys, time, os
import pynvml as nvml
nvml.nvmlInit()
sel = sys.argv[1]
h = nvml.nvmlDeviceGetHandleByIndex(int(sel)) if sel.isdigit() else nvml.nvmlDeviceGetHandleByUUID(sel)
smax = nvml.nvmlDeviceGetMaxClockInfo(h, nvml.NVML_CLOCK_SM)
out = open(sys.argv[2], "w", buffering=1)
while True:
    out.write("%.6f %d %d %d\n" % (time.time(), nvml.nvmlDeviceGetClockInfo(h, nvml.NVML_CLOCK_SM), smax,
                                     nvml.nvmlDeviceGetCurrentClocksEventReasons(h)))
    time.sleep(0.001)
"""


class ClockSampler:
    """SM clock and throttle-reason samples taken while the timed region runs, by a separate NVML
    polling process (about one sample per millisecond; the samples are cut to the timed window)."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            sel = vis.split(",")[self.gpu_index].strip() if vis else str(self.gpu_index)
            fd, self.path = tempfile.mkstemp(suffix=".clk")
            os.close(fd)
            self.proc = subprocess.Popen([sys.executable, "-c", _POLLER, sel, self.path], stdout=subprocess.DEVNULL,
                                         stderr=subprocess.DEVNULL)
            deadline = time.time() + 10.0
            while time.time() < deadline and os.path.getsize(self.path) == 0 and self.proc.poll() is None:
                time.sleep(0.01)  # first sample written: the poller is running
        except OSError:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "samples_under_load": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, bits = [], None, 0
        try:
            with open(self.path) as f:
                for line in f:
                    parts = line.split()
                    if len(parts) != 4:
                        continue
                    ts = float(parts[0])
                    if t_begin is not None and not (t_begin <= ts <= t_end):
                        continue
                    sm.append(int(parts[1]))
                    smax = int(parts[2])
                    bits |= int(parts[3])
            os.unlink(self.path)
        except (OSError, ValueError):
            pass
        if sm:
            out.update(sm_mhz=float(statistics.median(sm)), sm_min_mhz=float(min(sm)), sm_max_mhz=float(smax),
                       samples=len(sm), samples_under_load=len(sm),
                       reasons=sorted(n for bit, n in self.REASONS.items() if bits & bit))
        return out


def dist_setup(backend="nccl"):
    """(dist or None, rank, world, local_rank) from the torchrun environment."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        if not dist.is_initialized():
            if backend == "nccl":
                torch.cuda.set_device(local_rank)
                dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
            else:
                dist.init_process_group(backend)
        return dist, rank, world, local_rank
    return None, 0, 1, 0


# --------------------------------------------------------------------------------------------
# Oracle legs (the only places that touch oracle/)
# --------------------------------------------------------------------------------------------
def _oracle_sample_throughput(seconds_budget=12.0):
    """Time the float64 oracle on a bounded sample of the decode-attention workload: whole kv heads
    of one config-3 sequence (32768 tokens, 4 query heads each), as many as fit in the budget."""
    from oracle import polarquant_oracle as orc
    from paper_2502_02617_b200 import synthetic
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    cb = orc.fit_codebooks()
    S = orc.make_rotation(D, 0)
    K, V = synthetic.kv_like(10, CTX, 1, D, torch.bfloat16, "cpu")
    q = synthetic.queries(10, 1, HQ // HKV, D, torch.bfloat16, "cpu").float().double().numpy()
    Kc, Vc = K.float().double().numpy()[:, 0], V.float().double().numpy()[:, 0]
    t0 = time.perf_counter()
    kc, kr, _ = orc.encode(Kc, S, cb)
    vc, vr, _ = orc.encode(Vc, S, cb)
    t_enc = time.perf_counter() - t0
    heads, t_dec = 0, 0.0
    while t_dec < seconds_budget and heads < 64:
        t0 = time.perf_counter()
        orc.decode_attention(q, kc[None, None], kr[None, None], vc[None, None], vr[None, None], [CTX], cb, S, D ** -0.5)
        t_dec += time.perf_counter() - t0
        heads += 1
    gbs = heads * CTX * BYTES_PER_TOKEN_HEAD / t_dec / 1e9
    return {"value": gbs, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": f"{heads} kv head(s) x {CTX} tokens x {HQ // HKV} query heads of one config-3 sequence "
                      f"({t_dec:.1f} s); oracle encode of {2 * CTX} vectors took {t_enc:.1f} s "
                      f"= {CTX / t_enc:.0f} token-positions/s per kv head",
            "encode_vectors_per_s": 2 * CTX / t_enc}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals, samples = [], None
    per_step_budget = max(2.0, min(12.0, 150.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        r = _oracle_sample_throughput(per_step_budget)
        if i >= args.warmup:
            vals.append(r["value"])
        samples = r
    value = float(np.mean(vals))
    ms = CTX * BATCH * HKV * BYTES_PER_TOKEN_HEAD / (value * 1e9) * 1e3
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD, "note": "ms_per_step extrapolated "
                                                             "from the sample to the full decode-attention workload"},
            "cpu_baseline": dict(samples, value=value),
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def _oracle_setup(cache):
    from oracle import polarquant_oracle as orc
    cb = orc.codebooks_from_arrays((4, 2, 2, 2), cache.centroids.numpy(), cache.boundaries.numpy())
    return orc, cb, cache.S_host.double().numpy()


def _attention_units_error(pq, cache, cache_buf, batch, capacity, lens, q, out, units):
    """Relative L2 error of the (sequence, kv head) units `units` of `out`, taken together, against the oracle run on
    the codes that the GPU stored in `cache_buf` (a packed cache of `batch` sequences of `capacity` tokens each)."""
    orc, cb, S = _oracle_setup(cache)
    per_seq = cache_buf.numel() // batch
    g = HQ // HKV
    got, want = [], []
    for b, hk in units:
        n = int(lens[b])
        codes, radii = pq.pq_unpack_codes(D, HKV, cache_buf[b * per_seq:(b + 1) * per_seq], 1, capacity, n)
        c, r = codes[0, hk].cpu().numpy(), radii[0, hk].cpu().numpy()
        qq = q[b, hk * g:(hk + 1) * g].float().cpu().double().numpy()[None]
        want.append(orc.decode_attention(qq, c[0][None, None], r[0][None, None], c[1][None, None], r[1][None, None], [n],
                                         cb, S, D ** -0.5)[0])
        got.append(out[b, hk * g:(hk + 1) * g].float().cpu().double().numpy())
    got, want = np.concatenate(got), np.concatenate(want)
    return float(np.linalg.norm(got - want) / np.linalg.norm(want))


def _oracle_match(pq, cache, enc_buf, b_enc, K_chunk, V_chunk, dec_buf, dec_lens, q, out, units):
    """Sampled parity at the benchmark's full size: codes of sampled vectors of the chunk just encoded as sequence
    `b_enc` of `enc_buf`, and the attention output of sampled (sequence, kv head) units of the cache that was decoded."""
    orc, cb, S = _oracle_setup(cache)
    rng = np.random.default_rng(0)
    per_seq = enc_buf.numel() // BATCH
    codes, _ = pq.pq_unpack_codes(D, HKV, enc_buf[b_enc * per_seq:(b_enc + 1) * per_seq], 1, cache.capacity, CTX)
    toks = np.sort(rng.choice(CTX, 512, replace=False))
    res = {"codes_checked": 0, "codes_mismatch_inside_window": 0, "codes_mismatch_outside_window": 0}
    for kv, X in ((0, K_chunk), (1, V_chunk)):
        for h in range(HKV):
            x = X[torch.as_tensor(toks, device=X.device), h].float().cpu().double().numpy()
            want, _, angles = orc.encode(x, S, cb)
            got = codes[0, h, kv][torch.as_tensor(toks, device=codes.device)].cpu().numpy()
            diff = got != want
            dist = orc.boundary_distance(angles, cb)
            res["codes_checked"] += int(want.size)
            res["codes_mismatch_inside_window"] += int(np.count_nonzero(diff & (dist <= 1e-6)))
            res["codes_mismatch_outside_window"] += int(np.count_nonzero(diff & (dist > 1e-6)))
    err = _attention_units_error(pq, cache, dec_buf, BATCH, cache.capacity, dec_lens, q, out, units)
    res["attention_rel_l2_of_%d_units" % len(units)] = err
    res["ok"] = bool(res["codes_mismatch_outside_window"] == 0 and err < 2e-3)
    return res


# --------------------------------------------------------------------------------------------
# The CUDA arm: local measurements of one rank
# --------------------------------------------------------------------------------------------
def _event():
    return torch.cuda.Event(enable_timing=True)


def measure_headline(args, pq, synthetic, dev, rank, barrier):
    """Configs 2 + 3 (+ append): returns the local timings of this rank."""
    capacity = CTX + 256
    cache = pq.PolarQuantCache(BATCH, HQ, HKV, D, capacity, seed=0, device=dev)
    stream = torch.cuda.current_stream()
    bufs = [cache.cache, torch.empty_like(cache.cache)]      # two resident caches
    lens = [cache.lens, torch.zeros_like(cache.lens)]

    # Resident state: both caches filled by the encoder itself (2 distinct prefill chunks, each 128 MiB of bf16
    # K+V, so successive encode passes never find their input in L2).
    chunks = [synthetic.kv_like(1000 * rank + 10 + i, CTX, HKV, D, torch.bfloat16, dev) for i in range(2)]
    cu_all = torch.zeros(BATCH + 1, dtype=torch.int32, device=dev)
    for w in range(2):
        for b in range(BATCH):
            cu_all.zero_()
            cu_all[b + 1:] = CTX
            Kb, Vb = chunks[(b + w) % 2]
            pq.pq_encode_kv(cache.S, cache.tables, Kb, Vb, cu_all, bufs[w], lens[w], capacity, cache.status)
    torch.cuda.synchronize()
    cache.check_status()
    assert lens[0].cpu().tolist() == [CTX] * BATCH and lens[1].cpu().tolist() == [CTX] * BATCH

    q_all = [synthetic.queries(77 + i + 1000 * rank, BATCH, HQ, D, torch.bfloat16, dev) for i in range(4)]
    new_all = [synthetic.kv_like(99 + i + 1000 * rank, BATCH, HKV, D, torch.bfloat16, dev) for i in range(4)]
    out = torch.empty_like(q_all[0])
    cu_step, lens_step = [], []
    for b in range(BATCH):
        c = torch.zeros(BATCH + 1, dtype=torch.int32, device=dev)
        c[b + 1:] = CTX
        cu_step.append(c)
        l = torch.full((BATCH,), CTX, dtype=torch.int32, device=dev)
        l[b] = 0
        lens_step.append(l)

    # pinned host copies for the end-to-end leg
    host_chunks = [(k.cpu().pin_memory(), v.cpu().pin_memory()) for k, v in chunks]
    host_q = [t.cpu().pin_memory() for t in q_all]
    host_new = [(k.cpu().pin_memory(), v.cpu().pin_memory()) for k, v in new_all]
    host_out = torch.empty_like(out, device="cpu").pin_memory()
    dK, dV = torch.empty_like(chunks[0][0]), torch.empty_like(chunks[0][1])
    dq, dk1, dv1 = torch.empty_like(q_all[0]), torch.empty_like(new_all[0][0]), torch.empty_like(new_all[0][1])

    def one_pass(i, ev=None, e2e=False):
        """ev: four events -> [encode incl. its H2D | append incl. its H2D | decode incl. H2D of q and D2H of out]."""
        b_enc, w = (i // 2) % BATCH, i % 2      # write cache w, read cache 1 - w
        lens[w].copy_(lens_step[b_enc])
        if ev: ev[0].record(stream)
        if e2e:
            dK.copy_(host_chunks[i % 2][0], non_blocking=True)
            dV.copy_(host_chunks[i % 2][1], non_blocking=True)
            Kb, Vb = dK, dV
        else:
            Kb, Vb = chunks[i % 2]
        pq.pq_encode_kv(cache.S, cache.tables, Kb, Vb, cu_step[b_enc], bufs[w], lens[w], capacity, cache.status)
        if ev: ev[1].record(stream)
        if e2e:
            dk1.copy_(host_new[i % 4][0], non_blocking=True)
            dv1.copy_(host_new[i % 4][1], non_blocking=True)
            k1, v1 = dk1, dv1
        else:
            k1, v1 = new_all[i % 4]
        pq.pq_append_kv(cache.S, cache.tables, k1, v1, bufs[w], lens[w], capacity, cache.status)
        if ev: ev[2].record(stream)
        if e2e:
            dq.copy_(host_q[i % 4], non_blocking=True)
            qq = dq
        else:
            qq = q_all[i % 4]
        pq.pq_decode_attention(cache.S, cache.tables, qq, bufs[1 - w], lens[1 - w], HKV, capacity, CTX + 1,
                               D ** -0.5, out, cache.workspace, cache.status)
        if e2e:
            host_out.copy_(out, non_blocking=True)
        if ev: ev[3].record(stream)
        return b_enc, w, qq

    def timed(e2e, inner, max_samples=400):
        n_pass = args.steps * inner
        stride = max(1, n_pass // max_samples)
        evs = {}
        for i in range(args.warmup * min(inner, 8)):
            one_pass(i, None, e2e)
        barrier()
        wall0 = time.time()
        t_start, t_end = _event(), _event()
        t_start.record(stream)
        last = None
        for i in range(n_pass):
            ev = None
            if i % stride == 0:
                ev = evs[i] = [_event() for _ in range(4)]
            last = one_pass(i, ev, e2e)
        t_end.record(stream)
        barrier()
        wall1 = time.time()
        seg = np.array([[e[k].elapsed_time(e[k + 1]) for k in range(3)] for e in evs.values()])  # encode, append, decode
        return t_start.elapsed_time(t_end), seg, last, (wall0, wall1)

    # size the timed region: about TARGET_REGION_S seconds
    probe = [_event() for _ in range(2)]
    for i in range(4):
        one_pass(i)
    torch.cuda.synchronize()
    probe[0].record(stream)
    for i in range(16):
        one_pass(i)
    probe[1].record(stream)
    torch.cuda.synchronize()
    pass_ms = probe[0].elapsed_time(probe[1]) / 16
    inner = args.inner if args.inner > 0 else max(1, math.ceil(TARGET_REGION_S * 1e3 / (args.steps * pass_ms)))

    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    total_ms, seg, last, wall = timed(False, inner)
    clocks = sampler.stop(wall[0], wall[1])
    cache.check_status()
    match = None
    if rank == 0 and not args.skip_match:
        b_enc, w, qq = last
        n_pass = args.steps * inner
        Kb, Vb = chunks[(n_pass - 1) % 2]
        dec_lens = lens[1 - w].cpu().tolist()
        match = _oracle_match(pq, cache, bufs[w], b_enc, Kb, Vb, bufs[1 - w], dec_lens, qq, out,
                              [(b, (3 * b + 1) % HKV) for b in range(BATCH)])  # one unit of every sequence
    if args.skip_e2e:
        e2e_total_ms, e2e_seg, e2e_inner = total_ms, seg, inner
    else:
        e2e_inner = max(1, math.ceil(1.0e3 / (args.steps * 3.0)))   # a pass with its 128 MiB of H2D takes about 3 ms
        e2e_total_ms, e2e_seg, _, _ = timed(True, e2e_inner, 200)
    cache.check_status()
    return {
        "inner": inner, "e2e_inner": e2e_inner, "total_ms": total_ms, "e2e_total_ms": e2e_total_ms,
        "seg_ms": seg.mean(0).tolist(), "seg_best_ms": seg.min(0).tolist(), "e2e_seg_ms": e2e_seg.mean(0).tolist(),
        "seg_samples": int(seg.shape[0]), "clocks": clocks, "match": match,
        "h2d_decode_bytes": int(2 * new_all[0][0].numel() * 2 + q_all[0].numel() * 2),
        "h2d_encode_bytes": int(2 * chunks[0][0].numel() * 2), "d2h_bytes": int(out.numel() * 2),
    }


def measure_config4(args, pq, synthetic, dev, rank):
    """Config 4: 36 layers x (batch 1, 131072 tokens), every layer encoded on the device from its own seed and kept
    packed (4.68 GB); one decode step = 36 sequential pq_decode_attention launches."""
    layers, n = 36, 131072
    base = pq.PolarQuantCache(1, HQ, HKV, D, n, seed=4, device=dev)
    caches = [base.cache] + [torch.empty_like(base.cache) for _ in range(layers - 1)]
    lens = [torch.zeros(1, dtype=torch.int32, device=dev) for _ in range(layers)]
    cu = torch.tensor([0, n], dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    enc_ev = []
    for l in range(layers):
        K, V = synthetic.kv_like(4000 + 100 * rank + l, n, HKV, D, torch.bfloat16, dev)
        e = (_event(), _event())
        e[0].record(stream)
        pq.pq_encode_kv(base.S, base.tables, K, V, cu, caches[l], lens[l], n, base.status)
        e[1].record(stream)
        enc_ev.append(e)
        del K, V
    torch.cuda.synchronize()
    base.check_status()
    qs = [synthetic.queries(4500 + l, 1, HQ, D, torch.bfloat16, dev) for l in range(layers)]
    outs = [torch.empty_like(qs[0]) for _ in range(layers)]

    def step():
        for l in range(layers):
            pq.pq_decode_attention(base.S, base.tables, qs[l], caches[l], lens[l], HKV, n, n, D ** -0.5, outs[l],
                                   base.workspace, base.status)
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    reps = 30
    evs = [(_event(), _event()) for _ in range(reps)]
    for a, b in evs:
        a.record(stream)
        step()
        b.record(stream)
    torch.cuda.synchronize()
    base.check_status()
    t = [a.elapsed_time(b) for a, b in evs]
    res = {"layers": layers, "ctx": n, "batch": 1, "decode_step_ms": float(np.mean(t)), "decode_step_best_ms": float(min(t)),
           "launches_per_step": layers, "compressed_bytes_per_step": layers * n * HKV * BYTES_PER_TOKEN_HEAD,
           "encode_ms_per_layer": float(np.mean([a.elapsed_time(b) for a, b in enc_ev[1:]]))}
    if rank == 0 and not args.skip_match:
        res["attention_rel_l2_layers_5_17_30"] = float(np.sqrt(np.mean([_attention_units_error(
            pq, base, caches[l], 1, n, [n], qs[l], outs[l], [(0, hk)]) ** 2 for l, hk in ((5, 1), (17, 3), (30, 6))])))
    return res


def measure_multi_query(args, pq, synthetic, dev, rank):
    """A chunk of 64 queries per sequence over a config-3 cache (batch 8 x 32768 tokens): multi-query attention."""
    n_q = 64
    cache = pq.PolarQuantCache(BATCH, HQ, HKV, D, CTX, seed=0, device=dev)
    for b in range(BATCH):
        K, V = synthetic.kv_like(1000 * rank + 10 + b % 2, CTX, HKV, D, torch.bfloat16, dev)
        cu = torch.zeros(BATCH + 1, dtype=torch.int32, device=dev)
        cu[b + 1:] = CTX
        cache.encode(K, V, cu)
    g = torch.Generator(device=dev)
    g.manual_seed(640 + rank)
    q = torch.randn((BATCH, n_q, HQ, D), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream()
    for _ in range(2):
        cache.attend_multi(q, out=out)
    evs = [(_event(), _event()) for _ in range(8)]
    for a, b in evs:
        a.record(stream)
        cache.attend_multi(q, out=out)
        b.record(stream)
    torch.cuda.synchronize()
    cache.check_status()
    t = float(np.mean([a.elapsed_time(b) for a, b in evs]))
    pairs = BATCH * n_q * HQ * (CTX - (n_q - 1) / 2.0)          # (query head, visible token) pairs
    return {"batch": BATCH, "ctx": CTX, "n_q": n_q, "ms": t, "us_per_query": t / n_q * 1e3,
            "mma_tflops": pairs * 512 * 2 / (t * 1e-3) / 1e12,
            "mma_flops_definition": "4 x 128 multiply-adds per (query head, visible token): Q'K^T with the key as fp16 value + "
                                    "residual and the query likewise (3 products), and PV"}


def measure_online_codebook(args, pq, synthetic, dev, rank):
    """Section 4.1's online codebook on the config-2 chunk (32768 tokens x 8 kv heads, K and V): angle histograms on
    the device, k-means on the binned angles and the table build on the host, then the encode with the fitted codebook;
    device times from CUDA events, host times from the wall clock."""
    cache = pq.PolarQuantCache(1, HQ, HKV, D, CTX, seed=0, device=dev)
    Ks = [synthetic.kv_like(1000 * rank + 1 + i, CTX, HKV, D, torch.bfloat16, dev) for i in range(2)]
    cu = torch.tensor([0, CTX], dtype=torch.int32, device=dev)
    hist = torch.zeros((pq.N_LEVELS, pq.HIST_MAX_BINS), dtype=torch.int64, device=dev)
    stream = torch.cuda.current_stream()

    def timed(fn, n=20):
        for i in range(3):
            fn(i)
        evs = [(_event(), _event()) for _ in range(n)]
        for i, (a, b) in enumerate(evs):
            a.record(stream)
            fn(i)
            b.record(stream)
        torch.cuda.synchronize()
        return float(np.median([a.elapsed_time(b) for a, b in evs])) * 1e3

    def encode(i):
        cache.lens.zero_()
        cache.encode(*Ks[i % 2], cu)

    analytic_us = timed(encode)
    hist_us = timed(lambda i: pq.pq_angle_histograms(cache.S, *Ks[i % 2], hist, cache.status))
    pq.pq_fit_codebooks_from_histograms(hist.cpu())  # the first call of a process also computes the analytic start (60 ms)
    hist.zero_()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    pq.pq_angle_histograms(cache.S, *Ks[0], hist, cache.status)
    h = hist.cpu()
    t1 = time.perf_counter()
    cen, bnd = pq.pq_fit_codebooks_from_histograms(h)
    t2 = time.perf_counter()
    tables = pq.pq_build_tables(cen, bnd)
    t3 = time.perf_counter()
    cache.set_codebooks(cen, bnd)
    torch.cuda.synchronize()
    t4 = time.perf_counter()
    fitted_us = timed(encode)
    st = cache.check_status()
    return {"tokens": CTX, "kv_heads": HKV, "bins": pq.HIST_MAX_BINS, "histogram_us": hist_us,
            "histogram_gbs": 2 * CTX * HKV * D * 2 / (hist_us * 1e-6) / 1e9,
            "histogram_and_d2h_wall_us": (t1 - t0) * 1e6, "kmeans_host_us": (t2 - t1) * 1e6,
            "tables_host_us": (t3 - t2) * 1e6, "tables_again_and_h2d_wall_us": (t4 - t3) * 1e6,
            "encode_fitted_codebook_us": fitted_us, "encode_analytic_codebook_us": analytic_us,
            "max_centroid_shift_rad": float((cen - pq.pq_fit_codebooks()[0]).abs().max()),
            "float64_decisions": st[3], "rank": rank}


def measure_paged(args, pq, synthetic, dev, rank):
    """Config 3 behind a block table: 8 x 32768 tokens in 256-token pages drawn in random order from one pool; the
    same decode-attention kernel with one table lookup per 128-token stage."""
    P = 256
    pages_per_seq = CTX // P
    n_pages = BATCH * pages_per_seq
    rng = np.random.default_rng(7 + rank)
    table = torch.from_numpy(rng.permutation(n_pages).reshape(BATCH, pages_per_seq).astype(np.int32))
    caches = [pq.PagedPolarQuantCache(BATCH, HQ, HKV, D, P, n_pages, table, seed=0, device=dev) for _ in range(2)]
    for c, cache in enumerate(caches):
        for b in range(BATCH):
            K, V = synthetic.kv_like(1000 * rank + 10 + (b + c) % 2, CTX, HKV, D, torch.bfloat16, dev)
            cu = torch.zeros(BATCH + 1, dtype=torch.int32, device=dev)
            cu[b + 1:] = CTX
            cache.encode(K, V, cu)
    q = synthetic.queries(3, BATCH, HQ, D, torch.bfloat16, dev)
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream()
    for i in range(4):
        caches[i % 2].attend(q, out=out)
    evs = [(_event(), _event()) for _ in range(40)]
    for i, (a, b) in enumerate(evs):   # the two caches (520 MB) alternate: no block is still in L2 when it is read again
        a.record(stream)
        caches[i % 2].attend(q, out=out)
        b.record(stream)
    torch.cuda.synchronize()
    for cache in caches:
        cache.check_status()
    t = float(np.median([a.elapsed_time(b) for a, b in evs]))
    comp = BATCH * HKV * CTX * 124
    return {"batch": BATCH, "ctx": CTX, "page_tokens": P, "pages": n_pages, "decode_us": t * 1e3,
            "gbs": comp / (t * 1e-3) / 1e9, "rank": rank}


def measure_tail_window(args, pq, synthetic, dev, rank):
    """Config 3 with the 1024 most recent tokens of every sequence kept in bf16 (Section 5.3's protocol for generated
    tokens): partial attention over the packed cache with its log-sum-exp, exact attention over the window, merge --
    three launches, float32 partials."""
    T = 1024
    cache = pq.PolarQuantCache(BATCH, HQ, HKV, D, CTX, seed=0, device=dev)
    for b in range(BATCH):
        K, V = synthetic.kv_like(1000 * rank + 10 + b % 2, CTX, HKV, D, torch.bfloat16, dev)
        cu = torch.zeros(BATCH + 1, dtype=torch.int32, device=dev)
        cu[b + 1:] = CTX
        cache.encode(K, V, cu)
    kt, vt = synthetic.kv_like(1000 * rank + 77, BATCH * T, HKV, D, torch.bfloat16, dev, n_outliers=0)
    kt, vt = kt.view(BATCH, T, HKV, D).contiguous(), vt.view(BATCH, T, HKV, D).contiguous()
    tail_lens = torch.full((BATCH,), T, dtype=torch.int32, device=dev)
    q = synthetic.queries(3, BATCH, HQ, D, torch.bfloat16, dev)
    q32 = q.float()
    n_splits = 8
    parts_out = torch.empty((1 + n_splits,) + q32.shape, dtype=torch.float32, device=dev)
    parts_lse = torch.empty((1 + n_splits, BATCH, HQ), dtype=torch.float32, device=dev)
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream()
    scale = D ** -0.5

    def step(evs=None):
        marks = []
        for fn in (lambda: pq.pq_decode_attention_lse(cache.S, cache.tables, q32, cache.cache, cache.lens, HKV, CTX, CTX, scale,
                                                      parts_out[0], parts_lse[0], cache.workspace, cache.status),
                   lambda: pq.pq_tail_attention(q32, kt, vt, tail_lens, scale, parts_out[1:], parts_lse[1:], cache.status, n_splits),
                   lambda: pq.pq_merge_attention(parts_out, parts_lse, out, cache.status)):
            a, b = _event(), _event()
            a.record(stream)
            fn()
            b.record(stream)
            marks.append((a, b))
        return marks

    for _ in range(3):
        step()
    runs = [step() for _ in range(20)]
    torch.cuda.synchronize()
    cache.check_status()
    med = [float(np.median([r[i][0].elapsed_time(r[i][1]) for r in runs])) * 1e3 for i in range(3)]
    return {"batch": BATCH, "ctx": CTX, "window_tokens": T, "window_splits": n_splits, "decode_with_lse_us": med[0], "window_attention_us": med[1],
            "merge_us": med[2], "window_bytes": 2 * BATCH * T * HKV * D * 2, "rank": rank}


def measure_general(args, pq, synthetic, dev, rank):
    """The general entry points on the full recursion of Section 4 (d = 128, log2 d = 7 levels, 3 bits per angle:
    16 + 127 x 3 bits per vector): encode of 4096 tokens x 8 kv heads and decode attention over batch 8 x 4096 tokens.
    Reference-speed kernels (float64 encoder, one thread block per sequence and kv head in attention)."""
    n, bits = 4096, (3,) * 7
    cache = pq.GeneralPolarQuantCache(BATCH, HQ, HKV, D, bits, n, seed=0, device=dev)
    K, V = synthetic.kv_like(1000 * rank + 5, n, HKV, D, torch.bfloat16, dev)
    stream = torch.cuda.current_stream()
    enc = []
    for b in range(BATCH):
        cu = torch.zeros(BATCH + 1, dtype=torch.int32, device=dev)
        cu[b + 1:] = n
        e = (_event(), _event())
        e[0].record(stream)
        cache.encode(K, V, cu)
        e[1].record(stream)
        enc.append(e)
    q = synthetic.queries(3, BATCH, HQ, D, torch.bfloat16, dev)
    out = torch.empty_like(q)
    cache.attend(q, out=out)
    dec = [(_event(), _event()) for _ in range(5)]
    for a, b in dec:
        a.record(stream)
        cache.attend(q, out=out)
        b.record(stream)
    torch.cuda.synchronize()
    cache.check_status()
    t_enc = float(np.median([a.elapsed_time(b) for a, b in enc[1:]]))
    t_dec = float(np.median([a.elapsed_time(b) for a, b in dec]))
    comp = BATCH * HKV * n * 2 * cache.row_bytes
    return {"head_dim": D, "levels": 7, "bits_per_angle": 3, "row_bytes": cache.row_bytes, "tokens": n, "batch": BATCH,
            "encode_ms": t_enc, "encode_vectors_per_s": 2 * n * HKV / (t_enc * 1e-3), "decode_ms": t_dec,
            "decode_gbs": comp / (t_dec * 1e-3) / 1e9, "rank": rank}


def measure_config5(args, pq, synthetic, dev, rank):
    """Config 5: batch 16, ragged contexts in [4096, 65536], prefill in 4096-token chunks, then 128 steps of
    (append one token per sequence, decode attention)."""
    B, steps, chunk = 16, 128, 4096
    lens0 = synthetic.ragged_lengths(5, B, 4096, 65536)
    cap = max(lens0) + steps
    cache = pq.PolarQuantCache(B, HQ, HKV, D, cap, seed=5, device=dev)
    stream = torch.cuda.current_stream()
    done, c_idx, prefill_ms, pre_ev = [0] * B, 0, 0.0, []
    while any(d < n for d, n in zip(done, lens0)):
        take = [min(chunk, n - d) for d, n in zip(done, lens0)]
        K, V = synthetic.kv_like(500 + c_idx + 1000 * rank, sum(take), HKV, D, torch.bfloat16, dev)
        cu = torch.tensor(np.concatenate(([0], np.cumsum(take))), dtype=torch.int32, device=dev)
        e = (_event(), _event())
        e[0].record(stream)
        cache.encode(K, V, cu)
        e[1].record(stream)
        pre_ev.append((e, sum(take)))
        done = [d + t for d, t in zip(done, take)]
        c_idx += 1
    torch.cuda.synchronize()
    cache.check_status()
    prefill_ms = sum(e[0].elapsed_time(e[1]) for e, _ in pre_ev[1:])
    prefill_tokens = sum(t for _, t in pre_ev[1:])
    lens_base = cache.lens.clone()
    new = [synthetic.kv_like(9000 + s, B, HKV, D, torch.bfloat16, dev) for s in range(8)]
    qs = [synthetic.queries(9500 + s, B, HQ, D, torch.bfloat16, dev) for s in range(8)]
    out = torch.empty_like(qs[0])
    totals, app, dec = [], [], []
    for rep in range(3):          # the first repetition warms up
        cache.lens.copy_(lens_base)
        evs = [[_event() for _ in range(3)] for _ in range(steps)]
        for s in range(steps):
            evs[s][0].record(stream)
            cache.append(*new[s % 8])
            evs[s][1].record(stream)
            cache.attend(qs[s % 8], out=out, max_len=cap)
            evs[s][2].record(stream)
        torch.cuda.synchronize()
        cache.check_status()
        if rep:
            totals.append(evs[0][0].elapsed_time(evs[-1][2]))
            app.append(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
            dec.append(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    mean_tokens = sum(lens0) + B * (steps + 1) / 2
    return {"batch": B, "steps": steps, "context_lengths": [min(lens0), max(lens0)], "cached_tokens_at_start": sum(lens0),
            "total_ms_128_steps": float(np.mean(totals)), "ms_per_step": float(np.mean(totals)) / steps,
            "append_ms": float(np.mean(app)), "decode_ms": float(np.mean(dec)),
            "compressed_bytes_per_step": int(mean_tokens * HKV * BYTES_PER_TOKEN_HEAD),
            "prefill_chunk_tokens": chunk, "prefill_tokens_per_s": prefill_tokens / (prefill_ms * 1e-3)}


# --------------------------------------------------------------------------------------------
# Reduction over ranks and the JSON line (no CUDA calls: covered by a two-rank gloo test)
# --------------------------------------------------------------------------------------------
def reduce_and_format(local, steps, warmup, rank, world, dist=None, device="cpu", cpu_baseline=None):
    """Max over ranks of every timing of `local` (the slowest rank's time counts), then the JSON line (rank 0
    returns it, the other ranks return None)."""
    from paper_2502_02617_b200 import sharding
    head = local["headline"]
    keys = ["total_ms", "e2e_total_ms"]
    flat = [head[k] for k in keys] + head["seg_ms"] + head["seg_best_ms"] + head["e2e_seg_ms"]
    c4, c5, mq = local.get("cfg4"), local.get("cfg5"), local.get("multi_query")
    if c4:
        flat += [c4["decode_step_ms"], c4["decode_step_best_ms"], c4["encode_ms_per_layer"]]
    if c5:
        flat += [c5["total_ms_128_steps"], c5["append_ms"], c5["decode_ms"]]
    if mq:
        flat += [mq["ms"]]
    red = sharding.max_over_ranks(flat, dist, device)
    total_ms, e2e_total_ms = red[0], red[1]
    enc_ms, app_ms, dec_ms = red[2:5]
    enc_best, app_best, dec_best = red[5:8]
    e_enc_ms, e_app_ms, e_dec_ms = red[8:11]
    pos = 11
    if rank != 0:
        return None
    inner, batch = head["inner"], local["batch"]
    n_pass = steps * inner
    comp_bytes = batch * HKV * (CTX + 1) * BYTES_PER_TOKEN_HEAD
    peak, peak_src = _peaks()
    achieved = comp_bytes / (dec_ms * 1e-3) / 1e9
    value = world * achieved
    e2e_region_ms = e_app_ms + e_dec_ms
    enc_bytes = CTX * HKV * 2 * ENCODE_BYTES_PER_VECTOR
    clocks = head["clocks"]
    mhz = clocks.get("sm_mhz") or 0.0
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": total_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch": batch, "per_gpu": True, "inner": inner,
                   "step_definition": f"{inner} consecutive passes of (encode chunk, append, decode attention); times below are per pass",
                   "ms_per_pass": total_ms / n_pass, "timed_region_s": total_ms * 1e-3,
                   "l2": "inputs larger than L2 and rotated: two resident 260 MB caches alternate (a pass encodes and appends into one "
                         "and decodes the other, which was last written two passes earlier), two alternating 128 MiB prefill chunks",
                   "compressed_bytes_per_decode": comp_bytes, "decode_ms": dec_ms, "append_ms": app_ms, "encode_ms": enc_ms,
                   "decode_best_ms": dec_best, "encode_best_ms": enc_best, "event_samples": head["seg_samples"],
                   "decode_ms_x_sm_mhz": dec_ms * mhz, "encode_ms_x_sm_mhz": enc_ms * mhz,
                   "value_definition": "compressed bytes / mean CUDA-event time of pq_decode_attention (one persistent kernel)"},
        "encode": {"tokens_per_s": world * CTX / (enc_ms * 1e-3), "vectors_per_s": world * CTX * HKV * 2 / (enc_ms * 1e-3),
                   "gbs": enc_bytes / (enc_ms * 1e-3) / 1e9, "hbm_frac_measured": enc_bytes / (enc_ms * 1e-3) / 1e9 / peak,
                   "frac_of_nominal_8TBs": enc_bytes / (enc_ms * 1e-3) / 1e9 / 8000.0,
                   "e2e_tokens_per_s": world * CTX / (e_enc_ms * 1e-3), "e2e_h2d_bytes_per_chunk": head["h2d_encode_bytes"]},
        "roofline": {"kernel": "decode_attention_fast_kernel", "bound": "hbm", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "frac_of_nominal_8TBs": achieved / 8000.0,
                     "peak_source": peak_src, "traffic": _decode_traffic(batch)},
        "e2e": {"value": world * comp_bytes / (e2e_region_ms * 1e-3) / 1e9, "unit": UNIT,
                "h2d_bytes_per_step": head["h2d_decode_bytes"], "d2h_bytes_per_step": head["d2h_bytes"],
                "region_ms": e2e_region_ms,
                "definition": "compressed bytes / time of [H2D of the new k, v from pinned memory, pq_append_kv, H2D of q, "
                              "pq_decode_attention, D2H of the output]; the byte counts are the copies inside that region.  "
                              "The prefill chunk's own H2D (e2e_h2d_bytes_per_chunk) and encode are timed as encode.e2e_tokens_per_s",
                "ms_per_pass_with_prefill_h2d": e2e_total_ms / (steps * head["e2e_inner"])},
        "gpu_launches": 5 * n_pass,  # encode + lens, append + lens, decode attention
        "clocks": clocks,
        "oracle_match": head["match"],
        "configs": {},
    }
    if c4:
        t, tb, te = red[pos:pos + 3]
        pos += 3
        gbs = c4["compressed_bytes_per_step"] / (t * 1e-3) / 1e9
        line["configs"]["cfg4"] = dict(c4, decode_step_ms=t, decode_step_best_ms=tb, encode_ms_per_layer=te,
                                       per_layer_us=t / c4["layers"] * 1e3, gbs=gbs, hbm_frac_measured=gbs / peak,
                                       frac_of_nominal_8TBs=gbs / 8000.0)
    if c5:
        t, ta, td = red[pos:pos + 3]
        pos_mq = pos + 3
        gbs = c5["compressed_bytes_per_step"] / (td * 1e-3) / 1e9
        line["configs"]["cfg5"] = dict(c5, total_ms_128_steps=t, ms_per_step=t / c5["steps"], append_ms=ta, decode_ms=td,
                                       decode_gbs=gbs, hbm_frac_measured=gbs / peak, frac_of_nominal_8TBs=gbs / 8000.0)
    if mq:
        t = red[pos_mq if c5 else pos]
        line["configs"]["multi_query_chunk"] = dict(mq, ms=t, us_per_query=t / mq["n_q"] * 1e3,
                                                    mma_tflops=mq["mma_tflops"] * mq["ms"] / t)
    if local.get("paged"):
        line["configs"]["paged_decode"] = dict(local["paged"], hbm_frac_measured=local["paged"]["gbs"] / peak)
    if local.get("general"):
        line["configs"]["general_full_recursion_3bit"] = local["general"]
    if local.get("tail"):
        line["configs"]["tail_window"] = local["tail"]
    if local.get("online"):
        line["configs"]["online_codebook"] = local["online"]  # this rank's own figures (not reduced over ranks)
    if cpu_baseline is not None:
        line["cpu_baseline"] = cpu_baseline
    return line


def run_cuda(args):
    import paper_2502_02617_b200 as pq
    from paper_2502_02617_b200 import synthetic
    dist, rank, world, local_rank = dist_setup("nccl")
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    pq.lib()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    extra = {"cfg4": measure_config4, "cfg5": measure_config5, "multi_query": measure_multi_query,
             "online": measure_online_codebook, "paged": measure_paged, "tail": measure_tail_window, "general": measure_general}
    if args.only:   # one of the side measurements by itself (profiling captures): its own figures, this rank's
        print(json.dumps({"only": args.only, "n_gpus": world, "rank": rank, **extra[args.only](args, pq, synthetic, dev, rank)}))
        return
    local = {"batch": BATCH, "headline": measure_headline(args, pq, synthetic, dev, rank, barrier)}
    torch.cuda.empty_cache()
    if not args.skip_configs:
        local["cfg4"] = measure_config4(args, pq, synthetic, dev, rank)
        torch.cuda.empty_cache()
        local["cfg5"] = measure_config5(args, pq, synthetic, dev, rank)
        torch.cuda.empty_cache()
        local["multi_query"] = measure_multi_query(args, pq, synthetic, dev, rank)
        torch.cuda.empty_cache()
        local["online"] = measure_online_codebook(args, pq, synthetic, dev, rank)
        torch.cuda.empty_cache()
        local["paged"] = measure_paged(args, pq, synthetic, dev, rank)
        torch.cuda.empty_cache()
        local["tail"] = measure_tail_window(args, pq, synthetic, dev, rank)
        torch.cuda.empty_cache()
        local["general"] = measure_general(args, pq, synthetic, dev, rank)
        torch.cuda.empty_cache()
    cpu = _oracle_sample_throughput(12.0) if rank == 0 and world == 1 and not args.no_cpu_baseline else None
    line = reduce_and_format(local, args.steps, args.warmup, rank, world, dist, dev, cpu)
    if line is not None:
        print(json.dumps(line))


def main():
    global BATCH
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--inner", type=int, default=0, help="passes per step (0: sized for a timed region of about two seconds)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=BATCH, help="sequences in the resident batch (profiling captures use fewer)")
    ap.add_argument("--skip-e2e", action="store_true", help="skip the host-buffer leg (profiling captures)")
    ap.add_argument("--skip-match", action="store_true", help="skip the sampled oracle checks (profiling captures)")
    ap.add_argument("--skip-configs", action="store_true", help="skip configs 4 and 5 (profiling captures)")
    ap.add_argument("--only", default="", choices=["", "cfg4", "cfg5", "multi_query", "online", "paged", "tail", "general"],
                    help="run one of the side measurements alone and print its figures (profiling captures)")
    args = ap.parse_args()
    BATCH = args.batch
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
