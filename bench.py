#!/usr/bin/env python
"""Benchmark of the PolarQuant hot path on B200.

One step = one pass of the whole path on synthetic Llama-3.1-8B-shaped data:
  (1) pq_encode_kv   : a prefill chunk of 32768 tokens x 8 KV heads x d=128, bf16 K and V
                       (re-encodes one sequence of the resident batch),
  (2) pq_append_kv   : one new token for each of the 8 sequences,
  (3) pq_decode_attention : 32 query heads / 8 KV heads over batch 8 x ~32769 cached tokens.
The headline `value` is the decode-attention throughput on compressed bytes (62 B per token per
KV head for K and again for V), from CUDA events around call (3); the encoder's tokens/s and the
whole-step time are reported beside it.  With --gpus N every rank runs the same per-GPU workload
on its own sequences (no data-path collective; weak scaling) and the slowest rank's time counts.

`--impl reference` times the float64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
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
METRIC = "decode_attention_compressed_kv_throughput"
UNIT = "GB/s"
WORKLOAD = ("decode attention: batch 8 x ctx 32768, 32 q / 8 kv heads, d=128 (config 3); encode chunk 32768 tokens x "
            "8 kv heads (config 2); append 1 token/sequence")


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (earlier pool measurement)"


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
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
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
            out.update(sm_mhz=float(statistics.median(sm)), sm_max_mhz=float(smax), samples=len(sm),
                       reasons=sorted(n for bit, n in self.REASONS.items() if bits & bit))
        return out


def _dist_setup(n_gpus):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
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


def _oracle_match(cache, K_chunk, V_chunk, b_enc, q, out):
    """Sampled parity at the benchmark's full size: codes of sampled vectors of the chunk just
    encoded, and the attention output of two (sequence, kv head) units."""
    from oracle import polarquant_oracle as orc
    rng = np.random.default_rng(0)
    cb = orc.codebooks_from_arrays((4, 2, 2, 2), cache.centroids.numpy(), cache.boundaries.numpy())
    S = cache.S_host.double().numpy()
    n_tok = CTX + 1
    codes, radii = cache.unpack(n_tok)
    toks = np.sort(rng.choice(CTX, 512, replace=False))
    res = {"codes_checked": 0, "codes_mismatch_inside_window": 0, "codes_mismatch_outside_window": 0}
    for kv, X in ((0, K_chunk), (1, V_chunk)):
        for h in range(HKV):
            x = X[torch.as_tensor(toks, device=X.device), h].float().cpu().double().numpy()
            want, _, angles = orc.encode(x, S, cb)
            got = codes[b_enc, h, kv][torch.as_tensor(toks, device=codes.device)].cpu().numpy()
            diff = got != want
            dist = orc.boundary_distance(angles, cb)
            res["codes_checked"] += int(want.size)
            res["codes_mismatch_inside_window"] += int(np.count_nonzero(diff & (dist <= 1e-6)))
            res["codes_mismatch_outside_window"] += int(np.count_nonzero(diff & (dist > 1e-6)))
    lens = cache.lens.cpu().numpy()
    worst = 0.0
    for (b, hk) in ((b_enc, 0), ((b_enc + 3) % BATCH, 5 % HKV)):
        n = int(lens[b])
        c = codes[b, hk, :, :n].cpu().numpy()
        r = radii[b, hk, :, :n].cpu().numpy()
        g = HQ // HKV
        qq = q[b, hk * g:(hk + 1) * g].float().cpu().double().numpy()[None]
        want = orc.decode_attention(qq, c[0][None, None], r[0][None, None], c[1][None, None], r[1][None, None], [n],
                                    cb, S, D ** -0.5)[0]
        got = out[b, hk * g:(hk + 1) * g].float().cpu().double().numpy()
        worst = max(worst, float(np.linalg.norm(got - want) / np.linalg.norm(want)))
    res["attention_rel_l2_worst_of_2_units"] = worst
    res["ok"] = bool(res["codes_mismatch_outside_window"] == 0 and worst < 2e-3)
    return res


# --------------------------------------------------------------------------------------------
# The CUDA arm
# --------------------------------------------------------------------------------------------
def run_cuda(args):
    import paper_2502_02617_b200 as pq
    from paper_2502_02617_b200 import synthetic
    dist, rank, world, local_rank = _dist_setup(args.gpus)
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    pq.lib()
    capacity = CTX + 256
    cache = pq.PolarQuantCache(BATCH, HQ, HKV, D, capacity, seed=0, device=dev)
    stream = torch.cuda.current_stream()

    # Resident state: the batch's cache, filled by the encoder itself (2 distinct prefill chunks,
    # each 128 MiB of bf16 K+V, so successive encode steps never find their input in L2).
    chunks = [synthetic.kv_like(1000 * rank + 10 + i, CTX, HKV, D, torch.bfloat16, dev) for i in range(2)]
    cu = torch.tensor([0, CTX], dtype=torch.int32, device=dev)
    cu_all = torch.zeros(BATCH + 1, dtype=torch.int32, device=dev)
    for b in range(BATCH):
        cu_all.zero_()
        cu_all[b + 1:] = CTX
        Kb, Vb = chunks[b % 2]
        pq.pq_encode_kv(cache.S, cache.tables, Kb, Vb, cu_all, cache.cache, cache.lens, capacity, cache.status)
    torch.cuda.synchronize()
    cache.check_status()
    assert cache.lens.cpu().tolist() == [CTX] * BATCH

    n_total = args.warmup + args.steps
    q_all = [synthetic.queries(77 + i + 1000 * rank, BATCH, HQ, D, torch.bfloat16, dev) for i in range(4)]
    new_all = [synthetic.kv_like(99 + i + 1000 * rank, BATCH, HKV, D, torch.bfloat16, dev) for i in range(4)]
    out = torch.empty_like(q_all[0])
    lens_base = torch.full((BATCH,), CTX, dtype=torch.int32, device=dev)
    cu_step = []
    lens_step = []
    for b in range(BATCH):
        c = torch.zeros(BATCH + 1, dtype=torch.int32, device=dev)
        c[b + 1:] = CTX
        cu_step.append(c)
        l = lens_base.clone()
        l[b] = 0
        lens_step.append(l)

    # pinned host copies for the end-to-end leg
    host_chunks = [(k.cpu().pin_memory(), v.cpu().pin_memory()) for k, v in chunks]
    host_q = [t.cpu().pin_memory() for t in q_all]
    host_new = [(k.cpu().pin_memory(), v.cpu().pin_memory()) for k, v in new_all]
    host_out = torch.empty_like(out, device="cpu").pin_memory()
    dK, dV = torch.empty_like(chunks[0][0]), torch.empty_like(chunks[0][1])
    dq, dk1, dv1 = torch.empty_like(q_all[0]), torch.empty_like(new_all[0][0]), torch.empty_like(new_all[0][1])

    def step(i, ev=None, e2e=False):
        b_enc = i % BATCH
        cache.lens.copy_(lens_step[b_enc])
        if e2e:
            if ev: ev[0].record(stream)
            dK.copy_(host_chunks[i % 2][0], non_blocking=True)
            dV.copy_(host_chunks[i % 2][1], non_blocking=True)
            Kb, Vb = dK, dV
        else:
            Kb, Vb = chunks[i % 2]
            if ev: ev[0].record(stream)
        pq.pq_encode_kv(cache.S, cache.tables, Kb, Vb, cu_step[b_enc], cache.cache, cache.lens, capacity, cache.status)
        if ev: ev[1].record(stream)
        if e2e:
            dk1.copy_(host_new[i % 4][0], non_blocking=True)
            dv1.copy_(host_new[i % 4][1], non_blocking=True)
            k1, v1 = dk1, dv1
        else:
            k1, v1 = new_all[i % 4]
        pq.pq_append_kv(cache.S, cache.tables, k1, v1, cache.cache, cache.lens, capacity, cache.status)
        if ev: ev[2].record(stream)
        if e2e:
            dq.copy_(host_q[i % 4], non_blocking=True)
            qq = dq
        else:
            qq = q_all[i % 4]
        pq.pq_decode_attention(cache.S, cache.tables, qq, cache.cache, cache.lens, HKV, capacity, CTX + 1,
                               D ** -0.5, out, cache.workspace, cache.status)
        if e2e:
            host_out.copy_(out, non_blocking=True)
        if ev: ev[3].record(stream)
        return b_enc, qq

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(e2e):
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
        for i in range(args.warmup):
            step(i, None, e2e)
        barrier()
        wall = [time.time(), None]
        t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_start.record(stream)
        last = None
        for i in range(args.steps):
            last = step(args.warmup + i, evs[i], e2e)
        t_end.record(stream)
        barrier()
        wall[1] = time.time()
        total_ms = t_start.elapsed_time(t_end)
        seg = np.array([[e[k].elapsed_time(e[k + 1]) for k in range(3)] for e in evs])  # encode, append, decode
        return total_ms, seg, last, wall

    sampler = ClockSampler(local_rank)
    sampler.start()
    total_ms, seg, last, wall = timed(e2e=False)
    clocks = sampler.stop(wall[0], wall[1])
    cache.check_status()
    match = None
    if rank == 0 and not args.skip_match:
        b_enc, qq = last
        Kb, Vb = chunks[(n_total - 1) % 2]
        match = _oracle_match(cache, Kb, Vb, b_enc, qq, out)
    e2e_total_ms, e2e_seg, _, _ = (total_ms, seg, None, None) if args.skip_e2e else timed(e2e=True)
    cache.check_status()

    def reduce_max(x):
        if dist is None:
            return x
        t = torch.tensor(x, dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return t.cpu().numpy() if t.ndim else float(t)

    enc_ms, app_ms, dec_ms = (float(v) for v in reduce_max(seg.mean(0)))
    e_enc_ms, e_app_ms, e_dec_ms = (float(v) for v in reduce_max(e2e_seg.mean(0)))
    step_ms = float(reduce_max(total_ms)) / args.steps
    comp_bytes = BATCH * HKV * (CTX + 1) * BYTES_PER_TOKEN_HEAD
    value = world * comp_bytes / (dec_ms * 1e-3) / 1e9
    e2e_value = world * comp_bytes / ((e_app_ms + e_dec_ms) * 1e-3) / 1e9
    peak, peak_src = _peaks()
    achieved = comp_bytes / (dec_ms * 1e-3) / 1e9
    enc_bytes = CTX * HKV * 2 * (256 + 62)

    if rank != 0:
        return
    # DRAM bytes of one decode-attention launch: ncu capture at batch 4 (profiles/decode_attention_fast_kernel_
    # batch4_ctx32768.md: 130.47 MB read + 3.45 MB written), scaled by the batch (traffic is proportional to it)
    traffic = (130.47e6 + 3.45e6) * BATCH / 4.0
    cpu = _oracle_sample_throughput(12.0) if world == 1 and not args.no_cpu_baseline else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f16",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch": BATCH, "per_gpu": True, "l2": "inputs larger than L2 (260 MB cache per decode, "
                   "two alternating 128 MiB prefill chunks)", "compressed_bytes_per_decode": comp_bytes,
                   "decode_ms": dec_ms, "append_ms": app_ms, "encode_ms": enc_ms,
                   "value_definition": "compressed bytes / CUDA-event time of pq_decode_attention (one persistent kernel)"},
        "encode": {"tokens_per_s": world * CTX / (enc_ms * 1e-3), "vectors_per_s": world * CTX * HKV * 2 / (enc_ms * 1e-3),
                   "gbs": enc_bytes / (enc_ms * 1e-3) / 1e9, "hbm_frac_measured": enc_bytes / (enc_ms * 1e-3) / 1e9 / peak,
                   "e2e_tokens_per_s": world * CTX / (e_enc_ms * 1e-3)},
        "roofline": {"kernel": "decode attention main kernel", "bound": "hbm", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "frac_of_nominal_8TBs": achieved / 8000.0,
                     "peak_source": peak_src, "traffic": traffic},
        "e2e": {"value": e2e_value, "unit": UNIT,
                "h2d_bytes_per_step": int(2 * chunks[0][0].numel() * 2 + 2 * new_all[0][0].numel() * 2 + q_all[0].numel() * 2),
                "d2h_bytes_per_step": int(out.numel() * 2),
                "definition": "compressed bytes / (H2D of new k,v and q + append + decode attention + D2H of the output); "
                              "the 128 MiB prefill chunk's H2D is charged to encode.e2e_tokens_per_s",
                "ms_per_step": float(reduce_max(e2e_total_ms)) / args.steps},
        "gpu_launches": 5 * args.steps,  # encode + lens, append + lens, decode attention
        "clocks": clocks,
        "oracle_match": match,
    }
    if cpu is not None:
        line["cpu_baseline"] = cpu
    print(json.dumps(line))


def main():
    global BATCH
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=BATCH, help="sequences in the resident batch (profiling captures use fewer)")
    ap.add_argument("--skip-e2e", action="store_true", help="skip the host-buffer leg (profiling captures)")
    ap.add_argument("--skip-match", action="store_true", help="skip the sampled oracle check (profiling captures)")
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
