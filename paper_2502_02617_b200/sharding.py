"""Multi-GPU plumbing.  The hot path has no exchange step: (sequence, kv head) units are independent
(Algorithm 1 works per vector, Eq. 3 per query head), S and the codebooks are replicated.  Ranks
therefore own disjoint sequences and never communicate on the data path; torch.distributed is used
only to agree on timings (max over ranks) and to gather results for checks.

The one optional exchange: a cache whose TOKENS are sharded over ranks (contexts too long for one GPU).  Each rank
attends over its own tokens and the partial results -- d + 1 floats per query head -- are all-gathered and merged
(shard_positions, gather_partials; the merge itself is the library's pq_merge_attention)."""
from __future__ import annotations

import torch


def shard_range(n_units: int, rank: int, world: int) -> range:
    """Contiguous, balanced shard of `n_units` independent units (sequences) for `rank`."""
    base, extra = divmod(n_units, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def gather_shards(local: torch.Tensor, n_units: int, dist=None) -> torch.Tensor:
    """Concatenate per-rank results along dim 0 in rank order (shards from shard_range)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local
    world = dist.get_world_size()
    sizes = [len(shard_range(n_units, r, world)) for r in range(world)]
    pad = max(sizes)
    buf = torch.zeros((pad,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    buf[: local.shape[0]] = local
    out = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(out, buf)
    return torch.cat([o[:s] for o, s in zip(out, sizes)], dim=0)


def shard_positions(n_tokens: int, world: int, rank: int, granule: int = 128) -> torch.Tensor:
    """Token-sharded cache: position p of a sequence lives on rank (p // granule) % world, in order.  The positions
    (int64) of the first n_tokens that `rank` holds."""
    p = torch.arange(n_tokens, dtype=torch.int64)
    return p[(p // granule) % world == rank]


def gather_partials(out, lse, dist, group=None):
    """All-gather every rank's partial attention (out [B, Hq, d] float32, lse [B, Hq]) into [W, ...] tensors, rank order."""
    world = dist.get_world_size(group)
    outs = [torch.empty_like(out) for _ in range(world)]
    lses = [torch.empty_like(lse) for _ in range(world)]
    dist.all_gather(outs, out.contiguous(), group=group)
    dist.all_gather(lses, lse.contiguous(), group=group)
    return torch.stack(outs), torch.stack(lses)
