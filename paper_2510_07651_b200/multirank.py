"""Host-side logic for running the path on several GPUs, one process per GPU.

Every (batch item, KV head) unit is independent through score, select and compact (App. A.5 keeps a
group's query heads with their KV head), so the units are partitioned across ranks and no collective
touches the data path.  `torch.distributed` is only used to agree on a step time (max over ranks) and,
if the caller wants the whole index tensor on every rank, to gather the per-unit results.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def partition_units(n_units: int, world: int) -> list[tuple[int, int]]:
    """Contiguous, balanced [begin, end) ranges of the units, one per rank (earlier ranks get the
    extra unit when the division leaves a remainder; ranks beyond the units get empty ranges)."""
    base, extra = divmod(n_units, world)
    out, lo = [], 0
    for r in range(world):
        hi = lo + base + (1 if r < extra else 0)
        out.append((lo, hi))
        lo = hi
    return out


def kv_head_shard(n_kv_heads: int, group: int, rank: int, world: int) -> tuple[slice, slice]:
    """Slices of the KV-head axis and of the query-head axis that `rank` owns when the KV heads of
    one layer are split across `world` ranks (each KV head travels with its `group` query heads)."""
    lo, hi = partition_units(n_kv_heads, world)[rank]
    return slice(lo, hi), slice(lo * group, hi * group)


def max_over_ranks(ms: float, device: torch.device | str = "cpu") -> float:
    """The slowest rank's time: the time of the whole job."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gather_head_shards(local: torch.Tensor, n_kv_heads: int) -> torch.Tensor:
    """All-gather of per-head results `[B, heads_of_this_rank, ...]` into `[B, n_kv_heads, ...]` on
    every rank (ranks may own different numbers of heads)."""
    world = dist.get_world_size()
    parts = partition_units(n_kv_heads, world)
    most = max(hi - lo for lo, hi in parts)
    dtype = local.dtype
    raw = local.contiguous().view(torch.uint8)          # bytes: every backend can move them
    pad = torch.zeros((raw.shape[0], most) + tuple(raw.shape[2:]), dtype=torch.uint8, device=raw.device)
    pad[:, :raw.shape[1]] = raw
    bufs = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(bufs, pad)
    return torch.cat([bufs[r][:, :parts[r][1] - parts[r][0]] for r in range(world)], dim=1).view(dtype)
