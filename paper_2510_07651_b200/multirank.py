"""Host-side logic for running the path on several GPUs, one process per GPU.

Every (batch item, KV head) unit is independent through score, select and compact (App. A.5 keeps a
group's query heads with their KV head), so the units are partitioned across ranks and no collective
touches the data path.  `torch.distributed` is only used to agree on a step time (max over ranks) and,
if the caller wants the whole index tensor on every rank, to gather the per-unit results.

A cache sharded by TOKEN range instead (context parallelism: a sequence too long for one GPU) has one
real exchange: the window attention of Sec. 3 is a softmax over all cached tokens, so the ranks
all-gather their shards' (o, lse) of the R window rows, merge them, and then score their own tokens
(`context_parallel_scores`); the scores are gathered before the selection (`gather_token_shards`).
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


def token_shards(n_tokens: int, world: int) -> list[tuple[int, int]]:
    """Contiguous, balanced [begin, end) token ranges of a sequence, one per rank."""
    return partition_units(n_tokens, world)


def context_parallel_scores(q, k_local, v_local, *, offset: int, total_len: int, variants=("VK",), causal=True,
                            scale=0.0, path="auto", group=None, ops=None):
    """This rank's scores [n_variants,B,Hkv,n_local] of a cache sharded by token range.

    q [B,Hq,W,d] are the window queries (the last W positions of the whole sequence, the same on every
    rank); k_local, v_local [B,Hkv,n_local,d] hold tokens offset .. offset + n_local - 1 of a sequence of
    total_len tokens.  Steps: the shard's own window attention; all-gather of (o, lse) over `group`
    (B*Hq*W*(d+1) floats per rank); merge; scores of the local tokens from the merged attention.
    `ops` supplies obc_window_attention / obc_merge_attention / obc_score_given (default: the library)."""
    if ops is None:
        from . import api as ops
    B = q.shape[0]
    mask = torch.full((B,), int(total_len) - int(offset), dtype=torch.int32, device=q.device)
    o, lse = ops.obc_window_attention(q, k_local, v_local, mask_lens=mask, scale=scale, causal=causal, path=path)
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world > 1:
        o_parts = [torch.empty_like(o) for _ in range(world)]
        lse_parts = [torch.empty_like(lse) for _ in range(world)]
        dist.all_gather(o_parts, o.contiguous(), group=group)
        dist.all_gather(lse_parts, lse.contiguous(), group=group)
        o_parts, lse_parts = torch.stack(o_parts), torch.stack(lse_parts)
    else:
        o_parts, lse_parts = o.unsqueeze(0).contiguous(), lse.unsqueeze(0).contiguous()
    o_all, lse_all = ops.obc_merge_attention(o_parts, lse_parts)
    return ops.obc_score_given(q, k_local, v_local, o_all, lse_all, mask_lens=mask, variants=variants, causal=causal,
                               scale=scale, path=path)


def gather_token_shards(local: torch.Tensor, total_len: int, group=None) -> torch.Tensor:
    """All-gather of per-token results `[..., n_local]` (this rank's token range of `token_shards`) into
    `[..., total_len]` on every rank, e.g. the scores before a selection that every rank repeats."""
    world = dist.get_world_size(group)
    parts = token_shards(total_len, world)
    most = max(hi - lo for lo, hi in parts)
    pad = torch.zeros(tuple(local.shape[:-1]) + (most,), dtype=local.dtype, device=local.device)
    pad[..., :local.shape[-1]] = local
    bufs = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(bufs, pad, group=group)
    return torch.cat([bufs[r][..., :parts[r][1] - parts[r][0]] for r in range(world)], dim=-1)
