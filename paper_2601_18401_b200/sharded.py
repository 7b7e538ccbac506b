"""Sequence-sharded decode step: the KV cache of a sequence is split by position across the ranks of a
process group; one step is three library calls per rank with two all-gathers between them.  Argument
marshalling and the two exchanges only: every arithmetic step runs in the library's kernels."""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as B


def shard_range(cache_len: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous position range [lo, lo + len) of `rank` when `cache_len` positions are dealt to `world`
    ranks in equal shares (the last ranks may get less)."""
    per = (cache_len + world - 1) // world
    lo = min(rank * per, cache_len)
    return lo, min(per, cache_len - lo)


def _gather(t: torch.Tensor, group) -> torch.Tensor:
    """All ranks' copies of `t`, stacked in rank order: [world, ...].  With a backend that has no device
    collectives (gloo) a device tensor is staged through the host."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    src = t.contiguous()
    staged = src.is_cuda and dist.get_backend(group) == "gloo"
    if staged:
        src = src.cpu()
    parts = [torch.empty_like(src) for _ in range(world)]
    dist.all_gather(parts, src, group=group)
    out = torch.stack(parts)
    return out.to(t.device) if staged else out


def decode_step_sharded(handle: B.Handle, q_s: torch.Tensor, q: torch.Tensor, k_local: torch.Tensor,
                        v_local: torch.Tensor, shard_lo: int, n_ctx: int, params: B.sla_params_t, *,
                        shard_len: Optional[int] = None, group=None):
    """One decode step on this rank's slice of the cache (positions shard_lo .. shard_lo + shard_len - 1).
    Every rank passes the same q_s, q [B,Hq,D] and gets the same out, lse, anchors and scores, equal to
    sla_decode_step on the whole cache.  `group`: a torch.distributed process group (default group when
    None and torch.distributed is initialised; a single rank otherwise)."""
    import torch.distributed as dist
    multi = dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1
    cand_a, cand_s = B.sla_decode_shard_search(handle, q_s, k_local, shard_lo, n_ctx, params, shard_len=shard_len)
    all_a = _gather(cand_a, group) if multi else cand_a[None]
    all_s = _gather(cand_s, group) if multi else cand_s[None]
    anchor, score, partial = B.sla_decode_shard_attend(handle, q, k_local, v_local, shard_lo, n_ctx, params,
                                                      all_a.contiguous(), all_s.contiguous(), shard_len=shard_len)
    all_p = _gather(partial, group) if multi else partial[None]
    out, lse = B.sla_decode_shard_merge(handle, all_p.contiguous(), q)
    return out, lse, anchor, score
