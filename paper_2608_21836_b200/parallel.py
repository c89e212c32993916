"""Context-parallel decode: one sequence's KV cache sharded over the ranks of a process group.

The attention path has no exchange step when sequences or KV heads are sharded (replicas). Only when ONE sequence's
cache is split across GPUs do the ranks have to talk: each decodes over its shard and returns (o, lse); the partials
are all-gathered (NCCL over NVLink on GPUs) and merged with the same log-sum-exp formula the split decode kernel uses
between its pieces. This module is the host-side plumbing; the arithmetic is in the library (`l4l_attn_decode`,
`l4l_attn_merge`) and is passed in, so that the plumbing can be exercised on CPU ranks with stand-in functions.
"""
from __future__ import annotations

from typing import Callable, Optional, Tuple

import torch
import torch.distributed as dist


def shard_bounds(kv_len: int, world: int, rank: int, granule: int = 128) -> Tuple[int, int]:
    """Token range [begin, end) of `rank`'s shard of a sequence of kv_len cached tokens: contiguous ranges of whole
    `granule`-token blocks (the decode kernel's tile), as even as whole blocks allow; the last block may be ragged."""
    blocks = (kv_len + granule - 1) // granule
    per, extra = divmod(blocks, world)
    b0 = rank * per + min(rank, extra)
    b1 = b0 + per + (1 if rank < extra else 0)
    return min(b0 * granule, kv_len), min(b1 * granule, kv_len)


def context_parallel_decode(local_decode: Callable[[], Tuple[torch.Tensor, torch.Tensor]],
                            merge: Callable[[torch.Tensor, torch.Tensor], Tuple[torch.Tensor, torch.Tensor]],
                            group: Optional[dist.ProcessGroup] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """local_decode() -> (o [B,Hq,D], lse [B,Hq]) over this rank's shard; merge(o_parts [R,B,Hq,D], lse_parts [R,B,Hq])
    -> (o, lse). Returns the merged result on every rank. Without an initialised process group (or world size 1) the
    local result is the result."""
    o, lse = local_decode()
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return o, lse
    world = dist.get_world_size(group)
    # gathered along dimension 0 (the form every backend accepts), then seen as [R, ...]
    o_cat = torch.empty((world * o.shape[0],) + tuple(o.shape[1:]), dtype=o.dtype, device=o.device)
    lse_cat = torch.empty((world * lse.shape[0],) + tuple(lse.shape[1:]), dtype=lse.dtype, device=lse.device)
    dist.all_gather_into_tensor(o_cat, o.contiguous(), group=group)
    dist.all_gather_into_tensor(lse_cat, lse.contiguous(), group=group)
    return merge(o_cat.view((world,) + tuple(o.shape)), lse_cat.view((world,) + tuple(lse.shape)))


def gpu_context_parallel_decode(q, o, cache_k_shard, cache_v_shard, kv_lens_shard, max_kv_len: int, scale: float,
                                workspace, group: Optional[dist.ProcessGroup] = None):
    """The GPU form: this rank's shard of every sequence's cache in cache_*_shard (slots 0 .. kv_lens_shard[b] - 1).
    Writes the merged output to `o` and returns its log-sum-exp [B, Hq]."""
    from . import binding as l4l

    B, Hq, _ = q.shape

    def local():
        o_loc = torch.empty_like(q)
        lse_loc = torch.empty(B, Hq, dtype=torch.float32, device=q.device)
        l4l.l4l_attn_decode(q, o_loc, cache_k_shard, cache_v_shard, kv_lens_shard, max_kv_len, scale, workspace, lse=lse_loc)
        return o_loc, lse_loc

    def merge(o_parts, lse_parts):
        lse_out = torch.empty(B, Hq, dtype=torch.float32, device=q.device)
        l4l.l4l_attn_merge(o_parts, lse_parts, o, lse=lse_out)
        return o, lse_out

    o_res, lse_res = context_parallel_decode(local, merge, group)
    if o_res is not o:
        o.copy_(o_res)
    return lse_res
