"""Plumbing for a context sharded over devices (torch.distributed, one process per GPU).

Every rank runs xy_attn_run over its own slice of the keys (see xy_attn_shard_context), then
calls `gather_and_merge`: one all-gather of (O_k bf16, LSE_k fp32) into local memory, followed by
the local merge kernel xy_attn_merge_shards.  The merge kernel reads local memory only; the
collective is the library's (NCCL on GPUs; gloo moves the same layout on CPU ranks in the tests).
No arithmetic of the method happens here.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding as xb


def gather_shards(o_local: torch.Tensor, lse_local: torch.Tensor, group=None):
    """All-gather of the per-rank results.  o_local [rows, D] bf16, lse_local [rows] fp32 ->
    (o_shards [world, rows, D], lse_shards [world, rows]) in rank order, on the inputs' device."""
    world = dist.get_world_size(group)
    o_local = o_local.contiguous()
    lse_local = lse_local.contiguous()
    o_shards = torch.empty((world,) + tuple(o_local.shape), dtype=o_local.dtype, device=o_local.device)
    lse_shards = torch.empty((world,) + tuple(lse_local.shape), dtype=lse_local.dtype, device=lse_local.device)
    if o_local.is_cuda:
        dist.all_gather_into_tensor(o_shards, o_local, group=group)
        dist.all_gather_into_tensor(lse_shards, lse_local, group=group)
    else:  # gloo: list form
        dist.all_gather(list(o_shards.unbind(0)), o_local, group=group)
        dist.all_gather(list(lse_shards.unbind(0)), lse_local, group=group)
    return o_shards, lse_shards


def gather_and_merge(o_local: torch.Tensor, lse_local: torch.Tensor, group=None, stream=None):
    """o_local bf16 [T, Hq, D] and lse_local fp32 [T, Hq] of this rank's slice -> merged
    (o bf16 [T, Hq, D], lse fp32 [T, Hq]), identical on every rank.  CUDA tensors only: the
    merge is the library's kernel and there is no CPU fallback."""
    if not o_local.is_cuda:
        raise RuntimeError("gather_and_merge needs CUDA tensors; there is no CPU fallback")
    T, Hq, D = o_local.shape
    o_shards, lse_shards = gather_shards(o_local.reshape(T * Hq, D), lse_local.reshape(T * Hq), group)
    o = torch.empty_like(o_local)
    lse = torch.empty_like(lse_local)
    xb.xy_attn_merge_shards(o_shards, lse_shards, o.view(T * Hq, D), lse.view(T * Hq), stream)
    return o, lse
