"""A long sequence's KV split over several ranks: partial attention per rank, one small all-gather, log-sum-exp merge.

The report moves part of a long sequence's KV blocks to another DP group, computes attention there and gathers the
external results with an aggregation operator (Hierarchical DP Load Balance, partial migration at block granularity).
Here every rank of ``group`` holds one part of every sequence of the call in its own slots (rank order = position order,
the last rank holds the end of each sequence with the query tokens) and the only exchange is an all-gather of the fp32
partial outputs and their log-sum-exp values: ``rows * H_q * (D + 1) * 4`` bytes per rank.
"""
from __future__ import annotations

from typing import Optional, Sequence, Tuple

import torch
import torch.distributed as dist


def gather_parts(out_part: torch.Tensor, lse_part: torch.Tensor, group=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """All-gather the ranks' partial results: returns ([n_parts, rows, H_q, D], [n_parts, rows, H_q]) in rank order.

    Works on any backend (NCCL on GPUs, gloo on CPU tensors); without an initialised process group the one local part
    is returned as a stack of one."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return out_part.unsqueeze(0), lse_part.unsqueeze(0)
    world = dist.get_world_size(group)
    outs = torch.empty((world,) + tuple(out_part.shape), dtype=out_part.dtype, device=out_part.device)
    lses = torch.empty((world,) + tuple(lse_part.shape), dtype=lse_part.dtype, device=lse_part.device)
    if out_part.is_cuda:
        dist.all_gather_into_tensor(outs, out_part.contiguous(), group=group)
        dist.all_gather_into_tensor(lses, lse_part.contiguous(), group=group)
    else:  # gloo has no all_gather_into_tensor for every version: gather into views
        dist.all_gather(list(outs.unbind(0)), out_part.contiguous(), group=group)
        dist.all_gather(list(lses.unbind(0)), lse_part.contiguous(), group=group)
    return outs, lses


def split_attention(ctx, slots: Sequence[int], q_lens: Sequence[int], q: torch.Tensor, out: torch.Tensor,
                    lse_out: Optional[torch.Tensor] = None, scale: float = 1.0, group=None, holds_tail: Optional[bool] = None):
    """Attention of ``q`` over sequences whose KV is spread over the ranks of ``group``; every rank gets the full result.

    ``slots`` are this rank's ranges (one part of every sequence); ``holds_tail``: whether they end with the query
    tokens (default: the last rank does).  All kernels and the collective run on torch's current stream."""
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    rank = dist.get_rank(group) if world > 1 else 0
    if holds_tail is None:
        holds_tail = rank == world - 1
    rows, hq, d = q.shape
    stream = torch.cuda.current_stream().cuda_stream
    out_part = torch.empty((rows, hq, d), dtype=torch.float32, device=q.device)
    lse_part = torch.empty((rows, hq), dtype=torch.float32, device=q.device)
    ctx.partial_attention(slots, q_lens, [1 if holds_tail else 0] * len(slots), q, out_part, lse_part, scale, stream)
    outs, lses = gather_parts(out_part, lse_part, group)
    ctx.merge_partials(outs.contiguous(), lses.contiguous(), out, lse_out, stream)
