"""Sampled BN with statistics shared by the GPUs of a process group (Sec. 4.3 of the paper, "Micro-BN":
Sync-BN combined with Feature or Batch Sampling).

One process per GPU; every rank holds its slice of the batch.  The arithmetic is in the library
(``bns_sync_*``); this module only moves the two small per-channel messages between ranks with
``torch.distributed`` (NCCL on GPUs): an all-gather of 3C floats in the forward, an all-reduce of 2C
floats in the backward.  Both are latency-bound; nothing else crosses GPUs.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import bns


def all_gather_rows(rows: torch.Tensor, group=None) -> torch.Tensor:
    """[3, C] per rank -> [world, 3, C], rank-major, identical on every rank."""
    world = dist.get_world_size(group)
    parts = [torch.empty_like(rows) for _ in range(world)]
    dist.all_gather(parts, rows.contiguous(), group=group)
    return torch.stack(parts)


def all_reduce_rows(rows: torch.Tensor, group=None) -> torch.Tensor:
    """Sum of a [2, C] tensor over the ranks (a copy; the input keeps this rank's share)."""
    total = rows.clone()
    dist.all_reduce(total, op=dist.ReduceOp.SUM, group=group)
    return total


def forward(x, gamma, beta, eps, sampling, group=None):
    """Returns (y, mean, invstd, count): statistics of the union of all ranks' sampled sets and the number of
    sampled points per channel in that union (a device tensor; nothing is read back to the host).
    ``sampling`` is this rank's rule - FULL, BATCH or FEATURE on its slice, a VIRTUAL rule on the one rank that
    is fed the virtual samples, or None on a rank that contributes no statistics."""
    local = bns.sync_local_moments(x, sampling, eps)
    gathered = all_gather_rows(local, group)
    mean, invstd, count = bns.sync_merge_moments(gathered, eps)
    y = bns.sync_normalize(x, gamma, beta, mean, invstd)
    if sampling is not None and sampling.rule == bns.RULE_VIRTUAL and sampling.yv is not None:
        bns.sync_normalize(sampling.xv, gamma, beta, mean, invstd, y=sampling.yv)
    return y, mean, invstd, count


def backward(x, dy, gamma, mean, invstd, sampling, count, group=None):
    """Returns (dx, dgamma_local, dbeta_local): dx uses the sums of all ranks; the parameter gradients are
    this rank's share (a data-parallel wrapper reduces them with the other gradients).  On the rank that holds
    virtual samples their gradient dyv joins the sums and dxv is written."""
    virtual = sampling if (sampling is not None and sampling.rule == bns.RULE_VIRTUAL) else None
    dx, local = bns.sync_backward_sums(x, dy, gamma, mean, invstd, virtual_rows=virtual)
    total = all_reduce_rows(local, group)
    bns.sync_backward_apply(x, dy, gamma, mean, invstd, sampling, total, count, dx)
    return dx, local[1], local[0]
