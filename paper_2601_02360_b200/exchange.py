"""Replica-per-GPU form of the outer step: the one cross-replica exchange of Eq. 2.

In the paper's deployment (section 2, Fig. 1) every replica lives on its own machine; what crosses
the data-parallel axis at an outer step is the sparse message of Eq. 2 line 3, and every replica
then forms the same average (line 5) on its own copy of theta_global.  Here a rank is a replica:

    sl_compress (own replica)  ->  all-gather of (idx, codes, scales)  ->  sl_aggregate_apply

The gather is a plain `torch.distributed.all_gather` of bytes (NCCL on GPUs, gloo on CPU); the
gathered messages land in this rank's own memory before any kernel reads them.  Messages are
listed in rank order, which fixes the order of the additions, so every rank computes bit-identical
parameters.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def _gather_bytes(t: torch.Tensor, world: int, group=None) -> List[torch.Tensor]:
    flat = t.contiguous().view(torch.uint8).reshape(-1)
    out = [torch.empty_like(flat) for _ in range(world)]
    dist.all_gather(out, flat, group=group)
    return [o.view(t.dtype).reshape(t.shape) for o in out]


def all_gather_messages(idx: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor,
                        group=None) -> Tuple[List[torch.Tensor], List[torch.Tensor], List[torch.Tensor]]:
    """This rank's message in, every rank's message out (lists in rank order)."""
    world = dist.get_world_size(group)
    return (_gather_bytes(idx, world, group), _gather_bytes(codes, world, group),
            _gather_bytes(scales, world, group))


def message_bytes(idx: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor) -> int:
    """Bytes one replica sends per outer step."""
    return sum(t.numel() * t.element_size() for t in (idx, codes, scales))


def outer_step_replica(theta_local, theta_global, err, layout, beta: float, chunk: int, k: int, bits: int,
                       outer_lr: float, idx, codes, scales, flags=None, group=None, stream=None):
    """One outer step of the replica this rank hosts.  err, idx, codes, scales and theta_global are
    updated; returns the gathered messages (idx, codes, scales lists in rank order)."""
    from . import api
    api.sl_compress(theta_local, theta_global, err, layout, beta, chunk, k, bits, idx, codes, scales, flags, stream)
    g_idx, g_codes, g_scales = all_gather_messages(idx, codes, scales, group)
    api.sl_aggregate_apply(g_idx, g_codes, g_scales, layout, chunk, k, bits, theta_global, outer_lr, flags, stream)
    return g_idx, g_codes, g_scales
