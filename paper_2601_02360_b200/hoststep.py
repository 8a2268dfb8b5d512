"""The outer step (Eq. 2 of section 2.1) for callers whose replicas' parameters sit in HOST memory.

A replica's parameters after its H inner steps may live on the host (the replicas of one GPU are
time-multiplexed, or were received from other machines).  The whole step is then bound by the
host-to-device copies (12 R bytes of kernel traffic per parameter against 4 R bytes over PCIe, which is
two orders of magnitude slower than HBM), so what matters is that nothing else adds to them: the arena is
cut into groups of consecutive tensors (chunks never straddle tensors, so a group is an outer step of its
own) and group g's kernels and device-to-host copies run while group g+1 is still being copied in - three
streams, both PCIe directions busy at once.  Marshalling only: every step of the path is one of the
library's calls on a sub-arena.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch

from . import api
from .exchange import TensorGroup, group_slices, plan_groups  # noqa: F401  (plan_groups is re-exported for callers)


class HostStepStreams:
    def __init__(self, device=None):
        self.h2d = torch.cuda.Stream(device)
        self.d2h = torch.cuda.Stream(device)


def outer_step_from_host(host_theta_local: Sequence[torch.Tensor], theta_local: Sequence[torch.Tensor],
                         theta_global: torch.Tensor, err: Sequence[torch.Tensor], groups: Sequence[TensorGroup],
                         beta: float, chunk: int, k: int, bits: int, outer_lr: float, idx: Sequence[torch.Tensor],
                         codes: Sequence[torch.Tensor], scales: Sequence[torch.Tensor],
                         host_theta_global: Optional[torch.Tensor] = None,
                         host_messages: Optional[Sequence[Sequence[torch.Tensor]]] = None, flags=None,
                         streams: Optional[HostStepStreams] = None) -> None:
    """One outer step for R replicas whose parameters are in pinned host tensors `host_theta_local[r]`
    (staged through the device tensors `theta_local[r]`).  err, idx, codes, scales and theta_global (all
    on the device) are updated exactly as by sl_outer_step; if given, `host_theta_global` receives the new
    theta_global and `host_messages` = (idx, codes, scales) lists of pinned tensors receive the messages.
    Asynchronous: on return everything is enqueued and the current stream waits for all of it."""
    R = len(theta_local)
    cur = torch.cuda.current_stream()
    s = streams or HostStepStreams(theta_global.device)
    stride = api.sl_codes_stride(k, bits)
    s.h2d.wait_stream(cur)
    s.d2h.wait_stream(cur)
    for g in groups:
        lay = api.Layout(g.offsets, g.cols)
        with torch.cuda.stream(s.h2d):
            for r in range(R):
                theta_local[r][g.e0:g.e1].copy_(host_theta_local[r][g.e0:g.e1], non_blocking=True)
            arrived = torch.cuda.Event()
            arrived.record(s.h2d)
        cur.wait_event(arrived)
        parts = [group_slices(g, k, stride, idx[r], codes[r], scales[r]) for r in range(R)]
        g_idx, g_codes, g_scales = [p[0] for p in parts], [p[1] for p in parts], [p[2] for p in parts]
        api.sl_outer_step([t[g.e0:g.e1] for t in theta_local], theta_global[g.e0:g.e1], [e[g.e0:g.e1] for e in err], lay,
                          beta, chunk, k, bits, outer_lr, g_idx, g_codes, g_scales, flags, cur)
        if host_theta_global is not None or host_messages is not None:
            done = torch.cuda.Event()
            done.record(cur)
            with torch.cuda.stream(s.d2h):
                s.d2h.wait_event(done)
                if host_theta_global is not None:
                    host_theta_global[g.e0:g.e1].copy_(theta_global[g.e0:g.e1], non_blocking=True)
                if host_messages is not None:
                    for r in range(R):
                        for dst, src in zip(group_slices(g, k, stride, host_messages[0][r], host_messages[1][r],
                                                         host_messages[2][r]), parts[r]):
                            dst.copy_(src, non_blocking=True)
    cur.wait_stream(s.h2d)
    cur.wait_stream(s.d2h)
