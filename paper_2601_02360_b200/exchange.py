"""Replica-per-GPU form of the outer step: the one cross-replica exchange of Eq. 2.

In the paper's deployment (section 2, Fig. 1) every replica lives on its own machine; what crosses
the data-parallel axis at an outer step is the sparse message of Eq. 2 line 3, and every replica
then forms the same average (line 5) on its own copy of theta_global.  Here a rank is a replica:

    sl_compress (own replica)  ->  all-gather of (idx, codes, scales)  ->  sl_aggregate_apply

The gather is a plain `torch.distributed.all_gather` of bytes (NCCL on GPUs, gloo on CPU); the
gathered messages land in this rank's own memory before any kernel reads them.  Messages are
listed in rank order, which fixes the order of the additions, so every rank computes bit-identical
parameters.

`outer_step_replica_peer` is the form without a gather: every rank writes its message into a
buffer that all ranks of the node have mapped (symmetric memory over NVLink), and after one
barrier `sl_aggregate_apply` is handed the PEERS' buffers as its message tables, so the
averaging kernel pulls each chunk's messages over NVLink with plain loads while it works through
the chunks - the transfer and the arithmetic overlap chunk by chunk, nothing is staged, and every
load from a peer is an ordinary read-only load issued by the thread that needs the value.

`outer_step_replica_pipelined` cuts the arena into groups of consecutive tensors and overlaps the
gather of one group's message with the compression of the next group (two CUDA streams); the
result is the same bit for bit, because chunks never straddle tensors and every chunk is handled
by the same kernels as in the one-shot form.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence, Tuple

import numpy as np

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


def all_gather_messages_idx12(idx: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor, layout, chunk: int,
                              k: int, group=None, flags=None):
    """The same exchange with the positions sent as 12 bits each (sl_pack_idx12 before the gather,
    sl_unpack_idx12 of every rank's part after it, both on the current stream).  Returns the lists in
    rank order (positions back in their uint16 form) and the bytes this rank sent."""
    from . import api
    world = dist.get_world_size(group)
    nc = scales.numel()
    packed = torch.empty(nc * api.sl_idx12_stride(k), dtype=torch.uint8, device=idx.device)
    api.sl_pack_idx12(idx, nc, k, packed, flags)
    g_packed = _gather_bytes(packed, world, group)
    g_codes = _gather_bytes(codes, world, group)
    g_scales = _gather_bytes(scales, world, group)
    g_idx = [torch.empty_like(idx) for _ in range(world)]
    for r in range(world):
        api.sl_unpack_idx12(g_packed[r], layout, chunk, k, g_idx[r])
    return g_idx, g_codes, g_scales, message_bytes(packed, codes, scales)


def outer_step_replica(theta_local, theta_global, err, layout, beta: float, chunk: int, k: int, bits: int,
                       outer_lr: float, idx, codes, scales, flags=None, group=None, stream=None, idx12: bool = False):
    """One outer step of the replica this rank hosts.  err, idx, codes, scales and theta_global are
    updated; returns the gathered messages (idx, codes, scales lists in rank order).  idx12: send the
    positions as 12 bits each (chunk <= 4096; `stream` must then be the current stream)."""
    from . import api
    api.sl_compress(theta_local, theta_global, err, layout, beta, chunk, k, bits, idx, codes, scales, flags, stream)
    if idx12:
        g_idx, g_codes, g_scales, _ = all_gather_messages_idx12(idx, codes, scales, layout, chunk, k, group, flags)
    else:
        g_idx, g_codes, g_scales = all_gather_messages(idx, codes, scales, group)
    api.sl_aggregate_apply(g_idx, g_codes, g_scales, layout, chunk, k, bits, theta_global, outer_lr, flags, stream)
    return g_idx, g_codes, g_scales


@dataclasses.dataclass
class TensorGroup:
    """A run of consecutive tensors of the arena with the element and chunk ranges it owns."""
    t0: int
    t1: int
    e0: int
    e1: int
    c0: int
    c1: int
    offsets: np.ndarray           # the group's own offsets, starting at 0
    cols: Optional[np.ndarray]


def plan_groups(offsets: Sequence[int], chunk: int, n_groups: int,
                cols: Optional[Sequence[int]] = None) -> List[TensorGroup]:
    """Cuts the tensors into at most n_groups runs of about equal element counts (host logic only).
    A group never splits a tensor, so its chunks are exactly the arena's chunks c0..c1-1."""
    from . import api
    off = np.asarray(offsets, dtype=np.uint64)
    n_t = len(off) - 1
    assert n_t >= 1 and n_groups >= 1
    total = int(off[-1])
    cuts = [0]
    for g in range(1, n_groups):
        target = total * g // n_groups
        t = int(np.searchsorted(off, target, side="left"))
        t = min(max(t, cuts[-1] + 1), n_t)
        if t < n_t and t > cuts[-1]:
            cuts.append(t)
    cuts.append(n_t)
    groups, c0 = [], 0
    for t0, t1 in zip(cuts[:-1], cuts[1:]):
        if t1 <= t0:
            continue
        sub = (off[t0:t1 + 1] - off[t0]).astype(np.uint64)
        sub_cols = None if cols is None else np.asarray(cols, dtype=np.uint64)[t0:t1]
        nc = api.sl_num_chunks(api.Layout(sub, sub_cols), chunk)
        groups.append(TensorGroup(t0, t1, int(off[t0]), int(off[t1]), c0, c0 + nc, sub, sub_cols))
        c0 += nc
    return groups


def group_slices(g: TensorGroup, k: int, codes_stride: int, idx, codes, scales):
    """The part of one replica's message arrays that belongs to group g (views, no copy)."""
    return (idx[g.c0 * k:g.c1 * k], codes[g.c0 * codes_stride:g.c1 * codes_stride], scales[g.c0:g.c1])


def outer_step_replica_pipelined(theta_local, theta_global, err, groups: Sequence[TensorGroup], beta: float,
                                 chunk: int, k: int, bits: int, outer_lr: float, idx, codes, scales,
                                 flags=None, group=None, comm_stream=None):
    """The same step as outer_step_replica with the gather of group g overlapped with the
    compression of group g+1.  Compression and the final aggregate-and-apply run on the current
    stream, the gathers on `comm_stream` (created if not given)."""
    from . import api
    st = api.sl_codes_stride(k, bits)
    cur = torch.cuda.current_stream()
    comm = comm_stream or torch.cuda.Stream()
    gathered = []
    for g in groups:
        lay = api.Layout(g.offsets, g.cols)
        gi, gc, gs = group_slices(g, k, st, idx, codes, scales)
        api.sl_compress(theta_local[g.e0:g.e1], theta_global[g.e0:g.e1], err[g.e0:g.e1], lay, beta, chunk, k, bits,
                        gi, gc, gs, flags, cur)
        ready = torch.cuda.Event()
        ready.record(cur)
        with torch.cuda.stream(comm):
            comm.wait_event(ready)
            out = all_gather_messages(gi, gc, gs, group)
            done = torch.cuda.Event()
            done.record(comm)
        gathered.append((g, lay, out, done))
    for g, lay, (a_idx, a_codes, a_scales), done in gathered:
        cur.wait_event(done)
        api.sl_aggregate_apply(a_idx, a_codes, a_scales, lay, chunk, k, bits, theta_global[g.e0:g.e1], outer_lr,
                               flags, cur)
    return gathered


def _align(n: int, a: int = 256) -> int:
    return (n + a - 1) // a * a


class PeerMessages:
    """One replica's message buffers in symmetric memory, with views of every peer's copy.

    The three arrays of a message sit in one flat buffer (256-byte aligned sections) that
    `torch.distributed._symmetric_memory` maps into every rank of `group` (one node: NVLink peer
    mappings).  idx[r] / codes[r] / scales[r] are views of rank r's buffer; this rank writes only
    its own (index `rank`) and reads all of them after `barrier()`."""

    def __init__(self, layout, chunk: int, k: int, bits: int, group=None, device=None):
        import torch.distributed._symmetric_memory as symm
        from . import api
        group = group or dist.group.WORLD
        device = device or torch.device("cuda", torch.cuda.current_device())
        nc = api.sl_num_chunks(layout, chunk)
        st = api.sl_codes_stride(k, bits)
        self.sections = self.plan(nc, k, st)
        total = self.sections[-1][1]
        self.buf = symm.empty(total, dtype=torch.uint8, device=device)
        self.handle = symm.rendezvous(self.buf, group)
        self.rank, self.world = self.handle.rank, self.handle.world_size
        self.idx, self.codes, self.scales = [], [], []
        for r in range(self.world):
            b = self.buf if r == self.rank else self.handle.get_buffer(r, (total,), torch.uint8)
            (i0, i1), (c0, c1), (s0, s1) = self.sections
            self.idx.append(b[i0:i0 + nc * k * 2].view(torch.uint16))
            self.codes.append(b[c0:c0 + nc * st])
            self.scales.append(b[s0:s0 + nc * 4].view(torch.float32))

    @staticmethod
    def plan(n_chunks: int, k: int, codes_stride: int):
        """Byte ranges (start, end) of idx, codes, scales in the flat buffer (host logic only)."""
        i1 = _align(n_chunks * k * 2)
        c1 = i1 + _align(n_chunks * codes_stride)
        s1 = c1 + _align(n_chunks * 4)
        return (0, i1), (i1, c1), (c1, s1)

    def barrier(self) -> None:
        """All ranks' work enqueued so far on their current streams is complete and visible."""
        self.handle.barrier()


def outer_step_replica_peer(theta_local, theta_global, err, layout, beta: float, chunk: int, k: int, bits: int,
                            outer_lr: float, pm: PeerMessages, flags=None):
    """One outer step of the replica this rank hosts, with the exchange folded into the averaging
    kernel: compress into this rank's symmetric buffer, barrier, aggregate-and-apply reading every
    rank's message in place through its peer mapping (rank order, so all ranks end bit-identical),
    barrier again so that nobody overwrites a message a peer may still be reading."""
    from . import api
    r = pm.rank
    api.sl_compress(theta_local, theta_global, err, layout, beta, chunk, k, bits, pm.idx[r], pm.codes[r],
                    pm.scales[r], flags)
    pm.barrier()
    api.sl_aggregate_apply(pm.idx, pm.codes, pm.scales, layout, chunk, k, bits, theta_global, outer_lr, flags)
    pm.barrier()
