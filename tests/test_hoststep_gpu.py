"""hoststep.outer_step_from_host: the outer step for replicas whose parameters sit in pinned host memory,
tensor group by tensor group with the copies and the kernels overlapped.  Same bits as the checker's
one-shot step, over two rounds carrying the error buffers; the host receives the messages and the new
theta_global."""
import numpy as np
import pytest
import torch

from oracle import slo
from paper_2601_02360_b200 import api, hoststep, synth
from parity_util import GpuStep, assert_close, assert_exact

pytestmark = pytest.mark.gpu
f32 = np.float32


@pytest.mark.parametrize("n_groups,tiles", [(1, False), (4, False), (9, False), (3, True)])
def test_host_step_matches_the_checker(n_groups, tiles):
    wl = synth.sub_arena(synth.workload("180m"), list(range(10))).replace(R=3)
    off = wl.offsets()
    cols = [c if r > 1 else 0 for _, r, c in wl.tensors] if tiles else None
    groups = hoststep.plan_groups(off, wl.chunk, n_groups, cols)
    assert 1 <= len(groups) <= n_groups and groups[0].e0 == 0 and groups[-1].e1 == wl.n_total
    gs = GpuStep(off, wl.R, wl.chunk, wl.k, wl.bits, cols=cols)
    tgt = synth.gen_theta_global(wl)
    gs.theta_global.copy_(tgt)
    want = tgt.numpy().copy()
    h_err = [np.zeros(wl.n_total, f32) for _ in range(wl.R)]
    host_tl = [torch.empty(wl.n_total, dtype=torch.float32).pin_memory() for _ in range(wl.R)]
    host_tg = torch.zeros(wl.n_total, dtype=torch.float32).pin_memory()
    host_msgs = [[torch.zeros(t.shape, dtype=t.dtype).pin_memory() for t in grp] for grp in (gs.idx, gs.codes, gs.scales)]
    streams = hoststep.HostStepStreams()
    for rnd in range(2):
        tls = [synth.gen_theta_local(wl, torch.from_numpy(want), rnd, r) for r in range(wl.R)]
        for r in range(wl.R):
            host_tl[r].copy_(tls[r])
        hoststep.outer_step_from_host(host_tl, gs.theta_local, gs.theta_global, gs.err, groups, wl.beta, wl.chunk, wl.k,
                                      wl.bits, wl.outer_lr, gs.idx, gs.codes, gs.scales, host_tg, host_msgs, gs.flags,
                                      streams)
        torch.cuda.synchronize()
        msgs, _, _ = slo.outer_round([t.numpy() for t in tls], want, h_err, off, wl.beta, wl.chunk, wl.k, wl.bits,
                                     wl.outer_lr, cols)
        nc = gs.nc
        for r in range(wl.R):
            assert_exact(host_msgs[0][r].numpy().reshape(nc, wl.k), msgs[r][0], f"round {rnd} idx[{r}] on the host")
            assert_exact(host_msgs[1][r].numpy().reshape(nc, -1), msgs[r][1], f"round {rnd} codes[{r}] on the host")
            assert_close(host_msgs[2][r].numpy(), msgs[r][2], f"round {rnd} scales[{r}] on the host")
            assert_close(gs.err[r].cpu().numpy(), h_err[r], f"round {rnd} err[{r}]")
        assert_close(host_tg.numpy(), want, f"round {rnd} theta_global on the host")
        assert_close(gs.theta_global.cpu().numpy(), want, f"round {rnd} theta_global on the device")
    assert int(gs.flags.item()) == 0
