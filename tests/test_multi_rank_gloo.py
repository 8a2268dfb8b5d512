"""The N > 1 host logic of bench.py on CPU: two gloo ranks, no GPU.

The path has no exchange step (ranks run independent parameter sets), so what N > 1 adds is
plumbing: rendezvous, per-rank seeds, barrier, max-over-ranks timing, whole-job throughput, and
the reference arm printing from rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import bench
    r, l, w = bench.init_dist("gloo")
    assert (r, w) == (rank, world)
    bench.barrier(w)
    local_ms = 10.0 + 5.0 * rank           # rank 1 is the slow one
    worst = bench.max_over_ranks(local_ms, w)
    seed = bench.rank_seed(0, rank)
    out.put((rank, worst, seed, bench.job_value(1000, w, worst)))
    bench.barrier(w)


def test_two_ranks_max_timing_and_seeds():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]            # both ranks see the slowest rank's time
    assert res[0][2] != res[1][2]                         # independent parameter sets
    assert res[0][3] == 2 * 1000 / 15e-3                  # whole-job units over the slowest time


def test_reference_arm_prints_once_under_two_ranks():
    port = _free_port()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--workload", "tiny", "--gpus", "2", "--steps", "1", "--warmup", "0"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0


def _exchange_worker(rank, world, port, out):
    """Each rank hosts one replica: its message is made by the CPU checker, exchanged with the
    package's gather, and averaged by the checker on every rank."""
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import numpy as np
    import torch
    import torch.distributed as dist
    from oracle import slo
    from paper_2601_02360_b200 import exchange, synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = synth.workload("tiny").replace(R=world)
    off = wl.offsets()
    tg = synth.gen_theta_global(wl).numpy().copy()
    tl = synth.gen_theta_local(wl, torch.from_numpy(tg), 0, rank).numpy()
    err = np.zeros(wl.n_total, np.float32)
    i, c, s, _ = slo.compress(tl, tg, err, off, wl.beta, wl.chunk, wl.k, wl.bits)
    gi, gc, gs = exchange.all_gather_messages(torch.from_numpy(i), torch.from_numpy(c), torch.from_numpy(s))
    msgs = [(a.numpy(), b.numpy(), d.numpy()) for a, b, d in zip(gi, gc, gs)]
    upd = slo.aggregate(msgs, off, wl.chunk, wl.k, wl.bits)
    slo.outer_apply(tg, upd, wl.outer_lr)
    sent = exchange.message_bytes(torch.from_numpy(i), torch.from_numpy(c), torch.from_numpy(s))
    out.put((rank, tg.tobytes(), sent))
    dist.barrier()


def test_replica_per_rank_exchange_gives_every_rank_the_single_process_result():
    import numpy as np
    import torch
    from oracle import slo
    from paper_2601_02360_b200 import synth
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_exchange_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # the same step in one process
    wl = synth.workload("tiny").replace(R=2)
    tg = synth.gen_theta_global(wl).numpy().copy()
    tls = [synth.gen_theta_local(wl, torch.from_numpy(tg), 0, r).numpy() for r in range(2)]
    errs = [np.zeros(wl.n_total, np.float32) for _ in range(2)]
    slo.outer_round(tls, tg, errs, wl.offsets(), wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr)
    assert res[0][1] == res[1][1] == tg.tobytes()
    assert res[0][2] == wl.n_chunks() * (2 * wl.k + wl.k * wl.bits // 8 + 4)


def test_group_plan_covers_the_arena_without_splitting_tensors():
    import numpy as np
    from paper_2601_02360_b200 import api, exchange, synth
    wl = synth.sub_arena(synth.workload("180m"), list(range(12)))
    off = wl.offsets()
    whole = api.sl_num_chunks(api.Layout(off), wl.chunk)
    for n in (1, 2, 3, 7, 12, 40):
        gs = exchange.plan_groups(off, wl.chunk, n)
        assert 1 <= len(gs) <= min(n, len(off) - 1)
        assert gs[0].t0 == 0 and gs[0].e0 == 0 and gs[0].c0 == 0
        assert gs[-1].t1 == len(off) - 1 and gs[-1].e1 == int(off[-1]) and gs[-1].c1 == whole
        for a, b in zip(gs, gs[1:]):
            assert a.t1 == b.t0 and a.e1 == b.e0 and a.c1 == b.c0
        for g in gs:
            assert g.t1 > g.t0 and int(g.offsets[0]) == 0 and int(g.offsets[-1]) == g.e1 - g.e0
            assert np.array_equal(g.offsets, off[g.t0:g.t1 + 1] - off[g.t0])
    # tiles: the per-tensor chunk counts come from the library's own geometry
    cols = [c if r > 1 else 0 for _, r, c in wl.tensors]
    gs = exchange.plan_groups(off, wl.chunk, 3, cols)
    assert gs[-1].c1 == api.sl_num_chunks(api.Layout(off, cols), wl.chunk)


def _group_exchange_worker(rank, world, port, out):
    """Gathering the message group by group (the slices the pipelined step exchanges) must give
    every rank the same arrays as gathering it whole."""
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import numpy as np
    import torch
    import torch.distributed as dist
    from oracle import slo
    from paper_2601_02360_b200 import api, exchange, synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = synth.sub_arena(synth.workload("180m"), [0, 7, 8, 9]).replace(R=world)
    off = wl.offsets()
    tg = synth.gen_theta_global(wl).numpy().copy()
    tl = synth.gen_theta_local(wl, torch.from_numpy(tg), 0, rank).numpy()
    err = np.zeros(wl.n_total, np.float32)
    i, c, s, _ = slo.compress(tl, tg, err, off, wl.beta, wl.chunk, wl.k, wl.bits)
    ti, tc, ts = torch.from_numpy(i).reshape(-1), torch.from_numpy(c).reshape(-1), torch.from_numpy(s)
    whole = exchange.all_gather_messages(ti, tc, ts)
    st = api.sl_codes_stride(wl.k, wl.bits)
    parts = [exchange.all_gather_messages(*exchange.group_slices(g, wl.k, st, ti, tc, ts))
             for g in exchange.plan_groups(off, wl.chunk, 3)]
    ok = len(parts) >= 2
    for r in range(world):
        for a in range(3):
            ok = ok and torch.equal(torch.cat([p[a][r] for p in parts]), whole[a][r])
    out.put((rank, bool(ok)))
    dist.barrier()


def test_group_by_group_gather_equals_the_whole_gather():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_group_exchange_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == [(0, True), (1, True)]


def test_peer_message_buffer_plan():
    # the flat symmetric buffer: three aligned, non-overlapping sections that hold the three arrays
    from paper_2601_02360_b200 import api, exchange, synth
    wl = synth.workload("tiny")
    nc = api.sl_num_chunks(api.Layout(wl.offsets()), wl.chunk)
    for k, bits in ((64, 2), (5, 4), (32, 32), (1, 8)):
        st = api.sl_codes_stride(k, bits)
        (i0, i1), (c0, c1), (s0, s1) = exchange.PeerMessages.plan(nc, k, st)
        assert i0 == 0 and c0 == i1 and s0 == c1
        assert i1 - i0 >= nc * k * 2 and c1 - c0 >= nc * st and s1 - s0 >= nc * 4
        assert all(x % 256 == 0 for x in (i0, c0, s0, s1))      # 16-byte alignment of every array and more
