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
