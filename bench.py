#!/usr/bin/env python
"""Benchmark of the SparseLoCo outer step (paper §2.1, Eq. 2) on B200.

A step = one whole outer round (all of Eq. 2) over one synthetic parameter set for R replicas
resident on the device: sl_compress_batch (lines 1-4), then sl_aggregate_apply (line 5) on the
messages it wrote.  (sl_outer_step is the same two launches behind one call; the bench issues
them separately so that an event between them gives the dominant kernel's own time.)
Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1b|0p5b|180m|tiny]
  python bench.py --impl reference ...     # the CPU checker timed on the host cores

Between steps the replicas' parameters are re-drawn around the new theta_global (untimed);
every step is timed on the device with CUDA events on the launching stream.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time
from concurrent.futures import ThreadPoolExecutor

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2601_02360_b200 import synth

METRIC = "sparseloco_outer_step_params_per_s"
UNIT = "params/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of compress_c4096_kernel on the captured small case
# (51,384,320 parameters x 8 replicas, k = 64, 2-bit codes), per replica-parameter
COMPRESS_DRAM_BYTES_PER_REPLICA_PARAM = 12.43
MIN_ROW_SECONDS = 1.0          # a row of short launches runs at least this long, so that nvidia-smi (100 ms period) samples it
E2E_GROUPS = 24               # tensor groups of the host-buffer step (hoststep.outer_step_from_host)
KERNEL_LAUNCHES_PER_STEP = 4   # compress (full chunks, tails) + aggregate-apply (full chunks, tails)


# --------------------------------------------------------------------------- byte counts
def message_bytes(wl: synth.Workload) -> int:
    """Bytes of ONE replica's message: idx u16[k] + packed codes + one float scale per chunk."""
    stride = 4 * wl.k if wl.bits == 32 else (wl.k * wl.bits + 7) // 8
    return wl.n_chunks() * (2 * wl.k + stride + 4)


def compress_bytes(wl: synth.Workload) -> int:
    """Algorithmic bytes of one sl_compress_batch launch: per replica theta_local read, e read,
    e written (12 B/element); theta_global read once for all replicas; messages written."""
    return wl.n_total * (12 * wl.R + 4) + wl.R * message_bytes(wl)


def aggregate_apply_bytes(wl: synth.Workload) -> int:
    """theta_global read and written once, every message read once."""
    return wl.n_total * 8 + wl.R * message_bytes(wl)


def step_bytes_api(wl: synth.Workload) -> int:
    """Per-call count: N(16R + 8), every replica's compress reading theta_global itself, plus the messages."""
    return wl.n_total * (16 * wl.R + 8) + 2 * wl.R * message_bytes(wl)


def step_bytes_strict(wl: synth.Workload) -> int:
    """Least traffic of a whole step: N(12R + 8) + messages written once and read once."""
    return wl.n_total * (12 * wl.R + 8) + 2 * wl.R * message_bytes(wl)


# --------------------------------------------------------------------------- distributed plumbing
def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), \
        int(os.environ.get("WORLD_SIZE", "1"))


def init_dist(backend: str):
    import torch.distributed as dist
    rank, local, world = dist_env()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local, world


def barrier(world: int) -> None:
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """The slowest rank's time: the job is as slow as its slowest shard."""
    if world <= 1:
        return float(value)
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank owns an independent shard of the job (no exchange between shards): its own
    parameter set drawn from its own seed."""
    return base_seed + 1000003 * rank


def job_value(params_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput: parameters all ranks pushed through one outer step per second."""
    return params_per_rank * world / (ms_per_step * 1e-3)


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.path = tempfile.mktemp(prefix="sl_clocks_", suffix=".csv")
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 7:
                    continue
                try:
                    sm.append(float(f[0]))
                    smax.append(float(f[1]))
                except ValueError:
                    continue
                for nm, v in zip(names, f[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            os.unlink(self.path)
        except OSError:
            pass
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(smax)) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def measured_peak_gbs():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


# --------------------------------------------------------------------------- the CPU checker, timed
def cpu_sample_workload(wl: synth.Workload) -> synth.Workload:
    """Bounded sample of the workload for the CPU timing: the first transformer layer (its
    seven matrices and two norm vectors) when the set has one, else the whole set."""
    if len(wl.tensors) > 9:
        return synth.sub_arena(wl, list(range(9)), wl.name + "_layer0")
    return wl


def oracle_round(slo, tls, tg, errs, off, wl, threads):
    """One outer step on the CPU checker as it stands; replicas spread over host threads."""
    def one(r):
        return slo.compress(tls[r], tg, errs[r], off, wl.beta, wl.chunk, wl.k, wl.bits)
    with ThreadPoolExecutor(max_workers=threads) as ex:
        res = list(ex.map(one, range(len(tls))))
    upd = slo.aggregate([(i, c, s) for i, c, s, _ in res], off, wl.chunk, wl.k, wl.bits)
    slo.outer_apply(tg, upd, wl.outer_lr)


def time_oracle(wl_sample: synth.Workload, steps: int, warmup: int, seed: int, inputs=None):
    """Times `steps` outer steps of the CPU checker on the sample.  Returns (ms list, threads)."""
    from oracle import slo
    slo.build()
    cores = os.cpu_count() or 1
    threads = max(1, min(cores, wl_sample.R))
    off = wl_sample.offsets()
    if inputs is None:
        tg_t = synth.gen_theta_global(wl_sample, "cpu", seed)
        rho = synth.row_scales(wl_sample, seed)
        tg = tg_t.numpy().copy()
    else:
        tg = inputs[0].copy()
    errs = [np.zeros(wl_sample.n_total, np.float32) for _ in range(wl_sample.R)]
    times = []
    for t in range(warmup + steps):
        if inputs is None:
            tls = [synth.gen_theta_local(wl_sample, torch.from_numpy(tg), t, r, seed, rho=rho).numpy()
                   for r in range(wl_sample.R)]
        else:
            tls = inputs[1]
        t0 = time.perf_counter()
        oracle_round(slo, tls, tg, errs, off, wl_sample, threads)
        dt = (time.perf_counter() - t0) * 1e3
        if t >= warmup:
            times.append(dt)
    return times, threads


def run_reference_embed(args) -> None:
    """--impl reference --embed: the float64 numpy checker of Eqs. 3-4 on a bounded sample of the rows."""
    from oracle import embed as oe
    wl = synth.workload(args.workload)
    name, V, d = next(t for t in wl.tensors if t[0].startswith("embed"))
    k = args.k or d // 8
    rows = min(V, 4000)
    U = synth.gen_subspace_basis(d, k, args.seed)
    T_S, T_perp = synth.gen_embedding_pair(rows, d, args.seed)
    times = []
    for s in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        oe.embed_reproject(T_S, T_perp, U)
        if s >= args.warmup:
            times.append(time.perf_counter() - t0)
    sec = float(np.mean(times))
    desc = f"{rows} rows of a {V}x{d} table, k={k}, float64 numpy"
    print(json.dumps({
        "impl": "reference", "metric": "embed_reproject_rows_per_s", "value": rows / sec, "unit": "rows/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{wl.name} token embedding {V}x{d}, k={k}", "sample": desc},
        "cpu_baseline": {"value": rows / sec, "unit": "rows/s", "cores": os.cpu_count(), "kind": "oracle", "sample": desc},
        "e2e": {"value": rows / sec, "unit": "rows/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def run_reference_subspace(args) -> None:
    """--impl reference --subspace: the float64 numpy checker of section 2.3 on a bounded sample of the tokens."""
    from oracle import subspace as osub
    wl = synth.workload(args.workload)
    name, V, d = next(t for t in wl.tensors if t[0].startswith("embed"))
    k = args.k or d // 8
    L, rows = 2048, min(args.tokens, 2048)
    U = synth.gen_subspace_basis(d, k, args.seed)
    X, ids, T_perp, pos = synth.gen_stage_boundary(rows, L, V, d, args.seed)
    times = []
    for s in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        xt = osub.project(X, ids, T_perp, pos, U, L)
        osub.reconstruct(xt, ids, T_perp, pos, U, L)
        if s >= args.warmup:
            times.append(time.perf_counter() - t0)
    sec = float(np.mean(times))
    desc = f"{rows} tokens x d={d}, k={k}, float64 numpy, both directions"
    print(json.dumps({
        "impl": "reference", "metric": "subspace_roundtrip_tokens_per_s", "value": rows / sec, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{wl.name} stage boundary: {args.tokens} tokens x d={d}, k={k}, L={L}, vocab {V}",
                   "sample": desc},
        "cpu_baseline": {"value": rows / sec, "unit": "tokens/s", "cores": os.cpu_count(), "kind": "oracle", "sample": desc},
        "e2e": {"value": rows / sec, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def run_reference(args) -> None:
    rank, _, world = dist_env()
    if rank != 0:
        return
    if args.embed:
        return run_reference_embed(args)
    if args.subspace:
        return run_reference_subspace(args)
    wl = synth.workload(args.workload)
    sample = cpu_sample_workload(wl)
    times, threads = time_oracle(sample, args.steps, args.warmup, args.seed)
    ms = float(np.mean(times))
    value = sample.n_total / (ms * 1e-3)
    desc = (f"{sample.name}: {len(sample.tensors)} tensors, {sample.n_total} params x R={sample.R}, "
            f"one outer step per timed step")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "R": wl.R, "k": wl.k, "bits": wl.bits, "chunk": wl.chunk,
                   "beta": wl.beta, "outer_lr": wl.outer_lr, "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- the CUDA path, timed
class DeviceState:
    def __init__(self, wl: synth.Workload, seed: int, device, tiles: bool = False, bf16: bool = False):
        from paper_2601_02360_b200 import api
        self.api = api
        self.wl = wl
        self.seed = seed
        self.dev = device
        # --tiles: matrices are cut into sqrt(chunk) x sqrt(chunk) tiles (the paper's literal 64 x 64
        # chunks); vectors keep consecutive chunks
        cols = [c if r > 1 else 0 for _, r, c in wl.tensors] if tiles else None
        self.layout = api.Layout(wl.offsets(), cols)
        self.n_chunks = api.sl_num_chunks(self.layout, wl.chunk)
        n = wl.n_total
        self.bf16 = bf16          # parameters stored as bfloat16 (error buffers stay float32)
        self.theta_global = synth.gen_theta_global(wl, device, seed)
        self.rho = synth.row_scales(wl, seed)
        th_dtype = torch.bfloat16 if bf16 else torch.float32
        if bf16:
            self.theta_global = self.theta_global.to(torch.bfloat16)
            self._tmp = torch.empty(n, dtype=torch.float32, device=device)     # a replica is drawn in float32, then rounded
        self.theta_local = [torch.empty(n, dtype=th_dtype, device=device) for _ in range(wl.R)]
        self.err = [torch.zeros(n, dtype=torch.float32, device=device) for _ in range(wl.R)]
        self.idx, self.codes, self.scales = api.alloc_messages(self.layout, wl.chunk, wl.k, wl.bits,
                                                               wl.R, device)
        self.flags = torch.zeros(1, dtype=torch.int32, device=device)

    def redraw_locals(self, rnd: int) -> None:
        if self.bf16:
            tg32 = self.theta_global.float()
            for r in range(self.wl.R):
                synth.gen_theta_local(self.wl, tg32, rnd, r, self.seed, out=self._tmp, rho=self.rho)
                self.theta_local[r].copy_(self._tmp)
            return
        for r in range(self.wl.R):
            synth.gen_theta_local(self.wl, self.theta_global, rnd, r, self.seed,
                                  out=self.theta_local[r], rho=self.rho)

    def compress(self) -> None:
        w = self.wl
        if self.bf16:
            self.api.sl_compress_batch_bf16(self.theta_local, self.theta_global, self.err, self.layout, w.beta,
                                            w.chunk, w.k, w.bits, self.idx, self.codes, self.scales, self.flags)
            return
        self.api.sl_compress_batch(self.theta_local, self.theta_global, self.err, self.layout, w.beta,
                                   w.chunk, w.k, w.bits, self.idx, self.codes, self.scales, self.flags)

    def outer_step(self) -> None:
        w = self.wl
        self.api.sl_outer_step(self.theta_local, self.theta_global, self.err, self.layout, w.beta, w.chunk,
                               w.k, w.bits, w.outer_lr, self.idx, self.codes, self.scales, self.flags)

    def aggregate_apply(self) -> None:
        w = self.wl
        if self.bf16:
            self.api.sl_aggregate_apply_bf16(self.idx, self.codes, self.scales, self.layout, w.chunk, w.k, w.bits,
                                             self.theta_global, w.outer_lr, self.flags)
            return
        self.api.sl_aggregate_apply(self.idx, self.codes, self.scales, self.layout, w.chunk, w.k, w.bits,
                                    self.theta_global, w.outer_lr, self.flags)


def host_memory_available() -> int:
    try:
        import psutil
        avail = psutil.virtual_memory().available
    except Exception:
        avail = 8 << 30
    for p in ("/sys/fs/cgroup/memory.max", "/sys/fs/cgroup/memory/memory.limit_in_bytes"):
        try:
            v = open(p).read().strip()
            if v.isdigit():
                used = 0
                try:
                    used = int(open(os.path.join(os.path.dirname(p), "memory.current")).read())
                except Exception:
                    pass
                avail = min(avail, int(v) - used)
        except OSError:
            pass
    return avail


def run_e2e(st: DeviceState, steps: int, world: int):
    """The same step with HOST inputs and outputs through the package's host-buffer call
    (hoststep.outer_step_from_host): every step copies the replicas' parameters from pinned host memory to
    the device, runs Eq. 2, and reads the messages and the new theta_global back, group of tensors by group
    of tensors so that the copies in, the kernels and the copies out overlap.  Returns (ms per step, h2d
    bytes, d2h bytes, note)."""
    wl = st.wl
    n = wl.n_total
    need = n * 4
    budget = int(host_memory_available() * 0.5 / max(1, world))   # the ranks of a node share its memory
    pool = max(1, min(wl.R, budget // need - 1))
    host_tl = [torch.empty(n, dtype=torch.float32).pin_memory() for _ in range(pool)]
    for p in range(pool):
        host_tl[p].copy_(st.theta_local[p])
    host_tg = torch.empty(n, dtype=torch.float32).pin_memory()
    host_msgs = [[torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in grp]
                 for grp in (st.idx, st.codes, st.scales)]
    torch.cuda.synchronize()
    h2d = wl.R * n * 4
    d2h = n * 4 + sum(t.numel() * t.element_size() for grp in host_msgs for t in grp)
    from paper_2601_02360_b200 import hoststep
    cols = None if st.layout.cols is None else st.layout.cols
    groups = hoststep.plan_groups(wl.offsets(), wl.chunk, E2E_GROUPS, cols)
    streams = hoststep.HostStepStreams(st.dev)
    host_list = [host_tl[r % pool] for r in range(wl.R)]
    times = []
    for s in range(steps + 1):
        barrier(world)
        torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        hoststep.outer_step_from_host(host_list, st.theta_local, st.theta_global, st.err, groups, wl.beta, wl.chunk,
                                      wl.k, wl.bits, wl.outer_lr, st.idx, st.codes, st.scales, host_tg, host_msgs,
                                      st.flags, streams)
        e1.record()
        torch.cuda.synchronize()
        if s > 0:   # the first pass warms the pinned pages and the copy engines
            times.append(e0.elapsed_time(e1))
    note = (f"hoststep.outer_step_from_host over {len(groups)} tensor groups (copies in, kernels and copies out overlap); "
            f"pinned pool of {pool} distinct replica buffers" + ("" if pool == wl.R else f" reused for R={wl.R}"))
    del host_tl, host_tg, host_msgs
    return float(np.mean(times)), h2d, d2h, note


def run_exchange(args) -> None:
    """Replica-per-GPU form (the paper's deployment): every rank hosts ONE replica of the same
    parameter set; a step = sl_compress of the own replica, NCCL all-gather of the sparse
    messages, sl_aggregate_apply on the own copy of theta_global.  R = number of ranks."""
    import torch.distributed as dist
    from paper_2601_02360_b200 import api, exchange
    rank, local, world = dist_env()
    assert world == args.gpus, f"--gpus {args.gpus} but WORLD_SIZE={world}: launch with torchrun"
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29500")
    if not dist.is_initialized():
        dist.init_process_group(backend="nccl", rank=rank, world_size=world, device_id=dev)
    wl = synth.workload(args.workload).replace(R=world)
    if args.k:
        wl = wl.replace(k=args.k)
    if args.bits:
        wl = wl.replace(bits=args.bits)
    if args.first_tensors:
        wl = synth.sub_arena(wl, list(range(args.first_tensors)), f"{wl.name}[:{args.first_tensors}]")
    lay = api.Layout(wl.offsets())
    theta_global = synth.gen_theta_global(wl, dev, args.seed)          # the same on every rank
    rho = synth.row_scales(wl, args.seed)
    theta_local = torch.empty_like(theta_global)
    err = torch.zeros_like(theta_global)
    idx, codes, scales = api.alloc_messages(lay, wl.chunk, wl.k, wl.bits, 1, dev)
    flags = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    groups = exchange.plan_groups(wl.offsets(), wl.chunk, args.groups) if args.groups > 1 else None
    comm = torch.cuda.Stream() if groups else None
    pm = exchange.PeerMessages(lay, wl.chunk, wl.k, wl.bits) if args.peer else None
    if pm is not None:
        idx, codes, scales = [pm.idx[rank]], [pm.codes[rank]], [pm.scales[rank]]
    times = []
    for s in range(args.warmup + args.steps):
        synth.gen_theta_local(wl, theta_global, s, rank, args.seed, out=theta_local, rho=rho)
        if s == args.warmup:
            dist.barrier()
            torch.cuda.synchronize()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        if pm is not None:
            exchange.outer_step_replica_peer(theta_local, theta_global, err, lay, wl.beta, wl.chunk, wl.k, wl.bits,
                                             wl.outer_lr, pm, flags)
        elif groups is None:
            exchange.outer_step_replica(theta_local, theta_global, err, lay, wl.beta, wl.chunk, wl.k, wl.bits,
                                        wl.outer_lr, idx[0], codes[0], scales[0], flags, idx12=args.idx12)
        else:
            exchange.outer_step_replica_pipelined(theta_local, theta_global, err, groups, wl.beta, wl.chunk, wl.k,
                                                  wl.bits, wl.outer_lr, idx[0], codes[0], scales[0], flags,
                                                  comm_stream=comm)
        e1.record(stream)
        torch.cuda.synchronize()
        if s >= args.warmup:
            times.append(e0.elapsed_time(e1))
    dist.barrier()
    ms = max_over_ranks(float(np.sum(times)), world, dev) / args.steps
    # every rank must hold the same parameters after the step
    chk = theta_global.double().sum().reshape(1)
    lo, hi = chk.clone(), chk.clone()
    dist.all_reduce(lo, op=dist.ReduceOp.MIN)
    dist.all_reduce(hi, op=dist.ReduceOp.MAX)
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": wl.n_total / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "params": wl.n_total, "R": world, "k": wl.k, "bits": wl.bits,
                       "chunk": wl.chunk,
                       "mode": ("one replica per GPU, messages in symmetric memory, the averaging kernel reads "
                                "the peers' buffers over NVLink (no gather)") if args.peer else
                               "one replica per GPU, NCCL all-gather of the sparse messages",
                       "tensor_groups": len(groups) if groups else 1,
                       "positions": "12 bits on the wire" if args.idx12 else "uint16",
                       "message_bytes_per_replica": exchange.message_bytes(idx[0], codes[0], scales[0])
                       - (idx[0].numel() * 2 - wl.n_chunks() * api.sl_idx12_stride(wl.k) if args.idx12 else 0)},
            "replicas_agree": bool(lo.item() == hi.item()), "device_flags": int(flags.item()),
            "gpu_launches": (4 * len(groups) if groups else 4) * args.steps}))
    dist.destroy_process_group()


def run_subspace(args) -> None:
    """Stage-boundary activation compression (§2.3): sl_subspace_project and sl_subspace_reconstruct on
    one micro-batch of the chosen model (batch 32 x sequence 2048 tokens of the paper's local batch
    would be 64 K tokens; 16 K tokens here keep the buffers small), k = d/8.  One GPU, own JSON line."""
    from paper_2601_02360_b200 import api
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    wl = synth.workload(args.workload)
    name, V, d = next(t for t in wl.tensors if t[0].startswith("embed"))
    k = args.k or d // 8
    L, n_tok = 2048, args.tokens
    Xh, idsh, Tph, posh = synth.gen_stage_boundary(n_tok, L, V, d, args.seed)
    X, ids, T_perp, pos = (torch.from_numpy(a).to(dev) for a in (Xh, idsh, Tph, posh))
    U = torch.from_numpy(synth.gen_subspace_basis(d, k, args.seed)).to(dev)
    api.sl_round_tf32(U, U.numel())
    Xt = torch.empty(n_tok, k, dtype=torch.float32, device=dev)
    Xhat = torch.empty(n_tok, d, dtype=torch.float32, device=dev)
    flags = torch.zeros(1, dtype=torch.int32, device=dev)
    flush = torch.empty(64 << 20, dtype=torch.float32, device=dev)     # 256 MB > L2, written between steps
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(0)
    t_p, t_r = [], []
    for s in range(args.warmup + args.steps):
        if s == args.warmup:
            sampler.start()
        torch.cuda.synchronize()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        flush.fill_(float(s))                 # no synchronize after it: the launch below is queued while this
        flush.fill_(float(s) + 0.5)           # runs, so the host's launch work stays outside the timed interval
        e[0].record(stream)
        api.sl_subspace_project(X, ids, T_perp, pos, U, n_tok, L, V, d, k, Xt, flags)
        e[1].record(stream)
        api.sl_subspace_reconstruct(Xt, ids, T_perp, pos, U, n_tok, L, V, d, k, Xhat, flags)
        e[2].record(stream)
        torch.cuda.synchronize()
        if s >= args.warmup:
            t_p.append(e[0].elapsed_time(e[1]))
            t_r.append(e[1].elapsed_time(e[2]))
    clocks = sampler.stop()
    ms_p, ms_r = float(np.median(t_p)), float(np.median(t_r))     # short kernels: the median is robust to clock ramps
    # the same two launches for activation gradients (no embedding terms), outside the headline figures
    t_gp, t_gr = [], []
    for s in range(min(args.steps, 50) + 3):
        torch.cuda.synchronize()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        flush.fill_(float(s))
        flush.fill_(float(s) + 0.5)
        e[0].record(stream)
        api.sl_subspace_project(X, None, None, None, U, n_tok, L, 0, d, k, Xt, flags)
        e[1].record(stream)
        api.sl_subspace_reconstruct(Xt, None, None, None, U, n_tok, L, 0, d, k, Xhat, flags)
        e[2].record(stream)
        torch.cuda.synchronize()
        if s >= 3:
            t_gp.append(e[0].elapsed_time(e[1]))
            t_gr.append(e[1].elapsed_time(e[2]))
    # compress reads X and one gathered T_perp row per token, writes Xt; Pos and U are L2-resident (counted once)
    bytes_p = n_tok * d * 8 + n_tok * k * 4 + L * d * 4 + d * k * 4
    bytes_r = n_tok * k * 4 + n_tok * d * 8 + L * d * 4 + d * k * 4
    peak, peak_src = measured_peak_gbs()
    ms = ms_p + ms_r
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    line = {
        "metric": "subspace_roundtrip_tokens_per_s", "value": n_tok / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "tf32 contraction, f32 gather terms", "data": "synthetic",
        "config": {"workload": f"{wl.name} stage boundary: {n_tok} tokens x d={d}, k={k}, L={L}, vocab {V}",
                   "l2": "a 256 MB buffer is written between timed steps"},
        "kernels_ms": {"sl_subspace_project": ms_p, "sl_subspace_reconstruct": ms_r,
                       "gradient form (ids = NULL), project": float(np.median(t_gp)),
                       "gradient form (ids = NULL), reconstruct": float(np.median(t_gr))},
        "roofline": {"bound": "hbm", "kernel": "sl_subspace_reconstruct", "achieved": bytes_r / (ms_r * 1e-3) / 1e9,
                     "peak": peak, "unit": "GB/s", "frac": bytes_r / (ms_r * 1e-3) / 1e9 / peak, "traffic": None,
                     "peak_source": peak_src, "algorithmic_bytes": bytes_r,
                     "project": {"achieved": bytes_p / (ms_p * 1e-3) / 1e9, "frac": bytes_p / (ms_p * 1e-3) / 1e9 / peak,
                                 "algorithmic_bytes": bytes_p},
                     "tensor_tflops": 4 * n_tok * d * k / (ms * 1e-3) / 1e12,
                     # what an SM takes in, per SM and second: every 128-token sub-tile streams all of U again
                     # (the figure both launches run into is about 68 GB/s per SM, whatever the path)
                     "sm_intake_gbs": {
                         "project": (3 * n_tok * d * 4 + -(-n_tok // 128) * d * k * 4) / sms / (ms_p * 1e-3) / 1e9,
                         "reconstruct": (2 * n_tok * d * 4 + n_tok * k * 4 + -(-n_tok // 128) * d * k * 4) / sms
                                        / (ms_r * 1e-3) / 1e9}},
        "clocks": clocks, "device_flags": int(flags.item()), "gpu_launches": 2 * args.steps,
    }
    if not args.no_cpu:
        from oracle import subspace as osub
        rows = min(n_tok, 2048)
        Uh = U.cpu().numpy()
        t0 = time.perf_counter()
        xt = osub.project(Xh[:rows], idsh[:rows], Tph, posh, Uh, L)
        osub.reconstruct(xt, idsh[:rows], Tph, posh, Uh, L)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": rows / dt, "unit": "tokens/s", "cores": os.cpu_count(), "kind": "oracle",
                                "sample": f"first {rows} tokens, float64 numpy, both directions"}
    print(json.dumps(line))


def run_embed(args) -> None:
    """The step right after the outer step for replicas that compress activations (§2.4, Eqs. 3-4):
    sl_embed_reproject on the token-embedding table of the chosen model (vocab x d, k = d/8, the
    paper's 87.5 % setting).  One GPU; its own JSON line, not the default bench line."""
    from paper_2601_02360_b200 import api
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    wl = synth.workload(args.workload)
    name, V, d = next(t for t in wl.tensors if t[0].startswith("embed"))
    k = args.k or d // 8
    U = torch.from_numpy(synth.gen_subspace_basis(d, k, args.seed)).to(dev)
    api.sl_round_tf32(U, U.numel())          # once, as the header asks: U never changes
    T_S_h, T_perp_h = synth.gen_embedding_pair(V, d, args.seed)
    T_S0 = torch.from_numpy(T_S_h).to(dev)
    T_S, T_perp = T_S0.clone(), torch.from_numpy(T_perp_h).to(dev)
    flags = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(0)
    times = []
    for s in range(args.warmup + args.steps):
        torch.cuda.synchronize()
        if s == args.warmup:
            sampler.start()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        T_S.copy_(T_S0)                      # a table that has drifted out of the subspace again; no synchronize
        e0.record(stream)                    # after it: the launch is queued while the copy runs (host work untimed)
        api.sl_embed_reproject(T_S, T_perp, U, V, d, k, flags)
        e1.record(stream)
        torch.cuda.synchronize()
        if s >= args.warmup:
            times.append(e0.elapsed_time(e1))
    clocks = sampler.stop()
    ms = float(np.mean(times))
    alg_bytes = 16 * V * d + 4 * d * k      # read T_S and T_perp, write both, read U once
    # DRAM bytes of one launch from the ncu capture of this very case (profiles/): T_S is read twice
    traffic = 1.259e9 if (V, d, k) == (32000, 2048, 256) else None
    flops = 4 * V * d * k
    peak, peak_src = measured_peak_gbs()
    line = {
        "metric": "embed_reproject_rows_per_s", "value": V / (ms * 1e-3), "unit": "rows/s", "n_gpus": 1,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "tf32 contraction, f32 update", "data": "synthetic",
        "config": {"workload": f"{wl.name} token embedding {V}x{d}, k={k}",
                   "l2": "the two tables (2 x %.0f MB) exceed the 126 MB L2" % (V * d * 4 / 1e6)},
        "roofline": {"bound": "hbm", "achieved": alg_bytes / (ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                     "frac": alg_bytes / (ms * 1e-3) / 1e9 / peak, "traffic": traffic, "peak_source": peak_src,
                     "algorithmic_bytes": alg_bytes, "tensor_tflops": flops / (ms * 1e-3) / 1e12},
        "clocks": clocks, "device_flags": int(flags.item()), "gpu_launches": args.steps,
    }
    if not args.no_e2e:
        hs, hp = torch.from_numpy(T_S_h).pin_memory(), torch.from_numpy(T_perp_h).pin_memory()
        t_e2e = []
        for _ in range(max(1, args.e2e_steps)):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            T_S.copy_(hs, non_blocking=True)
            T_perp.copy_(hp, non_blocking=True)
            api.sl_embed_reproject(T_S, T_perp, U, V, d, k, flags)
            hs.copy_(T_S, non_blocking=True)
            hp.copy_(T_perp, non_blocking=True)
            torch.cuda.synchronize()
            t_e2e.append(time.perf_counter() - t0)
        e = float(np.mean(t_e2e))
        line["e2e"] = {"value": V / e, "unit": "rows/s", "ms": e * 1e3, "h2d_bytes_per_step": 8 * V * d,
                       "d2h_bytes_per_step": 8 * V * d}
    if not args.no_cpu:
        from oracle import embed as oe
        rows = min(V, 4000)
        Uh = U.cpu().numpy()
        t0 = time.perf_counter()
        oe.embed_reproject(T_S_h[:rows], T_perp_h[:rows], Uh)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": rows / dt, "unit": "rows/s", "cores": os.cpu_count(), "kind": "oracle",
                                "sample": f"first {rows} rows of the table, float64 numpy"}
    print(json.dumps(line))


# --------------------------------------------------------------------------- the other rows, outside the headline
def _median_row(ms_list, alg_bytes, peak, clocks, extra=None, burst_n=0):
    """ms / frac: median over all timed launches.  burst_n > 0: the row ran for at least MIN_ROW_SECONDS, during
    which a launch-after-launch loop may reach the power cap and lower clocks (see `clocks`); `ms_burst` /
    `frac_burst` are then the median of the first burst_n launches, taken before that happens."""
    ms = float(np.median(ms_list))
    row = {"ms": ms, "launches": len(ms_list), "algorithmic_bytes": int(alg_bytes),
           "achieved_gbs": alg_bytes / (ms * 1e-3) / 1e9, "frac": alg_bytes / (ms * 1e-3) / 1e9 / peak, "clocks": clocks}
    if burst_n and len(ms_list) > burst_n:
        mb = float(np.median(ms_list[:burst_n]))
        row["ms_burst"] = mb
        row["frac_burst"] = alg_bytes / (mb * 1e-3) / 1e9 / peak
    if extra:
        row.update(extra)
    return row


def row_outer_step(wl: synth.Workload, seed: int, dev, peak: float, steps: int, tiles: bool = False,
                   bf16: bool = False) -> dict:
    """One whole outer step (both launches) of another configuration: median of `steps` steps, theta_local
    re-drawn between steps (untimed); frac = strict step bytes / time / peak, like step_hbm.frac_of_peak."""
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info(dev)
    need = (2 * wl.R + 1) * wl.n_total * 4 + (3 << 30)
    if free < need:
        return {"skipped": f"needs {need >> 30} GiB of device memory, {free >> 30} GiB free"}
    st = DeviceState(wl, seed, dev, tiles=tiles, bf16=bf16)
    # bfloat16 parameters: theta_local 2 + e 8 bytes per replica-parameter, theta_global 2 + 2
    strict = step_bytes_strict(wl) - (wl.n_total * (2 * wl.R + 4) if bf16 else 0)
    comp_b = compress_bytes(wl) - (wl.n_total * (2 * wl.R + 2) if bf16 else 0)
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(dev.index or 0)
    t_step, t_comp = [], []
    for s in range(3 + steps):
        st.redraw_locals(s)
        if s == 3:
            torch.cuda.synchronize()
            sampler.start()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        ev[0].record(stream)
        st.compress()
        ev[1].record(stream)
        st.aggregate_apply()
        ev[2].record(stream)
        torch.cuda.synchronize()
        if s >= 3:
            t_step.append(ev[0].elapsed_time(ev[2]))
            t_comp.append(ev[0].elapsed_time(ev[1]))
    clocks = sampler.stop()
    flags = int(st.flags.item())
    comp = float(np.median(t_comp))
    row = _median_row(t_step, strict, peak, clocks,
                      {"R": wl.R, "k": wl.k, "bits": wl.bits, "geometry": "64x64 tiles" if tiles else "consecutive chunks",
                       "parameters": "bfloat16, float32 error buffers" if bf16 else "float32",
                       "params_per_s": wl.n_total / (float(np.median(t_step)) * 1e-3),
                       "compress_ms": comp, "compress_frac": comp_b / (comp * 1e-3) / 1e9 / peak,
                       "device_flags": flags})
    del st
    torch.cuda.empty_cache()
    return row


def row_embed(wl: synth.Workload, seed: int, dev, peak: float, launches: int, k: int) -> dict:
    """sl_embed_reproject on the workload's embedding table (Eqs. 3-4); the launch is queued behind the copy
    that restores T_S, so the host's launch work is outside the timed interval."""
    from paper_2601_02360_b200 import api
    name, V, d = next(t for t in wl.tensors if t[0].startswith("embed"))
    U = torch.from_numpy(synth.gen_subspace_basis(d, k, seed)).to(dev)
    api.sl_round_tf32(U, U.numel())
    T_S_h, T_perp_h = synth.gen_embedding_pair(V, d, seed)
    T_S0 = torch.from_numpy(T_S_h).to(dev)
    T_S, T_perp = T_S0.clone(), torch.from_numpy(T_perp_h).to(dev)
    flags = torch.zeros(1, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(dev.index or 0)
    times = []
    sampler.start()
    t_begin, s = time.perf_counter(), -1
    while s + 1 < 5 + launches or time.perf_counter() - t_begin < MIN_ROW_SECONDS:   # long enough for the clock sampler
        s += 1
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        T_S.copy_(T_S0)
        e0.record(stream)
        api.sl_embed_reproject(T_S, T_perp, U, V, d, k, flags)
        e1.record(stream)
        torch.cuda.synchronize()
        if s >= 5:
            times.append(e0.elapsed_time(e1))
    return _median_row(times, 16 * V * d + 4 * d * k, peak, sampler.stop(),
                       {"shape": f"{V}x{d}, k={k}", "device_flags": int(flags.item())}, burst_n=launches)


def row_subspace(wl: synth.Workload, seed: int, dev, peak: float, launches: int, n_tok: int, k: int) -> dict:
    """sl_subspace_project / sl_subspace_reconstruct at a stage boundary (section 2.3), with the embedding
    terms and in the gradient form (ids = NULL); a 256 MB buffer is written between launches (L2 flush)."""
    from paper_2601_02360_b200 import api
    name, V, d = next(t for t in wl.tensors if t[0].startswith("embed"))
    L = 2048
    Xh, idsh, Tph, posh = synth.gen_stage_boundary(n_tok, L, V, d, seed)
    X, ids, T_perp, pos = (torch.from_numpy(a).to(dev) for a in (Xh, idsh, Tph, posh))
    U = torch.from_numpy(synth.gen_subspace_basis(d, k, seed)).to(dev)
    api.sl_round_tf32(U, U.numel())
    Xt = torch.empty(n_tok, k, dtype=torch.float32, device=dev)
    Xhat = torch.empty(n_tok, d, dtype=torch.float32, device=dev)
    flags = torch.zeros(1, dtype=torch.int32, device=dev)
    flush = torch.empty(64 << 20, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    out = {}
    for form, args in (("with_embedding_terms", (ids, T_perp, pos, V)), ("gradient_form", (None, None, None, 0))):
        sampler = ClockSampler(dev.index or 0)
        t_p, t_r = [], []
        sampler.start()
        t_begin, s = time.perf_counter(), -1
        while s + 1 < 5 + launches or time.perf_counter() - t_begin < MIN_ROW_SECONDS:
            s += 1
            torch.cuda.synchronize()
            e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            flush.fill_(float(s))
            e[0].record(stream)
            api.sl_subspace_project(X, args[0], args[1], args[2], U, n_tok, L, args[3], d, k, Xt, flags)
            e[1].record(stream)
            flush.fill_(float(s) + 0.5)
            e[2].record(stream)
            api.sl_subspace_reconstruct(Xt, args[0], args[1], args[2], U, n_tok, L, args[3], d, k, Xhat, flags)
            e[3].record(stream)
            torch.cuda.synchronize()
            if s >= 5:
                t_p.append(e[0].elapsed_time(e[1]))
                t_r.append(e[2].elapsed_time(e[3]))
        clocks = sampler.stop()
        gather = n_tok * d * 4 + L * d * 4 if args[0] is not None else 0      # one T_perp row per token, the position table once
        bytes_p = n_tok * d * 4 + gather + n_tok * k * 4 + d * k * 4
        bytes_r = n_tok * k * 4 + gather + n_tok * d * 4 + d * k * 4
        out[form] = {"project": _median_row(t_p, bytes_p, peak, clocks, burst_n=launches),
                     "reconstruct": _median_row(t_r, bytes_r, peak, clocks, burst_n=launches)}
    out["shape"] = f"{n_tok} tokens x d={d}, k={k}, L={L}, vocab {V}"
    out["device_flags"] = int(flags.item())
    return out


def measured_rows(args, wl: synth.Workload, dev, peak: float) -> dict:
    """Everything else this library times, appended to the default line (outside its timed region)."""
    n = args.row_launches
    rows = {"note": "medians of CUDA-event times; frac = algorithmic bytes / time / peak"}
    rows["config_180m"] = row_outer_step(synth.workload("180m"), args.seed, dev, peak, n)     # benchmark configuration 2
    rows["config_0p5b"] = row_outer_step(synth.workload("0p5b"), args.seed, dev, peak, n)     # benchmark configuration 3
    rows["tiles"] = row_outer_step(wl, args.seed, dev, peak, n, tiles=True)
    rows["r2"] = row_outer_step(wl.replace(R=2), args.seed, dev, peak, n)
    rows["r16_k128"] = row_outer_step(wl.replace(R=16, k=128), args.seed, dev, peak, n)
    rows["bf16_params"] = row_outer_step(wl, args.seed, dev, peak, n, bf16=True)
    has_embed = any(t[0].startswith("embed") for t in wl.tensors)
    if has_embed:
        d = next(t for t in wl.tensors if t[0].startswith("embed"))[2]
        m = 4 * n                 # these launches take a quarter of a millisecond: more of them, so that the clock sampler sees some
        rows["embed"] = row_embed(wl, args.seed, dev, peak, m, d // 8)
        rows["embed_k128"] = row_embed(wl, args.seed, dev, peak, m, 128)
        rows["subspace"] = row_subspace(wl, args.seed, dev, peak, m, 65536, d // 8)
        rows["subspace_k128"] = row_subspace(wl, args.seed, dev, peak, m, 65536, 128)
    return rows


def run_ours(args) -> None:
    from paper_2601_02360_b200 import api
    rank, local, world = init_dist("nccl")
    assert world == args.gpus, f"--gpus {args.gpus} but WORLD_SIZE={world}: launch with torchrun"
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    api.load()
    wl = synth.workload(args.workload)
    if args.R:
        wl = wl.replace(R=args.R)
    if args.k:
        wl = wl.replace(k=args.k)
    if args.bits:
        wl = wl.replace(bits=args.bits)
    if args.variant != "plain":
        wl = wl.replace(variant=args.variant)
    if args.first_tensors:
        wl = synth.sub_arena(wl, list(range(args.first_tensors)), f"{wl.name}[:{args.first_tensors}]")
    st = DeviceState(wl, rank_seed(args.seed, rank), dev, tiles=args.tiles, bf16=args.bf16)
    stream = torch.cuda.current_stream()

    sampler = ClockSampler(local)
    t_step, t_comp, t_agg = [], [], []
    for s in range(args.warmup + args.steps):
        st.redraw_locals(s)
        if s == args.warmup:
            barrier(world)
            torch.cuda.synchronize()
            if rank == 0:
                sampler.start()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        ev[0].record(stream)
        st.compress()
        ev[1].record(stream)
        st.aggregate_apply()
        ev[2].record(stream)
        torch.cuda.synchronize()
        if s >= args.warmup:
            t_comp.append(ev[0].elapsed_time(ev[1]))
            t_agg.append(ev[1].elapsed_time(ev[2]))
            t_step.append(ev[0].elapsed_time(ev[2]))
    torch.cuda.synchronize()
    barrier(world)
    clocks = sampler.stop() if rank == 0 else None
    total_ms = max_over_ranks(float(np.sum(t_step)), world, dev)
    ms_per_step = total_ms / args.steps
    flags = int(st.flags.item())

    e2e = None
    if not args.no_e2e:
        e_ms, h2d, d2h, note = run_e2e(st, args.e2e_steps, world)
        e_ms = max_over_ranks(e_ms, world, dev)
        e2e = {"value": job_value(wl.n_total, world, e_ms), "unit": UNIT, "ms_per_step": e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps, "note": note}

    if rank != 0:
        return
    peak, peak_src = measured_peak_gbs()
    step_ms = float(np.mean(t_step))
    comp_ms = float(np.mean(t_comp))
    agg_ms = float(np.mean(t_agg))
    # bfloat16 parameters: theta_local 2 instead of 4 bytes per replica-parameter, theta_global 2 + 2 instead of 4 + 4
    comp_bytes = compress_bytes(wl) - (wl.n_total * (2 * wl.R + 2) if args.bf16 else 0)
    strict_bytes = step_bytes_strict(wl) - (wl.n_total * (2 * wl.R + 4) if args.bf16 else 0)
    achieved = comp_bytes / (comp_ms * 1e-3) / 1e9
    strict = strict_bytes / (step_ms * 1e-3) / 1e9
    # ncu DRAM bytes of the tuned compress launch on the small capture (profiles/), per
    # replica-parameter, scaled to this launch's units
    traffic = COMPRESS_DRAM_BYTES_PER_REPLICA_PARAM * wl.n_total * wl.R if wl.chunk == 4096 and not args.bf16 else None
    line = {
        "metric": METRIC, "value": job_value(wl.n_total, world, ms_per_step), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": wl.name, "params": wl.n_total, "tensors": len(wl.tensors),
                   "chunks": wl.n_chunks(), "R": wl.R, "k": wl.k, "bits": wl.bits, "chunk": wl.chunk,
                   "beta": wl.beta, "outer_lr": wl.outer_lr, "variant": wl.variant,
                   "geometry": "64x64 tiles of each matrix" if args.tiles else "consecutive chunks",
                   "parameters": "bfloat16, float32 error buffers" if args.bf16 else "float32",
                   "l2": "inputs (GBs per launch) far larger than the 126 MB L2; no flush needed",
                   "sharding": "none: every rank runs an independent parameter set" if world > 1 else "single GPU",
                   "step": "sl_compress_batch + sl_aggregate_apply; theta_local re-drawn between steps (untimed)"},
        "roofline": {"kernel": "compress_c4096_kernel (sl_compress_batch)", "bound": "hbm",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": traffic,
                     "traffic_source": ("ncu dram__bytes_read.sum + dram__bytes_write.sum of this kernel on the "
                                        "51.4 M-parameter x 8-replica case (profiles/compress_c4096_1b_layer0.md), "
                                        "scaled by N*R; a constant, not re-captured by this run") if traffic else None,
                     "peak_source": peak_src, "algorithmic_bytes": comp_bytes,
                     "launch_ms": comp_ms},
        "step_hbm": {"bytes_strict": strict_bytes, "gbs_strict": strict, "frac_of_peak": strict / peak,
                     "frac_of_8tbs_nominal": strict / 8000.0,
                     # per-call count: every replica's compress re-reads theta_global, as on R separate machines
                     "bytes_api": step_bytes_api(wl), "gbs_api": step_bytes_api(wl) / (step_ms * 1e-3) / 1e9,
                     "frac_api": step_bytes_api(wl) / (step_ms * 1e-3) / 1e9 / peak},
        "kernels_ms": {"sl_compress_batch": comp_ms, "sl_aggregate_apply": agg_ms,
                       "aggregate_apply_gbs": aggregate_apply_bytes(wl) / (agg_ms * 1e-3) / 1e9},
        "clocks": clocks, "device_flags": flags,
        "gpu_launches": KERNEL_LAUNCHES_PER_STEP * args.steps,
    }
    if wl.variant != "plain":
        # how hard the tie-breaking is exercised: chunks of the first tensor whose k-th and (k+1)-th largest
        # pseudo-gradient magnitudes are equal (a fresh draw, error buffers left out)
        st.redraw_locals(10 ** 6)
        n0 = (wl.sizes[0] // wl.chunk) * wl.chunk
        dlt = (st.theta_global[:n0] - st.theta_local[0][:n0]).abs().view(-1, wl.chunk)
        top = torch.topk(dlt, wl.k + 1, dim=1).values
        line["config"]["tie_fraction"] = float((top[:, wl.k - 1] == top[:, wl.k]).float().mean())
        del dlt, top
    if e2e is not None:
        line["e2e"] = e2e
    if not args.no_cpu:
        sample = cpu_sample_workload(wl)
        n_s = sample.n_total
        inputs = (st.theta_global[:n_s].cpu().numpy(), [t[:n_s].cpu().numpy() for t in st.theta_local])
        times, threads = time_oracle(sample, 1, 0, args.seed, inputs=inputs)
        cpu_ms = float(np.mean(times))
        line["cpu_baseline"] = {
            "value": n_s / (cpu_ms * 1e-3), "unit": UNIT, "cores": threads, "kind": "oracle",
            "ms": cpu_ms,
            "sample": f"first {len(sample.tensors)} tensors of the workload ({n_s} params) x R={wl.R}, "
                      f"one outer step, replicas spread over {threads} host threads"}
        # the same checker on ONE host thread, on a smaller sample (the first two tensors)
        if len(wl.tensors) > 2:
            s1 = synth.sub_arena(wl, [0, 1], wl.name + "_first2")
            n1 = s1.n_total
            from oracle import slo
            tg1 = st.theta_global[:n1].cpu().numpy()
            tl1 = [t[:n1].cpu().numpy() for t in st.theta_local]
            e1 = [np.zeros(n1, np.float32) for _ in range(wl.R)]
            t0 = time.perf_counter()
            oracle_round(slo, tl1, tg1, e1, s1.offsets(), s1, 1)
            dt = time.perf_counter() - t0
            line["cpu_baseline_1core"] = {"value": n1 / dt, "unit": UNIT, "cores": 1, "kind": "oracle", "ms": dt * 1e3,
                                          "sample": f"first 2 tensors ({n1} params) x R={wl.R}, one outer step, one host thread"}
    plain_default = not (args.bf16 or args.tiles or args.R or args.k or args.bits or args.first_tensors or args.variant != "plain")
    if world == 1 and not args.no_rows and wl.name == "1b" and plain_default:
        del st
        line["rows"] = measured_rows(args, wl, dev, peak)
    print(json.dumps(line))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="1b", choices=["tiny", "180m", "0p5b", "1b"])
    ap.add_argument("--R", type=int, default=0)
    ap.add_argument("--k", type=int, default=0)
    ap.add_argument("--bits", type=int, default=0, choices=[0, 2, 4, 8, 32],
                    help="bits per kept value (32 = no quantisation, the paper's own runs)")
    ap.add_argument("--first-tensors", type=int, default=0,
                    help="keep only the first N tensors of the workload (small cases for profiling)")
    ap.add_argument("--exchange", action="store_true",
                    help="replica-per-GPU form: every rank hosts one replica and the sparse messages are "
                         "all-gathered over NCCL (R = number of ranks); not the default bench line")
    ap.add_argument("--peer", action="store_true",
                    help="with --exchange: no gather; messages live in symmetric memory and the averaging "
                         "kernel reads every rank's buffer through its NVLink peer mapping")
    ap.add_argument("--idx12", action="store_true",
                    help="with --exchange: send the positions as 12 bits each")
    ap.add_argument("--groups", type=int, default=1,
                    help="with --exchange: cut the arena into this many tensor groups and overlap the gather "
                         "of one group with the compression of the next")
    ap.add_argument("--embed", action="store_true",
                    help="time sl_embed_reproject (token-embedding adaptation, Eqs. 3-4) on the model's "
                         "embedding table instead of the outer step; one GPU, its own JSON line")
    ap.add_argument("--subspace", action="store_true",
                    help="time sl_subspace_project + sl_subspace_reconstruct (activation compression of a "
                         "pipeline-stage boundary) instead of the outer step; one GPU, its own JSON line")
    ap.add_argument("--tokens", type=int, default=16384, help="with --subspace: tokens per micro-batch")
    ap.add_argument("--tiles", action="store_true",
                    help="cut matrices into square tiles of `chunk` elements instead of consecutive chunks")
    ap.add_argument("--bf16", action="store_true",
                    help="parameters stored as bfloat16 (error buffers float32): the *_bf16 entry points")
    ap.add_argument("--variant", default="plain", choices=["plain", "ties_literal", "ties_dyadic"],
                    help="tie-heavy value laws of the density-sweep configuration")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-rows", action="store_true",
                    help="leave out the `rows` object (tiles, R = 2, R = 16 / k = 128, embedding, activation subspace)")
    ap.add_argument("--row-launches", type=int, default=50, help="timed launches per entry of `rows`")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.subspace:
        run_subspace(args)
    elif args.embed:
        run_embed(args)
    elif args.exchange:
        run_exchange(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
