"""GPU parity: the CUDA path, called through the C ABI, against the CPU checker, element by
element on the same seeded inputs (bar: see parity_util)."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import slo
from paper_2601_02360_b200 import api, synth
from parity_util import (GpuStep, assert_close, assert_exact, compare_messages, oracle_compress_all,
                         run_and_compare)

pytestmark = pytest.mark.gpu
f32 = np.float32
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rand(n, seed, noise=1e-3, err=5e-4):
    rng = np.random.default_rng(seed)
    tg = rng.normal(0, 0.02, n).astype(f32)
    return tg, rng, noise, err


def _case(n, R, seed, noise=1e-3, err=5e-4):
    tg, rng, _, _ = _rand(n, seed)
    tls = [(tg + rng.normal(0, noise, n).astype(f32)).astype(f32) for _ in range(R)]
    errs = [rng.normal(0, err, n).astype(f32) for _ in range(R)]
    return tg, tls, errs


def test_hand_worked_example_on_gpu():
    g = json.load(open(os.path.join(GOLD, "w1_dyadic.json")))
    tg = np.array(g["theta_global"], f32)
    tls = [np.array(r["theta_local"], f32) for r in g["replicas"]]
    errs = [np.array(r["err_in"], f32) for r in g["replicas"]]
    gs = GpuStep([0, 8], 2, g["chunk"], g["k"], g["bits"])
    gs.upload(tg, tls, errs)
    gs.compress(g["beta"])
    msgs = gs.messages_host()
    for r, rep in enumerate(g["replicas"]):
        assert msgs[r][0].tolist() == [rep["idx"]]
        assert msgs[r][1].tolist() == [rep["packed"]]
        assert msgs[r][2].tolist() == [rep["scale"]]
        assert gs.err[r].cpu().numpy().tolist() == rep["err_out"]
    gs.aggregate_apply(g["outer_lr"])
    assert gs.theta_global.cpu().numpy().tolist() == g["theta_global_out"]


def test_tiny_config():
    wl = synth.workload("tiny")
    tgt = synth.gen_theta_global(wl)
    tls = [synth.gen_theta_local(wl, tgt, 0, r).numpy() for r in range(wl.R)]
    errs = [np.zeros(wl.n_total, f32) for _ in range(wl.R)]
    run_and_compare(wl.offsets(), tgt.numpy(), tls, errs, wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr,
                    what="tiny")


def test_tiny_config_three_rounds_carrying_err():
    wl = synth.workload("tiny")
    tgt = synth.gen_theta_global(wl)
    tls = [synth.gen_theta_local(wl, tgt, 0, r).numpy() for r in range(wl.R)]
    errs = [synth.gen_error(wl, r).numpy() for r in range(wl.R)]
    nxt = lambda t, tg: [synth.gen_theta_local(wl, torch.from_numpy(tg), t, r).numpy() for r in range(wl.R)]
    run_and_compare(wl.offsets(), tgt.numpy(), tls, errs, wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr,
                    rounds=3, next_locals=nxt, what="tiny x3")


@pytest.mark.parametrize("chunk,k,bits", [
    (4096, 64, 2), (4096, 32, 2), (4096, 16, 2), (4096, 128, 2), (4096, 64, 4), (4096, 64, 8),
    (4096, 32, 32), (4096, 1, 2), (4096, 4096, 32), (4096, 4096, 2), (8192, 100, 4), (256, 8, 2),
    (100, 7, 8), (8, 2, 2), (1, 1, 32), (2048, 2048, 8), (4096, 60, 2), (4096, 63, 4),
])
def test_ragged_multi_tensor_arena(chunk, k, bits):
    # several tiles plus ragged tails; tensor sizes that are NOT multiples of 4 elements
    sizes = [3 * chunk + 5, 1, chunk, 7, 2 * chunk + chunk // 2 + 3, max(1, chunk // 3)]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), 3, seed=chunk * 131 + k * 7 + bits)
    run_and_compare(off, tg, tls, errs, 0.95, chunk, k, bits, 0.8, what=f"ragged C{chunk} k{k} b{bits}")


@pytest.mark.parametrize("k,bits", [(16, 2), (32, 2), (64, 2), (128, 2), (64, 4), (64, 8), (32, 32), (5, 32), (7, 32),
                                    (6, 32), (8, 4), (4, 8), (2, 32), (128, 32), (128, 8)])
def test_aligned_arena_fast_path_shapes(k, bits):
    # every tensor a multiple of 4 elements (the layout the tuned kernels accept), short tails included
    sizes = [5 * 4096, 1024, 4096 + 2048, 512, 4, 3 * 4096 + 4092, 4096]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), 4, seed=k * 3 + bits)
    run_and_compare(off, tg, tls, errs, 0.95, 4096, k, bits, 1.0, what=f"aligned k{k} b{bits}")


def _adversarial_chunks(chunk, k):
    """(name, e' target) chunks; built with theta_global = 0, err = 0, beta = 0 => e' = -theta_local."""
    rng = np.random.default_rng(99)
    out = {}
    out["all_equal"] = np.full(chunk, 0.125, f32)
    out["all_zero"] = np.zeros(chunk, f32)
    z = np.zeros(chunk, f32); z[::2] = -0.0
    out["signed_zeros"] = z
    s = np.zeros(chunk, f32); s[chunk // 3] = -7.0
    out["one_spike"] = s
    t = rng.normal(0, 1, chunk).astype(f32)
    kth = np.sort(np.abs(t))[-min(k, chunk)]
    t[np.abs(t) < kth] = 0
    dup = rng.choice(chunk, size=chunk // 4, replace=False)
    t[dup] = kth * np.where(rng.random(len(dup)) < 0.5, -1, 1).astype(f32)   # many ties exactly at the k-th key
    out["ties_at_boundary"] = t
    out["two_levels"] = np.where(rng.random(chunk) < 0.5, f32(1.0), f32(-0.5)).astype(f32)
    sub = (rng.integers(-50, 50, chunk) * f32(2.0 ** -149)).astype(f32)
    out["subnormals"] = sub
    d = np.round(rng.normal(0, 3, chunk)).astype(f32) * f32(2.0 ** -13)
    out["dyadic_grid"] = d
    big = rng.normal(0, 1, chunk).astype(f32) * f32(1e30)
    out["huge"] = big
    asc = np.arange(chunk, dtype=f32)
    out["ascending"] = asc
    out["descending"] = asc[::-1].copy()
    return out


@pytest.mark.parametrize("chunk,k,bits", [(4096, 64, 2), (4096, 128, 2), (4096, 16, 2), (4096, 64, 8),
                                          (4096, 64, 32), (512, 64, 2), (4096, 1000, 4)])
def test_adversarial_chunks(chunk, k, bits):
    cases = _adversarial_chunks(chunk, k)
    n = chunk * len(cases)
    ep = np.concatenate(list(cases.values()))
    tg = np.zeros(n, f32)
    tls = [(-ep).astype(f32), np.roll(-ep, chunk).astype(f32)]
    errs = [np.zeros(n, f32), np.zeros(n, f32)]
    run_and_compare([0, n], tg, tls, errs, 0.0, chunk, k, bits, 1.0, what=f"adversarial C{chunk} k{k} b{bits}")


def test_nonfinite_values_raise_the_flag_without_trapping():
    chunk, k = 4096, 64
    n = 3 * chunk
    tg, tls, errs = _case(n, 2, seed=5)
    tls[0][17] = np.inf
    tls[0][chunk + 5] = np.nan
    tls[1][2 * chunk + 100] = -np.inf
    gs, _, _ = run_and_compare([0, n], tg, tls, errs, 0.95, chunk, k, 2, 1.0, what="nonfinite")
    assert int(gs.flags.item()) & api.SL_FLAG_NONFINITE


def test_batched_equals_per_replica_calls():
    wl = synth.workload("tiny").replace(R=3)
    tgt = synth.gen_theta_global(wl)
    tls = [synth.gen_theta_local(wl, tgt, 0, r).numpy() for r in range(wl.R)]
    errs = [synth.gen_error(wl, r).numpy() for r in range(wl.R)]
    a = GpuStep(wl.offsets(), wl.R, wl.chunk, wl.k, wl.bits)
    b = GpuStep(wl.offsets(), wl.R, wl.chunk, wl.k, wl.bits)
    for g, batched in ((a, True), (b, False)):
        g.upload(tgt.numpy(), tls, errs)
        g.compress(wl.beta, batched=batched)
    compare_messages(a.messages_host(), b.messages_host(), "batched vs single")
    for r in range(wl.R):
        assert torch.equal(a.err[r], b.err[r])


def test_aggregate_then_apply_equals_fused_and_checker():
    wl = synth.workload("tiny").replace(R=4)
    off = wl.offsets()
    tgt = synth.gen_theta_global(wl)
    tls = [synth.gen_theta_local(wl, tgt, 0, r).numpy() for r in range(wl.R)]
    errs = [np.zeros(wl.n_total, f32) for _ in range(wl.R)]
    gs = GpuStep(off, wl.R, wl.chunk, wl.k, wl.bits)
    gs.upload(tgt.numpy(), tls, errs)
    gs.compress(wl.beta)
    upd = torch.full((wl.n_total,), 7.0, dtype=torch.float32, device="cuda")  # must be fully overwritten
    api.sl_aggregate(gs.idx, gs.codes, gs.scales, gs.layout, wl.chunk, wl.k, wl.bits, upd, gs.flags)
    ora = slo.aggregate(gs.messages_host(), off, wl.chunk, wl.k, wl.bits)
    assert_close(upd.cpu().numpy(), ora, "dense update")
    th2 = gs.theta_global.clone()
    api.sl_outer_apply(th2, upd, wl.n_total, 0.8)
    gs.aggregate_apply(0.8)
    assert torch.equal(th2, gs.theta_global)
    want = tgt.numpy().copy()
    slo.outer_apply(want, ora, 0.8)
    assert_close(gs.theta_global.cpu().numpy(), want, "theta_global")
    # a replica that dropped out: its message is left out, the caller passes fewer messages
    upd3 = torch.empty_like(upd)
    api.sl_aggregate(gs.idx[:3], gs.codes[:3], gs.scales[:3], gs.layout, wl.chunk, wl.k, wl.bits, upd3)
    assert_close(upd3.cpu().numpy(), slo.aggregate(gs.messages_host()[:3], off, wl.chunk, wl.k, wl.bits),
                 "three of four")
    assert int(gs.flags.item()) == 0


def test_aggregate_skips_out_of_range_positions_and_flags_them():
    chunk, k = 256, 8
    n = chunk + 40          # second chunk is 40 long
    tg, tls, errs = _case(n, 1, seed=3)
    gs = GpuStep([0, n], 1, chunk, k, 2)
    gs.upload(tg, tls, errs)
    gs.compress(0.9)
    torch.cuda.synchronize()
    idx = gs.idx[0].cpu().numpy().copy()
    idx[k + 2] = 200        # beyond the short chunk's 40 elements
    gs.idx[0].copy_(torch.from_numpy(idx))
    upd = torch.empty(n, dtype=torch.float32, device="cuda")
    api.sl_aggregate(gs.idx, gs.codes, gs.scales, gs.layout, chunk, k, 2, upd, gs.flags)
    assert int(gs.flags.item()) & api.SL_FLAG_BAD_INDEX
    idx[k + 2] = 0xFFFF     # the checker sees the slot as padding: same result
    msgs = [(idx.reshape(2, k), gs.codes[0].cpu().numpy().reshape(2, -1), gs.scales[0].cpu().numpy())]
    assert_close(upd.cpu().numpy(), slo.aggregate(msgs, [0, n], chunk, k, 2), "skipped slot")


def test_outer_apply_unaligned_and_tail():
    rng = np.random.default_rng(0)
    for n, shift in [(1, 0), (5, 1), (1027, 0), (4099, 3), (1 << 20, 0)]:
        th = rng.normal(0, 1, n + 4).astype(f32)
        up = rng.normal(0, 1, n + 4).astype(f32)
        dth = torch.from_numpy(th).cuda()
        dup = torch.from_numpy(up).cuda()
        api.sl_outer_apply(dth[shift:], dup[shift:], n, 0.8)
        want = th.copy()
        w = want[shift:shift + n]
        slo.outer_apply(w, up[shift:shift + n].copy(), 0.8)
        want[shift:shift + n] = w
        assert_close(dth.cpu().numpy(), want, f"outer_apply n={n} shift={shift}")


def test_checkpoint_resume_on_gpu_is_bit_identical():
    wl = synth.workload("tiny")
    off = wl.offsets()
    def run(rounds, state=None):
        gs = GpuStep(off, wl.R, wl.chunk, wl.k, wl.bits)
        if state is None:
            gs.theta_global.copy_(synth.gen_theta_global(wl))
            t0 = 0
        else:
            gs.theta_global.copy_(state[0])
            for r in range(wl.R):
                gs.err[r].copy_(state[1][r])
            t0 = state[2]
        for t in range(t0, t0 + rounds):
            for r in range(wl.R):
                synth.gen_theta_local(wl, gs.theta_global, t, r, out=gs.theta_local[r])
            gs.compress(wl.beta)
            gs.aggregate_apply(wl.outer_lr)
        torch.cuda.synchronize()
        return gs.theta_global.cpu(), [e.cpu() for e in gs.err], t0 + rounds
    a = run(4)
    b = run(2, run(2))
    assert torch.equal(a[0], b[0]) and all(torch.equal(x, y) for x, y in zip(a[1], b[1]))


def test_180m_sub_arena_three_rounds():
    full = synth.workload("180m")
    # one whole layer (7 matrices + 2 norm vectors) and the final norm; value law of the full config
    keep = list(range(9)) + [len(full.tensors) - 1]
    wl = synth.sub_arena(full, keep)
    tgt = synth.gen_theta_global(wl)
    rho = synth.row_scales(wl)
    tls = [synth.gen_theta_local(wl, tgt, 0, r, rho=rho).numpy() for r in range(wl.R)]
    errs = [np.zeros(wl.n_total, f32) for _ in range(wl.R)]
    nxt = lambda t, tg: [synth.gen_theta_local(wl, torch.from_numpy(tg), t, r, rho=rho).numpy()
                         for r in range(wl.R)]
    run_and_compare(wl.offsets(), tgt.numpy(), tls, errs, wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr,
                    rounds=3, next_locals=nxt, what="180m sub-arena")


@pytest.mark.parametrize("variant", ["ties_literal", "ties_dyadic"])
def test_tie_heavy_variants(variant):
    full = synth.workload("1b").replace(variant=variant, R=2)
    keep = [0, 4, 7, 8]     # q (2048x2048), gate (2048x5632), two norm vectors
    wl = synth.sub_arena(full, keep)
    tgt = synth.gen_theta_global(wl)
    rho = synth.row_scales(wl)
    tls = [synth.gen_theta_local(wl, tgt, 0, r, rho=rho).numpy() for r in range(wl.R)]
    errs = [np.zeros(wl.n_total, f32) for _ in range(wl.R)]
    nxt = lambda t, tg: [synth.gen_theta_local(wl, torch.from_numpy(tg), t, r, rho=rho).numpy()
                         for r in range(wl.R)]
    if variant == "ties_dyadic":
        # the stress is real only if the k-th and (k+1)-th magnitudes tie in most chunks
        d = (tgt.numpy() - tls[0])[: 2048 * 2048].reshape(-1, 4096)
        srt = np.sort(np.abs(d), axis=1)
        assert (srt[:, -wl.k] == srt[:, -wl.k - 1]).mean() > 0.5
    run_and_compare(wl.offsets(), tgt.numpy(), tls, errs, wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr,
                    rounds=2, next_locals=nxt, what=variant)


@pytest.mark.parametrize("k,R", [(16, 2), (32, 8), (128, 2)])
def test_density_sweep_cells_on_sub_arena(k, R):
    full = synth.workload("1b").replace(k=k, R=R)
    wl = synth.sub_arena(full, [0, 6, 7])     # q, down, one norm vector
    tgt = synth.gen_theta_global(wl)
    rho = synth.row_scales(wl)
    tls = [synth.gen_theta_local(wl, tgt, 0, r, rho=rho).numpy() for r in range(wl.R)]
    errs = [np.zeros(wl.n_total, f32) for _ in range(wl.R)]
    run_and_compare(wl.offsets(), tgt.numpy(), tls, errs, wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr,
                    what=f"sweep k{k} R{R}")


# ---------------------------------------------------------------- the one-call step (sl_outer_step)
def test_outer_step_tiny_three_rounds():
    wl = synth.workload("tiny")
    tgt = synth.gen_theta_global(wl)
    tls = [synth.gen_theta_local(wl, tgt, 0, r).numpy() for r in range(wl.R)]
    errs = [synth.gen_error(wl, r).numpy() for r in range(wl.R)]
    nxt = lambda t, tg: [synth.gen_theta_local(wl, torch.from_numpy(tg), t, r).numpy() for r in range(wl.R)]
    run_and_compare(wl.offsets(), tgt.numpy(), tls, errs, wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr,
                    rounds=3, next_locals=nxt, what="outer_step tiny", fused=True)


@pytest.mark.parametrize("k,bits,R", [(64, 2, 8), (16, 2, 3), (128, 2, 5), (64, 8, 2), (32, 32, 1), (64, 4, 16)])
def test_outer_step_aligned_arena(k, bits, R):
    sizes = [5 * 4096, 1024, 4096 + 2048, 512, 4, 3 * 4096 + 4092, 4096]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), R, seed=k + bits + R)
    run_and_compare(off, tg, tls, errs, 0.95, 4096, k, bits, 0.8, what=f"outer_step k{k} b{bits} R{R}", fused=True)


@pytest.mark.parametrize("chunk,k,bits", [(4096, 60, 2), (256, 8, 2), (100, 7, 8), (8192, 100, 4)])
def test_outer_step_falls_back_on_other_shapes(chunk, k, bits):
    sizes = [3 * chunk + 5, 1, chunk, 7, 2 * chunk + chunk // 2 + 3]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), 3, seed=chunk + k)
    run_and_compare(off, tg, tls, errs, 0.95, chunk, k, bits, 1.0, what=f"outer_step generic C{chunk}", fused=True)


def test_outer_step_adversarial_chunks():
    chunk, k, bits = 4096, 64, 2
    cases = _adversarial_chunks(chunk, k)
    n = chunk * len(cases)
    ep = np.concatenate(list(cases.values()))
    tg = np.zeros(n, f32)
    tls = [(-ep).astype(f32), np.roll(-ep, chunk).astype(f32), np.roll(-ep, 3 * chunk).astype(f32)]
    errs = [np.zeros(n, f32) for _ in range(3)]
    run_and_compare([0, n], tg, tls, errs, 0.0, chunk, k, bits, 1.0, what="outer_step adversarial", fused=True)


def test_outer_step_180m_sub_arena_three_rounds():
    full = synth.workload("180m")
    wl = synth.sub_arena(full, list(range(9)) + [len(full.tensors) - 1])
    tgt = synth.gen_theta_global(wl)
    rho = synth.row_scales(wl)
    tls = [synth.gen_theta_local(wl, tgt, 0, r, rho=rho).numpy() for r in range(wl.R)]
    errs = [np.zeros(wl.n_total, f32) for _ in range(wl.R)]
    nxt = lambda t, tg: [synth.gen_theta_local(wl, torch.from_numpy(tg), t, r, rho=rho).numpy()
                         for r in range(wl.R)]
    run_and_compare(wl.offsets(), tgt.numpy(), tls, errs, wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr,
                    rounds=3, next_locals=nxt, what="outer_step 180m sub-arena", fused=True)


# ---------------------------------------------------------------- less travelled code paths
@pytest.mark.parametrize("R,k", [(20, 64), (64, 16), (17, 128), (1, 64), (2, 128)])
def test_many_replicas_beyond_the_pointer_cache(R, k):
    # R > 16 reads the replicas' pointers from the kernel parameters instead of shared memory;
    # R * k > 2048 sends the aggregate to the generic kernel
    sizes = [6 * 4096, 2048, 3 * 4096 + 1024]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), R, seed=R * 7 + k)
    run_and_compare(off, tg, tls, errs, 0.95, 4096, k, 2, 1.0, rounds=1, what=f"R{R} k{k}")


def test_arena_with_more_than_256_tensors():
    # 300 tensors select the large by-value table (up to 2048 tensors)
    rng = np.random.default_rng(4)
    sizes = [int(x) * 4 for x in rng.integers(1, 3000, size=300)]
    sizes[10] = 4096 * 3
    sizes[200] = 4096 * 2 + 512
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), 3, seed=17)
    run_and_compare(off, tg, tls, errs, 0.95, 4096, 64, 2, 1.0, rounds=2,
                    next_locals=lambda t, g: [(g + np.random.default_rng(t * 10 + r).normal(0, 1e-3, g.size)).astype(f32)
                                              for r in range(3)], what="300 tensors")


def test_empty_tensors_inside_the_arena():
    sizes = [4096, 0, 0, 8192 + 100, 0, 512]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), 2, seed=23)
    run_and_compare(off, tg, tls, errs, 0.95, 4096, 64, 2, 1.0, what="empty tensors")


def test_more_chunks_than_resident_ctas():
    # the persistent grids hold 296 / 592 CTAs: 1500 chunks give every CTA several chunks and a ragged last wave
    n = 1500 * 4096 + 2048
    tg, tls, errs = _case(n, 3, seed=31)
    run_and_compare([0, n], tg, tls, errs, 0.95, 4096, 64, 2, 1.0, rounds=2,
                    next_locals=lambda t, g: [(g + np.random.default_rng(t * 10 + r).normal(0, 1e-3, g.size)).astype(f32)
                                              for r in range(3)], what="1500 chunks")


def test_replica_per_rank_step_on_one_gpu():
    # world size 1: the exchange degenerates to a copy, the step must equal the single-replica step
    import torch.distributed as dist
    from paper_2601_02360_b200 import exchange
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1)
    try:
        wl = synth.workload("tiny").replace(R=1)
        tgt = synth.gen_theta_global(wl)
        tl = synth.gen_theta_local(wl, tgt, 0, 0)
        gs = GpuStep(wl.offsets(), 1, wl.chunk, wl.k, wl.bits)
        gs.upload(tgt.numpy(), [tl.numpy()])
        # gloo moves host tensors: gather through the host, aggregate on the device
        api.sl_compress(gs.theta_local[0], gs.theta_global, gs.err[0], gs.layout, wl.beta, wl.chunk, wl.k, wl.bits,
                        gs.idx[0], gs.codes[0], gs.scales[0], gs.flags)
        torch.cuda.synchronize()
        gi, gc, gsc = exchange.all_gather_messages(gs.idx[0].cpu(), gs.codes[0].cpu(), gs.scales[0].cpu())
        d = lambda ts: [t.cuda() for t in ts]
        api.sl_aggregate_apply(d(gi), d(gc), d(gsc), gs.layout, wl.chunk, wl.k, wl.bits, gs.theta_global, wl.outer_lr, gs.flags)
        want = tgt.numpy().copy()
        slo.outer_round([tl.numpy()], want, [np.zeros(wl.n_total, f32)], wl.offsets(), wl.beta, wl.chunk, wl.k,
                        wl.bits, wl.outer_lr)
        assert_close(gs.theta_global.cpu().numpy(), want, "replica-per-rank, world 1")
    finally:
        dist.destroy_process_group()


def test_pipelined_replica_step_on_one_gpu():
    # gathers of one tensor group overlapped with the compression of the next (two streams, NCCL with
    # one rank): same bits as the checker's one-shot step, over two rounds
    import torch.distributed as dist
    from paper_2601_02360_b200 import exchange
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    try:
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                                device_id=torch.device("cuda", 0))
    except Exception as exc:  # an environment without a usable NCCL: nothing of ours has run yet
        pytest.skip(f"one-rank NCCL group unavailable: {exc}")
    try:
        wl = synth.sub_arena(synth.workload("180m"), list(range(10))).replace(R=1)
        off = wl.offsets()
        groups = exchange.plan_groups(off, wl.chunk, 4)
        assert len(groups) >= 3
        tgt = synth.gen_theta_global(wl)
        gs = GpuStep(off, 1, wl.chunk, wl.k, wl.bits)
        want = tgt.numpy().copy()
        h_err = [np.zeros(wl.n_total, f32)]
        for rnd in range(2):
            tl = synth.gen_theta_local(wl, torch.from_numpy(want), rnd, 0)
            if rnd == 0:
                gs.upload(tgt.numpy(), [tl.numpy()])
            else:
                gs.theta_local[0].copy_(tl)
            exchange.outer_step_replica_pipelined(gs.theta_local[0], gs.theta_global, gs.err[0], groups, wl.beta,
                                                  wl.chunk, wl.k, wl.bits, wl.outer_lr, gs.idx[0], gs.codes[0],
                                                  gs.scales[0], gs.flags)
            torch.cuda.synchronize()
            msgs, _, _ = slo.outer_round([tl.numpy()], want, h_err, off, wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr)
            nc = wl.n_chunks()
            assert (gs.idx[0].cpu().numpy().reshape(nc, wl.k) == msgs[0][0]).all()
            assert (gs.codes[0].cpu().numpy().reshape(nc, -1) == msgs[0][1]).all()
            assert_close(gs.scales[0].cpu().numpy(), msgs[0][2], "pipelined scales")
            assert_close(gs.err[0].cpu().numpy(), h_err[0], "pipelined error buffer")
            assert_close(gs.theta_global.cpu().numpy(), want, "pipelined theta_global")
        assert int(gs.flags.item()) == 0
    finally:
        dist.destroy_process_group()


def test_outer_step_captured_in_a_cuda_graph():
    # every entry point only enqueues kernels on the caller's stream (tables travel by value in the
    # kernel parameters), so a whole outer step can be captured once and replayed every H inner steps
    wl = synth.sub_arena(synth.workload("180m"), [0, 1, 7, 8]).replace(R=3)
    off = wl.offsets()
    tgt = synth.gen_theta_global(wl)
    gs = GpuStep(off, wl.R, wl.chunk, wl.k, wl.bits)
    want = tgt.numpy().copy()
    h_err = [np.zeros(wl.n_total, f32) for _ in range(wl.R)]
    tls = [synth.gen_theta_local(wl, tgt, 0, r) for r in range(wl.R)]
    gs.upload(tgt.numpy(), [t.numpy() for t in tls])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            api.sl_outer_step(gs.theta_local, gs.theta_global, gs.err, gs.layout, wl.beta, wl.chunk, wl.k, wl.bits,
                              wl.outer_lr, gs.idx, gs.codes, gs.scales, gs.flags, stream=side)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    # capture does not execute: nothing has changed yet
    assert_close(gs.theta_global.cpu().numpy(), want, "theta_global untouched by capture")
    for rnd in range(3):
        if rnd:
            tls = [synth.gen_theta_local(wl, torch.from_numpy(want), rnd, r) for r in range(wl.R)]
            for r in range(wl.R):
                gs.theta_local[r].copy_(tls[r])
        graph.replay()
        torch.cuda.synchronize()
        msgs, _, _ = slo.outer_round([t.numpy() for t in tls], want, h_err, off, wl.beta, wl.chunk, wl.k, wl.bits,
                                     wl.outer_lr)
        nc = wl.n_chunks()
        for r in range(wl.R):
            assert (gs.idx[r].cpu().numpy().reshape(nc, wl.k) == msgs[r][0]).all()
            assert (gs.codes[r].cpu().numpy().reshape(nc, -1) == msgs[r][1]).all()
            assert_close(gs.err[r].cpu().numpy(), h_err[r], f"graph replay {rnd}: error buffer {r}")
        assert_close(gs.theta_global.cpu().numpy(), want, f"graph replay {rnd}: theta_global")
    assert int(gs.flags.item()) == 0


def test_peer_memory_replica_step_on_one_gpu():
    # the gather-free form: the message lives in symmetric memory and the averaging kernel reads the
    # ranks' buffers through their peer mappings (with one rank: its own mapping).  Two rounds.
    import torch.distributed as dist
    from paper_2601_02360_b200 import exchange
    import socket
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    try:
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                                device_id=torch.device("cuda", 0))
    except Exception as exc:  # an environment without a usable NCCL: nothing of ours has run yet
        pytest.skip(f"one-rank NCCL group unavailable: {exc}")
    try:
        wl = synth.sub_arena(synth.workload("180m"), list(range(10))).replace(R=1)
        off = wl.offsets()
        lay = api.Layout(off)
        try:
            pm = exchange.PeerMessages(lay, wl.chunk, wl.k, wl.bits)
        except Exception as exc:  # symmetric memory is a torch facility that a box may lack
            pytest.skip(f"symmetric memory unavailable: {exc}")
        assert pm.world == 1 and pm.idx[0].data_ptr() % 16 == 0 and pm.scales[0].data_ptr() % 16 == 0
        tgt = synth.gen_theta_global(wl)
        d_tg = tgt.cuda()
        d_err = torch.zeros_like(d_tg)
        flags = torch.zeros(1, dtype=torch.int32, device="cuda")
        want = tgt.numpy().copy()
        h_err = [np.zeros(wl.n_total, f32)]
        for rnd in range(2):
            tl = synth.gen_theta_local(wl, torch.from_numpy(want), rnd, 0)
            exchange.outer_step_replica_peer(tl.cuda(), d_tg, d_err, lay, wl.beta, wl.chunk, wl.k, wl.bits,
                                             wl.outer_lr, pm, flags)
            torch.cuda.synchronize()
            msgs, _, _ = slo.outer_round([tl.numpy()], want, h_err, off, wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr)
            nc = wl.n_chunks()
            assert (pm.idx[0].cpu().numpy().reshape(nc, wl.k) == msgs[0][0]).all()
            assert (pm.codes[0].cpu().numpy().reshape(nc, -1) == msgs[0][1]).all()
            assert_close(d_err.cpu().numpy(), h_err[0], "peer form: error buffer")
            assert_close(d_tg.cpu().numpy(), want, "peer form: theta_global")
        assert int(flags.item()) == 0
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("k,bits,R", [
    (128, 2, 16),    # 8 pairs per thread, a thread owns 8 slots of one replica
    (128, 8, 16),    # ... whose codes span 8 bytes
    (128, 32, 12),   # ... unquantised
    (100, 2, 20),    # 8 pairs per thread, k not a multiple of 8: pairs 256 apart
    (36, 4, 20),     # 4 pairs per thread, grouped
    (6, 2, 64),      # 2 pairs per thread, grouped, codes start in mid-byte
    (5, 2, 64),      # 2 pairs per thread, odd k
    (7, 8, 40),
    (32, 2, 64),     # the most replicas a call takes: 64 rounds, 8 slots per thread
    (16, 4, 64),
])
def test_aggregate_instances_for_many_pairs_per_chunk(k, bits, R):
    sizes = [6 * 4096, 1024, 4096 + 2048, 4, 2 * 4096 + 4092, 4096]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), R, seed=1000 + k + bits + R)
    for fused in (True, False):
        gs, _, _ = run_and_compare(off, tg, tls, errs, 0.95, 4096, k, bits, 0.8,
                                   what=f"aggregate k{k} b{bits} R{R} fused={fused}", fused=fused)
    # the same instance without the fused outer update: the dense mean update on its own
    upd = torch.full((int(off[-1]),), 7.0, dtype=torch.float32, device="cuda")
    api.sl_aggregate(gs.idx, gs.codes, gs.scales, gs.layout, 4096, k, bits, upd, gs.flags)
    assert_close(upd.cpu().numpy(), slo.aggregate(gs.messages_host(), off, 4096, k, bits), f"dense update k{k} b{bits} R{R}")


@pytest.mark.parametrize("cols", [None, "tiles"])
def test_no_write_outside_the_callers_buffers(cols):
    # every buffer handed to the library sits between two sentinel bands inside one allocation; after
    # a whole outer step on a ragged arena (short chunks, a 3-element tensor, edge tiles) the bands
    # must be untouched.  (compute-sanitizer is not available on the GPUs this runs on.)
    sizes = [100 * 72, 4096 * 2 + 16, 4, 4096, 128 * 200, 8]     # multiples of 4: the tuned kernels take the full chunks
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    col_list = [72, 0, 0, 0, 200, 0] if cols else None
    n, R, chunk, k, bits = int(off[-1]), 3, 4096, 64, 2
    lay = api.Layout(off, col_list)
    nc, st = api.sl_num_chunks(lay, chunk), api.sl_codes_stride(k, bits)
    band = 1024                                  # bytes
    need = [n * 4] * (1 + 2 * R) + [nc * k * 2] * R + [nc * st] * R + [nc * 4] * R
    total = sum(band + (b + 255) // 256 * 256 for b in need) + band
    pool = torch.full((total,), 0xA5, dtype=torch.uint8, device="cuda")
    views, at = [], 0
    for b in need:
        at += band
        views.append(pool[at:at + b])
        at += (b + 255) // 256 * 256
    f32v = lambda v: v.view(torch.float32)
    tg_v, tl_v, err_v = f32v(views[0]), [f32v(v) for v in views[1:1 + R]], [f32v(v) for v in views[1 + R:1 + 2 * R]]
    m = views[1 + 2 * R:]
    idx_v = [v.view(torch.uint16) for v in m[:R]]
    codes_v, sc_v = m[R:2 * R], [f32v(v) for v in m[2 * R:]]
    tg, tls, errs = _case(n, R, seed=77)
    tg_v.copy_(torch.from_numpy(tg))
    for r in range(R):
        tl_v[r].copy_(torch.from_numpy(tls[r]))
        err_v[r].zero_()
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.sl_outer_step(tl_v, tg_v, err_v, lay, 0.95, chunk, k, bits, 0.8, idx_v, codes_v, sc_v, flags)
    torch.cuda.synchronize()
    # the result is the checker's ...
    want = tg.copy()
    h_err = [np.zeros(n, f32) for _ in range(R)]
    msgs = oracle_compress_all(tls, want.copy(), h_err, off, 0.95, chunk, k, bits, cols=col_list)
    upd = slo.aggregate([(i, c, s) for i, c, s, _ in msgs], off, chunk, k, bits, col_list)
    slo.outer_apply(want, upd, 0.8)
    assert_close(tg_v.cpu().numpy(), want, "guarded theta_global")
    # ... and nothing outside the buffers changed
    mask = torch.ones(total, dtype=torch.bool, device="cuda")
    at = 0
    for b in need:
        at += band
        mask[at:at + b] = False
        at += (b + 255) // 256 * 256
    assert bool((pool[mask] == 0xA5).all()), "a byte outside the caller's buffers was written"
    assert int(flags.item()) == 0


@pytest.mark.parametrize("seed", list(range(24)))
def test_random_configurations(seed):
    # seeded random arenas (aligned or not, with short and tiny tensors, sometimes tiled), k, code
    # width, R and beta: whichever kernels the dispatch picks, the step must match the checker
    rng = np.random.default_rng(1234 + seed)
    chunk = int(rng.choice([4096, 4096, 4096, 1024, 256, 100]))
    tiled = chunk in (4096, 1024, 256) and rng.random() < 0.35
    side = int(round(chunk ** 0.5))
    align = 4 if rng.random() < 0.7 else 1
    sizes, cols = [], []
    for _ in range(int(rng.integers(1, 7))):
        if tiled and rng.random() < 0.7:
            r, c = int(rng.integers(1, 3 * side)), int(rng.integers(1, 3 * side))
            c = max(align, c // align * align)
            sizes.append(r * c)
            cols.append(c)
        else:
            n = int(rng.integers(1, 3 * chunk + 50))
            sizes.append(max(align, n // align * align))
            cols.append(0)
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    k = int(rng.choice([1, 2, 5, 8, 16, 32, 64, 128]))
    k = min(k, chunk)
    bits = int(rng.choice([2, 4, 8, 32]))
    R = int(rng.choice([1, 2, 3, 5, 8, 16]))
    beta = float(rng.choice([0.0, 0.5, 0.95, 1.0]))
    tg, tls, errs = _case(int(off[-1]), R, seed=5000 + seed)
    errs = [(np.random.default_rng(seed * 31 + r).normal(0, 5e-4, int(off[-1]))).astype(f32) for r in range(R)]
    nxt = lambda t, g: [(g + np.random.default_rng(seed * 1000 + t * 10 + r).normal(0, 1e-3, g.size)).astype(f32)
                        for r in range(R)]
    run_and_compare(off, tg, tls, errs, beta, chunk, k, bits, 0.8, rounds=2, next_locals=nxt,
                    what=f"random #{seed}: chunk {chunk} k {k} b {bits} R {R} tiled {tiled} align {align}",
                    fused=bool(seed % 2), cols=cols if tiled else None)


@pytest.mark.parametrize("lr", [0.8, 1.0, -0.5, 0.0])
@pytest.mark.parametrize("R,k", [(2, 64), (1, 128), (4, 64), (2, 16), (5, 64), (2, 32), (3, 20), (1, 7)])
def test_theta_global_update_touches_only_what_was_sent(R, k, lr):
    # with few entries per chunk and a positive step the averaging kernel updates only the elements some
    # replica sent; every other element must keep its bits - signed zeros included - exactly as the
    # dense form theta - lr * 0 leaves them, and a negative or zero step takes the dense form
    sizes = [40 * 4096, 2048, 3 * 4096]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), R, seed=R * 100 + k)
    rng = np.random.default_rng(7)
    z = rng.choice(tg.size, size=tg.size // 5, replace=False)
    tg[z[: len(z) // 2]] = 0.0
    tg[z[len(z) // 2:]] = -0.0
    if R >= 2:                       # replica 1 mirrors replica 0 around theta_global on the first chunks: sums that cancel to +0
        tls[1][:8 * 4096] = (2 * tg[:8 * 4096] - tls[0][:8 * 4096]).astype(f32)
        errs[1][:8 * 4096] = -errs[0][:8 * 4096]
    gs, tg_o, _ = run_and_compare(off, tg, tls, errs, 0.95, 4096, k, 2, lr, what=f"sparse update R{R} k{k} lr{lr}")
    got = gs.theta_global.cpu().numpy()
    assert np.array_equal(np.signbit(got), np.signbit(tg_o)), "a signed zero changed its sign"


@pytest.mark.parametrize("R,k", [(2, 64), (4, 16), (1, 32)])
def test_theta_global_update_touches_only_what_was_sent_in_tiles(R, k):
    # the same with matrices cut into 64 x 64 tiles (the position of an entry is a row and a column of its tile)
    sizes = [320 * 192, 2048, 128 * 640, 4096 * 3]
    cols = [192, 0, 640, 0]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), R, seed=R * 10 + k)
    tg[::7] = -0.0
    gs, tg_o, _ = run_and_compare(off, tg, tls, errs, 0.95, 4096, k, 2, 0.8, rounds=2, cols=cols,
                                  next_locals=lambda t, g: [(g + np.random.default_rng(t * 10 + r).normal(0, 1e-3, g.size)).astype(f32)
                                                            for r in range(R)], what=f"sparse update in tiles R{R} k{k}")
    assert np.array_equal(np.signbit(gs.theta_global.cpu().numpy()), np.signbit(tg_o))
