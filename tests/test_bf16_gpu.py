"""GPU parity of the bfloat16 parameter storage mode (parameters bfloat16, error buffers float32)
against the CPU checker's reading of it: messages bit-exact, error buffers and the stored theta_global
bit-identical, over several rounds carrying the error buffers, through the one-call and the two-call
forms, on arenas that take the tuned kernels (consecutive chunks, offsets multiples of 8) and on ones
that take the generic kernels (ragged offsets, tiles)."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import slo
from paper_2601_02360_b200 import api, synth
from parity_util import assert_close, assert_exact, compare_messages

pytestmark = pytest.mark.gpu
f32 = np.float32
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 patterns by a library conversion (input preparation only)."""
    return torch.from_numpy(np.ascontiguousarray(x, dtype=f32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16).copy()


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def host_bits(t: torch.Tensor) -> np.ndarray:
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def run_and_compare_bf16(offsets, tg_bits, tl_bits, errs, beta, chunk, k, bits, lr, rounds=1, next_locals=None,
                         fused=False, cols=None, what=""):
    R = len(tl_bits)
    lay = api.Layout(offsets, cols)
    nc, stride = api.sl_num_chunks(lay, chunk), api.sl_codes_stride(k, bits)
    d_tg = dev_bf16(tg_bits)
    d_tl = [dev_bf16(b) for b in tl_bits]
    d_err = [torch.from_numpy(e).cuda() for e in errs]
    idx, codes, scales = api.alloc_messages(lay, chunk, k, bits, R)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    tg_o = tg_bits.copy()
    errs_o = [e.copy() for e in errs]
    flags_o = 0
    for t in range(rounds):
        if t > 0:
            tl_bits = next_locals(t, tg_o)
            for r in range(R):
                d_tl[r].copy_(dev_bf16(tl_bits[r]))
        if fused:
            api.sl_outer_step_bf16(d_tl, d_tg, d_err, lay, beta, chunk, k, bits, lr, idx, codes, scales, flags)
        else:
            api.sl_compress_batch_bf16(d_tl, d_tg, d_err, lay, beta, chunk, k, bits, idx, codes, scales, flags)
            api.sl_aggregate_apply_bf16(idx, codes, scales, lay, chunk, k, bits, d_tg, lr, flags)
        torch.cuda.synchronize()
        msgs, _, f = slo.outer_round_bf16(tl_bits, tg_o, errs_o, offsets, beta, chunk, k, bits, lr, cols)
        flags_o |= f
        gpu_msgs = [(idx[r].cpu().numpy().reshape(nc, k), codes[r].cpu().numpy().reshape(nc, stride), scales[r].cpu().numpy())
                    for r in range(R)]
        compare_messages(gpu_msgs, msgs, f"{what} round {t}")
        for r in range(R):
            assert_close(d_err[r].cpu().numpy(), errs_o[r], f"{what} round {t} err[{r}]")
        got = host_bits(d_tg)
        nan_o = (tg_o & 0x7FFF) > 0x7F80                       # NaN payloads are not compared (nor are they for float32)
        assert np.array_equal((got & 0x7FFF) > 0x7F80, nan_o), f"{what} round {t}: NaN positions differ"
        assert_exact(np.where(nan_o, 0, got), np.where(nan_o, 0, tg_o), f"{what} round {t} theta_global (bfloat16 patterns)")
    assert int(flags.item()) == flags_o
    return d_tg, d_err


def _case(n, R, seed):
    rng = np.random.default_rng(seed)
    tg = to_bf16_bits(rng.normal(0, 0.02, n))
    tls = [to_bf16_bits(slo.widen_bf16(tg) + rng.normal(0, 1e-3, n).astype(f32)) for _ in range(R)]
    errs = [rng.normal(0, 5e-4, n).astype(f32) for _ in range(R)]
    return tg, tls, errs


def _next(R, seed):
    return lambda t, tg: [to_bf16_bits(slo.widen_bf16(tg) + np.random.default_rng(seed + 100 * t + r).normal(0, 1e-3, tg.size).astype(f32))
                          for r in range(R)]


def test_hand_worked_example_in_bfloat16():
    g = json.load(open(os.path.join(GOLD, "w1_dyadic.json")))
    tg = to_bf16_bits(np.array(g["theta_global"], f32))
    tls = [to_bf16_bits(np.array(r["theta_local"], f32)) for r in g["replicas"]]
    errs = [np.array(r["err_in"], f32) for r in g["replicas"]]
    d_tg, d_err = run_and_compare_bf16([0, 8], tg, tls, errs, g["beta"], g["chunk"], g["k"], g["bits"], g["outer_lr"], what="w1")
    assert d_tg.float().cpu().numpy().tolist() == g["theta_global_out"]
    for r, rep in enumerate(g["replicas"]):
        assert d_err[r].cpu().numpy().tolist() == rep["err_out"]


@pytest.mark.parametrize("fused", [False, True], ids=["two_calls", "outer_step"])
@pytest.mark.parametrize("k,bits,R", [(64, 2, 8), (16, 2, 3), (128, 2, 2), (64, 8, 4), (32, 32, 2), (128, 4, 16)])
def test_tuned_path_three_rounds(k, bits, R, fused):
    # every tensor starts on a multiple of 8 elements: the tuned kernels take the full chunks, the generic
    # ones the short tails; 700 chunks give every resident CTA several
    sizes = [700 * 4096, 1024, 4096 + 2048, 512, 8, 3 * 4096 + 4088, 4096]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), R, seed=k + bits + R)
    run_and_compare_bf16(off, tg, tls, errs, 0.95, 4096, k, bits, 0.8, rounds=3, next_locals=_next(R, k), fused=fused,
                         what=f"bf16 tuned k{k} b{bits} R{R}")


@pytest.mark.parametrize("chunk,k,bits", [(4096, 64, 2), (4096, 60, 2), (256, 8, 2), (100, 7, 8), (8192, 100, 4), (4096, 4096, 32)])
def test_generic_path_on_ragged_arenas(chunk, k, bits):
    # offsets that are multiples of 4 but not of 8, or of nothing at all: the generic kernels
    sizes = [3 * chunk + 4, 1, chunk, 7, 2 * chunk + chunk // 2 + 3, max(1, chunk // 3)]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), 3, seed=chunk + k)
    run_and_compare_bf16(off, tg, tls, errs, 0.95, chunk, k, bits, 1.0, rounds=2, next_locals=_next(3, chunk),
                         fused=bool(k % 2), what=f"bf16 generic C{chunk} k{k}")


def test_aligned_to_four_but_not_eight_takes_the_generic_kernels():
    sizes = [5 * 4096 + 4, 4096 * 3, 1020, 4096]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), 4, seed=9)
    run_and_compare_bf16(off, tg, tls, errs, 0.95, 4096, 64, 2, 1.0, rounds=2, next_locals=_next(4, 9), what="bf16 offsets % 8 != 0")


def test_tiles_take_the_generic_kernels():
    sizes = [100 * 72, 4096 * 2 + 16, 8, 128 * 200]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    cols = [72, 0, 0, 200]
    tg, tls, errs = _case(int(off[-1]), 3, seed=10)
    run_and_compare_bf16(off, tg, tls, errs, 0.95, 4096, 64, 2, 0.8, rounds=2, next_locals=_next(3, 10), cols=cols,
                         fused=True, what="bf16 tiles")


def test_adversarial_chunks():
    chunk, k = 4096, 64
    rng = np.random.default_rng(99)
    cases = [np.full(chunk, 0.125, f32), np.zeros(chunk, f32), np.where(rng.random(chunk) < 0.5, f32(1.0), f32(-0.5)).astype(f32),
             (np.round(rng.normal(0, 3, chunk)) * 2.0 ** -7).astype(f32), np.arange(chunk, dtype=f32) / 64]
    ep = np.concatenate(cases)
    n = ep.size
    tg = to_bf16_bits(np.zeros(n, f32))
    tls = [to_bf16_bits(-ep), to_bf16_bits(np.roll(-ep, chunk))]
    errs = [np.zeros(n, f32), np.zeros(n, f32)]
    run_and_compare_bf16([0, n], tg, tls, errs, 0.0, chunk, k, 2, 1.0, what="bf16 adversarial")


def test_1b_sub_arena_with_the_benchmark_value_law_three_rounds():
    full = synth.workload("1b").replace(R=4)
    wl = synth.sub_arena(full, [0, 4, 6, 7, 8])          # q, gate, down, two norm vectors
    rho = synth.row_scales(wl)
    tg = to_bf16_bits(synth.gen_theta_global(wl).numpy())
    draw = lambda t, tgb: [to_bf16_bits(synth.gen_theta_local(wl, torch.from_numpy(slo.widen_bf16(tgb)), t, r, rho=rho).numpy())
                           for r in range(wl.R)]
    errs = [np.zeros(wl.n_total, f32) for _ in range(wl.R)]
    run_and_compare_bf16(wl.offsets(), tg, draw(0, tg), errs, wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr, rounds=3,
                         next_locals=draw, what="bf16 1b sub-arena")


def test_outer_apply_bf16_alone():
    rng = np.random.default_rng(5)
    for n, shift in [(1, 0), (5, 1), (4099, 3), (1 << 20, 0)]:
        th = to_bf16_bits(rng.normal(0, 1, n + 4))
        up = rng.normal(0, 1e-2, n + 4).astype(f32)
        d_th, d_up = dev_bf16(th), torch.from_numpy(up).cuda()
        api.sl_outer_apply_bf16(d_th[shift:], d_up[shift:], n, 0.8)
        want = th.copy()
        w = want[shift:shift + n].copy()
        slo.outer_apply_bf16(w, up[shift:shift + n].copy(), 0.8)
        want[shift:shift + n] = w
        assert_exact(host_bits(d_th), want, f"outer_apply_bf16 n={n}")


def test_nonfinite_parameters_keep_their_kind():
    n = 2 * 4096
    tg, tls, errs = _case(n, 2, seed=12)
    tls[0][17] = 0x7F80            # +inf
    tls[1][4096 + 5] = 0x7FC1      # a NaN
    d_tg, _ = run_and_compare_bf16([0, n], tg, tls, errs, 0.95, 4096, 64, 2, 1.0, what="bf16 nonfinite")
    out = host_bits(d_tg)
    assert (out[17] & 0x7FFF) >= 0x7F80 and (out[4096 + 5] & 0x7F80) == 0x7F80 and (out[4096 + 5] & 0x7F) != 0
