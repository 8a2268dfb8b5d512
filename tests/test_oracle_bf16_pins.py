"""Pins of the checker's bfloat16 storage mode (parameters held as bfloat16, error buffers float32).

The paper states no storage precision for Eq. 2 (section 2.1), so WHERE the parameters are rounded is
a reading of this build (bfloat16 arrays for the parameters, the pseudo-gradient formed in float32 from the widened
values, the float32 step rounded once more, to nearest-even, when it is stored); what is pinned here is that the checker does exactly that
reading: exact widening, round-to-nearest-even on storage, the float32 step in between."""
import json
import os

import numpy as np
import torch

from oracle import slo

f32 = np.float32
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _bf16_bits(x):
    """float32 array of bfloat16-exact values -> their uint16 patterns."""
    x = np.ascontiguousarray(x, dtype=f32)
    b = x.view(np.uint32)
    assert np.all((b & 0xFFFF) == 0), "not a bfloat16 value"
    return (b >> 16).astype(np.uint16)


def test_widening_is_exact_for_every_pattern():
    allp = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    w = slo.widen_bf16(allp)
    assert np.array_equal(w.view(np.uint32), allp.astype(np.uint32) << 16)


def test_rounding_hand_worked_cases():
    # 1 + 2^-8 lies half way between 1 and 1 + 2^-7: the tie goes to the even pattern 0x3F80
    assert slo.round_bf16(1.0 + 2.0 ** -8) == 0x3F80
    # 1 + 3 * 2^-8 lies half way between 0x3F81 and 0x3F82: the tie goes to the even 0x3F82
    assert slo.round_bf16(1.0 + 3 * 2.0 ** -8) == 0x3F82
    assert slo.round_bf16(1.0 + 2.0 ** -8 + 2.0 ** -20) == 0x3F81       # just above the tie: up
    assert slo.round_bf16(1.0 + 2.0 ** -8 - 2.0 ** -20) == 0x3F80       # just below: down
    assert slo.round_bf16(-(1.0 + 2.0 ** -8 + 2.0 ** -20)) == 0xBF81    # sign-magnitude: symmetric
    assert slo.round_bf16(0.0) == 0x0000 and slo.round_bf16(-0.0) == 0x8000
    assert slo.round_bf16(float(np.finfo(np.float32).max)) == 0x7F80     # above half way past the largest bfloat16: infinity
    assert slo.round_bf16(float(np.float32(3.3895e38))) == 0x7F7F       # the largest bfloat16 itself stays
    assert slo.round_bf16(float("inf")) == 0x7F80 and slo.round_bf16(float("-inf")) == 0xFF80
    nan = slo.round_bf16(float("nan"))
    assert (nan & 0x7F80) == 0x7F80 and (nan & 0x007F) != 0             # still a NaN
    assert slo.round_bf16(float(np.float32(2.0 ** -133))) == 0x0001     # subnormals are kept
    assert slo.round_bf16(float(np.float32(2.0 ** -134))) == 0x0000     # half of the smallest: tie to even = 0


def test_rounding_agrees_with_a_library_conversion():
    # torch's float32 -> bfloat16 conversion is round-to-nearest-even: an independent routine
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000).astype(f32) * f32(10.0) ** rng.integers(-30, 30, 20000),
                        (rng.integers(0, 1 << 32, 20000, dtype=np.uint64).astype(np.uint32)).view(f32)]).astype(f32)
    x = x[np.isfinite(x)]
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([slo.round_bf16(float(v)) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want)


def test_hand_worked_example_is_unchanged_by_bfloat16_storage():
    # every parameter of the hand-worked example is a bfloat16 value and so is every result: the
    # bfloat16 mode must reproduce it value for value
    g = json.load(open(os.path.join(GOLD, "w1_dyadic.json")))
    tg = _bf16_bits(g["theta_global"])
    tls = [_bf16_bits(r["theta_local"]) for r in g["replicas"]]
    errs = [np.array(r["err_in"], f32) for r in g["replicas"]]
    msgs, upd, flags = slo.outer_round_bf16(tls, tg, errs, [0, 8], g["beta"], g["chunk"], g["k"], g["bits"], g["outer_lr"])
    for r, rep in enumerate(g["replicas"]):
        assert msgs[r][0].tolist() == [rep["idx"]] and msgs[r][1].tolist() == [rep["packed"]]
        assert msgs[r][2].tolist() == [rep["scale"]] and errs[r].tolist() == rep["err_out"]
    assert upd.tolist() == g["update"]
    assert slo.widen_bf16(tg).tolist() == g["theta_global_out"] and flags == 0


def test_step_is_the_float32_step_followed_by_one_rounding():
    rng = np.random.default_rng(1)
    n = 5000
    tg32 = rng.normal(0, 0.02, n).astype(f32)
    tg = torch.from_numpy(tg32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16).copy()
    upd = rng.normal(0, 1e-3, n).astype(f32)
    th = slo.widen_bf16(tg)
    want32 = th.copy()
    slo.outer_apply(want32, upd, 0.8)                     # the float32 step of the pinned checker
    want = torch.from_numpy(want32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    slo.outer_apply_bf16(tg, upd, 0.8)
    assert np.array_equal(tg, want)
    # an update far below half a bfloat16 unit of the parameter leaves it where it is (what bfloat16
    # storage costs: the step is lost, the error buffers are not involved)
    one = _bf16_bits(np.ones(4, f32))
    slo.outer_apply_bf16(one, np.full(4, 2.0 ** -10, f32), 1.0)
    assert one.tolist() == [0x3F80] * 4


def test_k_equal_chunk_without_quantisation_is_rounded_local_sgd_averaging():
    # k = chunk, bits = 32, e = 0, beta = 0: everything is sent; with dyadic parameters every float32
    # operation is exact, so the result is the bfloat16 rounding of theta - mean_r(theta - theta_r)
    rng = np.random.default_rng(2)
    n, R, chunk = 64, 4, 16
    tg_v = (rng.integers(-64, 65, n) / 64.0).astype(f32)
    tl_v = [(tg_v + rng.integers(-8, 9, n) / 1024.0).astype(f32) for _ in range(R)]
    q = lambda v: torch.from_numpy(v).to(torch.bfloat16)
    tg = q(tg_v).view(torch.int16).numpy().view(np.uint16).copy()
    tls = [q(v).view(torch.int16).numpy().view(np.uint16).copy() for v in tl_v]
    errs = [np.zeros(n, f32) for _ in range(R)]
    th = slo.widen_bf16(tg).astype(np.float64)
    mean = np.mean([th - slo.widen_bf16(t).astype(np.float64) for t in tls], axis=0)
    slo.outer_round_bf16(tls, tg, errs, [0, n], 0.0, chunk, chunk, 32, 1.0)
    want = torch.from_numpy((th - mean).astype(f32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal((th - mean).astype(f32).astype(np.float64), th - mean)      # the float32 step was exact
    assert np.array_equal(tg, want)
    assert all(not e.any() for e in errs)


def test_error_feedback_is_conserved_in_float32():
    # Eq. 2 lines 2 + 4 with the pseudo-gradient formed from the widened parameters: off the kept set
    # e_new is bit-equal to fma(beta, e, delta); on it e_new + sent = e' within one unit in the last place
    rng = np.random.default_rng(3)
    n, chunk, k, bits, beta = 4096 * 2 + 100, 4096, 64, 2, 0.95
    to_bits = lambda v: torch.from_numpy(v.astype(f32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16).copy()
    tg, tl = to_bits(rng.normal(0, 0.02, n)), None
    tl = to_bits(slo.widen_bf16(tg) + rng.normal(0, 1e-3, n))
    e0 = rng.normal(0, 5e-4, n).astype(f32)
    e = e0.copy()
    slo.outer_round_bf16([tl], tg.copy(), [e], [0, n], beta, chunk, k, bits, 1.0)
    delta = slo.widen_bf16(tg) - slo.widen_bf16(tl)            # float32 subtraction of the widened values
    ep = (np.float64(f32(beta)) * e0.astype(np.float64) + delta.astype(np.float64)).astype(f32)   # one rounding = fma
    same = e == ep
    assert same.sum() == n - (2 * k + 64)                        # all but the kept positions (the short chunk keeps 64)
    sent = ep[~same].astype(np.float64) - e[~same]
    assert np.all(np.abs(sent) > 0)
