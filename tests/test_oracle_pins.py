"""Pins of the CPU checker against what the paper and the mathematics fix (Eq. 2, §2.1).

None of these retype the checker's formulas: they use a hand-worked example,
numpy library routines as independent brute force, closed forms on dyadic
inputs, invariants and special cases that reduce to textbook averaging.
"""
import json
import os

import numpy as np
import pytest

from oracle import slo
from paper_2601_02360_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
f32 = np.float32


def _rand_case(n, seed, scale=1e-3, err_scale=5e-4):
    rng = np.random.default_rng(seed)
    tg = rng.normal(0, 0.02, n).astype(f32)
    tl = (tg + rng.normal(0, scale, n).astype(f32)).astype(f32)
    e = rng.normal(0, err_scale, n).astype(f32)
    return tg, tl, e


def _unpack(codes_row, k, bits):
    """LSB-first unpacking written independently of the checker (numpy unpackbits)."""
    if bits == 32:
        return codes_row.view(f32)[:k]
    b = np.unpackbits(codes_row, bitorder="little")[: k * bits].reshape(k, bits)
    return (b.astype(np.uint32) << np.arange(bits, dtype=np.uint32)).sum(axis=1)


# ---------------------------------------------------------------- hand-worked example
def test_w1_hand_worked_example():
    g = json.load(open(os.path.join(GOLD, "w1_dyadic.json")))
    tg = np.array(g["theta_global"], f32)
    off = [0, 8]
    msgs = []
    for rep in g["replicas"]:
        e = np.array(rep["err_in"], f32)
        tl = np.array(rep["theta_local"], f32)
        idx, codes, scales, flags = slo.compress(tl, tg, e, off, g["beta"], g["chunk"], g["k"], g["bits"])
        assert flags == 0
        assert idx.tolist() == [rep["idx"]]
        assert codes.tolist() == [rep["packed"]]
        assert scales.tolist() == [rep["scale"]]
        assert e.tolist() == rep["err_out"]
        assert not np.signbit(e[6])  # the cancelled residual is +0
        msgs.append((idx, codes, scales))
    upd = slo.aggregate(msgs, off, g["chunk"], g["k"], g["bits"])
    assert upd.tolist() == g["update"]
    slo.outer_apply(tg, upd, g["outer_lr"])
    assert tg.tolist() == g["theta_global_out"]


# ---------------------------------------------------------------- selection (Top-k per chunk)
@pytest.mark.parametrize("n,chunk,k", [(1, 8, 2), (7, 8, 3), (64, 64, 64), (512, 4096, 64),
                                       (4096, 4096, 32), (4097, 4096, 64), (3 * 4096 + 100, 4096, 16),
                                       (1000, 128, 5)])
def test_selection_matches_numpy_brute_force(n, chunk, k):
    tg, tl, e0 = _rand_case(n, seed=n + k)
    beta = f32(0.95)
    e = e0.copy()
    idx, codes, scales, _ = slo.compress(tl, tg, e, [0, n], beta, chunk, k, 32)
    # e' recomputed in float64 then rounded once = the fused single rounding
    ep = (np.float64(beta) * e0.astype(np.float64) + (tg - tl).astype(np.float64)).astype(f32)
    nc = (n + chunk - 1) // chunk
    assert idx.shape == (nc, k)
    for c in range(nc):
        seg = ep[c * chunk:(c + 1) * chunk]
        keff = min(k, len(seg))
        key = np.abs(seg)
        order = np.lexsort((np.arange(len(seg)), -key.astype(np.float64)))  # magnitude desc, position asc
        want = np.sort(order[:keff])
        got = idx[c]
        assert got[:keff].tolist() == want.tolist()
        assert (got[keff:] == 0xFFFF).all()
        assert scales[c] == key.max()
        # bits = 32 sends the values verbatim
        assert _unpack(codes[c], keff, 32).tolist() == seg[want].tolist()


def test_selection_ties_lower_position_wins_and_signed_zero():
    n, k = 16, 4
    tg = np.zeros(n, f32)
    # e' = -theta_local: magnitudes 1 at positions 3, 5, 9, 12, 14 (five-way tie for four slots ... plus one 2)
    tl = np.zeros(n, f32)
    tl[[3, 5, 9, 12, 14]] = [1, -1, 1, -1, 1]
    tl[7] = -2
    e = np.zeros(n, f32)
    idx, codes, scales, _ = slo.compress(tl, tg, e, [0, n], 0.0, 16, k, 2)
    assert idx.tolist() == [[3, 5, 7, 9]]
    assert scales[0] == 2.0
    # all-zero chunk with mixed +0 / -0: every key ties, lowest positions win
    tl = np.zeros(n, f32)
    tl[::2] = -0.0
    e = np.zeros(n, f32)
    idx, codes, scales, _ = slo.compress(tl, tg, e, [0, n], 0.0, 16, k, 2)
    assert idx.tolist() == [[0, 1, 2, 3]]
    assert scales[0] == 0.0 and (e == 0).all()


def test_selection_properties_and_density():
    wl = synth.workload("tiny")
    tg = synth.gen_theta_global(wl).numpy()
    tl = synth.gen_theta_local(wl, synth.gen_theta_global(wl), 0, 0).numpy()
    e0 = synth.gen_error(wl, 0).numpy()
    k = 32  # the paper's setting: 32 of 4096 = 0.78 %
    e = e0.copy()
    idx, codes, scales, _ = slo.compress(tl, tg, e, wl.offsets(), 0.95, 4096, k, 2)
    assert idx.shape[0] == wl.n_chunks() == 65
    used = idx != 0xFFFF
    assert used.sum() == 64 * 32 + 32  # 64 full chunks + the 512-element bias keeps min(k, 512)
    assert abs(used[:64].sum() / (64 * 4096) - 0.0078125) < 1e-12
    ep = (np.float64(f32(0.95)) * e0.astype(np.float64) + (tg - tl).astype(np.float64)).astype(f32)
    off = wl.offsets()
    for c in range(65):
        lo = c * 4096 if c < 64 else int(off[1])
        ln = 4096 if c < 64 else 512
        row = idx[c].astype(np.int64)
        assert (np.diff(row) > 0).all() and row.max() < ln
        key = np.abs(ep[lo:lo + ln])
        kept = np.zeros(ln, bool)
        kept[row] = True
        kmin = key[kept].min()
        assert (key[~kept] <= kmin).all()
        # where a dropped element ties the smallest kept key, it sits after every kept one of that key
        tied_out = np.flatnonzero(~kept & (key == kmin))
        tied_in = np.flatnonzero(kept & (key == kmin))
        if len(tied_out):
            assert tied_out.min() > tied_in.max()


def test_chunks_do_not_straddle_tensors_and_are_independent():
    sizes = [4096 + 512, 100, 8192]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    n = int(off[-1])
    tg, tl, e0 = _rand_case(n, 5)
    e = e0.copy()
    idx, codes, scales, _ = slo.compress(tl, tg, e, off, 0.9, 4096, 64, 4)
    assert idx.shape[0] == 2 + 1 + 2
    # compressing each chunk alone gives the same rows
    bounds = [(0, 4096), (4096, 4608), (4608, 4708), (4708, 4708 + 4096), (4708 + 4096, n)]
    for g, (lo, hi) in enumerate(bounds):
        ee = e0[lo:hi].copy()
        i1, c1, s1, _ = slo.compress(tl[lo:hi].copy(), tg[lo:hi].copy(), ee, [0, hi - lo], 0.9, 4096, 64, 4)
        assert (i1[0] == idx[g]).all() and (c1[0] == codes[g]).all() and s1[0] == scales[g]
        assert (ee == e[lo:hi]).all()


# ---------------------------------------------------------------- error feedback and residual
@pytest.mark.parametrize("bits", [2, 4, 8, 32])
def test_conservation_of_the_error_buffer(bits):
    n, chunk, k = 3 * 4096 + 77 * 4, 4096, 64
    tg, tl, e0 = _rand_case(n, 11)
    beta = f32(0.95)
    e = e0.copy()
    idx, codes, scales, _ = slo.compress(tl, tg, e, [0, n], beta, chunk, k, bits)
    ep = (np.float64(beta) * e0.astype(np.float64) + (tg - tl).astype(np.float64)).astype(f32)
    sent = np.zeros(n, np.float64)
    kept = np.zeros(n, bool)
    for c in range(idx.shape[0]):
        row = idx[c][idx[c] != 0xFFFF].astype(np.int64) + c * chunk
        kept[row] = True
        cd = _unpack(codes[c], len(row), bits)
        if bits == 32:
            sent[row] = cd
        else:
            L = 1 << (bits - 1)
            q = cd & (L - 1)
            sg = np.where(cd >> (bits - 1), -1.0, 1.0)
            sent[row] = sg * np.float64(scales[c]) * (2 * q + 1) / (2 * L)
    # untouched positions carry e' bit for bit
    assert (e[~kept].view(np.uint32) == ep[~kept].view(np.uint32)).all()
    # kept positions: e_new + sent = e' up to one rounding of the subtraction
    ulp = np.spacing(np.maximum(np.abs(ep[kept]), np.abs(sent[kept]).astype(f32)))
    assert (np.abs(e[kept].astype(np.float64) + sent[kept] - ep[kept]) <= ulp).all()
    if bits == 32:
        assert (e[kept] == 0).all() and not np.signbit(e[kept]).any()


def test_beta_one_telescopes_over_rounds():
    # with beta = 1 the buffer plus everything sent equals the sum of all pseudo-gradients
    n, chunk, k = 4096, 4096, 64
    rng = np.random.default_rng(3)
    tg = rng.normal(0, 0.02, n).astype(f32)
    e = np.zeros(n, f32)
    total_delta = np.zeros(n, np.float64)
    total_sent = np.zeros(n, np.float64)
    for t in range(6):
        tl = (tg + rng.normal(0, 1e-3, n).astype(f32)).astype(f32)
        total_delta += (tg - tl).astype(np.float64)
        idx, codes, scales, _ = slo.compress(tl, tg, e, [0, n], 1.0, chunk, k, 32)
        vals = codes.view(f32)
        np.add.at(total_sent, idx[0].astype(np.int64), vals[0].astype(np.float64))
    assert np.abs(e.astype(np.float64) + total_sent - total_delta).max() < 6 * 2.0 ** -24 * 0.02


# ---------------------------------------------------------------- quantiser (implementation of the chosen Q)
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_quantiser_closed_form_on_dyadic_levels(bits):
    # scale 1: thresholds are j/L exactly; value (j + 1/2)/L sits in level j and is its own reconstruction
    L = 1 << (bits - 1)
    for j in range(L):
        v = (j + 0.5) / L
        for sign in (1.0, -1.0):
            code = slo.quantise(sign * v, 1.0, bits)
            assert code == ((L if sign < 0 else 0) | j)
            assert slo.dequantise(code, 1.0, bits) == sign * v
        # a value exactly on a threshold belongs to the upper level
        assert slo.quantise(j / L, 1.0, bits) & (L - 1) == j
        if j:
            assert slo.quantise(np.nextafter(f32(j / L), f32(0)), 1.0, bits) & (L - 1) == j - 1
    assert slo.quantise(1.0, 1.0, bits) & (L - 1) == L - 1  # the chunk maximum takes the top level
    assert slo.quantise(-0.0, 1.0, bits) == L  # raw sign bit, level 0


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_quantiser_error_bound_monotone_and_sign(bits):
    n, chunk, k = 4 * 4096, 4096, 128
    tg, tl, e0 = _rand_case(n, 21)
    e = e0.copy()
    idx, codes, scales, _ = slo.compress(tl, tg, e, [0, n], 0.95, chunk, k, bits)
    ep = (np.float64(f32(0.95)) * e0.astype(np.float64) + (tg - tl).astype(np.float64)).astype(f32)
    L = 1 << (bits - 1)
    for c in range(4):
        row = idx[c].astype(np.int64)
        v = ep[c * chunk + row]
        cd = _unpack(codes[c], k, bits)
        q = cd & (L - 1)
        assert (cd < (1 << bits)).all()
        assert ((cd >> (bits - 1)) == np.signbit(v)).all()
        order = np.argsort(np.abs(v), kind="stable")
        assert (np.diff(q[order].astype(np.int64)) >= 0).all()
        assert q[np.argmax(np.abs(v))] == L - 1
        s = np.float64(scales[c])
        rec = np.where(np.signbit(v), -1.0, 1.0) * s * (2 * q + 1) / (2 * L)
        assert (np.abs(rec) <= s).all()
        assert (np.abs(v - rec) <= s / (2 * L) * (1 + 1e-6)).all()
        # the residual the checker wrote is e' minus that reconstruction, rounded to float
        want = (v.astype(np.float64) - rec.astype(f32).astype(np.float64)).astype(f32)
        assert (e[c * chunk + row] == want).all()


def test_quantiser_refines_with_bits():
    n, chunk, k = 4096, 4096, 64
    tg, tl, e0 = _rand_case(n, 8)
    worst = []
    for bits in (2, 4, 8, 32):
        e = e0.copy()
        slo.compress(tl, tg, e, [0, n], 0.95, chunk, k, bits)
        ep = (np.float64(f32(0.95)) * e0.astype(np.float64) + (tg - tl).astype(np.float64)).astype(f32)
        changed = e != ep
        worst.append(np.abs(e[changed]).max() if changed.any() else 0.0)
    assert worst[0] > worst[1] > worst[2] > worst[3] == 0.0


# ---------------------------------------------------------------- metamorphic
@pytest.mark.parametrize("p", [-20, 7])
def test_power_of_two_scaling(p):
    n, chunk, k = 2 * 4096 + 512, 4096, 64
    tg, tl, e0 = _rand_case(n, 4)
    s = f32(2.0 ** p)
    e1, e2 = e0.copy(), (e0 * s).astype(f32)
    i1, c1, s1, _ = slo.compress(tl, tg, e1, [0, n], 0.95, chunk, k, 2)
    i2, c2, s2, _ = slo.compress((tl * s).astype(f32), (tg * s).astype(f32), e2, [0, n], 0.95, chunk, k, 2)
    assert (i1 == i2).all() and (c1 == c2).all()
    assert (s2 == s1 * s).all() and (e2 == e1 * s).all()


def test_sign_symmetry():
    n, chunk, k = 4096 + 256, 4096, 64
    tg, tl, e0 = _rand_case(n, 6)
    e1, e2 = e0.copy(), (-e0).copy()
    i1, c1, s1, _ = slo.compress(tl, tg, e1, [0, n], 0.95, chunk, k, 2)
    i2, c2, s2, _ = slo.compress(tg, tl, e2, [0, n], 0.95, chunk, k, 2)  # swapped: delta negated
    assert (i1 == i2).all() and (s1 == s2).all() and (e2 == -e1).all()
    for c in range(2):
        a, b = _unpack(c1[c], k, 2), _unpack(c2[c], k, 2)
        assert ((a & 1) == (b & 1)).all() and ((a >> 1) != (b >> 1)).all()


def test_chunk_permutation_permutes_messages():
    chunk, k, nc = 256, 8, 6
    n = chunk * nc
    tg, tl, e0 = _rand_case(n, 9)
    perm = np.random.default_rng(1).permutation(nc)
    P = (perm[:, None] * chunk + np.arange(chunk)[None, :]).ravel()
    e1, e2 = e0.copy(), e0[P].copy()
    i1, c1, s1, _ = slo.compress(tl, tg, e1, [0, n], 0.95, chunk, k, 4)
    i2, c2, s2, _ = slo.compress(tl[P].copy(), tg[P].copy(), e2, [0, n], 0.95, chunk, k, 4)
    assert (i2 == i1[perm]).all() and (c2 == c1[perm]).all() and (s2 == s1[perm]).all()
    assert (e2 == e1[P]).all()


# ---------------------------------------------------------------- aggregate and outer update
def _messages(R, n, chunk, k, bits, seed):
    msgs, eps = [], []
    rng = np.random.default_rng(seed)
    tg = rng.normal(0, 0.02, n).astype(f32)
    for r in range(R):
        tl = (tg + rng.normal(0, 1e-3, n).astype(f32)).astype(f32)
        e = np.zeros(n, f32)
        i, c, s, _ = slo.compress(tl, tg, e, [0, n], 0.0, chunk, k, bits)
        msgs.append((i, c, s))
        eps.append(((tg - tl).astype(f32), e))
    return tg, msgs, eps


def test_aggregate_brute_force_and_fixed_divisor():
    R, n, chunk, k = 3, 2 * 512 + 64, 512, 16
    tg, msgs, eps = _messages(R, n, chunk, k, 32, 2)
    upd = slo.aggregate(msgs, [0, n], chunk, k, 32)
    dense = np.zeros((R, n), f32)
    for r, (i, c, s) in enumerate(msgs):
        for g in range(i.shape[0]):
            row = i[g][i[g] != 0xFFFF].astype(np.int64)
            dense[r, g * chunk + row] = c[g].view(f32)[: len(row)]
    acc = np.zeros(n, f32)
    for r in range(R):
        acc = (acc + dense[r]).astype(f32)
    assert (upd == (acc / f32(R)).astype(f32)).all()
    hit = (dense != 0).sum(axis=0)
    once = hit == 1
    assert once.any()
    # a position sent by one replica only is still divided by R, not by the hit count
    assert (upd[once] == (dense.sum(axis=0)[once] / f32(R)).astype(f32)).all()
    assert (upd[hit == 0] == 0).all() and not np.signbit(upd[hit == 0]).any()


def test_aggregate_single_and_identical_replicas():
    n, chunk, k = 4096 + 128, 4096, 64
    tg, msgs, eps = _messages(1, n, chunk, k, 2, 7)
    one = slo.aggregate(msgs, [0, n], chunk, k, 2)
    delta, e = eps[0]
    assert (one == (delta - e).astype(f32)).all()  # R = 1: the update is exactly what was sent
    four = slo.aggregate(msgs * 4, [0, n], chunk, k, 2)
    assert (four == one).all()  # identical messages, power-of-two R: the mean is exact


def test_dense_special_case_is_plain_local_sgd_averaging():
    # k = chunk, no quantisation, empty buffers: Eq. 2 collapses to DiLoCo's average of the
    # pseudo-gradients followed by an SGD outer step
    R, n, chunk = 4, 3 * 256 + 64, 256
    rng = np.random.default_rng(12)
    tg0 = rng.normal(0, 0.02, n).astype(f32)
    tls = [(tg0 + rng.normal(0, 1e-3, n).astype(f32)).astype(f32) for _ in range(R)]
    errs = [np.zeros(n, f32) for _ in range(R)]
    tg = tg0.copy()
    msgs, upd, _ = slo.outer_round(tls, tg, errs, [0, n], 0.95, chunk, chunk, 32, 0.8)
    assert all((e == 0).all() for e in errs)
    deltas = np.stack([(tg0 - tl) for tl in tls]).astype(np.float64)
    want = tg0.astype(np.float64) - 0.8 * deltas.mean(axis=0)
    assert np.abs(tg - want).max() <= 2.0 ** -23 * np.abs(want).max()
    # one replica, unit outer rate: the global parameters become the local ones exactly
    # (theta_global - theta_local is exact by Sterbenz wherever the two are within a factor 2)
    tg = tg0.copy()
    slo.outer_round(tls[:1], tg, [np.zeros(n, f32)], [0, n], 0.0, chunk, chunk, 32, 1.0)
    close = (np.abs(tls[0]) <= 2 * np.abs(tg0)) & (np.abs(tg0) <= 2 * np.abs(tls[0])) & (tls[0] * tg0 > 0)
    assert close.sum() > n // 2 and (tg[close] == tls[0][close]).all()
    assert np.abs(tg - tls[0]).max() <= 2.0 ** -23 * 0.2


def test_dense_error_feedback_averaging_with_beta():
    # k = chunk with a non-empty buffer: everything (beta e + delta) is sent, the buffer empties
    R, n, chunk = 2, 512, 128
    rng = np.random.default_rng(13)
    tg0 = rng.normal(0, 0.02, n).astype(f32)
    tls = [(tg0 + rng.normal(0, 1e-3, n).astype(f32)).astype(f32) for _ in range(R)]
    e0 = [rng.normal(0, 5e-4, n).astype(f32) for _ in range(R)]
    errs = [e.copy() for e in e0]
    tg = tg0.copy()
    slo.outer_round(tls, tg, errs, [0, n], 0.5, chunk, chunk, 32, 1.0)
    assert all((e == 0).all() for e in errs)
    mean = np.mean([0.5 * e.astype(np.float64) + (tg0 - tl).astype(np.float64) for e, tl in zip(e0, tls)], axis=0)
    assert np.abs(tg - (tg0 - mean)).max() <= 2.0 ** -22 * 0.1


def test_outer_apply_is_sgd_without_momentum():
    rng = np.random.default_rng(1)
    th = rng.normal(0, 1, 1000).astype(f32)
    u = rng.normal(0, 1, 1000).astype(f32)
    a = th.copy()
    slo.outer_apply(a, u, 0.8)
    want = (th.astype(np.float64) - np.float64(f32(0.8)) * u.astype(np.float64)).astype(f32)
    assert (a == want).all()
    b = a.copy()
    slo.outer_apply(b, np.zeros(1000, f32), 0.8)  # zero update: no hidden state, nothing moves
    assert (a.view(np.uint32) == b.view(np.uint32)).all()


# ---------------------------------------------------------------- state and edge cases
def test_checkpoint_resume_is_bit_identical():
    wl = synth.workload("tiny").replace(R=2)
    off = wl.offsets()
    def run(rounds, state=None):
        if state is None:
            tg = synth.gen_theta_global(wl).numpy().copy()
            errs = [np.zeros(wl.n_total, f32) for _ in range(wl.R)]
            t0 = 0
        else:
            tg, errs, t0 = state[0].copy(), [e.copy() for e in state[1]], state[2]
        for t in range(t0, t0 + rounds):
            import torch
            tgt = torch.from_numpy(tg)
            tls = [synth.gen_theta_local(wl, tgt, t, r).numpy() for r in range(wl.R)]
            slo.outer_round(tls, tg, errs, off, wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr)
        return tg, errs, t0 + rounds
    a = run(4)
    b = run(2, run(2))
    assert (a[0].view(np.uint32) == b[0].view(np.uint32)).all()
    assert all((x.view(np.uint32) == y.view(np.uint32)).all() for x, y in zip(a[1], b[1]))


def test_nonfinite_inputs_raise_the_flag_and_order_by_bit_pattern():
    n = 16
    tg = np.zeros(n, f32)
    tl = np.arange(n, dtype=f32)
    tl[4] = np.inf
    tl[9] = np.nan
    e = np.zeros(n, f32)
    idx, codes, scales, flags = slo.compress(tl, tg, e, [0, n], 0.0, 16, 3, 32)
    assert flags & slo.FLAG_NONFINITE
    assert idx.tolist() == [[4, 9, 15]]  # NaN above Inf above every finite value
    assert np.isnan(scales[0])
    e = np.zeros(n, f32)
    _, _, _, flags = slo.compress(np.arange(n, dtype=f32), tg, e, [0, n], 0.0, 16, 3, 32)
    assert flags == 0


def test_subnormal_values_are_kept_not_flushed():
    n = 8
    tiny = f32(2.0 ** -140)
    tg = np.zeros(n, f32)
    tl = np.zeros(n, f32)
    tl[3] = -tiny * 3
    tl[5] = tiny
    e = np.zeros(n, f32)
    idx, codes, scales, _ = slo.compress(tl, tg, e, [0, n], 0.0, 8, 2, 32)
    assert idx.tolist() == [[3, 5]] and scales[0] == tiny * 3
    assert codes.view(f32).tolist() == [[tiny * 3, -tiny]]


def test_argument_checks():
    z = np.zeros(8, f32)
    for chunk, k, bits in [(0, 1, 2), (8, 0, 2), (8, 9, 2), (8, 2, 3), (70000, 2, 2)]:
        with pytest.raises(ValueError):
            slo.compress(z, z, z.copy(), [0, 8], 0.9, chunk, k, bits)
