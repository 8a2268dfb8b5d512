"""Pins of the CPU checker of the embedding adaptation (paper §2.4, Eqs. 3-4) against facts that do
not come from the checker itself: a hand-worked example, closed forms, invariants, brute force."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import embed as oe

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "embed_reproject_hand.json")


def _frac(rows):
    return np.array([[float(Fraction(x)) for x in r] for r in rows], dtype=np.float64)


def _basis(d, k, seed):
    rng = np.random.default_rng(seed)
    q, _ = np.linalg.qr(rng.standard_normal((d, k)))
    return q


def test_hand_worked_example():
    g = json.load(open(GOLDEN))
    U, T_S, T_perp = _frac(g["U"]), _frac(g["T_S"]), _frac(g["T_perp"])
    ts, tp = oe.embed_reproject(T_S, T_perp, U)
    np.testing.assert_allclose(ts, _frac(g["T_S_new"]), rtol=0, atol=1e-15)
    np.testing.assert_allclose(tp, _frac(g["T_perp_new"]), rtol=0, atol=1e-15)


def test_identity_columns_closed_form():
    # U = columns 1, 4, 2 of the 6 x 6 identity: the projection keeps exactly those coordinates.
    d, cols = 6, [1, 4, 2]
    U = np.zeros((d, len(cols)))
    for j, c in enumerate(cols):
        U[c, j] = 1.0
    rng = np.random.default_rng(0)
    T_S, T_perp = rng.standard_normal((5, d)), rng.standard_normal((5, d))
    keep = np.zeros(d)
    keep[cols] = 1.0
    ts, tp = oe.embed_reproject(T_S, T_perp, U)
    assert np.array_equal(ts, T_S * keep)
    assert np.array_equal(tp, T_perp + T_S * (1.0 - keep))


def test_full_rank_basis_is_identity_map():
    # k = d: S is the whole space, so nothing moves.
    U = _basis(7, 7, 1)
    rng = np.random.default_rng(2)
    T_S, T_perp = rng.standard_normal((4, 7)), rng.standard_normal((4, 7))
    ts, tp = oe.embed_reproject(T_S, T_perp, U)
    np.testing.assert_allclose(ts, T_S, atol=1e-13)
    np.testing.assert_allclose(tp, T_perp, atol=1e-13)


@pytest.mark.parametrize("d,k,V", [(16, 4, 9), (48, 6, 33), (64, 8, 5)])
def test_invariants(d, k, V):
    U = _basis(d, k, 3)
    rng = np.random.default_rng(4)
    T_S, T_perp = rng.standard_normal((V, d)), rng.standard_normal((V, d))
    ts, tp = oe.embed_reproject(T_S, T_perp, U)
    # the table TE = T_S + T_perp is unchanged (what the paper's closing sentence of §2.4 asks for)
    np.testing.assert_allclose(ts + tp, T_S + T_perp, atol=1e-13)
    # the new T_S lies in S: projecting again changes nothing, and T_perp then stays put
    ts2, tp2 = oe.embed_reproject(ts, tp, U)
    np.testing.assert_allclose(ts2, ts, atol=1e-13)
    np.testing.assert_allclose(tp2, tp, atol=1e-13)
    # what was moved into T_perp is orthogonal to S
    np.testing.assert_allclose((tp - T_perp) @ U, 0.0, atol=1e-13)
    # Pythagoras: |t|^2 = |Pi t|^2 + |t - Pi t|^2 row by row
    np.testing.assert_allclose((T_S ** 2).sum(1), (ts ** 2).sum(1) + ((T_S - ts) ** 2).sum(1), rtol=1e-12)


def test_rows_already_in_subspace_do_not_move():
    d, k = 24, 5
    U = _basis(d, k, 5)
    C = np.random.default_rng(6).standard_normal((7, k))
    T_S = C @ U.T
    T_perp = np.random.default_rng(7).standard_normal((7, d))
    ts, tp = oe.embed_reproject(T_S, T_perp, U)
    np.testing.assert_allclose(ts, T_S, atol=1e-13)
    np.testing.assert_allclose(tp, T_perp, atol=1e-13)


def test_against_loops():
    d, k, V = 5, 2, 3
    U = _basis(d, k, 8)
    rng = np.random.default_rng(9)
    T_S, T_perp = rng.standard_normal((V, d)), rng.standard_normal((V, d))
    ts, tp = oe.embed_reproject(T_S, T_perp, U)
    for v in range(V):
        coord = [sum(T_S[v, i] * U[i, j] for i in range(d)) for j in range(k)]
        for n in range(d):
            pi = sum(coord[j] * U[n, j] for j in range(k))
            assert abs(ts[v, n] - pi) < 1e-14
            assert abs(tp[v, n] - (T_perp[v, n] + (T_S[v, n] - pi))) < 1e-14


def test_init_split():
    d, k = 12, 3
    U = _basis(d, k, 10)
    TE = np.random.default_rng(11).standard_normal((6, d))
    T_S, T_perp = oe.embed_init(TE, U)
    np.testing.assert_allclose(T_S + T_perp, TE, atol=1e-14)
    np.testing.assert_allclose(T_perp @ U, 0.0, atol=1e-13)
    np.testing.assert_allclose(oe.project(T_S, U), T_S, atol=1e-13)


def test_float32_inputs_are_widened():
    d, k = 32, 4
    U = _basis(d, k, 12).astype(np.float32)
    T = np.random.default_rng(13).standard_normal((3, d)).astype(np.float32)
    ts, _ = oe.embed_reproject(T, np.zeros_like(T), U)
    assert ts.dtype == np.float64
    np.testing.assert_allclose(ts, (T.astype(np.float64) @ U.astype(np.float64)) @ U.astype(np.float64).T, atol=0)


def test_abs_bound_dominates():
    d, k = 20, 4
    U = _basis(d, k, 14)
    T = np.random.default_rng(15).standard_normal((4, d))
    assert np.all(oe.abs_bound(T, U) >= np.abs(oe.project(T, U)) - 1e-14)
