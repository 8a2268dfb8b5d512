"""Pins of the CPU checker of the activation subspace compression (paper §2.3)."""
import numpy as np
import pytest

from oracle import subspace as osub


def _basis(d, k, seed):
    q, _ = np.linalg.qr(np.random.default_rng(seed).standard_normal((d, k)))
    return q


def _case(n_tok, L, V, d, k, seed):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((n_tok, d)), rng.integers(0, V, n_tok), rng.standard_normal((V, d)),
            rng.standard_normal((L, d)), _basis(d, k, seed + 1))


def test_hand_worked_example():
    # d = 3, k = 2, U columns (1,2,2)/3 and (2,1,-2)/3; L = 2, two sequences of two tokens.
    U = np.array([[1, 2], [2, 1], [2, -2]]) / 3.0
    T_perp = np.array([[0.0, 0, 0], [3, 0, 0]])          # token 1 has a high-rank part (3,0,0)
    pos = np.array([[0.0, 0, 0], [0, 3, 3]])             # position 1 adds (0,3,3)
    ids = np.array([0, 1, 1, 0])
    X = np.array([[3.0, 0, 0],      # token 0, position 0: nothing subtracted -> (3,0,0) U = (1, 2)
                  [3, 3, 3],        # token 1, position 1: minus (3,0,0) minus (0,3,3) -> 0 -> (0, 0)
                  [6, 0, 0],        # token 1, position 0: minus (3,0,0) -> (3,0,0) -> (1, 2)
                  [0, 6, 6]])       # token 0, position 1: minus (0,3,3) -> (0,3,3) -> (4, -1)
    Xt = osub.project(X, ids, T_perp, pos, U, L=2)
    np.testing.assert_allclose(Xt, [[1, 2], [0, 0], [1, 2], [4, -1]], atol=1e-15)
    # reconstruction of those coordinates: 1*u1 + 2*u2 = (5,4,-2)/3, plus what was subtracted
    Xh = osub.reconstruct(Xt, ids, T_perp, pos, U, L=2)
    np.testing.assert_allclose(Xh[0], np.array([5, 4, -2]) / 3.0, atol=1e-15)
    np.testing.assert_allclose(Xh[1], [3, 3, 3], atol=1e-15)
    np.testing.assert_allclose(Xh[2], np.array([5, 4, -2]) / 3.0 + [3, 0, 0], atol=1e-15)
    np.testing.assert_allclose(Xh[3], np.array([2, 7, 10]) / 3.0 + [0, 3, 3], atol=1e-15)


def test_lossless_when_the_residual_lies_in_the_subspace():
    # §2.3: residual activations lie in Col(U), so compress followed by reconstruct gives X back
    n_tok, L, V, d, k = 12, 4, 7, 16, 5
    _, ids, T_perp, pos, U = _case(n_tok, L, V, d, k, 0)
    C = np.random.default_rng(9).standard_normal((n_tok, k))
    X = C @ U.T + T_perp[ids] + pos[np.arange(n_tok) % L]
    Xt = osub.project(X, ids, T_perp, pos, U, L)
    np.testing.assert_allclose(Xt, C, atol=1e-12)
    np.testing.assert_allclose(osub.reconstruct(Xt, ids, T_perp, pos, U, L), X, atol=1e-12)


def test_general_input_loses_exactly_the_out_of_subspace_part():
    n_tok, L, V, d, k = 10, 5, 6, 12, 4
    X, ids, T_perp, pos, U = _case(n_tok, L, V, d, k, 1)
    Xh = osub.reconstruct(osub.project(X, ids, T_perp, pos, U, L), ids, T_perp, pos, U, L)
    R = X - T_perp[ids] - pos[np.arange(n_tok) % L]
    np.testing.assert_allclose(X - Xh, R - (R @ U) @ U.T, atol=1e-12)
    np.testing.assert_allclose((X - Xh) @ U, 0.0, atol=1e-12)          # what is lost is orthogonal to S


def test_identity_columns_closed_form():
    d, cols = 6, [4, 0, 3]
    U = np.zeros((d, 3))
    U[cols, np.arange(3)] = 1.0
    X, ids, T_perp, pos, _ = _case(8, 4, 5, d, 3, 2)
    Xt = osub.project(X, ids, T_perp, pos, U, 4)
    want = (X - T_perp[ids] - pos[np.arange(8) % 4])[:, cols]
    assert np.array_equal(Xt, want)
    Xh = osub.reconstruct(Xt, ids, T_perp, pos, U, 4)
    base = T_perp[ids] + pos[np.arange(8) % 4]
    expect = base.copy()
    expect[:, cols] += want
    np.testing.assert_allclose(Xh, expect, atol=1e-15)


def test_gradients_use_no_embedding_terms():
    G, _, T_perp, pos, U = _case(9, 3, 4, 10, 3, 3)
    np.testing.assert_allclose(osub.project(G, None, T_perp, pos, U, 3), G @ U, atol=0)


def test_positions_follow_the_sequence_layout():
    # token t sits at position t mod L: two sequences get the same positional rows
    X, ids, T_perp, pos, U = _case(6, 3, 4, 8, 2, 4)
    a = osub.project(X, ids, T_perp, pos, U, 3)
    X2 = X.copy()
    X2[3:] += pos[:3] - np.roll(pos, 1, axis=0)[:3]       # what a wrong position table would subtract instead
    assert not np.allclose(osub.project(X2, ids, T_perp, pos, U, 3)[3:], a[3:])
    b = osub.project(X[3:], ids[3:], T_perp, pos, U, 3)   # the second sequence on its own
    np.testing.assert_allclose(a[3:], b, atol=1e-15)


def test_against_loops():
    n_tok, L, V, d, k = 4, 2, 3, 5, 2
    X, ids, T_perp, pos, U = _case(n_tok, L, V, d, k, 5)
    Xt = osub.project(X, ids, T_perp, pos, U, L)
    Xh = osub.reconstruct(Xt, ids, T_perp, pos, U, L)
    for t in range(n_tok):
        for j in range(k):
            s = sum((X[t, i] - T_perp[ids[t], i] - pos[t % L, i]) * U[i, j] for i in range(d))
            assert abs(Xt[t, j] - s) < 1e-13
        for n in range(d):
            s = sum(Xt[t, j] * U[n, j] for j in range(k)) + T_perp[ids[t], n] + pos[t % L, n]
            assert abs(Xh[t, n] - s) < 1e-13
