"""CPU checker of the token-embedding adaptation of §2.4 (test infrastructure, never the product path).

The embedding table is split as TE = T_S + T_perp, with T_S meant to lie in the
row space S = Col(U) of a fixed matrix U (d x k, orthonormal columns, §2.3).
The projection of a row vector t onto S is  Pi_S(t) = t U U^T.

  * before training (§2.4, first modification):  T_S <- TE U U^T,  T_perp <- TE - T_S
  * after every outer synchronisation (Eqs. 3-4):
        T_perp <- T_perp + (T_S - Pi_S(T_S))
        T_S    <- Pi_S(T_S)

Everything is the definition written out with numpy in float64: two matrix
products and two element-wise updates, no blocking and no reordering.  Inputs
may be float32 arrays; they are widened first and the results stay float64, so
that a float32/TF32 implementation is compared with the exact value.

Pinned by tests/test_oracle_embed_pins.py: a hand-worked example, the closed
form for U = columns of the identity, idempotence, TE conservation, the residual
being orthogonal to S, a row already in S staying put, and a loop-by-loop
restatement on tiny inputs.
"""
from __future__ import annotations

from typing import Tuple

import numpy as np


def project(T: np.ndarray, U: np.ndarray) -> np.ndarray:
    """Pi_S(T) = (T U) U^T for every row of T (§2.4; U is d x k with orthonormal columns)."""
    T = np.asarray(T, dtype=np.float64)
    U = np.asarray(U, dtype=np.float64)
    assert T.ndim == 2 and U.ndim == 2 and T.shape[1] == U.shape[0]
    P = T @ U            # V x k : coordinates of each row in the basis U
    return P @ U.T       # V x d


def embed_init(TE: np.ndarray, U: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """§2.4, before training: T_S = TE U U^T and T_perp = TE - T_S."""
    TE = np.asarray(TE, dtype=np.float64)
    T_S = project(TE, U)
    return T_S, TE - T_S


def embed_reproject(T_S: np.ndarray, T_perp: np.ndarray, U: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Eqs. 3-4: returns (T_S', T_perp') with T_perp' = T_perp + (T_S - Pi_S(T_S)), T_S' = Pi_S(T_S)."""
    T_S = np.asarray(T_S, dtype=np.float64)
    T_perp = np.asarray(T_perp, dtype=np.float64)
    assert T_S.shape == T_perp.shape
    Pi = project(T_S, U)
    return Pi, T_perp + (T_S - Pi)


def abs_bound(T_S: np.ndarray, U: np.ndarray) -> np.ndarray:
    """B[v, n] = sum_j (sum_i |T_S[v, i]| |U[i, j]|) |U[n, j]|: the sum of the magnitudes of every
    product that enters Pi_S(T_S)[v, n].  A rounding error of relative size eps on each operand
    of each product moves the result by at most a small multiple of eps * B."""
    A = np.abs(np.asarray(T_S, dtype=np.float64))
    W = np.abs(np.asarray(U, dtype=np.float64))
    return (A @ W) @ W.T
