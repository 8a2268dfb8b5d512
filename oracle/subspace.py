"""CPU checker of the subspace compression of stage-boundary activations (paper §2.3; test
infrastructure only, never the product path).

Activations X (n_tok x d; tokens of a batch laid out sequence after sequence, so token t sits at
position t mod L), token ids x (n_tok), the fixed high-rank embedding part T_perp (V x d), the
positional embedding Pos (L x d) and the orthonormal basis U (d x k):

    compress     Xt   = (X - T_perp[x] - Pos) U            (§2.3, first display: n_tok x k travel)
    reconstruct  Xhat = Xt U^T + T_perp[x] + Pos           (§2.3, second display)
    gradients    Gt   = G U                                (§2.3, third display: no embedding terms)

Each is the definition written out with numpy in float64 (a gather, an element-wise difference or
sum, one matrix product); inputs may be float32 and are widened first.  Pinned by
tests/test_oracle_subspace_pins.py.
"""
from __future__ import annotations

from typing import Optional

import numpy as np


def _rows(n_tok: int, L: int) -> np.ndarray:
    return np.arange(n_tok) % L


def project(X, ids: Optional[np.ndarray], T_perp, pos, U, L: int) -> np.ndarray:
    """Xt = (X - T_perp[ids] - pos[t mod L]) U; with ids None (gradients) Xt = X U."""
    X = np.asarray(X, dtype=np.float64)
    U = np.asarray(U, dtype=np.float64)
    if ids is not None:
        X = X - np.asarray(T_perp, dtype=np.float64)[np.asarray(ids)] - np.asarray(pos, dtype=np.float64)[_rows(len(X), L)]
    return X @ U


def reconstruct(Xt, ids: np.ndarray, T_perp, pos, U, L: int) -> np.ndarray:
    """Xhat = Xt U^T + T_perp[ids] + pos[t mod L]."""
    Xt = np.asarray(Xt, dtype=np.float64)
    U = np.asarray(U, dtype=np.float64)
    return Xt @ U.T + np.asarray(T_perp, dtype=np.float64)[np.asarray(ids)] + np.asarray(pos, dtype=np.float64)[_rows(len(Xt), L)]


def abs_bound_project(X, ids, T_perp, pos, U, L: int) -> np.ndarray:
    """Sum of the magnitudes of the products entering every output of `project` (the quantity a
    relative rounding error of the operands scales with)."""
    A = np.asarray(X, dtype=np.float64)
    if ids is not None:
        A = A - np.asarray(T_perp, dtype=np.float64)[np.asarray(ids)] - np.asarray(pos, dtype=np.float64)[_rows(len(A), L)]
    return np.abs(A) @ np.abs(np.asarray(U, dtype=np.float64))


def abs_bound_reconstruct(Xt, U) -> np.ndarray:
    return np.abs(np.asarray(Xt, dtype=np.float64)) @ np.abs(np.asarray(U, dtype=np.float64)).T
