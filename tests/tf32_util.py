"""Error model of the TF32 contractions (paper sections 2.3 and 2.4 kernels) and the checks built on it.

What the kernels do to a contraction  out[r, n] = sum_i a[r, i] w[i, n]:
  * the float32 operand `a` is rounded to the NEAREST TF32 value (11 significant bits): the error of
    an element is at most half a TF32 unit in the last place, |da| <= 2^-11 |a|, and - being a
    rounding to nearest of data that has nothing to do with the TF32 grid - it behaves like a
    uniform variable on [-ulp/2, ulp/2] with ulp <= 2^-10 |a|: zero mean, standard deviation
    ulp / sqrt(12) <= SIGMA |a| with SIGMA = 2^-11 / sqrt(3), independent between elements;
  * `w` (the basis U) is a TF32 value already when the caller rounded it (then it is exact); as drawn,
    the tensor cores cut it, a one-sided error below 2^-10 |w|;
  * products of two TF32 values are exact in float32; the accumulation is float32 (the tensor
    core adds the eight products of an instruction to the accumulator; whether it rounds or cuts
    the sum, an addition costs at most 2^-23 of the partial sum, d / 8 additions per output).

So, with B = |a| @ |w| (the sum of the magnitudes of the products) and Q = sqrt(a^2 @ w^2) (their sum
in quadrature), and a rounded basis:
  hard bound        |err| <= 2^-11 B  +  (d / 8) 2^-23 B                     always
  statistical bound |err| <= C_STAT * (SIGMA + (d / 8) 2^-23) * Q            C_STAT = 8: a sum of many
                    independent bounded terms has lighter tails than a Gaussian, for which 8 standard
                    deviations are exceeded with probability 1e-15 per entry; the partial sums of the
                    accumulation are of the size of Q as well (below C_STAT * Q), and each of the d / 8
                    additions costs at most 2^-23 of one, whichever way the hardware rounds
  RMS               rms(err) <= SIGMA * rms-like(Q), i.e. about 0.6 * 2^-11 of the RMS of the result for
                    Gaussian data (the average TF32 ulp is about 0.72 of its upper bound 2^-10 |a|).
The hard bound cannot catch a dropped K step at the benchmark's shapes (B is several times the
result's RMS); the statistical bound and the RMS can, and the tests assert that about themselves.
"""
from __future__ import annotations

import numpy as np

SIGMA = 2.0 ** -11 / np.sqrt(3.0)
C_STAT = 8.0
TINY = 1e-30


def tf32_rna(x: np.ndarray) -> np.ndarray:
    """float32 -> nearest TF32 value (10 explicit mantissa bits), ties away from zero: the definition."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    b = ((b + 0x1000) & ~np.uint64(0x1FFF)).astype(np.uint32)        # add half of the cut part, clear it
    return b.view(np.float32)


def is_tf32(x: np.ndarray) -> bool:
    return bool(np.all((np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) & 0x1FFF) == 0))


def accumulation_allowance(B: np.ndarray, depth: int) -> np.ndarray:
    """float32 accumulation over `depth` products, eight per tensor-core instruction."""
    return (max(1, depth // 8) + 1) * 2.0 ** -23 * B


def accumulation_sigma(depth: int) -> float:
    """The same as a relative error of partial sums of the size of the quadrature sum."""
    return (max(1, depth // 8) + 1) * 2.0 ** -23


def rms(x: np.ndarray) -> float:
    return float(np.sqrt(np.mean(np.square(np.asarray(x, dtype=np.float64)))))


def check_single_contraction(got, ref, a, w, what, rounded_basis=True, extra=0.0):
    """One contraction out = a @ w with `a` rounded by the kernel.  `extra`: an allowance for float32
    element-wise operations around it (array or scalar).  Returns (observed max / statistical bound)."""
    a = np.asarray(a, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    err = np.abs(np.asarray(got, dtype=np.float64) - ref)
    B = np.abs(a) @ np.abs(w)
    acc = accumulation_allowance(B, a.shape[1])
    hard = (2.0 ** -11 if rounded_basis else 2.0 ** -11 + 2.0 ** -10) * B + acc + extra + TINY
    assert np.all(err <= hard), f"{what}: worst-case bound exceeded, max err/bound {float((err / hard).max()):.3f}"
    if not rounded_basis:
        return None
    stat = C_STAT * (SIGMA + accumulation_sigma(a.shape[1])) * np.sqrt((a * a) @ (w * w)) + extra + TINY
    ratio = float((err / stat).max())
    assert ratio <= 1.0, f"{what}: statistical bound exceeded, max err/bound {ratio:.3f}"
    return ratio


def check_rms(got, ref, what, rounded_basis=True):
    """Norm check: with a rounded basis the error is pure rounding noise, below 2^-11 of the RMS of the
    result; with the basis as drawn the cut adds a systematic 7e-4, and the bound is 2^-9."""
    err = rms(np.asarray(got, dtype=np.float64) - ref)
    lim = (2.0 ** -11 if rounded_basis else 2.0 ** -9) * rms(ref)
    assert err <= lim, f"{what}: RMS error {err:.3e} above {lim:.3e}"
    return err / max(lim, TINY)


def check_projection(got, T, U, what, rounded_basis=True, rows=None):
    """The two chained contractions of the embedding re-projection, Pi = (T U) U^T, T and the
    coordinates P = T U both rounded to TF32 by the kernel:
        err = dT (U U^T) + dP U^T   =>   variance  SIGMA^2 [ T^2 @ (U U^T)^2  +  P^2 @ (U^2)^T ],
        |err| <= 2^-11 (|T| @ |U U^T| + |P| @ |U|^T) <= 2 * 2^-11 B, B = (|T| @ |U|) @ |U|^T.
    `rows`: check the statistical bound on these rows only (it needs a d x d product per row)."""
    T = np.asarray(T, dtype=np.float64)
    U = np.asarray(U, dtype=np.float64)
    P = T @ U
    ref = P @ U.T
    err = np.abs(np.asarray(got, dtype=np.float64) - ref)
    B = (np.abs(T) @ np.abs(U)) @ np.abs(U).T
    acc = accumulation_allowance(B, T.shape[1]) + accumulation_allowance(B, U.shape[1])
    # 5 * 2^-11: two roundings (T, P) of 2^-11 each, their second-order products, and room for the
    # float32 rounding of P before it is rounded to TF32
    hard = (5 * 2.0 ** -11 if rounded_basis else 2.0 ** -8) * B + acc + TINY
    assert np.all(err <= hard), f"{what}: worst-case bound exceeded, max err/bound {float((err / hard).max()):.3f}"
    if not rounded_basis:
        return None, ref
    sel = slice(None) if rows is None else rows
    M = U @ U.T
    var = (T[sel] ** 2) @ (M * M) + (P[sel] ** 2) @ (U * U).T
    stat = C_STAT * (SIGMA + accumulation_sigma(T.shape[1]) + accumulation_sigma(U.shape[1])) * np.sqrt(var) + TINY
    ratio = float((err[sel] / stat).max())
    assert ratio <= 1.0, f"{what}: statistical bound exceeded, max err/bound {ratio:.3f}"
    return (ratio, float(np.median(stat)) / rms(ref)), ref
