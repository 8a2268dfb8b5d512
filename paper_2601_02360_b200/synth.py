"""Seeded synthetic inputs for the SparseLoCo outer step.

This module only draws random parameter sets; it holds none of the method's
arithmetic (no pseudo-gradient, error feedback, selection, quantisation or
averaging).  Both the CUDA path's tests/bench and the CPU checker's tests take
their inputs from here, generated once on one device and copied.

The parameter sets are shaped like the LLaMA-style models of the paper's
Table 5 / Table 8 (decoder-only, SwiGLU, 32K vocabulary, tied embedding), with
the sizes fixed by the benchmark configuration list:

  per layer: q, k, v, o (d x d), gate, up (d x ffn), down (ffn x d),
             two RMSNorm vectors (d); then the embedding (vocab x d) and the
             final norm (d).

Value law: theta_global ~ N(0, 0.02) i.i.d.;  theta_local_r = theta_global +
z * 1e-3 * rho_row with z ~ N(0,1) per (round, replica, element) and rho_row ~
LogNormal(0, rho_sigma) drawn once per (tensor, row) and shared by all
replicas and rounds (a 1-D tensor is one row).  Optionally each element's
noise is multiplied by `outlier_mult` with probability `outlier_p`.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

TensorSpec = Tuple[str, int, int]  # (name, rows, cols); a vector is (name, 1, n)


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    tensors: Tuple[TensorSpec, ...]
    R: int
    k: int = 64
    bits: int = 2
    chunk: int = 4096
    beta: float = 0.95
    outer_lr: float = 1.0
    rounds: int = 1
    rho_sigma: float = 1.0
    outlier_p: float = 0.0
    outlier_mult: float = 50.0
    variant: str = "plain"  # "plain" | "ties_literal" | "ties_dyadic"

    @property
    def sizes(self) -> List[int]:
        return [r * c for _, r, c in self.tensors]

    @property
    def n_total(self) -> int:
        return sum(self.sizes)

    def offsets(self) -> np.ndarray:
        """Element offsets [n_tensors + 1], uint64, ascending, offsets[0] = 0."""
        off = np.zeros(len(self.tensors) + 1, dtype=np.uint64)
        off[1:] = np.cumsum(np.asarray(self.sizes, dtype=np.uint64))
        return off

    def n_chunks(self) -> int:
        return sum((n + self.chunk - 1) // self.chunk for n in self.sizes)

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def llama_tensors(d: int, n_layers: int, ffn: int, vocab: int = 32000) -> Tuple[TensorSpec, ...]:
    t: List[TensorSpec] = []
    for l in range(n_layers):
        for nm in ("q", "k", "v", "o"):
            t.append((f"l{l}.{nm}", d, d))
        t.append((f"l{l}.gate", d, ffn))
        t.append((f"l{l}.up", d, ffn))
        t.append((f"l{l}.down", ffn, d))
        t.append((f"l{l}.norm1", 1, d))
        t.append((f"l{l}.norm2", 1, d))
    t.append(("embed", vocab, d))
    t.append(("final_norm", 1, d))
    return tuple(t)


def workload(name: str) -> Workload:
    """The benchmark configurations, by name."""
    if name == "tiny":
        return Workload("tiny", (("w", 512, 512), ("bias", 1, 512)), R=2, rounds=1, rho_sigma=1.0)
    if name == "180m":
        return Workload("180m", llama_tensors(1024, 12, 2816), R=4, rounds=3, rho_sigma=1.0)
    if name == "0p5b":
        return Workload("0p5b", llama_tensors(1536, 16, 4096), R=8, rounds=3, rho_sigma=1.5,
                        outlier_p=1e-3)
    if name == "1b":
        return Workload("1b", llama_tensors(2048, 18, 5632), R=8, rounds=5, rho_sigma=1.5,
                        outlier_p=1e-3)
    raise KeyError(name)


def sub_arena(wl: Workload, keep: Sequence[int], name: Optional[str] = None) -> Workload:
    """A workload made of a subset of another one's tensors (same value law)."""
    return wl.replace(name=name or (wl.name + "_sub"), tensors=tuple(wl.tensors[i] for i in keep))


# --------------------------------------------------------------------------
# seeding: one integer per (purpose, round, replica, tensor), SplitMix64-mixed
# --------------------------------------------------------------------------
_MASK = (1 << 64) - 1


def _mix(*parts: int) -> int:
    x = 0x9E3779B97F4A7C15
    for p in parts:
        x = (x ^ (p & _MASK)) & _MASK
        x = (x + 0x9E3779B97F4A7C15) & _MASK
        z = x
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK
        x = z ^ (z >> 31)
    return x & ((1 << 63) - 1)


_P_THETA, _P_RHO, _P_NOISE, _P_OUTLIER, _P_ERR = 1, 2, 3, 4, 5


def _gen(device, *key: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_mix(*key))
    return g


def row_scales(wl: Workload, seed: int = 0) -> List[torch.Tensor]:
    """rho_row per tensor, always drawn on the CPU in float64 so that every
    device sees the same table; returned as float32 CPU tensors [rows]."""
    out = []
    for ti, (_, rows, _) in enumerate(wl.tensors):
        g = _gen("cpu", seed, _P_RHO, ti)
        z = torch.randn(rows, generator=g, dtype=torch.float64)
        out.append(torch.exp(wl.rho_sigma * z).to(torch.float32))
    return out


def gen_theta_global(wl: Workload, device="cpu", seed: int = 0) -> torch.Tensor:
    theta = torch.empty(wl.n_total, dtype=torch.float32, device=device)
    off = wl.offsets()
    for ti in range(len(wl.tensors)):
        v = theta[int(off[ti]):int(off[ti + 1])]
        v.normal_(0.0, 0.02, generator=_gen(device, seed, _P_THETA, ti))
    if wl.variant == "ties_dyadic":
        g = 2.0 ** -13
        theta.div_(g).round_().mul_(g)
    return theta


def gen_theta_local(wl: Workload, theta_global: torch.Tensor, rnd: int, replica: int,
                    seed: int = 0, out: Optional[torch.Tensor] = None,
                    rho: Optional[List[torch.Tensor]] = None) -> torch.Tensor:
    """theta_local of one replica for one outer round, around `theta_global`."""
    device = theta_global.device
    if out is None:
        out = torch.empty_like(theta_global)
    if rho is None:
        rho = row_scales(wl, seed)
    off = wl.offsets()
    for ti, (_, rows, cols) in enumerate(wl.tensors):
        lo, hi = int(off[ti]), int(off[ti + 1])
        v = out[lo:hi].view(rows, cols)
        v.normal_(0.0, 1.0, generator=_gen(device, seed, _P_NOISE, rnd, replica, ti))
        v.mul_(rho[ti].to(device).view(rows, 1) * 1e-3)
        if wl.outlier_p > 0.0:
            u = torch.rand(rows, cols, device=device,
                           generator=_gen(device, seed, _P_OUTLIER, rnd, replica, ti))
            v.mul_(torch.where(u < wl.outlier_p, float(wl.outlier_mult), 1.0))
            del u
        tg = theta_global[lo:hi].view(rows, cols)
        if wl.variant == "ties_literal":
            # noise rounded to the nearest multiple of 1e-4 before it is applied
            v.div_(1e-4).round_().mul_(1e-4)
            torch.sub(tg, v, out=v)
        elif wl.variant == "ties_dyadic":
            g = 2.0 ** -13
            v.div_(g).round_().mul_(g)
            torch.sub(tg, v, out=v)
        else:
            v.add_(tg)
    return out


def gen_error(wl: Workload, replica: int, device="cpu", seed: int = 0, std: float = 5e-4) -> torch.Tensor:
    """A non-zero starting error buffer (tests only; the configurations start from zero)."""
    e = torch.empty(wl.n_total, dtype=torch.float32, device=device)
    e.normal_(0.0, std, generator=_gen(device, seed, _P_ERR, replica))
    return e


def sample_chunks(wl: Workload, n: int, seed: int = 0) -> List[Tuple[int, int, int]]:
    """`n` chunks of the arena as (global chunk number, element start, length):
    every short chunk first (they are few), then full chunks spread at random."""
    off = wl.offsets()
    table = []
    g = 0
    for ti, sz in enumerate(wl.sizes):
        nc = (sz + wl.chunk - 1) // wl.chunk
        table.append((g, int(off[ti]), sz, nc))
        g += nc
    n_c = g
    rng = np.random.default_rng(_mix(seed, 77) % (1 << 32))
    short = [g0 + nc - 1 for g0, lo, sz, nc in table if nc and sz % wl.chunk]
    edges = sorted({g0 for g0, lo, sz, nc in table if nc} | {g0 + nc - 1 for g0, lo, sz, nc in table if nc})
    picks = set(short[:n])
    room = n - len(picks)
    if room > 0:
        rest = [e for e in edges if e not in picks]
        if len(rest) > room // 2:
            rest = list(rng.choice(rest, size=room // 2, replace=False))
        picks |= set(int(x) for x in rest)
    while len(picks) < min(n, n_c):
        picks.add(int(rng.integers(0, n_c)))
    picks = sorted(picks)
    out = []
    starts = np.asarray([t[0] for t in table])
    for gc in picks:
        ti = int(np.searchsorted(starts, gc, side="right") - 1)
        g0, lo, sz, nc = table[ti]
        c = gc - g0
        s = lo + c * wl.chunk
        out.append((gc, s, min(wl.chunk, lo + sz - s)))
    return out


# ---------------------------------------------------------------------------
# inputs of the token-embedding adaptation (paper §2.3-2.4)
# ---------------------------------------------------------------------------
def gen_subspace_basis(d: int, k: int, seed: int = 0) -> np.ndarray:
    """U (d x k, float32): a Gaussian matrix orthonormalised by QR, as §2.3 describes its creation."""
    rng = np.random.default_rng(_mix(0x5B5, d, k, seed))
    q, r = np.linalg.qr(rng.standard_normal((d, k)))
    q = q * np.sign(np.diag(r))  # fixes the sign convention of the factorisation
    return np.ascontiguousarray(q.astype(np.float32))


def gen_embedding_pair(V: int, d: int, seed: int = 0, std: float = 0.02) -> Tuple[np.ndarray, np.ndarray]:
    """(T_S, T_perp), V x d float32 each, N(0, std) i.i.d.: after an outer synchronisation with
    replicas that do not compress, T_S is a generic table with components outside the subspace."""
    rng = np.random.default_rng(_mix(0xE3B, V, d, seed))
    T_S = (rng.standard_normal((V, d), dtype=np.float32) * np.float32(std))
    T_perp = (rng.standard_normal((V, d), dtype=np.float32) * np.float32(std))
    return T_S, T_perp


def gen_stage_boundary(n_tok: int, L: int, V: int, d: int, seed: int = 0, std: float = 1.0):
    """Inputs of the activation compression of §2.3: (X n_tok x d, ids int32 n_tok, T_perp V x d,
    pos L x d), all float32 N(0, .) i.i.d. (activations of unit scale, embeddings of scale 0.02)."""
    rng = np.random.default_rng(_mix(0x5B9, n_tok, L, V, d, seed))
    X = rng.standard_normal((n_tok, d), dtype=np.float32) * np.float32(std)
    ids = rng.integers(0, V, size=n_tok).astype(np.int32)
    T_perp = rng.standard_normal((V, d), dtype=np.float32) * np.float32(0.02)
    pos = rng.standard_normal((L, d), dtype=np.float32) * np.float32(0.02)
    return X, ids, T_perp, pos
