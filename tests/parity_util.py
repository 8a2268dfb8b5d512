"""Helpers shared by the GPU parity tests: run one outer step on both sides, compare.

The acceptance bar (written here once, used by every parity test):
  * Top-k positions (idx) and quantisation codes: bit-exact;
  * float outputs (err, scales, update, theta_global): |a - b| <= 1e-6 * max(|a|, |b|),
    so exact zeros must match exactly.  Both sides round every operation once in
    the same order, so the float outputs are in fact expected to be bit-identical;
    `bitwise=True` (the default) asserts that as well.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

from oracle import slo
from paper_2601_02360_b200 import api

REL_TOL = 1e-6


def assert_close(a: np.ndarray, b: np.ndarray, what: str, bitwise: bool = True) -> None:
    a = np.asarray(a)
    b = np.asarray(b)
    assert a.shape == b.shape, (what, a.shape, b.shape)
    nan_a, nan_b = np.isnan(a), np.isnan(b)
    assert (nan_a == nan_b).all(), f"{what}: NaN positions differ"
    ok = ~nan_a
    with np.errstate(invalid="ignore"):
        diff = np.abs(a[ok].astype(np.float64) - b[ok].astype(np.float64))
        bound = REL_TOL * np.maximum(np.abs(a[ok]), np.abs(b[ok])).astype(np.float64)
        bad = ~((diff <= bound) | (a[ok] == b[ok]))
    assert not bad.any(), f"{what}: {int(bad.sum())} of {a.size} beyond rel {REL_TOL}, worst {diff[bad].max()}"
    if bitwise:
        same = (a.view(np.uint32) == b.view(np.uint32)) | nan_a   # NaN payloads are not compared
        assert same.all(), f"{what}: {int((~same).sum())} of {a.size} not bit-identical"


def assert_exact(a: np.ndarray, b: np.ndarray, what: str) -> None:
    a = np.asarray(a)
    b = np.asarray(b)
    assert a.shape == b.shape, (what, a.shape, b.shape)
    if not (a == b).all():
        w = np.argwhere(a != b)
        raise AssertionError(f"{what}: {len(w)} of {a.size} differ, first at {w[0].tolist()}: "
                             f"{a[tuple(w[0])]} vs {b[tuple(w[0])]}")


def oracle_compress_all(tls, tg, errs, offsets, beta, chunk, k, bits, threads: int = 8, cols=None):
    """Checker side of Eq. 2 lines 1-4 for every replica (errs updated in place)."""
    def one(r):
        return slo.compress(tls[r], tg, errs[r], offsets, beta, chunk, k, bits, cols)
    with ThreadPoolExecutor(max_workers=max(1, min(threads, len(tls)))) as ex:
        return list(ex.map(one, range(len(tls))))


class GpuStep:
    """Device buffers for one arena and R replicas, driven through the binding."""

    def __init__(self, offsets, R, chunk, k, bits, device="cuda", cols=None):
        self.layout = api.Layout(offsets, cols)
        self.R, self.chunk, self.k, self.bits = R, chunk, k, bits
        n = self.layout.n_total
        self.n = n
        self.dev = device
        self.nc = api.sl_num_chunks(self.layout, chunk)
        self.stride = api.sl_codes_stride(k, bits)
        self.theta_global = torch.empty(n, dtype=torch.float32, device=device)
        self.theta_local = [torch.empty(n, dtype=torch.float32, device=device) for _ in range(R)]
        self.err = [torch.zeros(n, dtype=torch.float32, device=device) for _ in range(R)]
        self.idx, self.codes, self.scales = api.alloc_messages(self.layout, chunk, k, bits, R, device)
        self.flags = torch.zeros(1, dtype=torch.int32, device=device)

    def upload(self, tg, tls, errs=None):
        if tg is not None:
            self.theta_global.copy_(torch.from_numpy(tg))
        for r in range(self.R):
            self.theta_local[r].copy_(torch.from_numpy(tls[r]))
            if errs is not None:
                self.err[r].copy_(torch.from_numpy(errs[r]))

    def compress(self, beta, batched=True):
        if batched:
            api.sl_compress_batch(self.theta_local, self.theta_global, self.err, self.layout, beta,
                                  self.chunk, self.k, self.bits, self.idx, self.codes, self.scales,
                                  self.flags)
        else:
            for r in range(self.R):
                api.sl_compress(self.theta_local[r], self.theta_global, self.err[r], self.layout, beta,
                                self.chunk, self.k, self.bits, self.idx[r], self.codes[r], self.scales[r],
                                self.flags)

    def aggregate_apply(self, outer_lr):
        api.sl_aggregate_apply(self.idx, self.codes, self.scales, self.layout, self.chunk, self.k,
                               self.bits, self.theta_global, outer_lr, self.flags)

    def outer_step(self, beta, outer_lr):
        api.sl_outer_step(self.theta_local, self.theta_global, self.err, self.layout, beta, self.chunk,
                          self.k, self.bits, outer_lr, self.idx, self.codes, self.scales, self.flags)

    def messages_host(self):
        torch.cuda.synchronize()
        out = []
        for r in range(self.R):
            out.append((self.idx[r].cpu().numpy().reshape(self.nc, self.k),
                        self.codes[r].cpu().numpy().reshape(self.nc, self.stride),
                        self.scales[r].cpu().numpy()))
        return out


def compare_messages(gpu_msgs, ora_msgs, what=""):
    for r, (gm, om) in enumerate(zip(gpu_msgs, ora_msgs)):
        assert_exact(gm[0], om[0], f"{what} idx[r={r}]")
        assert_exact(gm[1], om[1], f"{what} codes[r={r}]")
        assert_close(gm[2], om[2], f"{what} scales[r={r}]")


def run_and_compare(offsets, tg, tls, errs, beta, chunk, k, bits, outer_lr, rounds=1, next_locals=None,
                    batched=True, what="", fused=False, cols=None):
    """Runs `rounds` outer steps on the GPU and on the checker from the same inputs and compares
    everything after every round.  `next_locals(round, theta_global_numpy)` supplies the replicas'
    parameters for the rounds after the first.  fused=True drives the GPU through the single
    sl_outer_step call instead of sl_compress_batch + sl_aggregate_apply."""
    R = len(tls)
    gs = GpuStep(offsets, R, chunk, k, bits, cols=cols)
    tg_o = tg.copy()
    errs_o = [e.copy() for e in errs]
    gs.upload(tg, tls, errs)
    flags_o = 0
    for t in range(rounds):
        if t > 0:
            tls = next_locals(t, tg_o)
            gs.upload(None, tls)   # theta_global stays what each side computed itself
        if fused:
            gs.outer_step(beta, outer_lr)
        else:
            gs.compress(beta, batched=batched)
        res = oracle_compress_all(tls, tg_o, errs_o, offsets, beta, chunk, k, bits, cols=cols)
        ora_msgs = [(i, c, s) for i, c, s, _ in res]
        for _, _, _, f in res:
            flags_o |= f
        gpu_msgs = gs.messages_host()
        compare_messages(gpu_msgs, ora_msgs, f"{what} round {t}")
        for r in range(R):
            assert_close(gs.err[r].cpu().numpy(), errs_o[r], f"{what} round {t} err[r={r}]")
        upd = slo.aggregate(ora_msgs, offsets, chunk, k, bits, cols)
        slo.outer_apply(tg_o, upd, outer_lr)
        if not fused:
            gs.aggregate_apply(outer_lr)
        assert_close(gs.theta_global.cpu().numpy(), tg_o, f"{what} round {t} theta_global")
    assert int(gs.flags.item()) == flags_o, (what, int(gs.flags.item()), flags_o)
    return gs, tg_o, errs_o
