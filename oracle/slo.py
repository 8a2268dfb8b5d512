"""ctypes front end of the CPU checker (test infrastructure, never the product path).

Builds `libslo.so` from `sparseloco_oracle.cpp` with g++ on first use and
exposes the checker's functions on numpy arrays.  Nothing here computes: every
step of Eq. 2 runs inside the C++ file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sparseloco_oracle.cpp")
_LIB = os.path.join(_HERE, "libslo.so")
_lib = None

FLAG_NONFINITE = 1


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math",
                               "-fPIC", "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, u64, u32, i32, f32 = (ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int,
                                  ctypes.c_float)
        L.slo_num_chunks.restype = u64
        L.slo_num_chunks.argtypes = [vp, u32, i32]
        L.slo_codes_stride.restype = u64
        L.slo_codes_stride.argtypes = [i32, i32]
        L.slo_compress.restype = i32
        L.slo_compress.argtypes = [vp, vp, vp, vp, u32, f32, i32, i32, i32, vp, vp, vp, vp]
        L.slo_aggregate.restype = i32
        L.slo_aggregate.argtypes = [i32, vp, vp, vp, vp, u32, i32, i32, i32, vp]
        L.slo_chunk_lengths.restype = i32
        L.slo_chunk_lengths.argtypes = [vp, vp, u32, i32, vp]
        L.slo_num_chunks_tiled.restype = u64
        L.slo_num_chunks_tiled.argtypes = [vp, vp, u32, i32]
        L.slo_compress_tiled.restype = i32
        L.slo_compress_tiled.argtypes = [vp, vp, vp, vp, vp, u32, f32, i32, i32, i32, vp, vp, vp, vp]
        L.slo_aggregate_tiled.restype = i32
        L.slo_aggregate_tiled.argtypes = [i32, vp, vp, vp, vp, vp, u32, i32, i32, i32, vp]
        L.slo_outer_apply.restype = i32
        L.slo_outer_apply.argtypes = [vp, vp, u64, f32]
        L.slo_quantise.restype = u32
        L.slo_widen_bf16.argtypes = [vp, vp, u64]
        L.slo_widen_bf16.restype = i32
        L.slo_round_bf16.argtypes = [f32]
        L.slo_round_bf16.restype = ctypes.c_uint16
        L.slo_outer_apply_bf16.argtypes = [vp, vp, u64, f32]
        L.slo_outer_apply_bf16.restype = i32
        L.slo_quantise.argtypes = [f32, f32, i32]
        L.slo_dequantise.restype = f32
        L.slo_dequantise.argtypes = [u32, f32, i32]
        _lib = L
    return _lib


def _p(a: np.ndarray) -> int:
    return a.ctypes.data


def _off(offsets) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(offsets, dtype=np.uint64))


def _cols(cols, n_tensors):
    """None = consecutive chunks everywhere; else per-tensor column counts (0 = consecutive)."""
    if cols is None:
        return None
    c = np.ascontiguousarray(np.asarray(cols, dtype=np.uint64))
    assert c.shape == (n_tensors,)
    return c


def num_chunks(offsets, chunk: int, cols=None) -> int:
    off = _off(offsets)
    c = _cols(cols, len(off) - 1)
    if c is None:
        return int(lib().slo_num_chunks(_p(off), len(off) - 1, chunk))
    return int(lib().slo_num_chunks_tiled(_p(off), _p(c), len(off) - 1, chunk))


def chunk_lengths(offsets, chunk: int, cols=None) -> np.ndarray:
    """Existing positions of every chunk of the arena (uint32[n_chunks])."""
    off = _off(offsets)
    c = _cols(cols, len(off) - 1)
    out = np.zeros(num_chunks(off, chunk, cols), dtype=np.uint32)
    rc = lib().slo_chunk_lengths(_p(off), _p(c) if c is not None else None, len(off) - 1, chunk, _p(out))
    if rc != 0:
        raise ValueError("slo_chunk_lengths: bad arguments")
    return out


def codes_stride(k: int, bits: int) -> int:
    return int(lib().slo_codes_stride(k, bits))


def compress(theta_local: np.ndarray, theta_global: np.ndarray, err: np.ndarray, offsets,
             beta: float, chunk: int, k: int, bits: int, cols=None) -> Tuple[np.ndarray, np.ndarray, np.ndarray, int]:
    """Eq. 2 lines 1-4 for one replica.  `err` is updated in place.  `cols` switches matrices
    to square-tile chunks.  Returns (idx[n_c, k] u16, codes[n_c, stride] u8, scales[n_c] f32, flags)."""
    off = _off(offsets)
    c = _cols(cols, len(off) - 1)
    for a in (theta_local, theta_global, err):
        assert a.dtype == np.float32 and a.flags.c_contiguous
    if chunk < 1:
        raise ValueError("slo_compress rejected its arguments (chunk)")
    nc = num_chunks(off, chunk, cols)
    idx = np.empty((nc, k), dtype=np.uint16)
    codes = np.empty((nc, codes_stride(k, bits)), dtype=np.uint8)
    scales = np.empty(nc, dtype=np.float32)
    flags = np.zeros(1, dtype=np.uint32)
    rc = lib().slo_compress_tiled(_p(theta_local), _p(theta_global), _p(err), _p(off),
                                  _p(c) if c is not None else None, len(off) - 1,
                                  beta, chunk, k, bits, _p(idx), _p(codes), _p(scales), _p(flags))
    if rc != 0:
        raise ValueError(f"slo_compress rejected its arguments ({rc})")
    return idx, codes, scales, int(flags[0])


def aggregate(msgs: Sequence[Tuple[np.ndarray, np.ndarray, np.ndarray]], offsets, chunk: int, k: int,
              bits: int, cols=None) -> np.ndarray:
    """Dense mean update from the messages of the replicas, added in the order
    given; the divisor is always len(msgs)."""
    off = _off(offsets)
    n = len(msgs)
    keep: List[np.ndarray] = []
    def arr(i):
        a = (ctypes.c_void_p * n)()
        for r, m in enumerate(msgs):
            c = np.ascontiguousarray(m[i])
            keep.append(c)
            a[r] = _p(c)
        return a
    pi, pc, ps = arr(0), arr(1), arr(2)
    update = np.empty(int(off[-1]), dtype=np.float32)
    c = _cols(cols, len(off) - 1)
    rc = lib().slo_aggregate_tiled(n, pi, pc, ps, _p(off), _p(c) if c is not None else None, len(off) - 1,
                                   chunk, k, bits, _p(update))
    if rc != 0:
        raise ValueError(f"slo_aggregate rejected its arguments ({rc})")
    return update


def outer_apply(theta_global: np.ndarray, update: np.ndarray, outer_lr: float) -> None:
    assert theta_global.dtype == np.float32 and update.dtype == np.float32
    rc = lib().slo_outer_apply(_p(theta_global), _p(update), theta_global.size, outer_lr)
    if rc != 0:
        raise ValueError("slo_outer_apply rejected its arguments")


def widen_bf16(x: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> the float32 values they stand for (exact)."""
    assert x.dtype == np.uint16 and x.flags.c_contiguous
    out = np.empty(x.shape, dtype=np.float32)
    assert lib().slo_widen_bf16(_p(x), _p(out), x.size) == 0
    return out


def round_bf16(v: float) -> int:
    return int(lib().slo_round_bf16(v))


def outer_apply_bf16(theta_global: np.ndarray, update: np.ndarray, outer_lr: float) -> None:
    """theta_global: uint16 bfloat16 patterns, updated in place (float32 step, then one rounding to bfloat16)."""
    assert theta_global.dtype == np.uint16 and update.dtype == np.float32
    if lib().slo_outer_apply_bf16(_p(theta_global), _p(update), theta_global.size, outer_lr) != 0:
        raise ValueError("slo_outer_apply_bf16 rejected its arguments")


def outer_round_bf16(theta_locals, theta_global: np.ndarray, errs, offsets, beta: float, chunk: int, k: int,
                     bits: int, outer_lr: float, cols=None):
    """One whole outer step with the parameters stored as bfloat16 (uint16 patterns) and float32 error
    buffers: the pseudo-gradient is formed in float32 from the widened parameters (Eq. 2 line 1), lines
    2-5 are those of the float32 step, and theta_global is rounded to bfloat16 once, when it is stored."""
    tg32 = widen_bf16(theta_global)
    msgs, flags = [], 0
    for tl, e in zip(theta_locals, errs):
        i, c, s, f = compress(widen_bf16(tl), tg32, e, offsets, beta, chunk, k, bits, cols)
        msgs.append((i, c, s))
        flags |= f
    upd = aggregate(msgs, offsets, chunk, k, bits, cols)
    outer_apply_bf16(theta_global, upd, outer_lr)
    return msgs, upd, flags


def quantise(v: float, s: float, bits: int) -> int:
    return int(lib().slo_quantise(v, s, bits))


def dequantise(code: int, s: float, bits: int) -> float:
    return float(lib().slo_dequantise(code, s, bits))


def outer_round(theta_locals: Sequence[np.ndarray], theta_global: np.ndarray, errs: Sequence[np.ndarray],
                offsets, beta: float, chunk: int, k: int, bits: int, outer_lr: float, cols=None):
    """One whole outer step (all of Eq. 2) for R replicas; theta_global and the
    error buffers are updated in place.  Returns the R messages and the update."""
    msgs = []
    flags = 0
    for tl, e in zip(theta_locals, errs):
        i, c, s, f = compress(tl, theta_global, e, offsets, beta, chunk, k, bits, cols)
        msgs.append((i, c, s))
        flags |= f
    upd = aggregate(msgs, offsets, chunk, k, bits, cols)
    outer_apply(theta_global, upd, outer_lr)
    return msgs, upd, flags
