"""Thin Python binding of the C ABI in include/sparseloco.h (argument marshalling only).

Every function has the name and the meaning of the C entry point it forwards
to; tensors are torch CUDA tensors whose device pointers are passed through.
All work happens in the CUDA library `csrc/libsparseloco.so`; there is no
Python or CPU implementation behind these calls, and a missing or unloadable
library raises instead of falling back.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

from . import build as _build

SL_OK, SL_ERR_INVALID_ARG, SL_ERR_ALIGNMENT, SL_ERR_UNSUPPORTED, SL_ERR_CUDA = 0, -1, -2, -3, -4
SL_FLAG_NONFINITE, SL_FLAG_BAD_INDEX, SL_FLAG_TIMEOUT, SL_FLAG_BOUNDS = 1, 2, 4, 8
SL_MAX_CHUNK, SL_MAX_TENSORS, SL_MAX_REPLICAS = 8192, 1280, 64

EXPORTS = ("sl_num_chunks", "sl_codes_stride", "sl_codes_bytes", "sl_compress", "sl_compress_batch", "sl_aggregate",
           "sl_outer_apply", "sl_aggregate_apply", "sl_outer_step", "sl_compress_batch_bf16", "sl_aggregate_apply_bf16",
           "sl_outer_apply_bf16", "sl_outer_step_bf16", "sl_embed_reproject", "sl_round_tf32", "sl_subspace_project", "sl_subspace_reconstruct", "sl_idx12_stride",
           "sl_pack_idx12", "sl_unpack_idx12", "sl_debug_set_wait_limit", "sl_debug_bounds_selftest", "sl_strerror")


class SlLayout(ctypes.Structure):
    _fields_ = [("n_total", ctypes.c_uint64), ("n_tensors", ctypes.c_uint32),
                ("offset", ctypes.POINTER(ctypes.c_uint64)), ("cols", ctypes.POINTER(ctypes.c_uint64))]


class SparseLoCoError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {strerror(code)} ({code})")
        self.code = code


_lib = None


def load(path: Optional[str] = None) -> ctypes.CDLL:
    """Loads the CUDA library (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or _build.LIB_PATH
    if not os.path.exists(p):
        raise RuntimeError(f"{p} is missing: build it with `python -m paper_2601_02360_b200.build` "
                           "(there is no fallback path)")
    L = ctypes.CDLL(p)
    vp, u64, i32, f32 = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int, ctypes.c_float
    lp = ctypes.POINTER(SlLayout)
    L.sl_num_chunks.restype = u64
    L.sl_num_chunks.argtypes = [lp, i32]
    L.sl_codes_stride.restype = u64
    L.sl_codes_stride.argtypes = [i32, i32]
    L.sl_codes_bytes.restype = u64
    L.sl_codes_bytes.argtypes = [lp, i32, i32, i32]
    L.sl_compress.restype = i32
    L.sl_compress.argtypes = [vp, vp, vp, lp, f32, i32, i32, i32, vp, vp, vp, vp, vp]
    L.sl_compress_batch.restype = i32
    L.sl_compress_batch.argtypes = [i32, vp, vp, vp, lp, f32, i32, i32, i32, vp, vp, vp, vp, vp]
    L.sl_aggregate.restype = i32
    L.sl_aggregate.argtypes = [i32, vp, vp, vp, lp, i32, i32, i32, vp, vp, vp]
    L.sl_outer_apply.restype = i32
    L.sl_outer_apply.argtypes = [vp, vp, u64, f32, vp]
    L.sl_aggregate_apply.restype = i32
    L.sl_aggregate_apply.argtypes = [i32, vp, vp, vp, lp, i32, i32, i32, vp, f32, vp, vp]
    L.sl_outer_step.restype = i32
    L.sl_outer_step.argtypes = [i32, vp, vp, vp, lp, f32, i32, i32, i32, f32, vp, vp, vp, vp, vp]
    L.sl_compress_batch_bf16.restype = i32
    L.sl_compress_batch_bf16.argtypes = [i32, vp, vp, vp, lp, f32, i32, i32, i32, vp, vp, vp, vp, vp]
    L.sl_aggregate_apply_bf16.restype = i32
    L.sl_aggregate_apply_bf16.argtypes = [i32, vp, vp, vp, lp, i32, i32, i32, vp, f32, vp, vp]
    L.sl_outer_apply_bf16.restype = i32
    L.sl_outer_apply_bf16.argtypes = [vp, vp, u64, f32, vp]
    L.sl_outer_step_bf16.restype = i32
    L.sl_outer_step_bf16.argtypes = [i32, vp, vp, vp, lp, f32, i32, i32, i32, f32, vp, vp, vp, vp, vp]
    L.sl_embed_reproject.restype = i32
    L.sl_embed_reproject.argtypes = [vp, vp, vp, u64, ctypes.c_uint32, ctypes.c_uint32, vp, vp]
    u32 = ctypes.c_uint32
    L.sl_subspace_project.restype = i32
    L.sl_subspace_project.argtypes = [vp, vp, vp, vp, vp, u64, u32, u64, u32, u32, vp, vp, vp]
    L.sl_subspace_reconstruct.restype = i32
    L.sl_subspace_reconstruct.argtypes = [vp, vp, vp, vp, vp, u64, u32, u64, u32, u32, vp, vp, vp]
    L.sl_round_tf32.restype = i32
    L.sl_round_tf32.argtypes = [vp, u64, vp]
    L.sl_idx12_stride.restype = u64
    L.sl_idx12_stride.argtypes = [i32]
    L.sl_pack_idx12.restype = i32
    L.sl_pack_idx12.argtypes = [vp, u64, i32, vp, vp, vp]
    L.sl_unpack_idx12.restype = i32
    L.sl_unpack_idx12.argtypes = [vp, lp, i32, i32, vp, vp]
    L.sl_debug_set_wait_limit.restype = None
    L.sl_debug_set_wait_limit.argtypes = [ctypes.c_int32]
    L.sl_debug_bounds_selftest.restype = i32
    L.sl_debug_bounds_selftest.argtypes = [vp, vp, vp]
    L.sl_strerror.restype = ctypes.c_char_p
    L.sl_strerror.argtypes = [i32]
    if path is None:
        _lib = L
    return L


def strerror(code: int) -> str:
    return load().sl_strerror(code).decode()


class Layout:
    """Host description of an arena (`sl_layout`): element offsets of its tensors and, for the
    tensors cut into square tiles, their number of columns (`cols`, 0 = consecutive chunks)."""

    def __init__(self, offsets: Sequence[int], cols: Optional[Sequence[int]] = None):
        self.offsets = np.ascontiguousarray(np.asarray(offsets, dtype=np.uint64))
        assert self.offsets.ndim == 1 and len(self.offsets) >= 1
        u64p = ctypes.POINTER(ctypes.c_uint64)
        self.cols = None
        cols_p = ctypes.cast(None, u64p)
        if cols is not None:
            self.cols = np.ascontiguousarray(np.asarray(cols, dtype=np.uint64))
            assert self.cols.shape == (len(self.offsets) - 1,)
            cols_p = self.cols.ctypes.data_as(u64p)
        self.c = SlLayout(int(self.offsets[-1]), len(self.offsets) - 1, self.offsets.ctypes.data_as(u64p), cols_p)

    @property
    def n_total(self) -> int:
        return int(self.offsets[-1])

    def ref(self):
        return ctypes.byref(self.c)


def _layout(layout) -> Layout:
    return layout if isinstance(layout, Layout) else Layout(layout)


def _ptr(t) -> int:
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _ptr_table(ts: Sequence) -> ctypes.Array:
    a = (ctypes.c_void_p * len(ts))()
    for i, t in enumerate(ts):
        a[i] = _ptr(t)
    return a


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(rc: int, what: str) -> None:
    if rc != SL_OK:
        raise SparseLoCoError(rc, what)


def sl_num_chunks(layout, chunk: int) -> int:
    return int(load().sl_num_chunks(_layout(layout).ref(), chunk))


def sl_codes_stride(k: int, bits: int) -> int:
    return int(load().sl_codes_stride(k, bits))


def sl_codes_bytes(layout, chunk: int, k: int, bits: int) -> int:
    return int(load().sl_codes_bytes(_layout(layout).ref(), chunk, k, bits))


def sl_compress(theta_local, theta_global, err, layout, beta: float, chunk: int, k: int, bits: int,
                idx, codes, scales, flags=None, stream=None) -> None:
    _check(load().sl_compress(_ptr(theta_local), _ptr(theta_global), _ptr(err), _layout(layout).ref(),
                              beta, chunk, k, bits, _ptr(idx), _ptr(codes), _ptr(scales), _ptr(flags),
                              _stream(stream)), "sl_compress")


def sl_compress_batch(theta_local: Sequence, theta_global, err: Sequence, layout, beta: float, chunk: int,
                      k: int, bits: int, idx: Sequence, codes: Sequence, scales: Sequence, flags=None,
                      stream=None) -> None:
    R = len(theta_local)
    assert len(err) == len(idx) == len(codes) == len(scales) == R
    _check(load().sl_compress_batch(R, _ptr_table(theta_local), _ptr(theta_global), _ptr_table(err),
                                    _layout(layout).ref(), beta, chunk, k, bits, _ptr_table(idx),
                                    _ptr_table(codes), _ptr_table(scales), _ptr(flags), _stream(stream)),
           "sl_compress_batch")


def sl_aggregate(idx: Sequence, codes: Sequence, scales: Sequence, layout, chunk: int, k: int, bits: int,
                 update, flags=None, stream=None) -> None:
    R = len(idx)
    assert len(codes) == len(scales) == R
    _check(load().sl_aggregate(R, _ptr_table(idx), _ptr_table(codes), _ptr_table(scales),
                               _layout(layout).ref(), chunk, k, bits, _ptr(update), _ptr(flags),
                               _stream(stream)), "sl_aggregate")


def sl_outer_apply(theta_global, update, n: int, outer_lr: float, stream=None) -> None:
    _check(load().sl_outer_apply(_ptr(theta_global), _ptr(update), n, outer_lr, _stream(stream)),
           "sl_outer_apply")


def sl_aggregate_apply(idx: Sequence, codes: Sequence, scales: Sequence, layout, chunk: int, k: int,
                       bits: int, theta_global, outer_lr: float, flags=None, stream=None) -> None:
    R = len(idx)
    assert len(codes) == len(scales) == R
    _check(load().sl_aggregate_apply(R, _ptr_table(idx), _ptr_table(codes), _ptr_table(scales),
                                     _layout(layout).ref(), chunk, k, bits, _ptr(theta_global), outer_lr,
                                     _ptr(flags), _stream(stream)), "sl_aggregate_apply")


def sl_outer_step(theta_local: Sequence, theta_global, err: Sequence, layout, beta: float, chunk: int,
                  k: int, bits: int, outer_lr: float, idx: Sequence, codes: Sequence, scales: Sequence,
                  flags=None, stream=None) -> None:
    R = len(theta_local)
    assert len(err) == len(idx) == len(codes) == len(scales) == R
    _check(load().sl_outer_step(R, _ptr_table(theta_local), _ptr(theta_global), _ptr_table(err),
                                _layout(layout).ref(), beta, chunk, k, bits, outer_lr, _ptr_table(idx),
                                _ptr_table(codes), _ptr_table(scales), _ptr(flags), _stream(stream)),
           "sl_outer_step")


def sl_compress_batch_bf16(theta_local: Sequence, theta_global, err: Sequence, layout, beta: float, chunk: int,
                           k: int, bits: int, idx: Sequence, codes: Sequence, scales: Sequence, flags=None,
                           stream=None) -> None:
    """theta_local / theta_global: torch.bfloat16 (or uint16 pattern) tensors."""
    R = len(theta_local)
    assert len(err) == len(idx) == len(codes) == len(scales) == R
    _check(load().sl_compress_batch_bf16(R, _ptr_table(theta_local), _ptr(theta_global), _ptr_table(err),
                                         _layout(layout).ref(), beta, chunk, k, bits, _ptr_table(idx),
                                         _ptr_table(codes), _ptr_table(scales), _ptr(flags), _stream(stream)),
           "sl_compress_batch_bf16")


def sl_aggregate_apply_bf16(idx: Sequence, codes: Sequence, scales: Sequence, layout, chunk: int, k: int,
                            bits: int, theta_global, outer_lr: float, flags=None, stream=None) -> None:
    R = len(idx)
    assert len(codes) == len(scales) == R
    _check(load().sl_aggregate_apply_bf16(R, _ptr_table(idx), _ptr_table(codes), _ptr_table(scales),
                                          _layout(layout).ref(), chunk, k, bits, _ptr(theta_global), outer_lr,
                                          _ptr(flags), _stream(stream)), "sl_aggregate_apply_bf16")


def sl_outer_apply_bf16(theta_global, update, n: int, outer_lr: float, stream=None) -> None:
    _check(load().sl_outer_apply_bf16(_ptr(theta_global), _ptr(update), n, outer_lr, _stream(stream)),
           "sl_outer_apply_bf16")


def sl_outer_step_bf16(theta_local: Sequence, theta_global, err: Sequence, layout, beta: float, chunk: int,
                       k: int, bits: int, outer_lr: float, idx: Sequence, codes: Sequence, scales: Sequence,
                       flags=None, stream=None) -> None:
    R = len(theta_local)
    assert len(err) == len(idx) == len(codes) == len(scales) == R
    _check(load().sl_outer_step_bf16(R, _ptr_table(theta_local), _ptr(theta_global), _ptr_table(err),
                                     _layout(layout).ref(), beta, chunk, k, bits, outer_lr, _ptr_table(idx),
                                     _ptr_table(codes), _ptr_table(scales), _ptr(flags), _stream(stream)),
           "sl_outer_step_bf16")


def sl_embed_reproject(T_S, T_perp, U, V: int, d: int, k: int, flags=None, stream=None) -> None:
    _check(load().sl_embed_reproject(_ptr(T_S), _ptr(T_perp), _ptr(U), V, d, k, _ptr(flags), _stream(stream)),
           "sl_embed_reproject")


def sl_subspace_project(X, ids, T_perp, pos, U, n_tok: int, L: int, V: int, d: int, k: int, Xt, flags=None,
                        stream=None) -> None:
    _check(load().sl_subspace_project(_ptr(X), _ptr(ids), _ptr(T_perp), _ptr(pos), _ptr(U), n_tok, L, V, d, k, _ptr(Xt),
                                      _ptr(flags), _stream(stream)), "sl_subspace_project")


def sl_subspace_reconstruct(Xt, ids, T_perp, pos, U, n_tok: int, L: int, V: int, d: int, k: int, Xhat, flags=None,
                            stream=None) -> None:
    _check(load().sl_subspace_reconstruct(_ptr(Xt), _ptr(ids), _ptr(T_perp), _ptr(pos), _ptr(U), n_tok, L, V, d, k,
                                          _ptr(Xhat), _ptr(flags), _stream(stream)), "sl_subspace_reconstruct")


def sl_round_tf32(x, n: int, stream=None) -> None:
    _check(load().sl_round_tf32(_ptr(x), n, _stream(stream)), "sl_round_tf32")


def sl_idx12_stride(k: int) -> int:
    return int(load().sl_idx12_stride(k))


def sl_pack_idx12(idx, n_chunks: int, k: int, packed, flags=None, stream=None) -> None:
    _check(load().sl_pack_idx12(_ptr(idx), n_chunks, k, _ptr(packed), _ptr(flags), _stream(stream)), "sl_pack_idx12")


def sl_unpack_idx12(packed, layout, chunk: int, k: int, idx, stream=None) -> None:
    _check(load().sl_unpack_idx12(_ptr(packed), _layout(layout).ref(), chunk, k, _ptr(idx), _stream(stream)),
           "sl_unpack_idx12")


def sl_debug_set_wait_limit(polls: int) -> None:
    load().sl_debug_set_wait_limit(polls)


def sl_debug_bounds_selftest(flags, probe, stream=None) -> int:
    """Returns the status code (SL_ERR_UNSUPPORTED in the normal build) instead of raising."""
    return int(load().sl_debug_bounds_selftest(_ptr(flags), _ptr(probe), _stream(stream)))


def alloc_messages(layout, chunk: int, k: int, bits: int, R: int, device="cuda"):
    """Device buffers for R replicas' messages: lists (idx, codes, scales)."""
    nc = sl_num_chunks(layout, chunk)
    idx = [torch.empty(nc * k, dtype=torch.uint16, device=device) for _ in range(R)]
    codes = [torch.empty(sl_codes_bytes(layout, chunk, k, bits), dtype=torch.uint8, device=device) for _ in range(R)]
    scales = [torch.empty(nc, dtype=torch.float32, device=device) for _ in range(R)]
    return idx, codes, scales
