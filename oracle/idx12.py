"""CPU checker of the 12-bit wire form of the message positions (test infrastructure only).

A position of a chunk of at most 4096 elements fits 12 bits, so the uint16 positions of a message
(Eq. 2 line 3 sends "indices and values") can travel as 12 bits each: slot j of a chunk occupies
bits [12 j, 12 j + 12) of the chunk's ceil(12 k / 8) bytes, least-significant bits first (the same
bit order as the quantised codes).  The padding value 0xFFFF (a slot of a chunk that has fewer
than k elements) travels as 0xFFF.  0xFFF is also position 4095, which exists only in a chunk
that has all 4096 positions - and such a chunk has no padding (k <= 4096 of its elements are
kept) - so on the way back 0xFFF means position 4095 in a chunk of 4096 existing positions and
padding in every other chunk.

Written with numpy bit arrays, one step per sentence above; pinned by tests/test_oracle_idx12.py.
"""
from __future__ import annotations

import numpy as np

PAD16 = 0xFFFF
PAD12 = 0xFFF


def idx12_stride(k: int) -> int:
    """Bytes of 12-bit positions one chunk owns."""
    return (12 * k + 7) // 8


def pack_idx12(idx: np.ndarray, k: int) -> np.ndarray:
    """uint16 positions [n_chunks * k] (or [n_chunks, k]) -> uint8 [n_chunks, idx12_stride(k)]."""
    v = np.asarray(idx, dtype=np.uint16).reshape(-1, k).astype(np.uint32)
    v = np.where(v == PAD16, PAD12, v)
    if np.any(v > PAD12):
        raise ValueError("a position does not fit 12 bits")
    bits = ((v[:, :, None] >> np.arange(12, dtype=np.uint32)) & 1).astype(np.uint8)   # slot-major, LSB first
    bits = bits.reshape(v.shape[0], 12 * k)
    pad = idx12_stride(k) * 8 - 12 * k
    if pad:
        bits = np.concatenate([bits, np.zeros((v.shape[0], pad), np.uint8)], axis=1)
    return np.packbits(bits, axis=1, bitorder="little")


def unpack_idx12(packed: np.ndarray, k: int, chunk_len: np.ndarray) -> np.ndarray:
    """uint8 [n_chunks, idx12_stride(k)] -> uint16 [n_chunks, k]; chunk_len[g] = existing positions of
    chunk g (tells padding from position 4095)."""
    p = np.asarray(packed, dtype=np.uint8).reshape(-1, idx12_stride(k))
    bits = np.unpackbits(p, axis=1, bitorder="little")[:, :12 * k].reshape(p.shape[0], k, 12).astype(np.uint32)
    v = (bits << np.arange(12, dtype=np.uint32)).sum(axis=2)
    full = (np.asarray(chunk_len).reshape(-1, 1) == 4096)
    v = np.where((v == PAD12) & ~full, PAD16, v)
    return v.astype(np.uint16)
