"""Pins of the CPU checker of the 12-bit position format: hand-worked bytes, round trips, the
padding rule, and the chunk lengths it relies on."""
import numpy as np
import pytest

from oracle import idx12, slo


def test_hand_worked_bytes():
    # slots 0x123 and 0xABC: the 24-bit little-endian word 0xABC123 -> bytes 23 C1 AB
    out = idx12.pack_idx12(np.array([0x123, 0xABC], np.uint16), 2)
    assert out.tolist() == [[0x23, 0xC1, 0xAB]]
    # padding travels as 0xFFF: slots (5, pad) -> word 0xFFF005 -> bytes 05 F0 FF
    out = idx12.pack_idx12(np.array([5, 0xFFFF], np.uint16), 2)
    assert out.tolist() == [[0x05, 0xF0, 0xFF]]
    # odd k: 3 slots = 36 bits in 5 bytes, the last 4 bits zero: (1, 2, 3) -> 0x003002001 -> 01 20 00 03 00
    out = idx12.pack_idx12(np.array([1, 2, 3], np.uint16), 3)
    assert out.tolist() == [[0x01, 0x20, 0x00, 0x03, 0x00]]


def test_stride():
    assert [idx12.idx12_stride(k) for k in (1, 2, 3, 32, 64, 128)] == [2, 3, 5, 48, 96, 192]


def test_same_bit_order_as_a_plain_shift_loop():
    rng = np.random.default_rng(0)
    k = 7
    v = rng.integers(0, 4096, size=(5, k)).astype(np.uint16)
    out = idx12.pack_idx12(v, k)
    for g in range(5):
        word = 0
        for j in range(k):
            word |= int(v[g, j]) << (12 * j)
        assert out[g].tobytes() == word.to_bytes(idx12.idx12_stride(k), "little")


@pytest.mark.parametrize("k", [1, 2, 5, 32, 64])
def test_round_trip_with_padding(k):
    rng = np.random.default_rng(k)
    n = 40
    lens = rng.integers(1, 4097, size=n)
    lens[0], lens[1], lens[2] = 4096, 1, min(k, 3)
    idx = np.full((n, k), 0xFFFF, np.uint16)
    for g in range(n):
        keep = min(k, int(lens[g]))
        idx[g, :keep] = np.sort(rng.choice(int(lens[g]), size=keep, replace=False))
    idx[0, -1] = 4095 if k <= 4096 else idx[0, -1]       # a full chunk whose largest kept position is 4095
    idx[0] = np.sort(idx[0])
    back = idx12.unpack_idx12(idx12.pack_idx12(idx, k), k, lens)
    assert np.array_equal(back, idx)


def test_0xfff_is_position_4095_only_in_a_full_chunk():
    packed = idx12.pack_idx12(np.array([[7, 0xFFF]], np.uint16), 2)
    assert idx12.unpack_idx12(packed, 2, np.array([4096])).tolist() == [[7, 4095]]
    assert idx12.unpack_idx12(packed, 2, np.array([4095])).tolist() == [[7, 0xFFFF]]
    assert idx12.unpack_idx12(packed, 2, np.array([1])).tolist() == [[7, 0xFFFF]]


def test_positions_that_do_not_fit_are_refused():
    with pytest.raises(ValueError):
        idx12.pack_idx12(np.array([4096], np.uint16), 1)


def test_chunk_lengths_of_both_geometries():
    # consecutive chunks: 10000 = 2 * 4096 + 1808; a 5-element vector
    assert slo.chunk_lengths([0, 10000, 10005], 4096).tolist() == [4096, 4096, 1808, 5]
    # a 100 x 70 matrix in 64 x 64 tiles: (64x64, 64x6, 36x64, 36x6)
    assert slo.chunk_lengths([0, 7000], 4096, cols=[70]).tolist() == [4096, 384, 2304, 216]
    assert int(slo.chunk_lengths([0, 7000, 7010], 4096, cols=[70, 0]).sum()) == 7010


def test_round_trip_of_a_real_message():
    from paper_2601_02360_b200 import synth
    import torch
    wl = synth.workload("tiny")
    off = wl.offsets()
    tg = synth.gen_theta_global(wl).numpy()
    tl = synth.gen_theta_local(wl, torch.from_numpy(tg), 0, 0).numpy()
    err = np.zeros(wl.n_total, np.float32)
    i, _, _, _ = slo.compress(tl, tg, err, off, wl.beta, wl.chunk, wl.k, wl.bits)
    lens = slo.chunk_lengths(off, wl.chunk)
    back = idx12.unpack_idx12(idx12.pack_idx12(i, wl.k), wl.k, lens)
    assert np.array_equal(back.reshape(i.shape), i)
