"""Parity of sl_pack_idx12 / sl_unpack_idx12 with the CPU checker, byte for byte, on positions made
by the CUDA compress kernels of the same case (so padding, short chunks and edge tiles all occur)."""
import numpy as np
import pytest
import torch

from oracle import idx12, slo
from paper_2601_02360_b200 import api, synth

pytestmark = pytest.mark.gpu


def _positions(offsets, chunk, k, cols=None, seed=0):
    n = int(offsets[-1])
    rng = np.random.default_rng(seed)
    tg = rng.normal(0, 0.02, n).astype(np.float32)
    tl = (tg + rng.normal(0, 1e-3, n)).astype(np.float32)
    lay = api.Layout(offsets, cols)
    d = lambda a: torch.from_numpy(a).cuda()
    err = torch.zeros(n, dtype=torch.float32, device="cuda")
    idx, codes, scales = api.alloc_messages(lay, chunk, k, 2, 1)
    api.sl_compress(d(tl), d(tg), err, lay, 0.95, chunk, k, 2, idx[0], codes[0], scales[0])
    torch.cuda.synchronize()
    return lay, idx[0]


@pytest.mark.parametrize("offsets,chunk,k,cols", [
    ([0, 4096 * 3 + 17, 4096 * 3 + 20, 4096 * 5 + 20], 4096, 64, None),     # short tails, a 3-element tensor
    ([0, 4096 * 2 + 100], 4096, 5, None),                                     # odd k
    ([0, 9000], 4096, 1, None),
    ([0, 1000, 5000], 1024, 32, None),                                        # positions below 1024
    ([0, 100 * 70, 100 * 70 + 4096 + 9], 4096, 64, [70, 0]),                  # edge tiles of a 100 x 70 matrix
    ([0, 130 * 200], 4096, 128, [200]),
])
def test_pack_and_unpack_match_the_checker(offsets, chunk, k, cols):
    lay, idx = _positions(offsets, chunk, k, cols)
    nc = api.sl_num_chunks(lay, chunk)
    st = api.sl_idx12_stride(k)
    assert st == idx12.idx12_stride(k)
    packed = torch.full((nc * st,), 0xAA, dtype=torch.uint8, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.sl_pack_idx12(idx, nc, k, packed, flags)
    back = torch.full_like(idx, 0x1234)
    api.sl_unpack_idx12(packed, lay, chunk, k, back)
    torch.cuda.synchronize()
    h_idx = idx.cpu().numpy()
    want = idx12.pack_idx12(h_idx, k)
    assert np.array_equal(packed.cpu().numpy().reshape(nc, st), want)
    lens = slo.chunk_lengths(offsets, chunk, cols)
    assert np.array_equal(idx12.unpack_idx12(want, k, lens).reshape(-1), h_idx)
    assert torch.equal(back, idx)
    assert int(flags.item()) == 0
    assert (h_idx == 0xFFFF).any() or k <= min(lens)      # the cases above do contain padding


def test_full_chunk_keeps_position_4095():
    # make 4095 the largest magnitude of a full chunk, and a short chunk beside it
    offsets = [0, 4096, 4096 + 40]
    lay = api.Layout(offsets)
    tg = np.zeros(offsets[-1], np.float32)
    tl = np.linspace(1e-3, 2e-3, offsets[-1]).astype(np.float32)
    tl[4095] = 1.0
    d = lambda a: torch.from_numpy(a).cuda()
    err = torch.zeros(offsets[-1], dtype=torch.float32, device="cuda")
    idx, codes, scales = api.alloc_messages(lay, 4096, 64, 2, 1)
    api.sl_compress(d(tl), d(tg), err, lay, 0.95, 4096, 64, 2, idx[0], codes[0], scales[0])
    h = idx[0].cpu().numpy().reshape(2, 64)
    assert h[0, -1] == 4095 and (h[1, 40:] == 0xFFFF).all()
    packed = torch.empty(2 * 96, dtype=torch.uint8, device="cuda")
    api.sl_pack_idx12(idx[0], 2, 64, packed)
    back = torch.empty_like(idx[0])
    api.sl_unpack_idx12(packed, lay, 4096, 64, back)
    assert torch.equal(back, idx[0])
    p = packed.cpu().numpy().reshape(2, 96)
    assert np.array_equal(p, idx12.pack_idx12(h, 64))


def test_position_above_12_bits_raises_the_flag():
    idx = torch.tensor([5, 5000, 0xFFFF, 7], dtype=torch.int32).to(torch.uint16).cuda()
    packed = torch.empty(6, dtype=torch.uint8, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.sl_pack_idx12(idx, 2, 2, packed, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == api.SL_FLAG_BAD_INDEX


def test_exchange_with_12_bit_positions_on_one_gpu():
    import socket
    import torch.distributed as dist
    from paper_2601_02360_b200 import exchange
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    try:
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                                device_id=torch.device("cuda", 0))
    except Exception as exc:  # an environment without a usable NCCL: nothing of ours has run yet
        pytest.skip(f"one-rank NCCL group unavailable: {exc}")
    try:
        wl = synth.sub_arena(synth.workload("180m"), [0, 1, 7, 8, 9]).replace(R=1)
        off = wl.offsets()
        lay = api.Layout(off)
        tg = synth.gen_theta_global(wl)
        tl = synth.gen_theta_local(wl, tg, 0, 0)
        res = []
        for use12 in (False, True):
            d_tg, d_tl = tg.cuda(), tl.cuda()
            err = torch.zeros_like(d_tg)
            idx, codes, scales = api.alloc_messages(lay, wl.chunk, wl.k, wl.bits, 1)
            flags = torch.zeros(1, dtype=torch.int32, device="cuda")
            exchange.outer_step_replica(d_tl, d_tg, err, lay, wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr,
                                        idx[0], codes[0], scales[0], flags, idx12=use12)
            torch.cuda.synchronize()
            assert int(flags.item()) == 0
            res.append((d_tg.cpu(), err.cpu(), idx[0].cpu()))
        for a, b in zip(res[0], res[1]):
            assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
        want = tg.numpy().copy()
        slo.outer_round([tl.numpy()], want, [np.zeros(wl.n_total, np.float32)], off, wl.beta, wl.chunk, wl.k, wl.bits,
                        wl.outer_lr)
        assert np.array_equal(res[1][0].numpy().view(np.uint32), want.view(np.uint32))
    finally:
        dist.destroy_process_group()
