"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py times:
the ~1B set (164 tensors, 241,829 chunks, R = 8, k = 64, 2-bit) over its five outer rounds, the
0.5B and 180M sets over their three, and every cell of the density sweep, always carrying the error
buffers.  The checker cannot do 8 x 1e9 elements in a test, so it is run on sampled chunks (every
kind of tensor, first and last chunks, all short tails, random interior chunks), each compared bit
for bit; properties that hold at any size are checked on every chunk on the device."""
import numpy as np
import pytest
import torch

import bench
from oracle import slo
from paper_2601_02360_b200 import synth
from parity_util import assert_close, assert_exact

pytestmark = pytest.mark.gpu
f32 = np.float32


def sampled_parity(wl, rounds, fused, n_samples, seed=1, min_short=0):
    """Runs `rounds` outer steps of the whole workload on the device in the launch configuration
    bench.py times (bench.DeviceState), carrying the error buffers, and compares sampled chunks with
    the checker bit for bit after every round; size-independent properties are checked on every chunk."""
    torch.cuda.empty_cache()                 # blocks cached by earlier tests count as free
    free, _ = torch.cuda.mem_get_info()
    need = (2 * wl.R + 1) * wl.n_total * 4 + (2 << 30)
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of device memory, {free >> 30} GiB free")
    dev = torch.device("cuda", 0)
    st = bench.DeviceState(wl, 0, dev)
    picks = synth.sample_chunks(wl, n_samples, seed=seed)
    assert sum(1 for _, _, ln in picks if ln < wl.chunk) >= min_short      # the short tails are in
    stride = st.api.sl_codes_stride(wl.k, wl.bits)
    for rnd in range(rounds):
        st.redraw_locals(rnd)
        tg_in = _gather(st.theta_global, picks)
        tl_in = [_gather(st.theta_local[r], picks) for r in range(wl.R)]
        e_in = [_gather(st.err[r], picks) for r in range(wl.R)]
        if fused:
            st.outer_step()
        else:
            st.compress()
            st.aggregate_apply()
        torch.cuda.synchronize()
        assert int(st.flags.item()) == 0
        _check_properties(st, wl)
        tg_out = _gather(st.theta_global, picks)
        idx_h = [t.cpu().numpy() for t in st.idx]
        codes_h = [t.cpu().numpy() for t in st.codes]
        scales_h = [t.cpu().numpy() for t in st.scales]
        for ci, (g, s, ln) in enumerate(picks):
            msgs = []
            for r in range(wl.R):
                e = e_in[r][ci].copy()
                i_o, c_o, s_o, _ = slo.compress(tl_in[r][ci], tg_in[ci], e, [0, ln], wl.beta, wl.chunk, wl.k, wl.bits)
                msgs.append((i_o, c_o, s_o))
                what = f"{wl.name} k={wl.k} R={wl.R} round {rnd} chunk {g} replica {r}"
                assert_exact(idx_h[r][g * wl.k:(g + 1) * wl.k], i_o[0], what + " idx")
                assert_exact(codes_h[r][g * stride:(g + 1) * stride], c_o[0], what + " codes")
                assert_close(scales_h[r][g:g + 1], s_o, what + " scale")
                assert_close(st.err[r][s:s + ln].cpu().numpy(), e, what + " err")
            upd = slo.aggregate(msgs, [0, ln], wl.chunk, wl.k, wl.bits)
            want = tg_in[ci].copy()
            slo.outer_apply(want, upd, wl.outer_lr)
            assert_close(tg_out[ci], want, f"{wl.name} round {rnd} chunk {g} theta_global")
    return st, picks


def _gather(t, picks):
    return [t[s:s + ln].cpu().numpy() for _, s, ln in picks]


def _check_properties(st, wl):
    nc = wl.n_chunks()
    # chunk lengths in chunk order
    lens = []
    for sz in wl.sizes:
        full, rem = divmod(sz, wl.chunk)
        lens += [wl.chunk] * full + ([rem] if rem else [])
    lens = torch.tensor(lens, dtype=torch.int32, device=st.dev)
    keff = torch.clamp(lens, max=wl.k)
    for r in range(wl.R):
        idx = (st.idx[r].view(torch.int16).to(torch.int32) & 0xFFFF).view(nc, wl.k)
        used = idx != 0xFFFF
        assert torch.equal(used.sum(dim=1).to(torch.int32), keff), "kept count per chunk"
        slot = torch.arange(wl.k, device=st.dev).view(1, -1)
        assert torch.equal(used, slot < keff.view(-1, 1)), "padding only after the used slots"
        nxt = torch.where(used[:, 1:], idx[:, 1:], torch.full_like(idx[:, 1:], 1 << 20))
        assert bool((nxt > idx[:, :-1]).all()), "positions strictly ascending"
        assert bool((torch.where(used, idx, torch.zeros_like(idx)) < lens.view(-1, 1)).all()), "positions inside the chunk"
        assert bool((st.scales[r] >= 0).all()) and bool(torch.isfinite(st.scales[r]).all())
        del idx, used, nxt


@pytest.mark.parametrize("fused,rounds", [(False, 5), (True, 2)], ids=["two_calls_all_5_rounds", "outer_step"])
def test_1b_workload_sampled_chunks(fused, rounds):
    """Benchmark configuration 4: the 1B set, R = 8, k = 64, 2-bit, all five outer rounds carrying
    the error buffers (the one-call form over two)."""
    wl = synth.workload("1b")
    assert wl.rounds == 5
    sampled_parity(wl, rounds, fused, 220, min_short=30)


def test_0p5b_workload_sampled_chunks_three_rounds():
    """Benchmark configuration 3: d = 1536, 16 layers, R = 8, three rounds carrying the error buffers.
    Rows of 1536 elements do not divide the 4096-element chunk, so every chunk of a d x d or ffn x d
    matrix holds pieces of three or four rows with their own scales (checked on the samples)."""
    wl = synth.workload("0p5b")
    assert wl.rounds == 3 and wl.R == 8 and wl.n_total == 502_187_520
    _, picks = sampled_parity(wl, 3, False, 260, seed=2, min_short=30)
    off = wl.offsets()
    straddle = 0
    for g, s, ln in picks:
        ti = int(np.searchsorted(off, s, side="right") - 1)
        _, rows, cols = wl.tensors[ti]
        if rows > 1 and cols == 1536 and ln == wl.chunk:
            lo = s - int(off[ti])
            if lo // 1536 != (lo + ln - 1) // 1536 and lo % 1536 != 0:
                straddle += 1
    assert straddle >= 60, straddle


def test_180m_workload_sampled_chunks_three_rounds():
    """Benchmark configuration 2: the whole 180M set (110 tensors), R = 4, three rounds."""
    wl = synth.workload("180m")
    assert wl.rounds == 3 and wl.R == 4 and wl.n_total == 186_934_272
    sampled_parity(wl, 3, False, 200, seed=3, min_short=20)


def sweep_sub_arena(full):
    """The sub-arena of the density sweep: one whole layer, the embedding and every norm vector."""
    keep = list(range(9)) + [i for i, (nm, rows, _) in enumerate(full.tensors) if i >= 9 and (rows == 1 or nm == "embed")]
    return synth.sub_arena(full, keep, full.name + "_sweep")


@pytest.mark.parametrize("R", [2, 8, 16])
@pytest.mark.parametrize("k", [16, 32, 64, 128])
def test_density_sweep_every_cell(k, R):
    """Benchmark configuration 5: every (k, R) cell of the sweep with the benchmark's value law
    (LogNormal(0, 1.5) row scales, x50 outliers), two rounds, on one layer + embedding + all norms."""
    wl = sweep_sub_arena(synth.workload("1b").replace(k=k, R=R))
    assert sum(1 for _, r, _ in wl.tensors if r == 1) == 37
    sampled_parity(wl, 2, (k + R) % 3 == 0, 120, seed=k + R, min_short=30)


@pytest.mark.parametrize("k,R", [(16, 8), (128, 8), (64, 16)])
@pytest.mark.parametrize("variant", ["ties_literal", "ties_dyadic"])
def test_tie_heavy_variants_of_the_sweep(variant, k, R):
    wl = sweep_sub_arena(synth.workload("1b").replace(k=k, R=R, variant=variant))
    st, _ = sampled_parity(wl, 2, False, 120, seed=5, min_short=30)
    if variant == "ties_dyadic":
        # the stress is real only if the k-th and (k+1)-th magnitudes tie in most chunks (the law of outer round 0:
        # the pseudo-gradient of a fresh draw on the 2^-13 grid)
        st.redraw_locals(7)
        d = (st.theta_global[:2048 * 2048] - st.theta_local[0][:2048 * 2048]).abs().view(-1, 4096)
        srt = torch.sort(d, dim=1).values
        assert float((srt[:, -k] == srt[:, -k - 1]).float().mean()) > 0.5


def test_1b_workload_with_tiles_sampled_tiles():
    """The same workload with every matrix cut into 64 x 64 tiles (the tuned tile kernels at full
    size): sampled tiles of every kind of matrix against the checker, one replica set, one round."""
    free, _ = torch.cuda.mem_get_info()
    wl = synth.workload("1b")
    need = (2 * wl.R + 1) * wl.n_total * 4 + (2 << 30)
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of device memory, {free >> 30} GiB free")
    dev = torch.device("cuda", 0)
    st = bench.DeviceState(wl, 0, dev, tiles=True)
    st.redraw_locals(0)
    for r in range(wl.R):                      # a non-trivial error buffer
        st.err[r].normal_(0.0, 5e-4)
    off = wl.offsets()
    rng = np.random.default_rng(3)
    # (tensor, tile row, tile col) samples: first / last / random tiles of the first layer's matrices and the embedding
    picks = []
    first_chunk = 0
    chunk_of = {}
    for ti, (_, rows, cols) in enumerate(wl.tensors):
        n_t = rows * cols
        if rows > 1:
            tr, tc = rows // 64, cols // 64
            chunk_of[ti] = (first_chunk, tr, tc)
            first_chunk += tr * tc
        else:
            first_chunk += -(-n_t // wl.chunk)
    for ti in [0, 4, 6, len(wl.tensors) - 2, 9 * 7 + 5]:
        fc, tr, tc = chunk_of[ti]
        cand = {(0, 0), (tr - 1, tc - 1), (0, tc - 1)} | {(int(rng.integers(tr)), int(rng.integers(tc))) for _ in range(5)}
        picks += [(ti, a, b) for a, b in sorted(cand)]
    stride = st.api.sl_codes_stride(wl.k, wl.bits)

    def block(t, ti, a, b):
        _, rows, cols = wl.tensors[ti]
        m = t[int(off[ti]):int(off[ti + 1])].view(rows, cols)
        return m[a * 64:(a + 1) * 64, b * 64:(b + 1) * 64]

    ins = [(block(st.theta_global, *p).cpu().numpy().copy(),
            [block(st.theta_local[r], *p).cpu().numpy().copy() for r in range(wl.R)],
            [block(st.err[r], *p).cpu().numpy().copy() for r in range(wl.R)]) for p in picks]
    st.compress()
    st.aggregate_apply()
    torch.cuda.synchronize()
    assert int(st.flags.item()) == 0
    for (ti, a, b), (tg_in, tl_in, e_in) in zip(picks, ins):
        fc, tr, tc = chunk_of[ti]
        g = fc + a * tc + b
        msgs = []
        for r in range(wl.R):
            e = e_in[r].reshape(-1).copy()
            i_o, c_o, s_o, _ = slo.compress(tl_in[r].reshape(-1), tg_in.reshape(-1), e, [0, 4096], wl.beta, wl.chunk,
                                            wl.k, wl.bits, cols=[64])
            msgs.append((i_o, c_o, s_o))
            what = f"tensor {ti} tile ({a},{b}) replica {r}"
            assert_exact(st.idx[r][g * wl.k:(g + 1) * wl.k].cpu().numpy(), i_o[0], what + " idx")
            assert_exact(st.codes[r][g * stride:(g + 1) * stride].cpu().numpy(), c_o[0], what + " codes")
            assert_close(st.scales[r][g:g + 1].cpu().numpy(), s_o, what + " scale")
            assert_close(block(st.err[r], ti, a, b).cpu().numpy().reshape(-1), e, what + " err")
        upd = slo.aggregate(msgs, [0, 4096], wl.chunk, wl.k, wl.bits, cols=[64])
        want = tg_in.reshape(-1).copy()
        slo.outer_apply(want, upd, wl.outer_lr)
        assert_close(block(st.theta_global, ti, a, b).cpu().numpy().reshape(-1), want, f"tensor {ti} tile ({a},{b}) theta_global")
