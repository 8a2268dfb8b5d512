"""GPU parity for the square-tile chunk geometry (the paper's literal 64 x 64 chunks): matrices cut
into tiles, edge tiles smaller, vectors in consecutive chunks, all against the CPU checker."""
import numpy as np
import pytest
import torch

from oracle import slo
from paper_2601_02360_b200 import api, synth
from parity_util import GpuStep, assert_close, run_and_compare

pytestmark = pytest.mark.gpu
f32 = np.float32


def _case(n, R, seed):
    rng = np.random.default_rng(seed)
    tg = rng.normal(0, 0.02, n).astype(f32)
    tls = [(tg + rng.normal(0, 1e-3, n).astype(f32)).astype(f32) for _ in range(R)]
    errs = [rng.normal(0, 5e-4, n).astype(f32) for _ in range(R)]
    return tg, tls, errs


@pytest.mark.parametrize("shapes,chunk,k,bits", [
    ([(8, 12)], 16, 3, 2),
    ([(128, 192)], 4096, 64, 2),
    ([(70, 130)], 4096, 64, 2),                       # ragged right and bottom edges
    ([(65, 65), (1, 300), (64, 64), (200, 3)], 4096, 32, 4),
    ([(130, 70), (1, 5000), (3, 64)], 4096, 64, 32),
    ([(100, 100)], 64, 8, 8),                          # 8 x 8 tiles
    ([(256, 320), (1, 320), (320, 256)], 4096, 128, 2),
])
def test_tiles_match_the_checker(shapes, chunk, k, bits):
    sizes = [r * c for r, c in shapes]
    cols = [c if r > 1 else 0 for r, c in shapes]      # vectors keep consecutive chunks
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), 3, seed=sum(sizes) + k)
    nxt = lambda t, g: [(g + np.random.default_rng(t * 10 + r).normal(0, 1e-3, g.size)).astype(f32) for r in range(3)]
    run_and_compare(off, tg, tls, errs, 0.95, chunk, k, bits, 0.8, rounds=2, next_locals=nxt,
                    what=f"tiles {shapes}", cols=cols)


def test_tiles_through_the_single_call_and_the_dense_update():
    shapes = [(192, 128), (1, 128), (70, 66)]
    sizes = [r * c for r, c in shapes]
    cols = [128, 0, 66]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    tg, tls, errs = _case(int(off[-1]), 2, seed=5)
    gs, tg_o, _ = run_and_compare(off, tg, tls, errs, 0.95, 4096, 64, 2, 1.0, what="tiles outer_step", fused=True, cols=cols)
    upd = torch.full((int(off[-1]),), 3.0, dtype=torch.float32, device="cuda")
    api.sl_aggregate(gs.idx, gs.codes, gs.scales, gs.layout, 4096, 64, 2, upd, gs.flags)
    assert_close(upd.cpu().numpy(), slo.aggregate(gs.messages_host(), off, 4096, 64, 2, cols), "dense update, tiles")


def test_tiles_on_a_model_layer_with_the_benchmark_value_law():
    full = synth.workload("180m").replace(R=2)
    wl = synth.sub_arena(full, [0, 4, 6, 7])            # q 1024x1024, gate 1024x2816, down 2816x1024, a norm vector
    cols = [c if r > 1 else 0 for _, r, c in wl.tensors]
    tgt = synth.gen_theta_global(wl)
    rho = synth.row_scales(wl)
    tls = [synth.gen_theta_local(wl, tgt, 0, r, rho=rho).numpy() for r in range(wl.R)]
    errs = [np.zeros(wl.n_total, f32) for _ in range(wl.R)]
    nxt = lambda t, tg: [synth.gen_theta_local(wl, torch.from_numpy(tg), t, r, rho=rho).numpy() for r in range(wl.R)]
    run_and_compare(wl.offsets(), tgt.numpy(), tls, errs, wl.beta, wl.chunk, wl.k, wl.bits, wl.outer_lr,
                    rounds=2, next_locals=nxt, what="tiles 180m layer", cols=cols)


def test_bad_tile_geometry_is_rejected_before_any_launch():
    lay = api.Layout([0, 24], cols=[6])
    z = torch.zeros(24, device="cuda")
    idx, codes, scales = api.alloc_messages(api.Layout([0, 24]), 8, 2, 2, 1)
    with pytest.raises(api.SparseLoCoError, match="invalid argument"):
        api.sl_compress(z, z, z.clone(), lay, 0.9, 8, 2, 2, idx[0], codes[0], scales[0])   # 8 is not a square
