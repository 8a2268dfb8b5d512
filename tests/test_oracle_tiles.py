"""Pins of the CPU checker's square-tile chunk geometry (the paper's literal "64 x 64" chunks,
section 3 and Table 8): matrices cut into s x s tiles, position p = row p / s, column p % s of the tile."""
import numpy as np
import pytest

from oracle import slo

f32 = np.float32


def _case(n, seed):
    rng = np.random.default_rng(seed)
    tg = rng.normal(0, 0.02, n).astype(f32)
    tl = (tg + rng.normal(0, 1e-3, n).astype(f32)).astype(f32)
    e = rng.normal(0, 5e-4, n).astype(f32)
    return tg, tl, e


def _retile(x, rows, cols, s):
    """row-major matrix -> tiles laid out one after the other, each tile row-major"""
    return x.reshape(rows // s, s, cols // s, s).transpose(0, 2, 1, 3).reshape(-1).copy()


def _untile(x, rows, cols, s):
    return x.reshape(rows // s, cols // s, s, s).transpose(0, 2, 1, 3).reshape(-1).copy()


@pytest.mark.parametrize("rows,cols,s,k,bits", [(8, 12, 4, 3, 2), (128, 192, 64, 64, 2), (64, 64, 64, 32, 4),
                                                (192, 128, 64, 16, 32)])
def test_full_tiles_equal_consecutive_chunks_of_the_retiled_matrix(rows, cols, s, k, bits):
    n = rows * cols
    tg, tl, e0 = _case(n, rows + cols + k)
    ea = e0.copy()
    ia, ca, sa, _ = slo.compress(tl, tg, ea, [0, n], 0.95, s * s, k, bits, cols=[cols])
    eb = _retile(e0, rows, cols, s)
    ib, cb, sb, _ = slo.compress(_retile(tl, rows, cols, s), _retile(tg, rows, cols, s), eb, [0, n], 0.95, s * s, k, bits)
    assert (ia == ib).all() and (ca == cb).all() and (sa == sb).all()
    assert (ea == _untile(eb, rows, cols, s)).all()
    # and the averaged update lands on the matching elements
    ua = slo.aggregate([(ia, ca, sa)], [0, n], s * s, k, bits, cols=[cols])
    ub = slo.aggregate([(ib, cb, sb)], [0, n], s * s, k, bits)
    assert (ua == _untile(ub, rows, cols, s)).all()


@pytest.mark.parametrize("rows,cols,s,k", [(10, 7, 4, 3), (70, 130, 64, 64), (1, 100, 8, 5), (65, 65, 64, 64), (3, 3, 4, 16)])
def test_ragged_tiles_against_numpy_brute_force(rows, cols, s, k):
    n = rows * cols
    tg, tl, e0 = _case(n, rows * 3 + cols)
    beta = f32(0.9)
    e = e0.copy()
    idx, codes, scales, _ = slo.compress(tl, tg, e, [0, n], beta, s * s, k, 32, cols=[cols])
    ep = (np.float64(beta) * e0.astype(np.float64) + (tg - tl).astype(np.float64)).astype(f32).reshape(rows, cols)
    tr, tc = -(-rows // s), -(-cols // s)
    assert idx.shape[0] == tr * tc == slo.num_chunks([0, n], s * s, cols=[cols])
    g = 0
    want_err = ep.copy()
    for a in range(tr):
        for b in range(tc):
            tile = ep[a * s:(a + 1) * s, b * s:(b + 1) * s]
            h, w = tile.shape
            pos = (np.arange(h)[:, None] * s + np.arange(w)[None, :]).ravel()
            val = tile.ravel()
            keff = min(k, h * w)
            order = np.lexsort((pos, -np.abs(val).astype(np.float64)))[:keff]
            kept = np.sort(pos[order])
            assert idx[g][:keff].tolist() == kept.tolist()
            assert (idx[g][keff:] == 0xFFFF).all()
            assert scales[g] == np.abs(val).max()
            sent = codes[g].view(f32)[:keff]
            assert sent.tolist() == [tile[p // s, p % s] for p in kept]
            for p in kept:
                want_err[a * s + p // s, b * s + p % s] = 0.0
            g += 1
    assert (e.reshape(rows, cols) == want_err).all()


def test_mixed_arena_of_matrices_and_vectors():
    s, chunk, k = 4, 16, 2
    sizes = [8 * 8, 20, 6 * 12, 5]
    cols = [8, 0, 12, 0]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    n = int(off[-1])
    assert slo.num_chunks(off, chunk, cols=cols) == 4 + 2 + 2 * 3 + 1
    tg, tl, e0 = _case(n, 9)
    e = e0.copy()
    idx, codes, scales, _ = slo.compress(tl, tg, e, off, 0.95, chunk, k, 2, cols=cols)
    # every tensor on its own gives the same rows of the message
    g = 0
    for t in range(4):
        lo, hi = int(off[t]), int(off[t + 1])
        et = e0[lo:hi].copy()
        it, ct, st, _ = slo.compress(tl[lo:hi].copy(), tg[lo:hi].copy(), et, [0, hi - lo], 0.95, chunk, k, 2, cols=[cols[t]])
        m = it.shape[0]
        assert (idx[g:g + m] == it).all() and (codes[g:g + m] == ct).all() and (scales[g:g + m] == st).all()
        assert (e[lo:hi] == et).all()
        g += m


def test_tiled_aggregate_dense_brute_force_and_bad_positions():
    rows, cols, s, k, R = 6, 10, 4, 3, 3
    n = rows * cols
    rng = np.random.default_rng(2)
    tg = rng.normal(0, 0.02, n).astype(f32)
    msgs, dense = [], np.zeros((R, rows, cols), f32)
    for r in range(R):
        tl = (tg + rng.normal(0, 1e-3, n).astype(f32)).astype(f32)
        e = np.zeros(n, f32)
        i, c, sc, _ = slo.compress(tl, tg, e, [0, n], 0.0, s * s, k, 32, cols=[cols])
        msgs.append((i, c, sc))
        dense[r] = ((tg - tl).astype(f32) - e).reshape(rows, cols)      # what was sent = e' - residual
    upd = slo.aggregate(msgs, [0, n], s * s, k, 32, cols=[cols]).reshape(rows, cols)
    acc = np.zeros((rows, cols), f32)
    for r in range(R):
        acc = (acc + dense[r]).astype(f32)
    assert (upd == (acc / f32(R)).astype(f32)).all()
    # a slot naming a position outside an edge tile is rejected
    bad = (msgs[0][0].copy(), msgs[0][1], msgs[0][2])
    bad[0][2][0] = 3          # tile (0, 2) is 4 x 2: column 3 does not exist
    with pytest.raises(ValueError):
        slo.aggregate([bad], [0, n], s * s, k, 32, cols=[cols])


def test_geometry_argument_checks():
    z = np.zeros(24, f32)
    with pytest.raises(ValueError):
        slo.compress(z, z, z.copy(), [0, 24], 0.9, 8, 2, 2, cols=[6])      # 8 is not a square
    with pytest.raises(ValueError):
        slo.compress(z, z, z.copy(), [0, 24], 0.9, 16, 2, 2, cols=[5])     # 24 elements are not rows of 5
    i, c, s, _ = slo.compress(z, z, z.copy(), [0, 24], 0.9, 8, 2, 2, cols=[0])   # cols 0: consecutive chunks, any chunk size
    assert i.shape[0] == 3
