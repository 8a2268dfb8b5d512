"""Parity of sl_subspace_project / sl_subspace_reconstruct (paper §2.3) with the float64 CPU checker.

Tolerance (derived): the float32 operand of each contraction (the difference X - T_perp[x] - Pos,
resp. Xt) is rounded to the nearest TF32 value, relative error <= 2^-11; U is used as given, and
the tensor cores cut it to TF32, relative error < 2^-10 (none when the caller has rounded it);
float32 accumulation adds far less.  With B the sum of the magnitudes of all products entering an
output, the error is below (2^-11 + 2^-10 + ...) B < 2^-9 B; the differences / sums around the
contraction are float32 operations and add a few units of 2^-24 of the magnitudes involved.
"""
import numpy as np
import pytest
import torch

import tf32_util as tu
from oracle import subspace as osub
from paper_2601_02360_b200 import api, synth

pytestmark = pytest.mark.gpu

TOL = 2.0 ** -9          # worst case per entry in units of B with a basis that is not rounded (see tests/tf32_util.py)


def _f64(a):
    return np.asarray(a, dtype=np.float64)


def _check_project(xt, X, ids, T_perp, pos, U, L, what, pos_rows=None):
    """Every check of a projection output: worst case, statistical (rounded basis only), RMS.  The
    float32 differences X - T_perp[x] - Pos cost two roundings of 2^-24 of the magnitudes involved each,
    which enter every output through |U|."""
    n = len(X)
    a = _f64(X)
    extra = 0.0
    if ids is not None:
        pr = _f64(pos)[np.arange(n) % L] if pos_rows is None else _f64(pos_rows)
        tp = _f64(T_perp)[ids]
        a = a - tp - pr
        extra = 2.0 ** -23 * ((np.abs(_f64(X)) + np.abs(tp) + np.abs(pr)) @ np.abs(_f64(U)))
    ref = a @ _f64(U)
    rounded = tu.is_tf32(U)
    ratio = tu.check_single_contraction(xt, ref, a, U, what, rounded_basis=rounded, extra=extra)
    if ref.size >= 4096:
        tu.check_rms(xt, ref, what, rounded_basis=rounded)
    return ref, ratio


def _check_reconstruct(xh, Xt, ids, T_perp, pos, U, L, what, pos_rows=None):
    """The same for a reconstruction output; the two float32 additions after the contraction cost
    2^-24 of the magnitudes involved each and are NOT scaled by the contraction's tolerance."""
    n = len(Xt)
    c = _f64(Xt) @ _f64(U).T
    ref, extra = c, 0.0
    if ids is not None:
        pr = _f64(pos)[np.arange(n) % L] if pos_rows is None else _f64(pos_rows)
        tp = _f64(T_perp)[ids]
        ref = c + tp + pr
        extra = 2.0 ** -23 * (np.abs(c) + np.abs(tp) + np.abs(pr))
    rounded = tu.is_tf32(U)
    err = np.abs(_f64(xh) - ref)
    B = np.abs(_f64(Xt)) @ np.abs(_f64(U)).T
    hard = (2.0 ** -11 if rounded else 2.0 ** -11 + 2.0 ** -10) * B + tu.accumulation_allowance(B, Xt.shape[1]) + extra + tu.TINY
    assert np.all(err <= hard), f"{what}: worst-case bound exceeded, {float((err / hard).max()):.3f}"
    ratio = None
    if rounded:
        stat = tu.C_STAT * (tu.SIGMA + tu.accumulation_sigma(Xt.shape[1])) * np.sqrt((_f64(Xt) ** 2) @ (_f64(U) ** 2).T) + extra + tu.TINY
        ratio = float((err / stat).max())
        assert ratio <= 1.0, f"{what}: statistical bound exceeded, {ratio:.3f}"
    if ref.size >= 4096:                        # the norm is taken against the contraction's part of the result
        lim = (2.0 ** -11 if rounded else 2.0 ** -9) * tu.rms(c) + 2.0 ** -23 * tu.rms(ref)
        assert tu.rms(_f64(xh) - ref) <= lim, f"{what}: RMS error {tu.rms(_f64(xh) - ref):.3e} above {lim:.3e}"
    return ref, ratio


def _dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _project(X, ids, T_perp, pos, U, L):
    n_tok, d = X.shape
    k = U.shape[1]
    out = torch.full((n_tok, k), 7.0, dtype=torch.float32, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.sl_subspace_project(_dev(X), _dev(ids), _dev(T_perp), _dev(pos), _dev(U), n_tok, L,
                            0 if T_perp is None else T_perp.shape[0], d, k, out, flags)
    torch.cuda.synchronize()
    return out.cpu().numpy(), int(flags.item())


def _reconstruct(Xt, ids, T_perp, pos, U, L):
    n_tok, k = Xt.shape
    d = U.shape[0]
    out = torch.full((n_tok, d), 7.0, dtype=torch.float32, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.sl_subspace_reconstruct(_dev(Xt), _dev(ids), _dev(T_perp), _dev(pos), _dev(U), n_tok, L,
                                0 if T_perp is None else T_perp.shape[0], d, k, out, flags)
    torch.cuda.synchronize()
    return out.cpu().numpy(), int(flags.item())


def _scale_project(X, ids, T_perp, pos, U, L):
    A = np.abs(X.astype(np.float64))
    if ids is not None:
        A = A + np.abs(T_perp.astype(np.float64))[ids] + np.abs(pos.astype(np.float64))[np.arange(len(X)) % L]
    return A @ np.abs(U.astype(np.float64))


@pytest.mark.parametrize("n_tok,L,V,d,k", [(1000, 128, 500, 512, 64), (4096, 1024, 2000, 2048, 256), (333, 50, 77, 132, 12),
                                           (5, 2, 3, 8, 4), (129, 129, 10, 64, 64), (260, 64, 300, 1536, 192),
                                           (2048, 512, 100, 1024, 8)])
@pytest.mark.parametrize("rounded", [True, False], ids=["basis_rounded", "basis_as_drawn"])
def test_parity_both_directions(n_tok, L, V, d, k, rounded):
    U = synth.gen_subspace_basis(d, k, seed=1)
    if rounded:
        U = tu.tf32_rna(U)
    X, ids, T_perp, pos = synth.gen_stage_boundary(n_tok, L, V, d, seed=2)
    xt, f = _project(X, ids, T_perp, pos, U, L)
    assert f == 0
    ref, _ = _check_project(xt, X, ids, T_perp, pos, U, L, "project")
    assert np.array_equal(ref, osub.project(X, ids, T_perp, pos, U, L))          # the helper's reference is the checker's
    # reconstruction from the checker's coordinates (as float32)
    Xt = ref.astype(np.float32)
    xh, f = _reconstruct(Xt, ids, T_perp, pos, U, L)
    assert f == 0
    ref_h, _ = _check_reconstruct(xh, Xt, ids, T_perp, pos, U, L, "reconstruct")
    assert np.allclose(ref_h, osub.reconstruct(Xt, ids, T_perp, pos, U, L), rtol=1e-15, atol=0)


def test_gradient_form_has_no_embedding_terms():
    n_tok, d, k = 700, 1024, 128
    U = synth.gen_subspace_basis(d, k, seed=3)
    G, _, _, _ = synth.gen_stage_boundary(n_tok, 64, 10, d, seed=4)
    gt, f = _project(G, None, None, None, U, 64)
    ref = osub.project(G, None, None, None, U, 64)
    S = np.abs(G.astype(np.float64)) @ np.abs(U.astype(np.float64))
    assert f == 0 and np.all(np.abs(gt - ref) <= TOL * S + 1e-30)
    gh, f = _reconstruct(ref.astype(np.float32), None, None, None, U, 64)
    assert f == 0
    assert np.all(np.abs(gh - ref.astype(np.float32).astype(np.float64) @ U.astype(np.float64).T)
                  <= TOL * osub.abs_bound_reconstruct(ref, U) + 1e-30)


@pytest.mark.parametrize("n_tok,L,V,d,k", [(300, 7, 20, 256, 8), (130, 16, 9, 512, 32), (128, 128, 5, 2048, 256)])
def test_exact_when_tf32_is_exact(n_tok, L, V, d, k):
    # identity columns and dyadic values with few bits: every operation is exact, so both directions
    # must match the checker bit for bit (catches a mis-swizzled operand or a wrong gather row)
    rng = np.random.default_rng(5)
    cols = rng.permutation(d)[:k]
    U = np.zeros((d, k), dtype=np.float32)
    U[cols, np.arange(k)] = 1.0
    q = lambda shape: (rng.integers(-32, 33, size=shape) / 16.0).astype(np.float32)
    X, T_perp, pos = q((n_tok, d)), q((V, d)), q((L, d))
    ids = rng.integers(0, V, size=n_tok).astype(np.int32)
    xt, f = _project(X, ids, T_perp, pos, U, L)
    assert f == 0 and np.array_equal(xt, osub.project(X, ids, T_perp, pos, U, L).astype(np.float32))
    xh, f = _reconstruct(xt, ids, T_perp, pos, U, L)
    assert f == 0 and np.array_equal(xh, osub.reconstruct(xt, ids, T_perp, pos, U, L).astype(np.float32))


def _hadamard(n):
    H = np.array([[1.0]])
    while H.shape[0] < n:
        H = np.block([[H, H], [H, -H]])
    return H


@pytest.mark.parametrize("d,k", [(256, 64), (1024, 128)])
def test_exact_on_every_cta_with_two_sub_tiles_each(d, k):
    # at least two sub-tiles of 128 tokens on every CTA and a ragged rest; dyadic values and a basis of
    # +-1/sqrt(d) Hadamard columns (d a power of 4): the differences, their rounding to TF32, every product
    # and every sum are exact, so the projection with embedding terms, its two-sub-tile form without them
    # and the reconstruction must all match the checker bit for bit
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    n_tok, L, V = sms * 256 + 72, 96, 300
    rng = np.random.default_rng(d * 3 + k)
    U = (_hadamard(d)[:, rng.permutation(d)[:k]] / np.sqrt(d)).astype(np.float32)
    q = lambda shape, m: (rng.integers(-m, m + 1, size=shape) / 4.0).astype(np.float32)
    X, T_perp, pos = q((n_tok, d), 8), q((V, d), 8), q((L, d), 8)
    ids = rng.integers(0, V, size=n_tok).astype(np.int32)
    want = osub.project(X, ids, T_perp, pos, U, L)
    assert np.array_equal(want.astype(np.float32), want)
    xt, f = _project(X, ids, T_perp, pos, U, L)
    assert f == 0 and np.array_equal(xt, want.astype(np.float32))
    want_g = osub.project(X, None, None, None, U, L)
    gt, f = _project(X, None, None, None, U, L)                      # two sub-tiles share every slice of U
    assert f == 0 and np.array_equal(gt, want_g.astype(np.float32))
    Xt = q((n_tok, k), 16)                                           # TF32 values: the kernel's rounding is exact
    want_h = osub.reconstruct(Xt, ids, T_perp, pos, U, L)
    assert np.array_equal(want_h.astype(np.float32), want_h)
    xh, f = _reconstruct(Xt, ids, T_perp, pos, U, L)
    assert f == 0 and np.array_equal(xh, want_h.astype(np.float32))
    gh, f = _reconstruct(Xt, None, None, None, U, L)
    assert f == 0 and np.array_equal(gh, (Xt.astype(np.float64) @ U.astype(np.float64).T).astype(np.float32))


@pytest.mark.parametrize("extra_sub_tiles,extra_tokens,d,k", [
    (1, 0, 1024, 64),       # one sub-tile left over: shared by more CTAs than it has blocks, most get nothing of it
    (41, 17, 256, 64),      # 42 left over (the last ragged): three CTAs share each, two blocks do not split evenly
    (74, 0, 320, 32),       # half as many left over as CTAs: two share each; d ends in a 64-column block
    (-100, 5, 1024, 128),   # fewer sub-tiles than CTAs: nobody has a whole one
])
def test_reconstruction_exact_where_ctas_share_a_sub_tile(extra_sub_tiles, extra_tokens, d, k):
    # The reconstruction deals whole sub-tiles of 128 tokens evenly and cuts the remaining ones by 128-column
    # blocks among several CTAs.  Exact arithmetic (dyadic values, identity columns), so every entry must match
    # the checker bit for bit in both forms: a block done twice shows nothing here, but a block left out (the
    # output is filled with 7 beforehand) or gathered for the wrong rows does.
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    n_tok, L, V = (sms + extra_sub_tiles) * 128 + extra_tokens, 48, 200
    rng = np.random.default_rng(1000 + extra_sub_tiles)
    U = np.zeros((d, k), dtype=np.float32)
    U[rng.permutation(d)[:k], np.arange(k)] = 1.0
    q = lambda shape, m: (rng.integers(-m, m + 1, size=shape) / 4.0).astype(np.float32)
    Xt, T_perp, pos = q((n_tok, k), 16), q((V, d), 8), q((L, d), 8)
    ids = rng.integers(0, V, size=n_tok).astype(np.int32)
    xh, f = _reconstruct(Xt, ids, T_perp, pos, U, L)
    assert f == 0 and np.array_equal(xh, osub.reconstruct(Xt, ids, T_perp, pos, U, L).astype(np.float32))
    gh, f = _reconstruct(Xt, None, None, None, U, L)
    assert f == 0 and np.array_equal(gh, (Xt.astype(np.float64) @ U.astype(np.float64).T).astype(np.float32))


def test_round_trip_is_lossless_for_residuals_in_the_subspace():
    n_tok, L, V, d, k = 1500, 256, 400, 1024, 128
    u = _dev(synth.gen_subspace_basis(d, k, seed=6))
    api.sl_round_tf32(u, u.numel())
    U = u.cpu().numpy()
    _, ids, T_perp, pos = synth.gen_stage_boundary(n_tok, L, V, d, seed=7)
    C = np.random.default_rng(8).standard_normal((n_tok, k))
    X = (C @ U.astype(np.float64).T + T_perp[ids] + pos[np.arange(n_tok) % L]).astype(np.float32)
    xt, _ = _project(X, ids, T_perp, pos, U, L)
    xh, _ = _reconstruct(xt, ids, T_perp, pos, U, L)
    # U is orthonormal only up to the rounding of its entries, and both contractions are TF32
    assert np.sqrt(((xh - X) ** 2).mean()) <= 2.0 ** -9 * np.sqrt((X ** 2).mean())


def test_bad_token_id_is_flagged_and_gathers_nothing():
    n_tok, L, V, d, k = 64, 8, 5, 64, 8
    U = synth.gen_subspace_basis(d, k, seed=9)
    X, ids, T_perp, pos = synth.gen_stage_boundary(n_tok, L, V, d, seed=10)
    ids = ids.copy()
    ids[3], ids[40] = V, -1
    xt, f = _project(X, ids, T_perp, pos, U, L)
    assert f == api.SL_FLAG_BAD_INDEX
    good = np.ones(n_tok, bool)
    good[[3, 40]] = False
    ref = osub.project(X[good], ids[good], T_perp, pos[(np.arange(n_tok) % L)[good]], U, n_tok)   # per-row positions
    assert np.all(np.abs(xt[good] - ref) <= TOL * _scale_project(X, np.clip(ids, 0, V - 1), T_perp, pos, U, L)[good] + 1e-30)
    plain = X[[3, 40]].astype(np.float64) @ U.astype(np.float64)
    assert np.all(np.abs(xt[[3, 40]] - plain) <= TOL * (np.abs(X[[3, 40]].astype(np.float64)) @ np.abs(U.astype(np.float64))))


@pytest.mark.parametrize("L,extra_pairs,d,k", [
    (128, 2, 256, 64),      # four units of 32 positions in a sequence: passes cross from one pair of sequences to the next
    (96, 60, 256, 32),      # three units in a sequence: no pass is 128 consecutive tokens
    (2048, 0, 256, 64),     # the benchmark's sequence length: 64 units in a sequence, passes of 128 consecutive tokens
])
def test_projection_exact_where_a_pass_pairs_two_sequences(L, extra_pairs, d, k):
    # A batch that is a whole number of pairs of sequences, with two sub-tiles or more for every CTA: the
    # projection with embedding terms pairs the same positions of two sequences and fetches a position row once
    # for both.  Exact arithmetic (dyadic values, identity columns): bit for bit against the checker.  Then two
    # token ids out of range, one in each sequence of a pair at the SAME position: each leaves only its own row
    # without terms, the row that shares its position row keeps them.
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    pairs = -(-sms * 256 // (2 * L)) + extra_pairs
    n_tok, V = pairs * 2 * L, 300
    rng = np.random.default_rng(L + d)
    U = np.zeros((d, k), dtype=np.float32)
    U[rng.permutation(d)[:k], np.arange(k)] = 1.0
    q = lambda shape, m: (rng.integers(-m, m + 1, size=shape) / 4.0).astype(np.float32)
    X, T_perp, pos = q((n_tok, d), 8), q((V, d), 8), q((L, d), 8)
    ids = rng.integers(0, V, size=n_tok).astype(np.int32)
    want = osub.project(X, ids, T_perp, pos, U, L)
    xt, f = _project(X, ids, T_perp, pos, U, L)
    assert f == 0 and np.array_equal(xt, want.astype(np.float32))
    bad_a, bad_b = 2 * L * 3 + 17, 2 * L * 5 + L + 40 % L              # first sequence of pair 3, second of pair 5
    ids2 = ids.copy()
    ids2[bad_a], ids2[bad_b] = V + 7, -2
    xt2, f = _project(X, ids2, T_perp, pos, U, L)
    assert f == api.SL_FLAG_BAD_INDEX
    want2 = want.copy()
    want2[[bad_a, bad_b]] = X[[bad_a, bad_b]].astype(np.float64) @ U.astype(np.float64)     # no terms for those rows
    assert np.array_equal(xt2, want2.astype(np.float32))


@pytest.mark.parametrize("n_tok,L,V,d,k", [(50, 10, 7, 1536, 2), (33, 5, 4, 10, 3), (20, 4, 6, 64, 300)])
def test_shapes_outside_the_tensor_core_path(n_tok, L, V, d, k):
    rng = np.random.default_rng(11)
    U = synth.gen_subspace_basis(d, k, seed=11) if k <= d else (rng.standard_normal((d, k)) / np.sqrt(k)).astype(np.float32)
    X, ids, T_perp, pos = synth.gen_stage_boundary(n_tok, L, V, d, seed=12)
    xt, f = _project(X, ids, T_perp, pos, U, L)
    ref = osub.project(X, ids, T_perp, pos, U, L)
    assert f == 0 and np.all(np.abs(xt - ref) <= 2.0 ** -18 * _scale_project(X, ids, T_perp, pos, U, L) + 1e-30)
    xh, f = _reconstruct(ref.astype(np.float32), ids, T_perp, pos, U, L)
    ref_h = osub.reconstruct(ref.astype(np.float32), ids, T_perp, pos, U, L)
    S_h = osub.abs_bound_reconstruct(ref, U) + np.abs(T_perp)[ids] + np.abs(pos)[np.arange(n_tok) % L]
    assert f == 0 and np.all(np.abs(xh - ref_h) <= 2.0 ** -18 * S_h + 1e-30)


@pytest.mark.parametrize("n_tok", [16384, 65536])
def test_bench_size_on_sampled_tokens(n_tok):
    # the workload bench.py --subspace times (1B stage boundary), both launches at full size; tokens are
    # independent, so the checker computes a sample of them one by one: the first and last token, the
    # tokens around every boundary between two CTAs' shares and between sub-tiles, and random ones
    L, V, d, k = 2048, 32000, 2048, 256
    U = synth.gen_subspace_basis(d, k, seed=0)
    u = torch.from_numpy(U).cuda()
    api.sl_round_tf32(u, u.numel())
    U = u.cpu().numpy()
    X, ids, T_perp, pos = synth.gen_stage_boundary(n_tok, L, V, d, seed=0)
    dX, dids, dT, dP = _dev(X), _dev(ids), _dev(T_perp), _dev(pos)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    xt = torch.full((n_tok, k), 7.0, dtype=torch.float32, device="cuda")
    xh = torch.full((n_tok, d), 7.0, dtype=torch.float32, device="cuda")
    api.sl_subspace_project(dX, dids, dT, dP, u, n_tok, L, V, d, k, xt, flags)
    api.sl_subspace_reconstruct(xt, dids, dT, dP, u, n_tok, L, V, d, k, xh, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    rng = np.random.default_rng(5)
    groups = n_tok // 32
    edges = np.unique(np.array([(c * groups // 148) * 32 for c in range(149)]))
    near = np.concatenate([edges + o for o in (-1, 0, 1, 127, 128, 129)])
    rows = np.unique(np.clip(np.concatenate([[0, 1, n_tok - 2, n_tok - 1], near, rng.integers(0, n_tok, 300)]), 0, n_tok - 1))
    g_xt = xt[torch.from_numpy(rows).cuda()].cpu().numpy()
    g_xh = xh[torch.from_numpy(rows).cuda()].cpu().numpy()
    pos_rows = pos[rows % L]                               # the positions of the sampled tokens
    ref, r1 = _check_project(g_xt, X[rows], ids[rows], T_perp, pos, U, L, f"project {n_tok}", pos_rows=pos_rows)
    assert np.array_equal(ref, osub.project(X[rows], ids[rows], T_perp, pos_rows, U, len(rows)))
    _, r2 = _check_reconstruct(g_xh, g_xt, ids[rows], T_perp, pos, U, L, f"reconstruct {n_tok}", pos_rows=pos_rows)
    print(f"{n_tok} tokens: max err / statistical bound: project {r1:.3f}, reconstruct {r2:.3f}")
    # the per-entry bound is a small fraction of the results' RMS (a dropped K step would show)
    a = X[rows].astype(np.float64) - T_perp[ids[rows]] - pos_rows
    stat = tu.C_STAT * (tu.SIGMA + tu.accumulation_sigma(d)) * np.sqrt((a * a) @ (U.astype(np.float64) ** 2))
    assert float(np.median(stat)) <= 0.05 * tu.rms(ref)
    # every token was written (the fill value is gone) and nothing is NaN
    assert not bool(torch.isnan(xh).any()) and not bool((xt == 7.0).all(dim=1).any())


@pytest.mark.parametrize("n_tok,d,k", [(65536, 2048, 256), (40037, 1024, 192), (38000, 512, 64)])
def test_gradient_form_at_sizes_where_two_sub_tiles_share_the_basis(n_tok, d, k):
    # Gt = G U at sizes where every CTA has at least two sub-tiles (the launch that walks two sub-tiles
    # through K together), checked on sampled tokens: ends, sub-tile and CTA boundaries, random ones;
    # then back through the reconstruction without embedding terms
    U = synth.gen_subspace_basis(d, k, seed=6)
    u = torch.from_numpy(U).cuda()
    api.sl_round_tf32(u, u.numel())
    U = u.cpu().numpy()
    rng = np.random.default_rng(7)
    G = rng.standard_normal((n_tok, d), dtype=np.float32)
    dG = _dev(G)
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    gt = torch.full((n_tok, k), 7.0, dtype=torch.float32, device="cuda")
    gh = torch.full((n_tok, d), 7.0, dtype=torch.float32, device="cuda")
    api.sl_subspace_project(dG, None, None, None, u, n_tok, 1, 0, d, k, gt, flags)
    api.sl_subspace_reconstruct(gt, None, None, None, u, n_tok, 1, 0, d, k, gh, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    groups = (n_tok + 31) // 32
    edges = np.unique(np.array([(c * groups // 148) * 32 for c in range(149)]))
    near = np.concatenate([edges + o for o in (-1, 0, 1, 127, 128, 129, 255, 256, 257)])
    rows = np.unique(np.clip(np.concatenate([[0, 1, n_tok - 2, n_tok - 1], near, rng.integers(0, n_tok, 300)]), 0, n_tok - 1))
    sel = torch.from_numpy(rows).cuda()
    g_gt, g_gh = gt[sel].cpu().numpy(), gh[sel].cpu().numpy()
    ref, _ = _check_project(g_gt, G[rows], None, None, None, U, 1, f"gradient project {n_tok}x{d}")
    assert np.array_equal(ref, osub.project(G[rows], None, None, None, U, 1))
    _check_reconstruct(g_gh, g_gt, None, None, None, U, 1, f"gradient reconstruct {n_tok}x{d}")
    assert not bool((gt == 7.0).all(dim=1).any()) and not bool(torch.isnan(gt).any())


def _random_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        d = int(rng.integers(1, 300)) * 4 if i % 4 else int(rng.integers(3, 700))      # every fourth: any d (plain kernels)
        k = int(rng.integers(1, min(64, d // 4) + 1)) * 4 if i % 4 else int(rng.integers(1, min(d, 40) + 1))
        out.append((int(rng.integers(1, 3000)), int(rng.integers(1, 300)), int(rng.integers(1, 2000)), d, min(k, d)))
    return out


@pytest.mark.parametrize("n_tok,L,V,d,k", _random_shapes(24, 11))
def test_random_shapes_both_directions(n_tok, L, V, d, k):
    # seeded random sizes: ragged token counts, sequence lengths that do not divide them, widths and subspace
    # sizes off every tile boundary; three in four take the tensor-core kernels, the rest the plain ones
    rng = np.random.default_rng(n_tok * 7 + d)
    q, _ = np.linalg.qr(rng.standard_normal((d, k)))
    U = np.ascontiguousarray(q[:, :k], dtype=np.float32)
    X, ids, T_perp, pos = synth.gen_stage_boundary(n_tok, L, V, d, seed=n_tok)
    xt, f = _project(X, ids, T_perp, pos, U, L)
    assert f == 0
    ref = osub.project(X, ids, T_perp, pos, U, L)
    S = _scale_project(X, ids, T_perp, pos, U, L)
    assert np.all(np.abs(xt - ref) <= TOL * S + 1e-30)
    xh, f = _reconstruct(xt, ids, T_perp, pos, U, L)
    assert f == 0
    ref_h = osub.reconstruct(xt, ids, T_perp, pos, U, L)
    S_h = osub.abs_bound_reconstruct(xt, U) + np.abs(T_perp.astype(np.float64))[ids] + np.abs(pos.astype(np.float64))[np.arange(n_tok) % L]
    assert np.all(np.abs(xh - ref_h) <= TOL * S_h + 1e-30)
    # and the gradient form on the same activations
    gt, f = _project(X, None, None, None, U, L)
    assert f == 0
    assert np.all(np.abs(gt - osub.project(X, None, None, None, U, L)) <= TOL * (np.abs(X.astype(np.float64)) @ np.abs(U.astype(np.float64))) + 1e-30)
    # ... and back without embedding terms (the launch with two MMA-issuing warps; d / 128 odd, even or one block)
    gh, f = _reconstruct(gt, None, None, None, U, L)
    assert f == 0
    _check_reconstruct(gh, gt, None, None, None, U, L, f"gradient reconstruct {n_tok}x{d} k={k}")
