"""Parity of sl_embed_reproject (paper §2.4, Eqs. 3-4) with the float64 CPU checker.

Tolerances are derived in tests/tf32_util.py from the arithmetic (operands rounded to the nearest TF32
value, exact products, float32 accumulation): a worst-case bound per entry (5 * 2^-11 * B with the
basis rounded to TF32 by the caller, 2^-8 * B with the basis as drawn, which the tensor cores cut),
a statistical bound per entry (8 standard deviations of the rounding noise, a fraction of a percent
of the result's RMS: the check that catches a dropped K step) and an RMS bound (2^-11 of the result's
RMS with a rounded basis).  The element-wise part (the subtraction and the addition of Eq. 3) is
float32 with one rounding each and is checked bit for bit from the kernel's own T_S output.
"""
import numpy as np
import pytest
import torch

import tf32_util as tu
from oracle import embed as oe
from paper_2601_02360_b200 import api, synth

pytestmark = pytest.mark.gpu

TOL = 2.0 ** -8          # worst case per entry, in units of B, with a basis that is not rounded


def _run(T_S, T_perp, U):
    T_S, T_perp, U = (np.ascontiguousarray(a, dtype=np.float32) for a in (T_S, T_perp, U))
    V, d = T_S.shape
    k = U.shape[1]
    ts = torch.from_numpy(T_S).cuda()
    tp = torch.from_numpy(T_perp).cuda()
    u = torch.from_numpy(U).cuda()
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.sl_embed_reproject(ts, tp, u, V, d, k, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    assert torch.equal(u.cpu(), torch.from_numpy(U))
    return ts.cpu().numpy(), tp.cpu().numpy()


def _check(T_S, T_perp, U, ts_gpu, tp_gpu, stat_rows=None, what="embed"):
    """Every check an output of the tensor-core kernel must pass; the statistical and RMS checks need a
    basis of TF32 values (tu.tf32_rna) and are left out otherwise."""
    rounded = tu.is_tf32(U)
    stat, ref_ts = tu.check_projection(ts_gpu, T_S, U, what, rounded_basis=rounded, rows=stat_rows)
    if ref_ts.size >= 4096:                  # a norm over a handful of entries is not a norm
        tu.check_rms(ts_gpu, ref_ts, what, rounded_basis=rounded)
    _, ref_tp = oe.embed_reproject(T_S, T_perp, U)
    assert np.array_equal(oe.embed_reproject(T_S, T_perp, U)[0], ref_ts)
    tiny = 1e-30
    err_ts = np.abs(ts_gpu.astype(np.float64) - ref_ts)
    ulp = 2.0 ** -23 * (np.abs(ref_tp) + np.abs(T_S) + np.abs(ref_ts))
    err_tp = np.abs(tp_gpu.astype(np.float64) - ref_tp)
    assert np.all(err_tp <= err_ts + 2 * ulp + tiny)      # T_perp carries the same error, plus two float32 roundings
    # Eq. 3 in float32, one rounding per operation, from the very T_S that was stored
    expect_tp = (T_perp + (T_S - ts_gpu)).astype(np.float32)
    assert np.array_equal(expect_tp.view(np.uint32), tp_gpu.view(np.uint32))
    # the table T_S + T_perp is conserved to float32 rounding
    te_err = np.abs((ts_gpu.astype(np.float64) + tp_gpu) - (T_S.astype(np.float64) + T_perp))
    assert np.all(te_err <= 2 * ulp + tiny)
    if stat is not None:
        print(f"{what}: max err / statistical bound {stat[0]:.3f}; bound = {100 * stat[1]:.2f} % of RMS(Pi)")
    return err_ts, ref_ts, stat


def _basis(d, k, seed, rounded=True):
    U = synth.gen_subspace_basis(d, k, seed=seed)
    return tu.tf32_rna(U) if rounded else U


@pytest.mark.parametrize("rounded", [True, False], ids=["basis_rounded", "basis_as_drawn"])
@pytest.mark.parametrize("V,d,k", [(1000, 512, 64), (333, 2048, 256), (129, 132, 12), (5, 64, 4),
                                   (260, 1536, 192), (128, 128, 32), (257, 1000, 200), (64, 2048, 8)])
def test_parity_random(V, d, k, rounded):
    U = _basis(d, k, 1, rounded)
    T_S, T_perp = synth.gen_embedding_pair(V, d, seed=2)
    ts_gpu, tp_gpu = _run(T_S, T_perp, U)
    err, ref, _ = _check(T_S, T_perp, U, ts_gpu, tp_gpu, what=f"random {V}x{d} k={k}")
    # typical accuracy.  The tensor cores CUT a float32 operand to TF32 (they do not round).  The kernel
    # rounds T_S and the coordinates itself; U is used as given (not rounded in this test), so each of
    # its two uses loses between 0 and 2^-10 of its magnitude, about 0.75 * 2^-11 on average for these
    # values: the result comes out about 7e-4 short.  The difference stays in T_perp (checked above:
    # T_S + T_perp is conserved).  (_check holds the RMS error to 2^-9 of the result's RMS then, and to
    # 2^-11 with the rounded basis.)


@pytest.mark.parametrize("V,d,k", [(300, 256, 8), (130, 512, 32), (128, 2048, 256), (77, 384, 100)])
def test_exact_when_tf32_is_exact(V, d, k):
    # U = k columns of the identity and dyadic table entries with <= 10 significant bits: every
    # product and every sum is exact in TF32 / float32, so the result must match bit for bit.
    rng = np.random.default_rng(3)
    cols = rng.permutation(d)[:k]
    U = np.zeros((d, k), dtype=np.float32)
    U[cols, np.arange(k)] = 1.0
    T_S = (rng.integers(-512, 513, size=(V, d)) / 64.0).astype(np.float32)
    T_perp = (rng.integers(-512, 513, size=(V, d)) / 64.0).astype(np.float32)
    ts_gpu, tp_gpu = _run(T_S, T_perp, U)
    ref_ts, ref_tp = oe.embed_reproject(T_S, T_perp, U)
    assert np.array_equal(ts_gpu, ref_ts.astype(np.float32))
    assert np.array_equal(tp_gpu, ref_tp.astype(np.float32))


def test_signed_basis_exact():
    # columns of +-1/2-scaled Hadamard-like vectors keep everything dyadic: catches a transposed or
    # mis-swizzled operand that the identity columns (symmetric in their own way) could hide
    d, k, V = 64, 4, 200
    H = np.array([[1.0]])
    while H.shape[0] < d:
        H = np.block([[H, H], [H, -H]])
    U = (H[:, [1, 6, 11, 40]] / 8.0).astype(np.float32)          # orthonormal: |column|^2 = 64/64
    rng = np.random.default_rng(4)
    T_S = (rng.integers(-8, 9, size=(V, d)) / 4.0).astype(np.float32)
    T_perp = (rng.integers(-8, 9, size=(V, d)) / 4.0).astype(np.float32)
    ts_gpu, tp_gpu = _run(T_S, T_perp, U)
    ref_ts, ref_tp = oe.embed_reproject(T_S, T_perp, U)
    assert np.array_equal(ts_gpu, ref_ts.astype(np.float32))
    assert np.array_equal(tp_gpu, ref_tp.astype(np.float32))


def test_second_application_is_a_fixed_point_up_to_tf32():
    V, d, k = 256, 1024, 128
    U = _basis(d, k, 5)
    T_S, T_perp = synth.gen_embedding_pair(V, d, seed=6)
    ts1, tp1 = _run(T_S, T_perp, U)
    ts2, tp2 = _run(ts1, tp1, U)
    _check(ts1, tp1, U, ts2, tp2, what="second application")
    # a table already in the subspace moves by rounding noise only: 2^-10 of its RMS (two applications' noise)
    assert tu.rms(ts2.astype(np.float64) - ts1) <= 2.0 ** -10 * tu.rms(ts1)


def test_full_table_of_the_1b_model():
    # the table bench.py --embed times: 250 sub-tiles over all CTAs.  Worst-case and RMS bounds on every
    # entry; the statistical bound (which needs a d x d product per row) on the rows around every boundary
    # between two CTAs' shares and between sub-tiles plus random ones.
    V, d, k = 32000, 2048, 256
    U = _basis(d, k, 7)
    T_S, T_perp = synth.gen_embedding_pair(V, d, seed=8)
    ts_gpu, tp_gpu = _run(T_S, T_perp, U)
    G = (V + 31) // 32
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    edges = np.unique(np.array([(c * G // sms) * 32 for c in range(sms + 1)]))
    near = np.concatenate([edges + o for o in (-1, 0, 1, 127, 128, 129)])
    rows = np.unique(np.clip(np.concatenate([[0, V - 1], near, np.random.default_rng(1).integers(0, V, 1500)]), 0, V - 1))
    _, ref, stat = _check(T_S, T_perp, U, ts_gpu, tp_gpu, stat_rows=rows, what="1b table")
    # the check can fail where it matters: the per-entry bound is a small fraction of the result's RMS
    # (a dropped 32-column K step of the first contraction moves Pi by 12 % of its RMS)
    assert stat[1] <= 0.05, stat


def _hadamard(n):
    H = np.array([[1.0]])
    while H.shape[0] < n:
        H = np.block([[H, H], [H, -H]])
    return H


@pytest.mark.parametrize("d,k,kind", [(1024, 128, "hadamard"), (2048, 256, "identity"), (256, 64, "hadamard"),
                                      (640, 100, "identity")])
def test_exact_on_every_cta_with_two_sub_tiles_each(d, k, kind):
    # enough rows for at least two sub-tiles on every CTA (148 x 256 and a ragged rest), dyadic entries
    # and a basis of identity or +-1/sqrt(d) Hadamard columns (d a power of 4): every product, every sum
    # and both roundings to TF32 are exact, so all of T_S and T_perp must match the checker bit for bit
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    V = sms * 256 + 96
    rng = np.random.default_rng(d + k)
    if kind == "identity":
        U = np.zeros((d, k), dtype=np.float32)
        U[rng.permutation(d)[:k], np.arange(k)] = 1.0
        T_S = (rng.integers(-512, 513, size=(V, d)) / 64.0).astype(np.float32)
    else:
        U = (_hadamard(d)[:, rng.permutation(d)[:k]] / np.sqrt(d)).astype(np.float32)
        assert np.array_equal(U.astype(np.float64).T @ U, np.eye(k))
        T_S = (rng.integers(-8, 9, size=(V, d)) / 4.0).astype(np.float32)
        P = T_S.astype(np.float64) @ U
        assert tu.is_tf32(P.astype(np.float32)) and np.array_equal(P.astype(np.float32), P)   # the coordinates survive TF32
    T_perp = (rng.integers(-512, 513, size=(V, d)) / 64.0).astype(np.float32)
    ts_gpu, tp_gpu = _run(T_S, T_perp, U)
    ref_ts, ref_tp = oe.embed_reproject(T_S, T_perp, U)
    assert np.array_equal(ref_ts.astype(np.float32), ref_ts) and np.array_equal(ref_tp.astype(np.float32), ref_tp)
    assert np.array_equal(ts_gpu, ref_ts.astype(np.float32))
    assert np.array_equal(tp_gpu, ref_tp.astype(np.float32))


def test_captured_in_a_cuda_graph():
    # the tensor maps are built on the host at call time and travel in the kernel parameters, so the
    # call can be captured and replayed on the same buffers
    V, d, k = 500, 512, 64
    U = synth.gen_subspace_basis(d, k, seed=9)
    T_S, T_perp = synth.gen_embedding_pair(V, d, seed=10)
    ts, tp, u = torch.from_numpy(T_S).cuda(), torch.from_numpy(T_perp).cuda(), torch.from_numpy(U).cuda()
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            api.sl_embed_reproject(ts, tp, u, V, d, k, flags, stream=side)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    assert torch.equal(ts.cpu(), torch.from_numpy(T_S))
    graph.replay()
    torch.cuda.synchronize()
    _check(T_S, T_perp, U, ts.cpu().numpy(), tp.cpu().numpy())
    assert int(flags.item()) == 0


def test_initial_split_is_the_same_call_on_a_zero_t_perp():
    # §2.4, before training: T_S <- TE U U^T, T_perp <- TE - T_S.  With T_S = TE and T_perp = 0 the
    # re-projection computes exactly that.
    V, d, k = 640, 768, 96
    U = synth.gen_subspace_basis(d, k, seed=11)
    TE, _ = synth.gen_embedding_pair(V, d, seed=12)
    ts_gpu, tp_gpu = _run(TE, np.zeros_like(TE), U)
    ref_ts, ref_tp = oe.embed_init(TE, U)
    B = oe.abs_bound(TE, U)
    assert np.all(np.abs(ts_gpu - ref_ts) <= TOL * B + 1e-30)
    assert np.all(np.abs(tp_gpu - ref_tp) <= TOL * B + 1e-30)
    assert tu.rms(ts_gpu - ref_ts) <= 2.0 ** -9 * tu.rms(ref_ts)
    assert np.array_equal(tp_gpu, (TE - ts_gpu).astype(np.float32))
    # and the table is back exactly: T_S + T_perp == TE wherever the subtraction was exact, else 1 ulp
    assert np.all(np.abs((ts_gpu.astype(np.float64) + tp_gpu) - TE) <= 2.0 ** -23 * (np.abs(TE) + np.abs(ts_gpu)))


@pytest.mark.parametrize("V,d,k", [(1, 4, 4), (2, 8, 8), (31, 36, 4), (33, 60, 16), (127, 260, 256), (200, 124, 100),
                                   (96, 4096, 32), (385, 96, 96), (1000, 64, 64), (160, 2052, 252)])
def test_odd_shapes(V, d, k):
    # sizes below one tile, k = d (the projection is the identity up to TF32), d and k off the
    # 32 / 128 grids: everything outside the matrices is zero-filled on load and clipped on store
    U = _basis(d, k, 21)
    T_S, T_perp = synth.gen_embedding_pair(V, d, seed=22)
    ts_gpu, tp_gpu = _run(T_S, T_perp, U)
    _check(T_S, T_perp, U, ts_gpu, tp_gpu, what=f"odd {V}x{d} k={k}")


def test_neighbouring_memory_is_untouched():
    # the table sits in the middle of a larger allocation: rows before and after it must not change
    V, d, k = 130, 200, 40
    U = synth.gen_subspace_basis(d, k, seed=23)
    T_S, T_perp = synth.gen_embedding_pair(V + 64, d, seed=24)
    big_s, big_p = torch.from_numpy(T_S).cuda(), torch.from_numpy(T_perp).cuda()
    u = torch.from_numpy(U).cuda()
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.sl_embed_reproject(big_s[32:32 + V], big_p[32:32 + V], u, V, d, k, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    hs, hp = big_s.cpu().numpy(), big_p.cpu().numpy()
    assert np.array_equal(hs[:32], T_S[:32]) and np.array_equal(hs[32 + V:], T_S[32 + V:])
    assert np.array_equal(hp[:32], T_perp[:32]) and np.array_equal(hp[32 + V:], T_perp[32 + V:])
    _check(T_S[32:32 + V], T_perp[32:32 + V], U, hs[32:32 + V], hp[32:32 + V])


GEN_TOL = 2.0 ** -20      # float32 fused multiply-adds over d and k terms: far below (d + k) * 2^-24 of B in practice


@pytest.mark.parametrize("V,d,k", [(50, 1536, 2), (33, 10, 3), (9, 7, 7), (100, 62, 6), (20, 64, 300), (17, 5, 1),
                                   (300, 2048, 260)])
def test_shapes_outside_the_tensor_core_path(V, d, k):
    # the paper's smallest subspaces (k = 2 at d = 1536), odd d and k, k above 256: plain float32 kernel
    if k <= d:
        U = synth.gen_subspace_basis(d, k, seed=31)
    else:     # more columns than rows cannot be orthonormal; the call does not check, any matrix will do
        U = (np.random.default_rng(31).standard_normal((d, k)) / np.sqrt(k)).astype(np.float32)
    T_S, T_perp = synth.gen_embedding_pair(V, d, seed=32)
    ts_gpu, tp_gpu = _run(T_S, T_perp, U)
    ref_ts, ref_tp = oe.embed_reproject(T_S, T_perp, U)
    B = oe.abs_bound(T_S, U)
    assert np.all(np.abs(ts_gpu - ref_ts) <= GEN_TOL * B + 1e-30), float((np.abs(ts_gpu - ref_ts) / (B + 1e-30)).max())
    assert np.array_equal(tp_gpu, (T_perp + (T_S - ts_gpu)).astype(np.float32))
    assert np.all(np.abs(tp_gpu - ref_tp) <= GEN_TOL * B + 2.0 ** -22 * (np.abs(ref_tp) + np.abs(T_S) + np.abs(ref_ts)))


def test_unaligned_tables_take_the_plain_kernel():
    V, d, k = 40, 128, 32
    U = synth.gen_subspace_basis(d, k, seed=33)
    T_S, T_perp = synth.gen_embedding_pair(V, d, seed=34)
    buf = torch.zeros(V * d + 1, dtype=torch.float32, device="cuda")
    ts = buf[1:]                                   # 4-byte aligned only
    ts.copy_(torch.from_numpy(T_S).reshape(-1))
    tp, u = torch.from_numpy(T_perp).cuda(), torch.from_numpy(U).cuda()
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.sl_embed_reproject(ts, tp, u, V, d, k, flags)
    torch.cuda.synchronize()
    ref_ts, _ = oe.embed_reproject(T_S, T_perp, U)
    got = ts.cpu().numpy().reshape(V, d)
    assert np.all(np.abs(got - ref_ts) <= GEN_TOL * oe.abs_bound(T_S, U) + 1e-30)
    assert float(buf[0].item()) == 0.0 and int(flags.item()) == 0


_tf32_rna = tu.tf32_rna


def test_round_tf32_helper():
    rng = np.random.default_rng(41)
    x = np.concatenate([rng.standard_normal(5000).astype(np.float32) * np.float32(10.0) ** rng.integers(-20, 20, 5000),
                        np.array([0.0, -0.0, 1.0, 1.0 + 2.0 ** -11, 1.0 + 2.0 ** -11 + 2.0 ** -23, 1.0 + 2.0 ** -10,
                                  -(1.0 + 2.0 ** -11), 3.0e38, 1e-40, np.inf, -np.inf], dtype=np.float32)]).astype(np.float32)
    t = torch.from_numpy(x.copy()).cuda()
    api.sl_round_tf32(t, t.numel())
    got = t.cpu().numpy()
    want = _tf32_rna(x)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert np.all((got.view(np.uint32) & 0x1FFF) == 0)                 # representable in TF32
    assert got[5002] == 1.0 and got[5003] == np.float32(1.0 + 2.0 ** -10)   # the tie goes away from zero
    api.sl_round_tf32(t, t.numel())
    assert np.array_equal(t.cpu().numpy().view(np.uint32), got.view(np.uint32))   # idempotent


@pytest.mark.parametrize("V,d,k", [(2000, 2048, 256), (1000, 1024, 32)])
def test_no_systematic_shortening_with_a_rounded_basis(V, d, k):
    # with U rounded once (sl_round_tf32) every operand the tensor cores see is a TF32 value: what is
    # left are rounding errors of random sign, far smaller than the 7e-4 that a cut basis costs
    U = synth.gen_subspace_basis(d, k, seed=42)
    u = torch.from_numpy(U).cuda()
    api.sl_round_tf32(u, u.numel())
    Ur = u.cpu().numpy()
    assert np.array_equal(Ur.view(np.uint32), _tf32_rna(U).view(np.uint32))
    T_S, T_perp = synth.gen_embedding_pair(V, d, seed=43)
    ts_gpu, tp_gpu = _run(T_S, T_perp, Ur)
    err, ref, _ = _check(T_S, T_perp, Ur, ts_gpu, tp_gpu, what="rounded basis")
    rel = np.sqrt((err ** 2).mean()) / np.sqrt((ref ** 2).mean())
    assert rel <= 2.0 ** -11, rel
    # no bias: the result is neither systematically shorter nor longer than the exact projection
    ratio = float((ts_gpu.astype(np.float64) * ref).sum() / (ref * ref).sum())
    assert abs(ratio - 1.0) <= 1e-4, ratio
