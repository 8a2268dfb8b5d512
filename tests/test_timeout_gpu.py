"""The give-up path of the bounded on-chip waits, driven without any fault: the wait limit is set to
"no poll" (every wait gives up at once) or to one poll through the debugging aid of the C ABI, so the
copy a wait stood for still arrives and is drained like any other.  Each call must return SL_OK with
SL_FLAG_TIMEOUT raised (certain with "no poll", possible with one), the device must stay usable, and
the same call on the same buffers with the default limit must then match the CPU checker."""
import numpy as np
import pytest
import torch

from oracle import embed as oe
from oracle import slo
from oracle import subspace as osub
from paper_2601_02360_b200 import api, synth
from parity_util import GpuStep, assert_close, compare_messages, oracle_compress_all

pytestmark = pytest.mark.gpu
f32 = np.float32


@pytest.fixture
def wait_limit():
    """Sets the limit for the duration of a test and always restores the default."""
    yield api.sl_debug_set_wait_limit
    api.sl_debug_set_wait_limit(0)


def _arena(R, seed):
    sizes = [700 * 4096, 1024, 5 * 4096 + 2048]       # several chunks per resident CTA, short tails
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
    rng = np.random.default_rng(seed)
    n = int(off[-1])
    tg = rng.normal(0, 0.02, n).astype(f32)
    tls = [(tg + rng.normal(0, 1e-3, n).astype(f32)).astype(f32) for _ in range(R)]
    errs = [rng.normal(0, 5e-4, n).astype(f32) for _ in range(R)]
    return off, tg, tls, errs


@pytest.mark.parametrize("polls", [-1, 1])
def test_compress_and_aggregate_give_up_cleanly(wait_limit, polls):
    R, chunk, k, bits, beta, lr = 5, 4096, 64, 2, 0.95, 0.8      # R * k = 320: the averaging kernel that prefetches theta_global
    off, tg, tls, errs = _arena(R, 11)
    gs = GpuStep(off, R, chunk, k, bits)
    gs.upload(tg, tls, errs)
    wait_limit(polls)
    gs.compress(beta)                                  # returns SL_OK (the binding raises otherwise)
    torch.cuda.synchronize()
    f = int(gs.flags.item())
    assert f & ~api.SL_FLAG_TIMEOUT == 0
    if polls < 0:
        assert f & api.SL_FLAG_TIMEOUT, "no wait was allowed to succeed, yet no time-out was reported"
    # the same buffers, default limit: a normal compress matches the checker
    wait_limit(0)
    gs.flags.zero_()
    gs.upload(tg, tls, errs)
    gs.compress(beta)
    h_err = [e.copy() for e in errs]
    res = oracle_compress_all(tls, tg, h_err, off, beta, chunk, k, bits)
    msgs = [(i, c, s) for i, c, s, _ in res]
    compare_messages(gs.messages_host(), msgs, "after a give-up")
    for r in range(R):
        assert_close(gs.err[r].cpu().numpy(), h_err[r], f"err[{r}] after a give-up")
    # now the averaging kernel gives up ...
    wait_limit(polls)
    gs.aggregate_apply(lr)
    torch.cuda.synchronize()
    f = int(gs.flags.item())
    assert f & ~api.SL_FLAG_TIMEOUT == 0
    if polls < 0:
        assert f & api.SL_FLAG_TIMEOUT
    # ... and works again on the same buffers
    wait_limit(0)
    gs.flags.zero_()
    gs.theta_global.copy_(torch.from_numpy(tg))
    gs.aggregate_apply(lr)
    want = tg.copy()
    slo.outer_apply(want, slo.aggregate(msgs, off, chunk, k, bits), lr)
    assert_close(gs.theta_global.cpu().numpy(), want, "theta_global after a give-up")
    assert int(gs.flags.item()) == 0


@pytest.mark.parametrize("polls", [-1, 1])
def test_tensor_core_kernels_give_up_cleanly(wait_limit, polls):
    V, d, k, n_tok, L = 148 * 256 + 40, 256, 64, 148 * 256 + 72, 128
    U = synth.gen_subspace_basis(d, k, 3)
    T_S, T_perp = synth.gen_embedding_pair(V, d, 3)
    X, ids, Tp, pos = synth.gen_stage_boundary(n_tok, L, V, d, 3)
    d_u = torch.from_numpy(U).cuda()
    api.sl_round_tf32(d_u, d_u.numel())
    U = d_u.cpu().numpy()
    d_ts, d_tp = torch.from_numpy(T_S).cuda(), torch.from_numpy(T_perp).cuda()
    d_x, d_ids, d_tp2, d_pos = (torch.from_numpy(a).cuda() for a in (X, ids, Tp, pos))
    d_xt = torch.zeros(n_tok, k, dtype=torch.float32, device="cuda")
    d_xh = torch.zeros(n_tok, d, dtype=torch.float32, device="cuda")
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")

    def run_all():
        api.sl_embed_reproject(d_ts, d_tp, d_u, V, d, k, flags)
        api.sl_subspace_project(d_x, d_ids, d_tp2, d_pos, d_u, n_tok, L, V, d, k, d_xt, flags)
        api.sl_subspace_project(d_x, None, None, None, d_u, n_tok, L, 0, d, k, d_xt, flags)     # the two-sub-tile form
        api.sl_subspace_project(d_x, d_ids, d_tp2, d_pos, d_u, n_tok // (2 * L) * 2 * L, L, V, d, k, d_xt, flags)   # pairs of sequences
        api.sl_subspace_reconstruct(d_xt, d_ids, d_tp2, d_pos, d_u, n_tok, L, V, d, k, d_xh, flags)
        api.sl_subspace_reconstruct(d_xt, None, None, None, d_u, n_tok, L, 0, d, k, d_xh, flags)    # two MMA warps, two rings
        torch.cuda.synchronize()

    wait_limit(polls)
    run_all()
    f = int(flags.item())
    assert f & ~api.SL_FLAG_TIMEOUT == 0
    if polls < 0:
        assert f & api.SL_FLAG_TIMEOUT
    wait_limit(0)
    flags.zero_()
    d_ts.copy_(torch.from_numpy(T_S))
    d_tp.copy_(torch.from_numpy(T_perp))
    api.sl_embed_reproject(d_ts, d_tp, d_u, V, d, k, flags)
    api.sl_subspace_project(d_x, d_ids, d_tp2, d_pos, d_u, n_tok, L, V, d, k, d_xt, flags)
    api.sl_subspace_reconstruct(d_xt, d_ids, d_tp2, d_pos, d_u, n_tok, L, V, d, k, d_xh, flags)
    torch.cuda.synchronize()
    assert int(flags.item()) == 0
    ref_ts, _ = oe.embed_reproject(T_S, T_perp, U)
    assert (np.abs(d_ts.cpu().numpy() - ref_ts) <= 2.0 ** -9 * oe.abs_bound(T_S, U) + 1e-30).all()
    g_xt = d_xt.cpu().numpy()
    assert (np.abs(g_xt - osub.project(X, ids, Tp, pos, U, L))
            <= 2.0 ** -9 * osub.abs_bound_project(X, ids, Tp, pos, U, L) + 1e-30).all()
    assert (np.abs(d_xh.cpu().numpy() - osub.reconstruct(g_xt, ids, Tp, pos, U, L))
            <= 2.0 ** -9 * osub.abs_bound_reconstruct(g_xt, U) + 1e-6).all()
