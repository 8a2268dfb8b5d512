"""The byte counts behind the bench line's roofline figures (host only)."""
import importlib.util
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bench():
    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    mod = importlib.util.module_from_spec(spec)
    sys.modules["bench_module"] = mod
    spec.loader.exec_module(mod)
    return mod


def test_algorithmic_bytes_of_the_headline_configuration():
    from paper_2601_02360_b200 import synth
    b = _bench()
    wl = synth.workload("1b")
    n, R, nc = wl.n_total, wl.R, wl.n_chunks()
    assert (n, R, wl.k, wl.bits, nc) == (990455808, 8, 64, 2, 241829)
    msg = nc * (2 * 64 + 16 + 4)                       # 148 bytes per chunk: positions, codes, scale
    assert b.message_bytes(wl) == msg == 35790692
    assert b.compress_bytes(wl) == n * (12 * R + 4) + R * msg        # theta_local, e in and out per replica; theta_global once
    assert b.aggregate_apply_bytes(wl) == n * 8 + R * msg
    assert b.step_bytes_strict(wl) == n * (12 * R + 8) + 2 * R * msg
    assert round(b.compress_bytes(wl) / 1e9, 2) == 99.33
    assert round(b.aggregate_apply_bytes(wl) / 1e9, 2) == 8.21
    assert round(b.step_bytes_strict(wl) / 1e9, 2) == 103.58


def test_unquantised_messages():
    from paper_2601_02360_b200 import synth
    b = _bench()
    wl = synth.workload("tiny").replace(k=32, bits=32)
    assert b.message_bytes(wl) == wl.n_chunks() * (2 * 32 + 4 * 32 + 4)


def test_per_call_byte_count():
    from paper_2601_02360_b200 import synth
    b = _bench()
    wl = synth.workload("1b")
    n, R = wl.n_total, wl.R
    # every replica's compress reads theta_global itself: 16 bytes per replica-parameter instead of 12 + 4 / R
    assert b.step_bytes_api(wl) == n * (16 * R + 8) + 2 * R * b.message_bytes(wl)
    assert b.step_bytes_api(wl) - b.step_bytes_strict(wl) == 4 * n * R
    assert round(b.step_bytes_api(wl) / 1e9, 1) == 135.3


def test_host_step_groups_cover_the_arena():
    # the tensor groups of the host-buffer step are consecutive, never split a tensor and tile the arena and its chunks
    from paper_2601_02360_b200 import hoststep, synth
    wl = synth.workload("180m")
    off = wl.offsets()
    groups = hoststep.plan_groups(off, wl.chunk, 24)
    assert 1 < len(groups) <= 24
    assert groups[0].e0 == 0 and groups[-1].e1 == wl.n_total and groups[0].c0 == 0 and groups[-1].c1 == wl.n_chunks()
    for a, b_ in zip(groups[:-1], groups[1:]):
        assert a.e1 == b_.e0 and a.c1 == b_.c0 and a.t1 == b_.t0
    for g in groups:
        assert int(off[g.t0]) == g.e0 and int(off[g.t1]) == g.e1
        assert g.e0 % 4 == 0                    # a group starts on 16 bytes: its calls can take the tuned kernels
