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
