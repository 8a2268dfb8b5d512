"""Host-only checks of the C ABI: the library loads without a GPU, exports every symbol the
header declares, and rejects bad arguments before anything is launched."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2601_02360_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "sparseloco.h")


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.load()


def _declared():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(sl_[a-z0-9_]+)\s*\(", src)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert set(names) == set(api.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(RuntimeError, match="no fallback"):
        api.load(str(tmp_path / "absent.so"))


def test_sizes(lib):
    lay = api.Layout([0, 4096 * 3 + 5, 4096 * 3 + 5, 4096 * 4 + 5 + 100])
    assert api.sl_num_chunks(lay, 4096) == 4 + 0 + 2
    assert api.sl_num_chunks(lay, 0) == 0
    assert api.sl_codes_stride(64, 2) == 16
    assert api.sl_codes_stride(2, 2) == 1
    assert api.sl_codes_stride(63, 4) == 32
    assert api.sl_codes_stride(32, 32) == 128
    assert api.sl_codes_stride(64, 3) == 0
    lay = api.Layout([0, 4096 * 2 + 5, 4096 * 2 + 105])
    assert api.sl_codes_bytes(lay, 4096, 64, 2) == 4 * 16
    assert api.sl_codes_bytes(lay, 4096, 32, 32) == 4 * 128
    assert api.sl_codes_bytes(lay, 4096, 64, 3) == 0 and api.sl_codes_bytes(lay, 32, 64, 2) == 0
    assert api.strerror(api.SL_OK) == "ok" and "align" in api.strerror(api.SL_ERR_ALIGNMENT)


def test_tile_geometry_sizes(lib):
    lay = api.Layout([0, 24], cols=[6])                 # a 4 x 6 matrix
    assert api.sl_num_chunks(lay, 16) == 1 * 2          # 4 x 4 tiles: one tile row, two tile columns
    assert api.sl_num_chunks(lay, 4) == 2 * 3
    assert api.sl_num_chunks(lay, 8) == 0               # 8 is not a square
    assert api.sl_num_chunks(api.Layout([0, 24], cols=[5]), 16) == 0   # 24 elements are not rows of 5
    assert api.sl_num_chunks(api.Layout([0, 24, 30], cols=[6, 0]), 16) == 2 + 1
    assert api.sl_num_chunks(api.Layout([0, 24], cols=[0]), 8) == 3    # no tiles: any chunk size


def _call_compress(lib, lay, chunk=4096, k=64, bits=2, beta=0.95, ptr=0x1000, idx=0x1000, R=None):
    if R is None:
        return lib.sl_compress(ptr, 0x1000, 0x1000, lay.ref(), beta, chunk, k, bits, idx, 0x1000, 0x1000, 0, 0)
    tab = (ctypes.c_void_p * max(R, 1))(*([0x1000] * max(R, 1)))
    return lib.sl_compress_batch(R, tab, 0x1000, tab, lay.ref(), beta, chunk, k, bits, tab, tab, tab, 0, 0)


def test_bad_arguments_are_rejected_on_the_host(lib):
    # every call below must return before any CUDA work: the pointers are fake
    lay = api.Layout([0, 8192])
    E = api
    assert _call_compress(lib, lay, k=0) == E.SL_ERR_INVALID_ARG
    assert _call_compress(lib, lay, chunk=64, k=65) == E.SL_ERR_INVALID_ARG
    assert _call_compress(lib, lay, bits=3) == E.SL_ERR_INVALID_ARG
    assert _call_compress(lib, lay, chunk=0) == E.SL_ERR_INVALID_ARG
    assert _call_compress(lib, lay, beta=float("nan")) == E.SL_ERR_INVALID_ARG
    assert _call_compress(lib, lay, beta=float("inf")) == E.SL_ERR_INVALID_ARG
    assert _call_compress(lib, lay, ptr=0) == E.SL_ERR_INVALID_ARG
    assert _call_compress(lib, lay, chunk=api.SL_MAX_CHUNK + 1) == E.SL_ERR_UNSUPPORTED
    assert _call_compress(lib, lay, ptr=0x1002) == E.SL_ERR_ALIGNMENT
    assert _call_compress(lib, lay, idx=0x1001) == E.SL_ERR_ALIGNMENT
    assert _call_compress(lib, lay, R=0) == E.SL_ERR_INVALID_ARG
    assert _call_compress(lib, lay, R=api.SL_MAX_REPLICAS + 1) == E.SL_ERR_INVALID_ARG
    assert lib.sl_compress(0x1000, 0x1000, 0x1000, None, 0.9, 4096, 64, 2, 0x1000, 0x1000, 0x1000, 0, 0) \
        == E.SL_ERR_INVALID_ARG
    bad = api.Layout([0, 100, 50, 200])           # offsets go backwards
    assert _call_compress(lib, bad) == E.SL_ERR_INVALID_ARG
    wrong_total = api.Layout([0, 100, 200])
    wrong_total.c.n_total = 150
    assert _call_compress(lib, wrong_total) == E.SL_ERR_INVALID_ARG
    many = api.Layout(np.arange(api.SL_MAX_TENSORS + 2) * 4)
    assert _call_compress(lib, many) == E.SL_ERR_UNSUPPORTED
    assert _call_compress(lib, api.Layout([0, 24], cols=[6]), chunk=8, k=2) == E.SL_ERR_INVALID_ARG    # not a square
    assert _call_compress(lib, api.Layout([0, 24], cols=[5]), chunk=16, k=2) == E.SL_ERR_INVALID_ARG   # not whole rows
    tab = (ctypes.c_void_p * 2)(0x1000, 0x1000)
    assert lib.sl_aggregate(2, tab, tab, tab, lay.ref(), 4096, 64, 2, 0, 0, 0) == E.SL_ERR_INVALID_ARG
    assert lib.sl_aggregate(0, tab, tab, tab, lay.ref(), 4096, 64, 2, 0x1000, 0, 0) == E.SL_ERR_INVALID_ARG
    assert lib.sl_aggregate_apply(2, tab, tab, tab, lay.ref(), 4096, 64, 2, 0x1000, float("nan"), 0, 0) \
        == E.SL_ERR_INVALID_ARG
    assert lib.sl_aggregate_apply(2, tab, tab, tab, lay.ref(), 4096, 64, 5, 0x1000, 1.0, 0, 0) \
        == E.SL_ERR_INVALID_ARG
    assert lib.sl_outer_apply(0, 0x1000, 10, 1.0, 0) == E.SL_ERR_INVALID_ARG
    assert lib.sl_outer_apply(0x1001, 0x1000, 10, 1.0, 0) == E.SL_ERR_ALIGNMENT
    assert lib.sl_outer_apply(0x1000, 0x1000, 10, float("inf"), 0) == E.SL_ERR_INVALID_ARG


def test_binding_raises_with_the_library_message(lib):
    with pytest.raises(api.SparseLoCoError, match="invalid argument"):
        api.sl_compress(0x1000, 0x1000, 0x1000, [0, 8192], 0.9, 4096, 0, 2, 0x1000, 0x1000, 0x1000, None, 0)


def test_embed_reproject_argument_checks():
    L = api.load()
    fake = 0x10000
    call = lambda ts, tp, u, V, d, k: L.sl_embed_reproject(ts, tp, u, V, d, k, None, None)
    assert call(None, fake, fake, 8, 64, 8) == api.SL_ERR_INVALID_ARG
    assert call(fake, fake, None, 8, 64, 8) == api.SL_ERR_INVALID_ARG
    assert call(fake, fake, fake, 8, 64, 0) == api.SL_ERR_INVALID_ARG
    assert call(fake, fake, fake, 8, 0, 4) == api.SL_ERR_INVALID_ARG
    assert call(fake + 2, fake, fake, 8, 64, 8) == api.SL_ERR_ALIGNMENT
    assert call(fake, fake, fake + 1, 8, 64, 8) == api.SL_ERR_ALIGNMENT
    assert call(fake, fake, fake, 8, 64, 5000) == api.SL_ERR_UNSUPPORTED      # k above 4096
    assert call(fake, fake, fake, 1 << 31, 64, 8) == api.SL_ERR_UNSUPPORTED   # V at or above 2^31
    assert call(fake, fake, fake, 0, 64, 8) == api.SL_OK                      # an empty table is a no-op
    assert call(fake, fake, fake, 0, 62, 6) == api.SL_OK


def test_idx12_argument_checks():
    L = api.load()
    assert [api.sl_idx12_stride(k) for k in (0, 1, 2, 3, 64)] == [0, 2, 3, 5, 96]
    fake = 0x10000
    assert L.sl_pack_idx12(None, 4, 64, fake, None, None) == api.SL_ERR_INVALID_ARG
    assert L.sl_pack_idx12(fake, 4, 0, fake, None, None) == api.SL_ERR_INVALID_ARG
    assert L.sl_pack_idx12(fake + 1, 4, 64, fake, None, None) == api.SL_ERR_ALIGNMENT
    assert L.sl_pack_idx12(fake, 0, 64, fake, None, None) == api.SL_OK        # nothing to do
    lay = api.Layout([0, 100])
    assert L.sl_unpack_idx12(None, lay.ref(), 4096, 64, fake, None) == api.SL_ERR_INVALID_ARG
    assert L.sl_unpack_idx12(fake, lay.ref(), 8192, 64, fake, None) == api.SL_ERR_UNSUPPORTED   # 13-bit positions
    assert L.sl_unpack_idx12(fake, lay.ref(), 4096, 64, fake + 1, None) == api.SL_ERR_ALIGNMENT


def test_subspace_argument_checks():
    # all checks happen on the host before any launch, so fake addresses are enough
    L = api.load()
    fake = 0x10000
    for fn in (L.sl_subspace_project, L.sl_subspace_reconstruct):
        ok_args = [fake, fake, fake, fake, fake, 0, 64, 100, 256, 32, fake, None, None]     # n_tok = 0: nothing to do
        assert fn(*ok_args) == api.SL_OK
        def call(**kw):
            a = list(ok_args)
            a[5] = 128
            for i, v in kw.items():
                a[int(i[1:])] = v
            return fn(*a)
        assert call(_0=None) == api.SL_ERR_INVALID_ARG            # no input
        assert call(_4=None) == api.SL_ERR_INVALID_ARG            # no basis
        assert call(_10=None) == api.SL_ERR_INVALID_ARG           # no output
        assert call(_8=0) == api.SL_ERR_INVALID_ARG               # d = 0
        assert call(_9=0) == api.SL_ERR_INVALID_ARG               # k = 0
        assert call(_2=None) == api.SL_ERR_INVALID_ARG            # token ids without an embedding table
        assert call(_3=None) == api.SL_ERR_INVALID_ARG            # ... without positions
        assert call(_6=0) == api.SL_ERR_INVALID_ARG               # ... with sequence length 0
        assert call(_0=fake + 2) == api.SL_ERR_ALIGNMENT
        assert call(_1=fake + 1) == api.SL_ERR_ALIGNMENT
        assert call(_11=fake + 2) == api.SL_ERR_ALIGNMENT
        assert call(_9=4100) == api.SL_ERR_UNSUPPORTED            # k above 4096
        assert call(_5=1 << 31) == api.SL_ERR_UNSUPPORTED         # n_tok at or above 2^31
        assert call(_7=1 << 31) == api.SL_ERR_UNSUPPORTED         # V at or above 2^31


def test_header_is_valid_c_and_a_c_client_links(lib, tmp_path):
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no gcc")
    exe = str(tmp_path / "abi_c_client")
    libdir = os.path.dirname(build.LIB_PATH)
    cmd = ["gcc", "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(ROOT, "include"),
           os.path.join(ROOT, "tests", "support", "abi_c_client.c"), "-o", exe,
           "-L", libdir, "-lsparseloco", f"-Wl,-rpath,{libdir}"]
    built = subprocess.run(cmd, capture_output=True, text=True)
    assert built.returncode == 0, built.stderr[-2000:]
    run = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert run.returncode == 0, (run.returncode, run.stdout, run.stderr[-1000:])
    assert run.stdout.startswith("c client ok")
