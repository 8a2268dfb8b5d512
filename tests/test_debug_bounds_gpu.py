"""The bounds-checked debug build (-DSL_DEBUG_BOUNDS): every shared- and global-memory index of the
Eq. 2 kernels is range-checked, a violation raises SL_FLAG_BOUNDS and skips the access.  This is the
stand-in for a memory checker on GPUs where none may be run.  The small parity cases are run once more
against that build (in a child pytest, so that this process keeps the normal library): they compare
every output with the CPU checker AND require the device flags to equal the checker's, so any raised
SL_FLAG_BOUNDS fails them."""
import os
import subprocess
import sys

import pytest
import torch

from paper_2601_02360_b200 import api, build

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SMALL_CASES = ("test_hand_worked_example_on_gpu or test_tiny_config or test_ragged_multi_tensor_arena or "
               "test_aligned_arena_fast_path_shapes or test_adversarial_chunks or test_outer_step_aligned_arena or "
               "test_many_replicas_beyond_the_pointer_cache or test_more_chunks_than_resident_ctas or "
               "test_aggregate_instances_for_many_pairs_per_chunk or test_random_configurations or "
               "test_no_write_outside_the_callers_buffers or test_empty_tensors_inside_the_arena")


def test_small_parity_cases_raise_no_bounds_flag_in_the_debug_build():
    cmd = [sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_parity_gpu.py"),
           os.path.join(ROOT, "tests", "test_tiles_gpu.py"), "-m", "gpu", "-x", "-q", "--sl-debug-bounds",
           "-k", SMALL_CASES + " or tiles", "-p", "no:cacheprovider"]
    run = subprocess.run(cmd, capture_output=True, text=True, cwd=ROOT, timeout=1500)
    tail = run.stdout[-3000:] + run.stderr[-1500:]
    assert run.returncode == 0, tail
    assert " passed" in run.stdout and "failed" not in run.stdout, tail


def test_the_checks_are_compiled_in_and_skip_the_access():
    path = build.build(debug=True)
    lib = api.load(path)                       # a second handle; the process-wide one stays the normal build
    flags = torch.zeros(1, dtype=torch.int32, device="cuda")
    probe = torch.zeros(4, dtype=torch.int32, device="cuda")
    rc = lib.sl_debug_bounds_selftest(flags.data_ptr(), probe.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert rc == api.SL_OK
    assert int(flags.item()) == api.SL_FLAG_BOUNDS
    assert probe.cpu().tolist() == [0, 0, 0, 0]
    # the normal build has no such checks and says so
    assert api.sl_debug_bounds_selftest(flags, probe) == api.SL_ERR_UNSUPPORTED
