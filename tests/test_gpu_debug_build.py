"""The bounds-checked build (libdbw_dbg.so: the library's sources with -DDBW_BOUNDS) stands in for a memory
checker: every index a kernel reads from its own data (graph, mixing plan, worker order, links) is checked, a
violation sets DBW_STATUS_BOUNDS and the access is redirected.  The kernel-level parity tests are run against it
in a process of their own; each of them ends by asserting a clean status word, so a single out-of-range index
anywhere in those kernels fails the run."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_kernel_parity_tests_pass_against_the_bounds_checked_library():
    pytest.importorskip("torch")
    from paper_2102_06280_b200 import build
    build.build(debug=True)
    env = dict(os.environ, DBW_LIBRARY="debug")
    select = ("selection_bit_exact or mix_matches_oracle or tensor_core_kernel or staged_kernel or large_worker_count or "
              "update_backups or grad_fp32 or consensus_only_mix or degenerate or per_link_times")
    cmd = [sys.executable, "-m", "pytest", "tests/debug_bounds_checks.py", "tests/test_gpu_kernels.py", "tests/test_zz_no_alloc.py",
           "-m", "gpu", "-q", "-x", "-p", "no:cacheprovider", "-k", select + " or bounds_checked or bad_neighbour or static_selection"]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-4000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "skipped" not in r.stdout.splitlines()[-1]
