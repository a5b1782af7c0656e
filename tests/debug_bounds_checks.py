"""Checks that only make sense against the bounds-checked library (libdbw_dbg.so, DBW_LIBRARY=debug); run by
tests/test_gpu_debug_build.py in a process of its own.  In that build an index that a kernel reads from its own
data and that is out of range sets DBW_STATUS_BOUNDS and the access is redirected: nothing faults."""
import numpy as np
import pytest

from oracle import dbw_oracle as orc
from workloads import configs as wl

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def test_this_process_runs_the_bounds_checked_library():
    from paper_2102_06280_b200 import binding
    binding.lib()
    assert binding._LIB_PATH.endswith("libdbw_dbg.so")


def test_unvalidated_graph_with_a_bad_neighbour_index_is_caught():
    """dbw_select_static takes its CSR from device memory without validation.  A neighbour index past the last
    worker would make the regular build read beyond the arrival times; the bounds-checked build reports it and
    reads worker 0 instead."""
    import paper_2102_06280_b200 as p
    from paper_2102_06280_b200 import binding
    if not binding._LIB_PATH.endswith("libdbw_dbg.so"):
        pytest.skip("needs the bounds-checked library")
    rowptr, col = wl.ring(8)
    n, nnz = 8, len(col)
    bad = np.asarray(col, dtype=np.int32).copy()
    bad[3] = n + 5
    t = dev(1.0 + np.arange(n, dtype=np.float64))
    b = dev(np.zeros(n, dtype=np.int32))
    kept = torch.zeros(nnz, dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.select_static(dev(np.asarray(rowptr, dtype=np.int32)), dev(bad), t, b, kept, status_out=st)
    torch.cuda.synchronize()
    assert int(st.item()) & p.STATUS_BOUNDS
    good = torch.zeros(nnz, dtype=torch.uint8, device="cuda")
    binding.select_static(dev(np.asarray(rowptr, dtype=np.int32)), dev(np.asarray(col, dtype=np.int32)), t, b, good, status_out=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert np.array_equal(good.cpu().numpy(), orc.select_fastest(rowptr, col, 1.0 + np.arange(n, dtype=np.float64), np.zeros(n, dtype=np.int32)))
