"""The worker order of the structured-sparse tensor-core mix (dbw_graph_order_2of4), checked on the host against
its defining property by brute force: for every worker i, no aligned group of four consecutive positions
holds more than two members of {i} + N_i, every worker is placed exactly once, and the result is the same
on every call.  (Eq. 5 does not depend on how the workers are numbered.)"""
import numpy as np
import pytest

from workloads import configs as wl


def _check(rowptr, col, order):
    n = len(rowptr) - 1
    assert len(order) % 128 == 0 and len(order) <= 1024
    placed = order[order >= 0]
    assert sorted(placed.tolist()) == list(range(n))              # a permutation of the workers, padded with -1
    pos = np.empty(n, dtype=np.int64)
    pos[placed] = np.nonzero(order >= 0)[0]
    for i in range(n):
        support = np.concatenate([[i], col[rowptr[i]: rowptr[i + 1]]])
        groups, counts = np.unique(pos[support] // 4, return_counts=True)
        assert counts.max() <= 2, (i, groups[counts.argmax()])


@pytest.mark.parametrize("name,make", [
    ("ring8", lambda: wl.ring(8)),
    ("reg4_32", lambda: wl.random_regular(32, 4, 2)),
    ("complete40", lambda: wl.complete(40)),                      # every worker adjacent to every other: two per group
    ("er64", lambda: wl.erdos_renyi_connected(64, 0.2, 3)),
    ("reg32_256", lambda: wl.random_regular(256, 32, 11)),
    ("config4_graph", lambda: (wl.make_workload(4, d=64).rowptr, wl.make_workload(4, d=64).col)),
])
def test_order_has_the_two_of_four_property(name, make):
    from paper_2102_06280_b200 import binding
    rowptr, col = make()
    order = binding.graph_order_2of4(rowptr, col)
    assert order is not None
    _check(np.asarray(rowptr), np.asarray(col), order)
    again = binding.graph_order_2of4(rowptr, col)
    assert np.array_equal(order, again)


def test_order_reports_graphs_without_one():
    """A complete graph on 600 workers would need two workers per group of four, i.e. 1200 positions > 1024."""
    from paper_2102_06280_b200 import binding
    rowptr, col = wl.complete(600)
    assert binding.graph_order_2of4(rowptr, col) is None


def test_order_rejects_bad_arguments():
    from paper_2102_06280_b200 import binding
    lib = binding.lib()
    rowptr, col = wl.ring(8)
    rp = np.ascontiguousarray(rowptr, dtype=np.int32)
    c = np.ascontiguousarray(col, dtype=np.int32)
    out = np.zeros(1024, dtype=np.int32)
    assert lib.dbw_graph_order_2of4(8, None, c.ctypes.data, out.ctypes.data, 1024) == -1
    assert lib.dbw_graph_order_2of4(8, rp.ctypes.data, c.ctypes.data, out.ctypes.data, 0) == -3
    bad = c.copy(); bad[0] = 0                                    # self loop
    assert lib.dbw_graph_order_2of4(8, rp.ctypes.data, bad.ctypes.data, out.ctypes.data, 1024) == -2
    assert lib.dbw_graph_order_2of4(8, rp.ctypes.data, c.ctypes.data, out.ctypes.data, 64) == 0   # needs 128 positions
