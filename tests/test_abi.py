"""The C-ABI library builds, loads and exports every entry point that include/dbw.h declares;
host-side argument checks work without a GPU."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from workloads import configs as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def p():
    from paper_2102_06280_b200 import build
    build.build()
    import paper_2102_06280_b200 as pkg
    return pkg


def test_every_declared_symbol_is_exported(p):
    header = open(os.path.join(ROOT, "include", "dbw.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(dbw_[a-z_0-9]+)\s*\(", header))
    assert len(declared) >= 18
    handle = C.CDLL(os.path.join(ROOT, "paper_2102_06280_b200", "libdbw.so"))
    for name in declared:
        assert hasattr(handle, name), name
    from paper_2102_06280_b200 import binding
    assert declared == set(binding.exported_symbols())


def test_model_layout(p):
    m = p.model_layout([784, 200, 10], 64)
    assert m.d == 784 * 200 + 200 + 200 * 10 + 10 == 159010
    assert m.ld % 32 == 0 and all(o % 32 == 0 for o in m.w_off + m.b_off)
    assert m.w_off[0] == 0 and m.b_off[0] == 156800 and m.w_off[1] == 157024
    x = np.arange(m.d, dtype=np.float32)[None]
    packed = m.pack(x)
    assert packed.shape == (1, m.ld) and np.array_equal(m.unpack(packed), x)
    assert np.count_nonzero(packed) == m.d - 1
    with pytest.raises(p.DbwError):
        p.model_layout([784, 0, 10], 64)
    with pytest.raises(p.DbwError):
        p.model_layout([4] * 11, 8)


@pytest.mark.parametrize("breakage", ["self_loop", "asymmetric", "unsorted", "range", "disconnected"])
def test_init_rejects_bad_graphs_on_the_host(p, breakage):
    rowptr, col = wl.ring(6)
    rowptr, col = rowptr.copy(), col.copy()
    if breakage == "self_loop":
        col[0] = 0
    elif breakage == "asymmetric":
        col[1] = 3                      # 0 -> 3 without 3 -> 0
    elif breakage == "unsorted":
        col[0], col[1] = col[1], col[0]
    elif breakage == "range":
        col[0] = 6
    else:
        rowptr, col = wl._csr_from_edges(6, [(0, 1), (1, 2), (2, 0), (3, 4), (4, 5), (5, 3)])
    with pytest.raises(p.DbwError) as e:
        p.Dbw(rowptr, col, d=8)
    assert e.value.code == -2


def test_init_rejects_bad_shapes_and_models(p):
    rowptr, col = wl.ring(6)
    with pytest.raises(p.DbwError) as e:
        p.Dbw(rowptr, col, d=10, ld=8)
    assert e.value.code == -3
    with pytest.raises(p.DbwError) as e:
        p.Dbw(rowptr, col, d=10, ld=10)           # ld % 4 != 0
    assert e.value.code == -3
    m = p.model_layout([8, 4], 2)
    with pytest.raises(p.DbwError) as e:
        p.Dbw(rowptr, col, d=m.d + 1, ld=m.ld, model=m)
    assert e.value.code == -5
    m.desc.w_off[0] = 16                            # not a multiple of 32
    with pytest.raises(p.DbwError) as e:
        p.Dbw(rowptr, col, d=m.d, ld=m.ld, model=m)
    assert e.value.code == -5


def test_null_arguments(p):
    lib = p.lib()
    assert lib.dbw_destroy(None) == -1
    assert lib.dbw_status(None) == -1
    assert lib.dbw_select(None, None, None, None, None, None, None, None) == -1
    assert lib.dbw_launch_count() >= 0
