"""The C-ABI library loads, exports every symbol the header declares, and its host-only logic agrees with the oracle."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def mst():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2408_11746_b200 as m
    return m


def _declared():
    src = open(os.path.join(ROOT, "include", "mst.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(mst_[a-z0-9_]+)\s*\(", src)))


def test_every_declared_symbol_is_exported(mst):
    names = _declared()
    assert len(names) >= 15
    lib = ctypes.CDLL(mst.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(mst.EXPORTS) == names               # the binding covers the same surface
    for n in names:
        assert callable(getattr(mst, n, None)) or n == "mst_status_string"


def test_status_strings(mst):
    assert mst.status_string(0) == "ok"
    assert len({mst.status_string(i) for i in range(10)}) == 10


def test_host_side_argument_checks_need_no_gpu(mst):
    for args, status in [((0, 0, 8, mst.MST_F32, 4), 2), ((0, 8, 70000, mst.MST_F32, 4), 2),
                         ((0, 8, 8, 7, 4), 3), ((0, 8, 8, mst.MST_BF16, 0), 4), ((0, 8, 8, mst.MST_BF16, 65), 4)]:
        with pytest.raises(mst.MstError) as e:
            mst.mst_layer_create(*args)
        assert e.value.status == status


def test_update_counts_agree_with_oracle(mst):
    rng = np.random.default_rng(0)
    for _ in range(3000):
        N = int(rng.integers(1, 5_000_000))
        nnz = int(rng.integers(0, N + 1))
        tgt = int(rng.integers(-1, N + 1))
        zeta = float(rng.choice([0.0, 0.1, 0.3, 0.5, 1.0, rng.random()]))
        R = float(rng.choice([0.0, 0.25, 1.0, rng.random()]))
        assert mst.mst_update_counts(zeta, nnz, tgt, N, R) == oracle.mg_counts(zeta, nnz, tgt, N, R)
    with pytest.raises(mst.MstError) as e:
        mst.mst_update_counts(0.3, 10, 50, 40, 0.25)
    assert e.value.status == 5
    with pytest.raises(mst.MstError) as e:
        mst.mst_update_counts(-0.1, 10, 10, 40, 0.25)
    assert e.value.status == 1
