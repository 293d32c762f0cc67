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


def test_random_growth_bracket_holds_the_kth_smallest_of_uniform_keys(mst):
    # host logic of the bracket the update kernel lists its random candidates in: on uniform 64-bit keys the k-th
    # smallest falls inside, the list it implies fits, and the degenerate requests plan nothing
    rng = np.random.default_rng(5)
    for C, k in [(1000, 1), (1000, 1000), (5000, 37), (200_000, 1500), (1_000_000, 7500), (1_000_000, 999_000), (3_000_000, 31_457)]:
        br = mst.mst_rand_bracket(k, C, 6.0, 32768)
        assert br is not None
        lo, hi = br
        assert 0 <= lo < hi <= 2 ** 64 - 1
        for trial in range(3):
            keys = rng.integers(0, 2 ** 64, size=C, dtype=np.uint64)
            kth = int(np.partition(keys, k - 1)[k - 1])
            below = int((keys < np.uint64(lo)).sum())
            inside = int(((keys >= np.uint64(lo)) & (keys < np.uint64(hi))).sum())
            assert below < k <= below + inside            # what the kernel checks before it trusts the bracket
            assert lo <= kth < hi
            assert inside <= 32768
    assert mst.mst_rand_bracket(0, 100, 6.0, 32768) is None
    assert mst.mst_rand_bracket(101, 100, 6.0, 32768) is None
    assert mst.mst_rand_bracket(50, 100, 0.0, 32768) is None           # switched off
    assert mst.mst_rand_bracket(4_000_000, 8_000_000, 6.0, 32768) is None   # the list would not fit
    assert mst.mst_rand_bracket(50, 100, 6.0, 32768) == (0, 2 ** 64 - 1)     # k + m beyond the candidates: everything
    narrow, wide = mst.mst_rand_bracket(10_000, 1_000_000, 1.0, 32768), mst.mst_rand_bracket(10_000, 1_000_000, 6.0, 32768)
    assert wide[0] < narrow[0] < narrow[1] < wide[1]
