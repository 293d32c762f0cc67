"""Host-side Sparsity-Variation driver: library vs oracle, closed forms and invariants (CPU only)."""
import math

import pytest

import oracle.sv_schedule as ref
from oracle import flop_model


@pytest.fixture(scope="module")
def mst():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2408_11746_b200 as m
    return m


def test_stage_levels_closed_form(mst):
    sc = mst.SvSchedule()           # S_M = 0.96, N = 5, 2000-step stages, T_U = 100000
    warm = [mst.mst_sv_sparsity(sc, k * 2000) for k in range(6)]
    # S_M (1 - (1 - k/5)^3): 0, .96*.488, .96*.784, .96*.936, .96*.992, .96
    for got, want in zip(warm, [0.0, 0.46848, 0.75264, 0.89856, 0.95232, 0.96]):
        assert got == pytest.approx(want, abs=1e-12)
    rest = [mst.mst_sv_sparsity(sc, 110000 + k * 2000) for k in range(6)]
    for got, want in zip(rest, [0.96, 0.49152, 0.20736, 0.06144, 0.00768, 0.0]):
        assert got == pytest.approx(want, abs=1e-12)
    assert mst.mst_sv_sparsity(sc, 1999) == 0.0 and mst.mst_sv_sparsity(sc, 2000) > 0.4       # stepwise, not continuous
    assert mst.mst_sv_sparsity(sc, 50000) == 0.96 and mst.mst_sv_sparsity(sc, 10 ** 7) == 0.0


def test_schedule_matches_oracle_everywhere(mst):
    sc = mst.SvSchedule(0.9, 4, 7, 31, 5)
    prev = None
    for t in range(0, 4 * 7 + 31 + 4 * 5 + 10):
        s = mst.mst_sv_sparsity(sc, t)
        assert s == pytest.approx(ref.sparsity(t, 0.9, 4, 7, 31, 5), abs=1e-12)
        assert 0.0 <= s <= 0.9 + 1e-12
        if t < 4 * 7 + 31 and prev is not None:
            assert s >= prev - 1e-12                       # never densifies before restoration
        if t > 4 * 7 + 31 and prev is not None:
            assert s <= prev + 1e-12                       # never sparsifies during restoration
        prev = s
        for decay in (1.0, 0.5):
            z = mst.mst_sv_update_fraction(sc, t, 0.3, decay)
            assert z == pytest.approx(ref.update_fraction(t, 0.3, decay, 4, 7, 31, 5), abs=1e-12)
            assert 0.0 <= z <= 0.3 + 1e-12


def test_update_fraction_cosine_shape(mst):
    sc = mst.SvSchedule()
    T1 = 110000
    assert mst.mst_sv_update_fraction(sc, 0) == pytest.approx(0.3)                  # starts at zeta_1
    assert mst.mst_sv_update_fraction(sc, T1 // 2) == pytest.approx(0.15)          # half-way: zeta_1 / 2
    assert mst.mst_sv_update_fraction(sc, T1 - 1) < 1e-9                            # annealed to ~0
    assert mst.mst_sv_update_fraction(sc, T1) == pytest.approx(0.3)                 # reset at each restoration stage
    assert mst.mst_sv_update_fraction(sc, T1, 0.3, 0.5) == pytest.approx(0.15)      # decayed magnitude
    assert mst.mst_sv_update_fraction(sc, T1 + 2000, 0.3, 0.5) == pytest.approx(0.075)
    assert mst.mst_sv_update_fraction(sc, T1 + 1000) == pytest.approx(0.3 / 2 * (1 + math.cos(math.pi / 2)))
    assert mst.mst_sv_update_fraction(sc, 10 ** 7) == 0.0


def test_er_split(mst):
    shapes = [(2304, 768), (768, 768), (3072, 768), (768, 3072)]
    d = mst.mst_er_densities(shapes, 0.04)
    assert d == pytest.approx([0.04, 0.06, 0.0375, 0.0375], rel=1e-12)             # eps = 23.04
    assert d == pytest.approx(flop_model.erdos_renyi_densities(shapes, 0.04)[0], rel=1e-12)
    # total active count is preserved, capped layers become dense
    shapes = [(8, 8), (512, 512), (64, 2048)]
    for g in (0.0, 0.05, 0.3, 0.9, 1.0):
        d = mst.mst_er_densities(shapes, g)
        assert all(0.0 <= x <= 1.0 for x in d)
        assert sum(x * o * i for x, (o, i) in zip(d, shapes)) == pytest.approx(g * sum(o * i for o, i in shapes), rel=1e-9, abs=1e-9)
        assert d == pytest.approx(flop_model.erdos_renyi_densities(shapes, g)[0], rel=1e-9, abs=1e-12)
    assert mst.mst_er_densities(shapes, 0.3)[0] == 1.0                               # the tiny layer saturates


def test_bad_arguments(mst):
    with pytest.raises(mst.MstError):
        mst.mst_sv_sparsity(mst.SvSchedule(1.5, 5, 10, 10, 10), 0)
    with pytest.raises(mst.MstError):
        mst.mst_sv_sparsity(mst.SvSchedule(), -1)
    with pytest.raises(mst.MstError):
        mst.mst_er_densities([(0, 4)], 0.5)
