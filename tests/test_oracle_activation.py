"""Pins for the oracle's GELU and its derivative (CPU only)."""
import numpy as np

from oracle import activation as act


def test_phi_matches_integral_of_the_normal_density():
    # Phi(y) = 1/2 + int_0^y exp(-s^2/2)/sqrt(2 pi) ds, by a fine trapezoid rule: independent of erf
    for y in (-3.0, -0.75, 0.3, 1.0, 2.5):
        s = np.linspace(0.0, y, 200001)
        f = np.exp(-0.5 * s * s) / np.sqrt(2 * np.pi)
        integral = float(np.sum((f[1:] + f[:-1]) * 0.5 * np.diff(s)))
        assert abs(act.phi_cdf(y) - (0.5 + integral)) < 1e-10


def test_table_values():
    # standard normal table: Phi(1) = 0.841344746, Phi(2) = 0.977249868
    assert act.gelu(0.0) == 0.0
    assert abs(act.gelu(1.0) - 0.8413447461) < 1e-9
    assert abs(act.gelu(-1.0) + 0.1586552539) < 1e-9
    assert abs(act.gelu(2.0) - 2 * 0.9772498681) < 1e-9


def test_odd_part_is_identity_and_limits():
    y = np.linspace(-6, 6, 241)
    np.testing.assert_allclose(act.gelu(y) - act.gelu(-y), y, atol=1e-14)
    assert abs(act.gelu(12.0) - 12.0) < 1e-12 and abs(act.gelu(-12.0)) < 1e-12
    assert abs(act.gelu_grad(12.0) - 1.0) < 1e-12 and abs(act.gelu_grad(-12.0)) < 1e-12
    assert act.gelu_grad(0.0) == 0.5


def test_derivative_against_central_differences_and_minimum():
    y = np.linspace(-4, 4, 161)
    h = 1e-5
    fd = (act.gelu(y + h) - act.gelu(y - h)) / (2 * h)
    np.testing.assert_allclose(act.gelu_grad(y), fd, atol=1e-9)
    # GELU has one minimum, near y = -0.7518, value about -0.17
    ys = np.linspace(-1.0, -0.5, 500001)
    k = int(np.argmin(act.gelu(ys)))
    assert abs(ys[k] + 0.751792) < 1e-5 and abs(act.gelu(ys[k]) + 0.169971) < 1e-6
    assert abs(act.gelu_grad(ys[k])) < 1e-5
