"""Pins for the oracle's grids and quadrature weights (App. A.1; Eq. quadrature)."""
import math

import numpy as np
import pytest

from oracle import sna_oracle as orc

EQ, GL, TZ = orc.EQUIANGULAR, orc.LEGENDRE_GAUSS, orc.EQUIANGULAR_TRAPEZOID


def test_equiangular_colatitudes_include_both_poles():
    th = orc.colatitudes(EQ, 5)
    assert th[0] == 0.0 and abs(th[-1] - math.pi) < 1e-15
    assert np.allclose(np.diff(th), math.pi / 4, atol=1e-15)


@pytest.mark.parametrize("nlat, expected", [
    (2, [1.0, 1.0]),
    (3, [1 / 3, 4 / 3, 1 / 3]),
    (4, [1 / 9, 8 / 9, 8 / 9, 1 / 9]),
    (5, [1 / 15, 8 / 15, 12 / 15, 8 / 15, 1 / 15]),
])
def test_clenshaw_curtis_closed_forms(nlat, expected):
    # textbook closed forms of the Clenshaw-Curtis rule (n=3 is Simpson's rule)
    assert np.allclose(orc.latitude_weights(EQ, nlat), expected, rtol=0, atol=1e-15)


@pytest.mark.parametrize("nlat", [2, 3, 8, 33, 128, 257])
def test_clenshaw_curtis_polynomial_exactness(nlat):
    # an (nlat)-point interpolatory rule integrates x^p on [-1,1] exactly for p <= nlat-1
    w = orc.latitude_weights(EQ, nlat)
    x = np.cos(orc.colatitudes(EQ, nlat))
    assert np.all(w > 0) and np.allclose(w, w[::-1], atol=1e-15)
    for p in range(0, min(nlat, 24)):
        exact = (1 + (-1) ** p) / (p + 1)
        assert abs(np.sum(w * x ** p) - exact) < 1e-13, p


def test_gauss_legendre_closed_forms():
    assert np.allclose(np.cos(orc.colatitudes(GL, 2)), [1 / math.sqrt(3), -1 / math.sqrt(3)], atol=1e-15)
    assert np.allclose(orc.latitude_weights(GL, 2), [1, 1], atol=1e-15)
    assert np.allclose(np.cos(orc.colatitudes(GL, 3)), [math.sqrt(3 / 5), 0, -math.sqrt(3 / 5)], atol=1e-15)
    assert np.allclose(orc.latitude_weights(GL, 3), [5 / 9, 8 / 9, 5 / 9], atol=1e-15)


@pytest.mark.parametrize("nlat", [4, 17, 128, 361])
def test_gauss_legendre_matches_library_routine(nlat):
    x, w = np.polynomial.legendre.leggauss(nlat)      # ascending nodes
    th = orc.colatitudes(GL, nlat)
    assert np.all(np.diff(th) > 0), "colatitude must ascend (north to south)"
    assert np.allclose(np.cos(th), x[::-1], rtol=0, atol=2e-15)
    assert np.allclose(orc.latitude_weights(GL, nlat), w[::-1], rtol=1e-9, atol=1e-15)


@pytest.mark.parametrize("nlat", [3, 10, 64])
def test_gauss_legendre_polynomial_exactness(nlat):
    w = orc.latitude_weights(GL, nlat)
    x = np.cos(orc.colatitudes(GL, nlat))
    for p in range(0, min(2 * nlat, 30)):
        exact = (1 + (-1) ** p) / (p + 1)
        assert abs(np.sum(w * x ** p) - exact) < 1e-13, p


@pytest.mark.parametrize("grid, nlat, nlon", [(EQ, 32, 64), (EQ, 256, 512), (GL, 361, 720), (GL, 5, 10)])
def test_point_weights_sum_to_sphere_area(grid, nlat, nlon):
    omega = orc.quad_weights(grid, nlat, nlon)
    assert abs(np.sum(omega) * nlon - 4 * math.pi) < 1e-12


def test_quadrature_integrates_a_smooth_function():
    # int_{S^2} (1 + z + x^2) dmu = 4pi + 0 + 4pi/3
    for grid, nlat, nlon in [(EQ, 17, 32), (GL, 12, 24)]:
        th = orc.colatitudes(grid, nlat)
        om = orc.quad_weights(grid, nlat, nlon)
        phi = 2 * math.pi * np.arange(nlon) / nlon
        x = np.sin(th)[:, None] * np.cos(phi)[None, :]
        z = np.cos(th)[:, None] * np.ones_like(phi)[None, :]
        total = np.sum((1 + z + x * x) * om[:, None])
        assert abs(total - (4 * math.pi + 4 * math.pi / 3)) < 1e-12


def test_trapezoid_grid_has_the_north_pole_but_not_the_south_pole():
    # Eq. (latlon_grid): theta_i = pi i / nlat for i = 0 .. nlat-1
    th = orc.colatitudes(TZ, 6)
    assert th[0] == 0.0 and abs(th[-1] - (math.pi - math.pi / 6)) < 1e-15
    assert np.allclose(np.diff(th), math.pi / 6, rtol=0, atol=1e-15)


def test_trapezoid_weights_values_from_the_printed_formula():
    # Eq. (latlon_quad_weights) by hand for nlat = 4, nlon = 8: 2 pi^2/32 * sin(0, pi/4, pi/2, 3pi/4)
    om = orc.quad_weights(TZ, 4, 8)
    unit = 2 * math.pi ** 2 / 32
    assert om[0] == 0.0
    assert np.allclose(om, [0.0, unit * math.sqrt(0.5), unit, unit * math.sqrt(0.5)], rtol=1e-15, atol=0)


@pytest.mark.parametrize("nlat", [2, 5, 64, 361])
def test_trapezoid_weights_are_the_library_trapezoid_rule_in_theta(nlat):
    # int_0^pi f(theta) sin(theta) dtheta by the composite trapezoid rule on nlat intervals: the integrand
    # vanishes at both ends, so the rule needs no south-pole node and equals the weighted sum over the grid
    from scipy.integrate import trapezoid
    w, th = orc.latitude_weights(TZ, nlat), orc.colatitudes(TZ, nlat)
    nodes = np.linspace(0.0, math.pi, nlat + 1)
    for f in (lambda t: np.ones_like(t), lambda t: np.cos(t) ** 2, lambda t: np.exp(0.3 * t)):
        assert abs(np.sum(w * f(th)) - trapezoid(f(nodes) * np.sin(nodes), nodes)) < 1e-13


@pytest.mark.parametrize("nlat, nlon", [(4, 8), (33, 64), (361, 720)])
def test_trapezoid_point_weights_sum_only_approximately_to_sphere_area(nlat, nlon):
    # closed form: sum_i sin(pi i/n) = cot(pi/(2n)), so the total is (2 pi^2/n) cot(pi/(2n)) = 4 pi (1 - pi^2/(12 n^2) + ...)
    total = np.sum(orc.quad_weights(TZ, nlat, nlon)) * nlon
    assert abs(total - 2 * math.pi ** 2 / nlat / math.tan(math.pi / (2 * nlat))) < 1e-12
    lead = 4 * math.pi * math.pi ** 2 / (12 * nlat ** 2)          # x cot x = 1 - x^2/3 - x^4/45 - ... at x = pi/(2n)
    assert lead < 4 * math.pi - total < lead * 1.02


def test_invalid_arguments():
    with pytest.raises(orc.OracleError):
        orc.colatitudes(EQ, 1)
    with pytest.raises(orc.OracleError):
        orc.latitude_weights(7, 8)
