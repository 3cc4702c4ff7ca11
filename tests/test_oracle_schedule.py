"""Pins for oracle/schedule.py (dropout probability over the epochs, Sec. 5.3, Eq. 12-14).

What the mathematics fixes: Eq. 12 is the skew-normal density (a library routine gives the same values, and it
integrates to one), Eq. 13-14 are its first two moments (numerical integration of Eq. 12, and the library's
moments), shape 0 is the normal density, the scaled curve has the prescribed mean, and its shape is the one
Sec. 5.3 describes: low at the start, a single maximum, low again at the end.
"""
import math

import numpy as np
from scipy import integrate, stats

from oracle import schedule as S


def test_density_is_the_skew_normal_of_the_library_and_integrates_to_one():
    for mu, sigma, lam in [(0.0, 1.0, 0.0), (3.0, 2.5, 4.0), (-1.0, 0.7, -2.0), (10.0, 5.0, 0.5)]:
        for y in np.linspace(mu - 4 * sigma, mu + 4 * sigma, 23):
            assert math.isclose(S.density(y, mu, sigma, lam), stats.skewnorm.pdf(y, lam, loc=mu, scale=sigma),
                                rel_tol=1e-10, abs_tol=1e-300)
        area, _ = integrate.quad(S.density, mu - 12 * sigma, mu + 12 * sigma, args=(mu, sigma, lam))
        assert abs(area - 1.0) < 1e-9


def test_shape_zero_is_the_normal_density():
    for y in [-2.0, 0.3, 5.0]:
        assert math.isclose(S.density(y, 1.0, 2.0, 0.0), stats.norm.pdf(y, 1.0, 2.0), rel_tol=1e-13)
    assert S.mu0(0.0) == 0.0 and S.sigma0_sq(0.0) == 1.0


def test_moments_of_eq_13_and_14_by_integration():
    for E, D, lam in [(20.0, 36.0, 3.0), (5.0, 1.0, -1.5), (0.0, 4.0, 0.0), (50.0, 400.0, 8.0)]:
        mu, sigma = S.parameters(E, D, lam)
        lo, hi = mu - 14 * sigma, mu + 14 * sigma
        m1, _ = integrate.quad(lambda y: y * S.density(y, mu, sigma, lam), lo, hi)
        m2, _ = integrate.quad(lambda y: (y - E) ** 2 * S.density(y, mu, sigma, lam), lo, hi)
        assert abs(m1 - E) < 1e-7 * max(1.0, abs(E)) and abs(m2 - D) < 1e-6 * D
        assert math.isclose(stats.skewnorm.mean(lam, loc=mu, scale=sigma), E, rel_tol=1e-12, abs_tol=1e-12)
        assert math.isclose(stats.skewnorm.var(lam, loc=mu, scale=sigma), D, rel_tol=1e-12)


def test_schedule_has_the_prescribed_mean_and_the_described_shape():
    n = 60
    p = S.schedule(n, 0.4, 35.0, 150.0, -3.0)
    assert abs(np.mean(p) - 0.4) < 1e-12                     # nothing clipped here
    k = int(np.argmax(p))
    assert 0 < k < n - 1
    assert all(p[i] <= p[i + 1] for i in range(k)) and all(p[i] >= p[i + 1] for i in range(k, n - 1))
    assert p[0] < 0.1 * p[k] and p[-1] < 0.8 * p[k]            # low at the start, lower again at the end
    assert k > 35                                            # negative shape: the maximum lies after the mean
    q = S.schedule(n, 0.4, 35.0, 150.0, -3.0, p_max=0.6)
    assert max(q) == 0.6 and all(a == min(b, 0.6) for a, b in zip(q, p))
    assert all(v == 0.0 for v in S.schedule(5, 0.0, 2.0, 1.0, 1.0))
