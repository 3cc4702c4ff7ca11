"""Pins of the distribution search (Sec. 3.3, Algorithm 1) in oracle/search.py.

The paper prints no numbers for K, so the pins are what the mathematics fixes: the gradient against
finite differences, the shape of every stationary point (ln k_i affine in (i-1)/i with the slope the
loss dictates), the small-lambda limit (the maximum-entropy distribution at the target rate, computed
by an independent bisection in the input generators) and Eq. 2-3 (the expected per-unit drop rate of
the returned K equals its global rate).
"""
import numpy as np
import pytest

from oracle import search as OS
from oracle import pattern as OP
from paper_2203_05705_b200 import inputs
from distributions import max_entropy_K


def test_gradient_matches_central_differences():
    rng = np.random.default_rng(0)
    for _ in range(5):
        n = int(rng.integers(2, 12))
        v = rng.standard_normal(n)
        p, lam = float(rng.uniform(0.2, 0.8)), float(rng.uniform(1e-3, 1.0))
        _, g, _ = OS.loss_and_grad(v, p, lam)
        for i in range(n):
            h = 1e-6
            vp, vm = v.copy(), v.copy()
            vp[i] += h
            vm[i] -= h
            fd = (OS.loss_and_grad(vp, p, lam)[0] - OS.loss_and_grad(vm, p, lam)[0]) / (2 * h)
            assert abs(fd - g[i]) <= 1e-8 * max(1.0, abs(fd)), (i, fd, g[i])


@pytest.mark.parametrize("p,ndp,lam", [(0.5, 16, 1e-2), (0.3, 16, 1e-2), (0.7, 8, 1e-1), (0.5, 5, 1e-3)])
def test_result_is_a_stationary_point_of_the_gibbs_family(p, ndp, lam):
    K, iters = OS.search_K(p, ndp, lam=lam, tol=1e-18)
    assert iters < 200000
    assert abs(K.sum() - 1.0) <= 1e-12 and np.all(K > 0)
    pu = OS.p_u(ndp)
    A = np.vstack([pu, np.ones(ndp)]).T
    coef, *_ = np.linalg.lstsq(A, np.log(K), rcond=None)
    assert np.abs(A @ coef - np.log(K)).max() <= 1e-5            # ln k_i = beta (i-1)/i + c
    e = float(K @ pu) - p
    assert abs(coef[0] - (-2.0 * e / lam)) <= 1e-3 * max(1.0, abs(coef[0]))   # beta = -2 e / lam


def test_small_lambda_tends_to_the_maximum_entropy_distribution():
    errs = []
    for lam in (1e-1, 1e-2, 1e-3):
        K, _ = OS.search_K(0.5, 16, lam=lam, tol=1e-18)
        ref = np.asarray(max_entropy_K(0.5, 16))
        errs.append(np.abs(K - ref).max())
        assert abs(float(K @ OS.p_u(16)) - 0.5) <= 1.5 * lam     # |e| = lam |beta| / 2, |beta| < 3 here
    assert errs[0] > errs[1] > errs[2] and errs[2] <= 2e-3


def test_searched_K_gives_every_unit_the_global_rate():
    """Eq. 2-3 with the searched K, in exact rational arithmetic on the quantised table."""
    from fractions import Fraction
    K, _ = OS.search_K(0.6, 8, lam=1e-2)
    cdf = OP.quantise_K(K)
    N = 37
    probs = [Fraction(c - (cdf[i - 1] if i else 0), 1 << 32) for i, c in enumerate(cdf)]
    global_rate = sum(pr * Fraction(dp - 1, dp) for dp, pr in enumerate(probs, start=1))
    for unit in range(1, N + 1):
        drop = Fraction(0)
        for dp, pr in enumerate(probs, start=1):
            dropped_b = sum(1 for b in range(1, dp + 1) if (unit - b) % dp != 0)
            drop += pr * Fraction(dropped_b, dp)
        assert drop == global_rate
    assert abs(float(global_rate) - 0.6) <= 0.02
