"""Dropout probability as a function of the training epoch (Sec. 5.3, Eq. 12-14).

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  fp64.

Sec. 5.3 starts training with a low dropout probability, raises it, and lowers it again towards the end; it
says the curve over the epochs has the shape of a skew-normal density (Eq. 12) and that the density's two
parameters follow from a prescribed expectation (Eq. 13) and variance (Eq. 14).

Readings (the text does not say what the density is scaled by, nor what its axis is; PARITY UNPINNED):
  * the axis y is the epoch number e = 0 .. n_epochs-1;
  * the prescribed expectation E and variance D are those of the curve along the epoch axis (where the
    dropout effort is centred and how wide it is spread); sigma = sqrt(D / sigma0^2(lambda)),
    mu = E - mu0(lambda) * sigma are Eq. 13-14 solved for the parameters;
  * the curve is scaled so that its mean over the epochs is the overall dropout probability p_total, then
    clipped to [0, p_max]: p_e = min(p_max, p_total * n_epochs * f(e) / sum_e' f(e')).
"""
from __future__ import annotations

import math


def mu0(lam):
    """Eq. 13: mean of the standard skew-normal with shape lambda."""
    return math.sqrt(2.0 / math.pi) * lam / math.sqrt(1.0 + lam * lam)


def sigma0_sq(lam):
    """Eq. 14: variance of the standard skew-normal with shape lambda."""
    return 1.0 - (2.0 / math.pi) * lam * lam / (1.0 + lam * lam)


def parameters(E, D, lam):
    """(mu, sigma) of the density whose expectation is E and whose variance is D (Eq. 13-14 inverted)."""
    sigma = math.sqrt(D / sigma0_sq(lam))
    return E - mu0(lam) * sigma, sigma


def density(y, mu, sigma, lam):
    """Eq. 12: (2/sigma) * phi(z) * Phi(lambda z), z = (y - mu)/sigma."""
    z = (y - mu) / sigma
    phi = math.exp(-0.5 * z * z) / math.sqrt(2.0 * math.pi)
    Phi = 0.5 * math.erfc(-lam * z / math.sqrt(2.0))
    return 2.0 / sigma * phi * Phi


def schedule(n_epochs, p_total, E, D, lam, p_max=1.0):
    """Dropout probability of every epoch."""
    mu, sigma = parameters(E, D, lam)
    f = [density(float(e), mu, sigma, lam) for e in range(n_epochs)]
    total = sum(f)
    return [min(p_max, p_total * n_epochs * v / total) for v in f]
