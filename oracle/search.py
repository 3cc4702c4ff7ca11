"""Search for the distribution K over the pattern periods (Sec. 3.3, Algorithm 1).

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  numpy fp64.

The paper describes the algorithm in words; the listing's body is not printed.  What the text
fixes: a vector v of length N (arbitrary start), d = softmax(v) is the distribution, the constant
vector p_u = {(i-1)/i} holds the global dropout rate of pattern i, d . p_u is the expected global
rate and its difference from the target p is the objective, the negative entropy of d is added so
that d is dense, v is updated by gradient steps, and d is returned when the loss stops changing.

Reading used here (everything the text leaves open):
  loss(v) = (d . p_u - p)^2 + lam * sum_i d_i ln d_i,     d = softmax(v)
  v starts at 0 (uniform d); full-gradient steps v <- v - lr * dloss/dv (the loss has no data, so
  "SGD" has nothing to subsample); stop when |loss_t - loss_{t-1}| < tol or after max_iter steps.

Pins (tests/test_oracle_search.py): every stationary point of this loss has ln d_i affine in
(i-1)/i, with slope beta = -2 (d.p_u - p) / lam; as lam -> 0 the result tends to the maximum-entropy
distribution with d . p_u = p; sum d = 1, d > 0.
"""
from __future__ import annotations

import numpy as np


def p_u(ndp):
    """Global dropout rate of the pattern with period i, i = 1..ndp (Sec. 3.3)."""
    i = np.arange(1, ndp + 1, dtype=np.float64)
    return (i - 1.0) / i


def loss_and_grad(v, p, lam):
    """Loss of Algorithm 1 in the reading above and its gradient with respect to v."""
    v = np.asarray(v, dtype=np.float64)
    ex = np.exp(v - v.max())
    d = ex / ex.sum()
    pu = p_u(len(v))
    e = float(d @ pu) - p
    loss = e * e + lam * float(np.sum(d * np.log(d)))
    g_d = 2.0 * e * pu + lam * (np.log(d) + 1.0)      # d loss / d d_i
    g_v = d * (g_d - float(d @ g_d))                    # through the softmax
    return loss, g_v, d


def search_K(p, ndp, lam=1e-3, lr=10.0, max_iter=200000, tol=1e-16):
    """Returns (K, iterations).  K: ndp probabilities, K[i-1] for period i."""
    v = np.zeros(ndp, dtype=np.float64)
    prev = None
    d = None
    it = 0
    for it in range(1, max_iter + 1):
        loss, g_v, d = loss_and_grad(v, p, lam)
        if prev is not None and abs(prev - loss) < tol:
            break
        prev = loss
        v = v - lr * g_v
    return d, it
