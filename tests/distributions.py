"""Pattern distributions K used as test INPUTS and as the closed-form pin of the distribution search.

K is an input of the hot path (Sec. 3.3 produces it, Sec. 3.4 samples from it); this module belongs to the tests,
not to the library: the library never computes this closed form, and the benchmark keeps its own generator.
"""
import numpy as np
from scipy import optimize


def max_entropy_K(p, n_dp):
    """Maximum-entropy distribution over the periods dp = 1..n_dp whose global dropout rate
    sum_i k_i (i-1)/i (Eq. 2-3) equals p: k_i proportional to exp(beta (i-1)/i), beta the root of the rate
    equation.  It is the hard-constraint limit of the loss Sec. 3.3 describes (rate error plus negative entropy)."""
    if n_dp < 2:
        raise ValueError("need at least two periods")
    pu = np.array([(i - 1) / i for i in range(1, n_dp + 1)], dtype=np.float64)
    if not (0.0 < p < pu[-1]):
        raise ValueError("target rate must lie in (0, (n_dp-1)/n_dp)")

    def gibbs(beta):
        w = np.exp(beta * (pu - (pu[-1] if beta > 0 else 0.0)))
        return w / w.sum()

    beta = optimize.brentq(lambda bt: float(gibbs(bt) @ pu) - p, -200.0, 200.0, xtol=1e-14, rtol=1e-15, maxiter=500)
    k = gibbs(beta)
    return k / k.sum()
