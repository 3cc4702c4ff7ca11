"""Row-based sensitivity-aware dropout of a convolution layer's input matrix (Sec. 5.1, Sec. 5.2.1).

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  Integers and fp64 numpy.

The layer is a matrix product: the im2col transform (a library routine, not part of the method) turns the
input feature map into the input matrix A [M x Kc] (M = output positions, Kc = C*k*k) and the filters into the
weight W [Kc x N] (N = output channels), Y = A W.  Sec. 5.1 splits A into regions, looks at a random k% of a
region's values, calls the region sensitive if at least t% of them exceed a threshold and gives sensitive
regions a low and insensitive regions a high dropout probability; Sec. 5.2.1 drops whole rows of A with those
probabilities, multiplies only the kept rows and writes the results to the same rows of Y, the others zero.

Readings (the paper fixes none of this; PARITY UNPINNED):
  * regions: x consecutive rows by the whole width of A (the row is the granularity of Sec. 5.2.1);
  * the random k% of a region's values: every sampled value is drawn on its own, uniformly over the region's
    x*Kc positions and with replacement, one Philox word per value (`run_len` = 1, the default, is the text's
    statement).  `run_len` = c > 1 is an explicit departure, offered because a memory transaction delivers
    neighbouring values: the positions are then drawn as runs of c neighbouring values of a row (c divides Kc).
    In both cases the region has Cn = x*Kc/c runs, n_c = max(1, floor(k * Cn + 1/2)) of them are drawn,
    s = n_c * c values are looked at; run d of region g is chosen by word (d mod 4) of the Philox4x32-10 block
    with key (seed) and counter (iteration low, iteration high, g, stream_id * 65536 + d div 4) as run number
    floor(word * Cn / 2^32), runs numbered row-major; positions below the last row of A (ragged last region)
    count as not exceeding;
  * sensitive iff the count of values above the threshold is >= max(1, ceil(t * s)), the product taken
    exactly (t is the binary fraction the caller's double holds, s an integer);
  * a probability p becomes the integer P = min(floor(p * 2^32), 2^32 - 1); row r is dropped iff word 0 of the
    block with counter (iteration low, iteration high, r, stream_id * 65536 + 65535) is < P of its region;
  * no rescale is mentioned: alpha is an explicit argument, as for the other patterns;
  * the backward products are the exact adjoints of the forward map.
"""
from __future__ import annotations

import math
from fractions import Fraction

import numpy as np

from .pattern import philox4x32_10, MASK32

TWO32 = 1 << 32
MAX_BLOCKS = 65535


def transaction_run(Kc):
    """The run length at which every run of bf16 / fp32 values is one aligned piece of a row: gcd(Kc, 32).
    Not the default: pass it as `run_len` to ask for the clustered sample."""
    return math.gcd(Kc, 32)


def n_runs(k_frac, x, Kc, run_len=1):
    """How many runs of a region are drawn (run_len = 1: how many values)."""
    assert run_len >= 1 and Kc % run_len == 0
    return max(1, int(math.floor(k_frac * (x * (Kc // run_len)) + 0.5)))


def n_samples(k_frac, x, Kc, run_len=1):
    """How many values of a region are looked at."""
    return n_runs(k_frac, x, Kc, run_len) * run_len


def needed(t_frac, s):
    """Smallest count that reaches the fraction t of s sampled values: max(1, ceil(t * s)) in exact arithmetic."""
    return max(1, math.ceil(Fraction(t_frac) * s))


def quantise_probability(p):
    return min(int(math.floor(p * TWO32)), TWO32 - 1)


def region_sensitive(A, g, x, k_frac, t_frac, threshold, seed, iteration, stream_id, run_len=1):
    """Sec. 5.1, steps 2-3 for region g.  Returns (sensitive, count, samples)."""
    A = np.asarray(A)
    M, Kc = A.shape
    s = n_samples(k_frac, x, Kc, run_len)
    c = run_len
    per_row = Kc // c
    Cn = x * per_row
    n_c = n_runs(k_frac, x, Kc, run_len)
    assert (n_c + 3) // 4 <= MAX_BLOCKS
    count = 0
    for q in range((n_c + 3) // 4):
        words = philox4x32_10((iteration & MASK32, (iteration >> 32) & MASK32, g, ((stream_id << 16) | q) & MASK32),
                              (seed & MASK32, (seed >> 32) & MASK32))
        for w in range(4):
            if 4 * q + w >= n_c:
                break
            run = (words[w] * Cn) >> 32
            row, col = g * x + run // per_row, (run % per_row) * c
            if row < M:
                count += int(np.count_nonzero(np.asarray(A[row, col:col + c], dtype=np.float64) > threshold))
    return count >= needed(t_frac, s), count, s


def sensitivity_mask(A, x, k_frac, t_frac, threshold, m_prob, n_prob, seed, iteration, stream_id, run_len=1):
    """Sec. 5.1, step 4: the dropout probability of every region, as the integers the sampler compares with
    (sensitive regions get m_prob, the others n_prob; n_prob > m_prob)."""
    M = np.asarray(A).shape[0]
    regions = (M + x - 1) // x
    Pm, Pn = quantise_probability(m_prob), quantise_probability(n_prob)
    out = np.empty(regions, dtype=np.uint64)
    sens = np.empty(regions, dtype=bool)
    for g in range(regions):
        sens[g], _, _ = region_sensitive(A, g, x, k_frac, t_frac, threshold, seed, iteration, stream_id, run_len)
        out[g] = Pm if sens[g] else Pn
    return out, sens


def draw_rows(P_region, x, M, seed, iteration, stream_id):
    """Sec. 5.2.1: one Bernoulli draw per row with its region's probability.  Returns the kept rows, ascending."""
    keep = []
    for r in range(M):
        w0 = philox4x32_10((iteration & MASK32, (iteration >> 32) & MASK32, r, ((stream_id << 16) | 0xFFFF) & MASK32),
                           (seed & MASK32, (seed >> 32) & MASK32))[0]
        if not (w0 < int(P_region[r // x])):
            keep.append(r)
    return np.asarray(keep, dtype=np.int64)


def row_mask(M, keep):
    m = np.zeros(M)
    m[np.asarray(keep, dtype=np.int64)] = 1.0
    return m


# -- the three products; W in the math orientation [Kc x N] ------------------------------------------------
def fwd(A, W, keep, alpha=1.0):
    """Y = alpha * (rows of A kept) W; dropped rows of Y are zero (Sec. 5.2.1, step 3 and the fill-back)."""
    A = np.asarray(A, dtype=np.float64)
    return alpha * (A * row_mask(A.shape[0], keep)[:, None]) @ np.asarray(W, dtype=np.float64)


def bwd_data(dY, W, keep, alpha=1.0):
    dY = np.asarray(dY, dtype=np.float64)
    return alpha * (dY * row_mask(dY.shape[0], keep)[:, None]) @ np.asarray(W, dtype=np.float64).T


def bwd_weight(A, dY, keep, alpha=1.0):
    A = np.asarray(A, dtype=np.float64)
    dY = np.asarray(dY, dtype=np.float64)
    return alpha * (A * row_mask(A.shape[0], keep)[:, None]).T @ dY


def fwd_compact(A, W, keep, alpha=1.0):
    """The same through the dense, small input matrix of Sec. 5.2.1 (step 2): only the kept rows are touched."""
    keep = np.asarray(keep, dtype=np.int64)
    Y = np.zeros((np.asarray(A).shape[0], np.asarray(W).shape[1]))
    Y[keep] = alpha * np.asarray(A, dtype=np.float64)[keep] @ np.asarray(W, dtype=np.float64)
    return Y
