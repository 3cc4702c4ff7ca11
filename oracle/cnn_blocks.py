"""Block-based sensitivity-aware dropout of a convolution layer's input matrix (Sec. 5.1, Sec. 5.2.2).

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  Integers and fp64 numpy.

The input matrix A [M x Kc] (im2col of the feature map) is cut into ts x ts blocks; the Q = Kc/ts blocks that
share their rows form a group, there are G = M/ts groups.  A block is the dropout granularity (Sec. 5.2.2).
Dropping blocks by sensitivity alone leaves some rows of A with many more kept blocks than others; the
paper's remedy is to bound the number of sensitive blocks per group so that all groups have nearly the same
number, after which every group keeps nearly the same amount of work.

Readings (the paper fixes none of this, and the figure that shows the balancing is not available;
PARITY UNPINNED):
  * prediction is that of Sec. 5.1 with one block as the region: every sampled value is drawn on its own,
    uniformly over the block's ts*ts positions and with replacement, one Philox word per value (`run_len` = 1,
    the default, is the text's statement).  `run_len` = c > 1 is an explicit departure, offered because a memory
    transaction delivers neighbouring values: the positions are then drawn as runs of c neighbouring values of
    a row (c divides ts).  In both cases a block has Cn = ts*ts/c runs, n_c = max(1, floor(k * Cn + 1/2)) of
    them are drawn, s = n_c * c values are looked at; run d is chosen by word (d mod 4) of the Philox4x32-10
    block with key (seed) and counter (iteration low, iteration high, g*Q + j, stream_id * 65536 + d div 4) as
    run number floor(word * Cn / 2^32), runs numbered row-major; the block passes iff at least
    max(1, ceil(t * s)) of the values looked at exceed the threshold, the product taken exactly (t is the
    binary fraction the caller's double holds);
  * the bound: in every group at most `cap` blocks are labelled sensitive, namely the passing blocks with
    the highest counts (equal counts: the lower block index first);
  * a probability p becomes the integer P = min(floor(p * 2^32), 2^32 - 1); block (g, j) is dropped iff word 0
    of the block with counter (iteration low, iteration high, g*Q + j, stream_id * 65536 + 65535) is < P of
    its label (m for sensitive, n for the others, n > m);
  * no rescale is mentioned: alpha is an explicit argument; the backward products are the exact adjoints.
"""
from __future__ import annotations

import math
from fractions import Fraction

import numpy as np

from .pattern import philox4x32_10, MASK32

TWO32 = 1 << 32


def transaction_run(ts):
    """The run length at which every run of bf16 / fp32 values is one aligned piece of a row: gcd(ts, 32).
    Not the default: pass it as `run_len` to ask for the clustered sample."""
    return math.gcd(ts, 32)


def n_runs(k_frac, ts, run_len=1):
    """How many runs of a block are drawn (run_len = 1: how many values)."""
    assert run_len >= 1 and ts % run_len == 0
    return max(1, int(math.floor(k_frac * (ts * ts // run_len) + 0.5)))


def n_samples(k_frac, ts, run_len=1):
    """How many values of a block are looked at."""
    return n_runs(k_frac, ts, run_len) * run_len


def needed(t_frac, s):
    """Smallest count that reaches the fraction t of s sampled values: max(1, ceil(t * s)) in exact arithmetic."""
    return max(1, math.ceil(Fraction(t_frac) * s))


def quantise_probability(p):
    return min(int(math.floor(p * TWO32)), TWO32 - 1)


def block_count(A, g, j, ts, k_frac, threshold, seed, iteration, stream_id, run_len=1):
    """Sec. 5.1, step 2 for block j of group g: how many of the sampled values exceed the threshold."""
    A = np.asarray(A)
    Q = A.shape[1] // ts
    c = run_len
    Cn = ts * ts // c
    per_row = ts // c
    n_c = n_runs(k_frac, ts, run_len)
    assert (n_c + 3) // 4 <= 65535
    count = 0
    for q in range((n_c + 3) // 4):
        words = philox4x32_10((iteration & MASK32, (iteration >> 32) & MASK32, g * Q + j,
                               ((stream_id << 16) | q) & MASK32), (seed & MASK32, (seed >> 32) & MASK32))
        for w in range(4):
            if 4 * q + w >= n_c:
                break
            run = (words[w] * Cn) >> 32
            row, col = g * ts + run // per_row, j * ts + (run % per_row) * c
            for e in range(c):
                if float(A[row, col + e]) > threshold:
                    count += 1
    return count


def label_group(counts, need, cap):
    """Sec. 5.2.2: of the blocks of one group whose count reaches `need`, the `cap` with the highest counts
    are sensitive (ties: lower index first).  Returns a bool array."""
    counts = np.asarray(counts, dtype=np.int64)
    order = sorted(range(len(counts)), key=lambda j: (-int(counts[j]), j))
    sens = np.zeros(len(counts), dtype=bool)
    taken = 0
    for j in order:
        if taken == cap or counts[j] < need:
            break
        sens[j] = True
        taken += 1
    return sens


def predict(A, ts, k_frac, t_frac, threshold, cap, seed, iteration, stream_id, run_len=1):
    """Counts [G][Q] and sensitivity labels [G][Q] of all blocks."""
    A = np.asarray(A)
    M, Kc = A.shape
    assert M % ts == 0 and Kc % ts == 0
    G, Q = M // ts, Kc // ts
    need = needed(t_frac, n_samples(k_frac, ts, run_len))
    counts = np.zeros((G, Q), dtype=np.int64)
    sens = np.zeros((G, Q), dtype=bool)
    for g in range(G):
        for j in range(Q):
            counts[g, j] = block_count(A, g, j, ts, k_frac, threshold, seed, iteration, stream_id, run_len)
        sens[g] = label_group(counts[g], need, cap)
    return counts, sens


def draw_blocks(sens, m_prob, n_prob, seed, iteration, stream_id):
    """One Bernoulli draw per block with the probability of its label.  Returns keep [G][Q] (bool)."""
    sens = np.asarray(sens, dtype=bool)
    G, Q = sens.shape
    Pm, Pn = quantise_probability(m_prob), quantise_probability(n_prob)
    keep = np.zeros((G, Q), dtype=bool)
    for g in range(G):
        for j in range(Q):
            w0 = philox4x32_10((iteration & MASK32, (iteration >> 32) & MASK32, g * Q + j,
                                ((stream_id << 16) | 0xFFFF) & MASK32), (seed & MASK32, (seed >> 32) & MASK32))[0]
            keep[g, j] = not (w0 < (Pm if sens[g, j] else Pn))
    return keep


def block_lists(keep):
    """The index lists a device needs, all ascending.  With r = j (block along Kc) and c = g (group):
    idx = r*G + c of the kept blocks; per group the kept j (col_ptr [G+1], col_idx); per j the groups that keep
    it (row_ptr [Q+1], row_idx)."""
    keep = np.asarray(keep, dtype=bool)
    G, Q = keep.shape
    idx = [j * G + g for j in range(Q) for g in range(G) if keep[g, j]]
    col_ptr, col_idx = [0], []
    for g in range(G):
        col_idx += [j for j in range(Q) if keep[g, j]]
        col_ptr.append(len(col_idx))
    row_ptr, row_idx = [0], []
    for j in range(Q):
        row_idx += [g for g in range(G) if keep[g, j]]
        row_ptr.append(len(row_idx))
    return (np.asarray(idx, dtype=np.int64), np.asarray(col_ptr, dtype=np.int64), np.asarray(col_idx, dtype=np.int64),
            np.asarray(row_ptr, dtype=np.int64), np.asarray(row_idx, dtype=np.int64))


def block_mask(keep, ts):
    """keep [G][Q] expanded to the 0/1 mask of A [G*ts][Q*ts]."""
    return np.kron(np.asarray(keep, dtype=np.float64), np.ones((ts, ts)))


# -- the three products; W in the math orientation [Kc x N] ------------------------------------------------
def fwd(A, W, keep, ts, alpha=1.0):
    """Y = alpha * (A .* mask) W: dropped blocks of A contribute nothing."""
    return alpha * (np.asarray(A, dtype=np.float64) * block_mask(keep, ts)) @ np.asarray(W, dtype=np.float64)


def bwd_input(dY, W, keep, ts, alpha=1.0):
    """dA = alpha * (dY W^T) .* mask: dropped blocks receive no gradient."""
    return alpha * (np.asarray(dY, dtype=np.float64) @ np.asarray(W, dtype=np.float64).T) * block_mask(keep, ts)


def bwd_weight(A, dY, keep, ts, alpha=1.0):
    """dW = alpha * (A .* mask)^T dY."""
    return alpha * (np.asarray(A, dtype=np.float64) * block_mask(keep, ts)).T @ np.asarray(dY, dtype=np.float64)
