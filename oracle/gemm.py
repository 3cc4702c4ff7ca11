"""Masked dense products: what the compacted GEMMs must equal.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  fp64 numpy.

Orientation: X[B x K], W[K x N] (math orientation, Y = X W), dY[B x N].
Sec. 3.1: only the kept rows are fetched and multiplied and every other entry
of the output is zero, i.e. the result equals the product with the
dropped part of W replaced by zeros.  The backward products are the exact
adjoints of that forward map (the paper states only that forward and backward
are both accelerated).
"""
from __future__ import annotations

import numpy as np


def expand_mask(mask, K_dim, N_dim):
    """A row pattern's 0/1 vector over the N output neurons, or a tile
    pattern's [K x N] matrix, as a full [K x N] synapse mask."""
    mask = np.asarray(mask, dtype=np.float64)
    if mask.ndim == 1:
        assert mask.shape == (N_dim,)
        return np.broadcast_to(mask[None, :], (K_dim, N_dim))
    assert mask.shape == (K_dim, N_dim)
    return mask


def fwd(X, W, mask, alpha=1.0, in_mask=None):
    """Y = alpha * (X . m_in) (W . Mask)."""
    X = np.asarray(X, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    M = expand_mask(mask, *W.shape)
    if in_mask is not None:
        X = X * np.asarray(in_mask, dtype=np.float64)[None, :]
    return alpha * (X @ (W * M))


def bwd_data(dY, W, mask, alpha=1.0, in_mask=None):
    """dX = alpha * dY (W . Mask)^T, columns of dropped inputs zeroed."""
    dY = np.asarray(dY, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    M = expand_mask(mask, *W.shape)
    dX = alpha * (dY @ (W * M).T)
    if in_mask is not None:
        dX = dX * np.asarray(in_mask, dtype=np.float64)[None, :]
    return dX


def bwd_weight(X, dY, mask, alpha=1.0, in_mask=None):
    """dW = alpha * (X^T dY) . Mask  in the math orientation [K x N]."""
    X = np.asarray(X, dtype=np.float64)
    dY = np.asarray(dY, dtype=np.float64)
    if in_mask is not None:
        X = X * np.asarray(in_mask, dtype=np.float64)[None, :]
    M = expand_mask(mask, X.shape[1], dY.shape[1])
    return alpha * ((X.T @ dY) * M)


# -- sampled forms for sizes where the full fp64 product takes too long -------
def fwd_rows(X, W, mask, alpha, rows):
    """Rows `rows` of fwd(...)."""
    return fwd(np.asarray(X)[rows], W, mask, alpha)


def bwd_data_rows(dY, W, mask, alpha, rows):
    """Rows `rows` of bwd_data(...)."""
    return bwd_data(np.asarray(dY)[rows], W, mask, alpha)


def bwd_weight_cols(X, dY, mask, alpha, cols):
    """Columns `cols` (output neurons) of bwd_weight(...), shape [K x len(cols)]."""
    X = np.asarray(X, dtype=np.float64)
    dYc = np.asarray(dY, dtype=np.float64)[:, cols]
    M = expand_mask(mask, X.shape[1], np.asarray(dY).shape[1])[:, cols]
    return alpha * ((X.T @ dYc) * M)


# -- brute force on tiny shapes: scalar loops with an `if kept` ---------------
def fwd_bruteforce(X, W, kept, alpha=1.0):
    """kept(k, n) -> bool.  Pure-Python loops; only for tiny problems."""
    B, K = len(X), len(X[0])
    N = len(W[0])
    Y = [[0.0] * N for _ in range(B)]
    for i in range(B):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                if kept(k, n):
                    acc += float(X[i][k]) * float(W[k][n])
            Y[i][n] = alpha * acc
    return np.array(Y)


def bwd_data_bruteforce(dY, W, kept, alpha=1.0):
    B, N = len(dY), len(dY[0])
    K = len(W)
    dX = [[0.0] * K for _ in range(B)]
    for i in range(B):
        for k in range(K):
            acc = 0.0
            for n in range(N):
                if kept(k, n):
                    acc += float(dY[i][n]) * float(W[k][n])
            dX[i][k] = alpha * acc
    return np.array(dX)


def bwd_weight_bruteforce(X, dY, kept, alpha=1.0):
    B, K = len(X), len(X[0])
    N = len(dY[0])
    dW = [[0.0] * N for _ in range(K)]
    for k in range(K):
        for n in range(N):
            if kept(k, n):
                acc = 0.0
                for i in range(B):
                    acc += float(X[i][k]) * float(dY[i][n])
                dW[k][n] = alpha * acc
    return np.array(dW)


def rel_fro(G, O):
    """|G - O|_F / |O|_F  (0 if both are all-zero)."""
    G = np.asarray(G, dtype=np.float64)
    O = np.asarray(O, dtype=np.float64)
    den = np.linalg.norm(O)
    num = np.linalg.norm(G - O)
    if den == 0.0:
        return 0.0 if num == 0.0 else float("inf")
    return float(num / den)
