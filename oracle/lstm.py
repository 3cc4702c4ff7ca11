"""LSTM layer under a row pattern on its hidden units: forward and BPTT.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  fp64 numpy.

The paper gives no LSTM equations: it only notes that an LSTM step is again a
matrix product (Sec. 7, LSTM experiment) and that one pattern serves a whole
iteration.  Reading used here: the row pattern of Sec. 3.1 is applied to the H
hidden units (a dropped unit loses all of its synapses), the same pattern at
every time step; gate blocks are ordered i | f | g | o, no peepholes.

  z_t = [x_t, h_{t-1}] W + bias                W: [(I+H) x 4H]
  i, f, o = sigmoid(z_i, z_f, z_o);  g = tanh(z_g)
  c_t = m * (f * c_{t-1} + i * g)
  h_t = alpha * m * o * tanh(c_t)

with m the 0/1 mask over hidden units; h_0, c_0 are masked on entry.
"""
from __future__ import annotations

import numpy as np


def _sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


def cell_fwd(Z, c_prev, m, alpha):
    """Point-wise cell update from gate pre-activations Z[B x 4H]."""
    H = c_prev.shape[1]
    i = _sigmoid(Z[:, 0 * H:1 * H])
    f = _sigmoid(Z[:, 1 * H:2 * H])
    g = np.tanh(Z[:, 2 * H:3 * H])
    o = _sigmoid(Z[:, 3 * H:4 * H])
    c = m[None, :] * (f * c_prev + i * g)
    h = alpha * m[None, :] * o * np.tanh(c)
    return i, f, g, o, c, h


def cell_bwd(i, f, g, o, c_prev, c, m, alpha, dh, dc_in):
    """Adjoint of cell_fwd.  dh: gradient w.r.t. h_t (all sources summed);
    dc_in: gradient arriving at c_t from step t+1.  Returns dZ[B x 4H] and the
    gradient w.r.t. c_{t-1}."""
    tc = np.tanh(c)
    do = dh * alpha * m[None, :] * tc
    dc = dc_in + dh * alpha * m[None, :] * o * (1.0 - tc * tc)
    dc = dc * m[None, :]
    di = dc * g
    dg = dc * i
    df = dc * c_prev
    dc_prev = dc * f
    dZ = np.concatenate([di * i * (1.0 - i), df * f * (1.0 - f),
                         dg * (1.0 - g * g), do * o * (1.0 - o)], axis=1)
    return dZ, dc_prev


def fwd(X, W, bias, m, alpha=1.0, h0=None, c0=None):
    """X: [T x B x I].  Returns dict with Hs [T x B x H], c_T and the saved
    per-step quantities needed by bwd."""
    X = np.asarray(X, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    m = np.asarray(m, dtype=np.float64)
    T, B, I = X.shape
    H = m.shape[0]
    assert W.shape == (I + H, 4 * H)
    bias = np.zeros(4 * H) if bias is None else np.asarray(bias, dtype=np.float64)
    h = np.zeros((B, H)) if h0 is None else np.asarray(h0, dtype=np.float64) * m[None, :]
    c = np.zeros((B, H)) if c0 is None else np.asarray(c0, dtype=np.float64) * m[None, :]
    saved = []
    Hs = np.zeros((T, B, H))
    for t in range(T):
        xh = np.concatenate([X[t], h], axis=1)
        Z = xh @ W + bias[None, :]
        i, f, g, o, c_new, h_new = cell_fwd(Z, c, m, alpha)
        saved.append((xh, i, f, g, o, c, c_new))
        h, c = h_new, c_new
        Hs[t] = h
    return {"Hs": Hs, "cT": c, "saved": saved}


def bwd(fw, W, m, alpha, dHs, dhT=None, dcT=None):
    """Back-propagation through time of fwd().  dHs: [T x B x H] gradient
    w.r.t. every h_t.  Returns dX [T x B x I], dW, dbias, dh0, dc0."""
    W = np.asarray(W, dtype=np.float64)
    m = np.asarray(m, dtype=np.float64)
    dHs = np.asarray(dHs, dtype=np.float64)
    T, B, H = dHs.shape
    I = W.shape[0] - H
    dW = np.zeros_like(W)
    dbias = np.zeros(4 * H)
    dX = np.zeros((T, B, I))
    dh_next = np.zeros((B, H)) if dhT is None else np.asarray(dhT, dtype=np.float64)
    dc_next = np.zeros((B, H)) if dcT is None else np.asarray(dcT, dtype=np.float64)
    for t in reversed(range(T)):
        xh, i, f, g, o, c_prev, c = fw["saved"][t]
        dh = dHs[t] + dh_next
        dZ, dc_next = cell_bwd(i, f, g, o, c_prev, c, m, alpha, dh, dc_next)
        dW += xh.T @ dZ
        dbias += dZ.sum(axis=0)
        dxh = dZ @ W.T
        dX[t] = dxh[:, :I]
        dh_next = dxh[:, I:]
    # h_0 and c_0 enter masked
    return {"dX": dX, "dW": dW, "dbias": dbias,
            "dh0": dh_next * m[None, :], "dc0": dc_next * m[None, :]}
