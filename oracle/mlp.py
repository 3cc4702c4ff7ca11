"""Fully connected layer -> activation -> dropout as ONE layer step, for a stack of layers.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  fp64 numpy.

Sec. 3.2 (last paragraph) names the three steps of a layer: the fully connected product, the
activation and the dropout mask; under a dropout pattern the third step disappears and the first one
shrinks.  Sec. 3.1: a dropped neuron's output is zero, and the layer that consumes it may leave the
matching column of its input matrix and of its weight out as well, so that both matrices of the product
are compact.

Reading (the paper prints no formula for the activation): ReLU with relu'(0) = 0, a bias per neuron,
inverted dropout, i.e. for layer l with row mask m_l over its neurons and rescale alpha_l

    Z_l = A_{l-1} W_l + bias_l             (A_0 = X)
    A_l = alpha_l * relu(Z_l) . m_l        (hidden layers)
    A_L = Z_L                              (the last layer is linear and is not dropped)

and the backward pass is the exact adjoint of that map.  Orientation as in gemm.py: W_l [K_l x N_l].
"""
from __future__ import annotations

import numpy as np


def layer_fwd(A_prev, W, bias, m, alpha, relu=True):
    """One layer step on full-width operands.  Returns (Z, A)."""
    A_prev = np.asarray(A_prev, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    m = np.asarray(m, dtype=np.float64)
    Z = A_prev @ W
    if bias is not None:
        Z = Z + np.asarray(bias, dtype=np.float64)[None, :]
    H = np.maximum(Z, 0.0) if relu else Z
    return Z, alpha * H * m[None, :]


def layer_bwd(A_prev, W, m, alpha, Z, dA, relu=True):
    """Adjoint of layer_fwd.  Returns (dZ, dW [K x N], dbias [N], dA_prev)."""
    A_prev = np.asarray(A_prev, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    m = np.asarray(m, dtype=np.float64)
    dH = alpha * np.asarray(dA, dtype=np.float64) * m[None, :]
    dZ = dH * (np.asarray(Z) > 0.0) if relu else dH
    dW = A_prev.T @ dZ
    db = dZ.sum(axis=0)
    dA_prev = dZ @ W.T
    return dZ, dW, db, dA_prev


def fwd(X, Ws, biases, masks, alphas):
    """Stack of len(Ws) layers; the last one is linear.  Returns {"Z": [...], "A": [X, A_1, ..., A_L]}."""
    L = len(Ws)
    A = [np.asarray(X, dtype=np.float64)]
    Zs = []
    for l in range(L):
        Z, Al = layer_fwd(A[-1], Ws[l], None if biases is None else biases[l], masks[l], alphas[l], relu=(l < L - 1))
        Zs.append(Z)
        A.append(Al)
    return {"Z": Zs, "A": A}


def bwd(fw, Ws, masks, alphas, dOut):
    """Gradients of <dOut, A_L> with respect to every weight, bias and the input."""
    L = len(Ws)
    dA = np.asarray(dOut, dtype=np.float64)
    dWs, dbs, dZs = [None] * L, [None] * L, [None] * L
    for l in range(L - 1, -1, -1):
        dZs[l], dWs[l], dbs[l], dA = layer_bwd(fw["A"][l], Ws[l], masks[l], alphas[l], fw["Z"][l], dA, relu=(l < L - 1))
    return {"dW": dWs, "db": dbs, "dZ": dZs, "dX": dA}


# -- the same layer on compact matrices (Sec. 3.1: compact input matrix and compact weight matrix) ----
def layer_fwd_compact(Ac_prev, keep_in, W, bias, keep, alpha, relu=True):
    """Ac_prev [B x len(keep_in)] holds the kept input columns only (keep_in = None: all of them).
    Returns the compact activations [B x len(keep)] of the kept neurons."""
    W = np.asarray(W, dtype=np.float64)
    Wk = W if keep_in is None else W[np.asarray(keep_in), :]
    Wk = Wk[:, np.asarray(keep)]
    Z = np.asarray(Ac_prev, dtype=np.float64) @ Wk
    if bias is not None:
        Z = Z + np.asarray(bias, dtype=np.float64)[np.asarray(keep)][None, :]
    H = np.maximum(Z, 0.0) if relu else Z
    return alpha * H


def layer_bwd_compact(Ac_prev, keep_in, W, keep, dZc):
    """dZc [B x len(keep)]: gradient of the pre-activations of the kept neurons.  Returns the compact
    weight gradient [len(keep_in) x len(keep)], the compact bias gradient and the gradient of the kept inputs."""
    W = np.asarray(W, dtype=np.float64)
    Wk = W if keep_in is None else W[np.asarray(keep_in), :]
    Wk = Wk[:, np.asarray(keep)]
    dZc = np.asarray(dZc, dtype=np.float64)
    return np.asarray(Ac_prev, dtype=np.float64).T @ dZc, dZc.sum(axis=0), dZc @ Wk.T
