"""Stack of LSTM layers with dropout on the layer OUTPUTS only: forward and BPTT.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  fp64 numpy.

Second reading of the LSTM experiment of Sec. 7 (the paper prints no LSTM equations; its networks are stacks of two
and three LSTM layers).  Here dropout touches only the non-recurrent connections, the usual way of regularising a
stacked LSTM: every unit of a layer is computed at every step and the recurrent path h_{t-1} -> h_t is left alone;
what a layer hands to the layer above it (and the top layer to whatever follows the stack) is masked by that
layer's row pattern (Sec. 3.1, Eq. 1) and rescaled,

    (h^l_t, c^l_t) = LSTM cell of layer l on [y^{l-1}_t, h^l_{t-1}]        (no mask inside the layer)
    y^l_t          = alpha_l * m_l .* h^l_t                                 (y^{-1}_t = x_t)

one pattern per layer and iteration, the same at every time step.  A dropped unit of layer l multiplies the
matching fan-in row of layer l+1's weight by zero, so the consumer may contract over kept units only.
PARITY UNPINNED by the paper; pinned to a library LSTM (fp64) with the mask applied between the layers, to its
autograd gradients and to finite differences.  The layer itself is oracle/lstm.py with an all-ones mask.
"""
from __future__ import annotations

import numpy as np

from . import lstm as L1


def fwd(X, Ws, biases, masks, alphas):
    """X [T x B x I0]; Ws[l] [(I_l + H_l) x 4 H_l]; masks[l] 0/1 over the H_l units; alphas[l].
    Returns the masked outputs of every layer (Ys[l] [T x B x H_l]) and what bwd needs."""
    inp = np.asarray(X, dtype=np.float64)
    layers, Ys = [], []
    for l, W in enumerate(Ws):
        H = np.asarray(W).shape[1] // 4
        fw = L1.fwd(inp, W, None if biases is None else biases[l], np.ones(H), 1.0)
        y = alphas[l] * np.asarray(masks[l], dtype=np.float64)[None, None, :] * fw["Hs"]
        layers.append(fw)
        Ys.append(y)
        inp = y
    return {"Ys": Ys, "layers": layers}


def bwd(fw, Ws, masks, alphas, dY_top):
    """dY_top [T x B x H_top]: gradient with respect to the top layer's masked output.
    Returns dX [T x B x I0] and per layer dW, dbias."""
    dY = np.asarray(dY_top, dtype=np.float64)
    dWs, dbs = [None] * len(Ws), [None] * len(Ws)
    for l in reversed(range(len(Ws))):
        H = np.asarray(Ws[l]).shape[1] // 4
        dH = alphas[l] * np.asarray(masks[l], dtype=np.float64)[None, None, :] * dY
        bw = L1.bwd(fw["layers"][l], Ws[l], np.ones(H), 1.0, dH)
        dWs[l], dbs[l] = bw["dW"], bw["dbias"]
        dY = bw["dX"]
    return {"dX": dY, "dW": dWs, "dbias": dbs}
