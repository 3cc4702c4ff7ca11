"""Three-layer MLP training-step products under row patterns on both hidden
layers (the 784-2048-2048-10 experiment of Sec. 7).

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  fp64 numpy.

The paper's step is fully connected layer -> activation -> (skipped) dropout
layer (Sec. 3.2, last paragraph).  Reading: ReLU activation, no bias,
relu'(0) = 0; a dropped hidden neuron outputs exactly zero, so the consumer
layer may also skip the matching input column (Sec. 3.1 describes a
dropped neuron as removing its row of the next layer's weight).
"""
from __future__ import annotations

import numpy as np
from . import gemm


def fwd(X, W1, W2, W3, m1, m2, a1, a2):
    Z1 = gemm.fwd(X, W1, m1, a1)
    A1 = np.maximum(Z1, 0.0)
    Z2 = gemm.fwd(A1, W2, m2, a2, in_mask=m1)
    A2 = np.maximum(Z2, 0.0)
    Z3 = gemm.fwd(A2, W3, np.ones(W3.shape[1]), 1.0, in_mask=m2)
    return {"Z1": Z1, "A1": A1, "Z2": Z2, "A2": A2, "Z3": Z3}


def bwd(X, W1, W2, W3, m1, m2, a1, a2, fw, dZ3):
    ones3 = np.ones(W3.shape[1])
    dW3 = gemm.bwd_weight(fw["A2"], dZ3, ones3, 1.0, in_mask=m2)
    dA2 = gemm.bwd_data(dZ3, W3, ones3, 1.0, in_mask=m2)
    dZ2 = dA2 * (fw["Z2"] > 0.0)
    dW2 = gemm.bwd_weight(fw["A1"], dZ2, m2, a2, in_mask=m1)
    dA1 = gemm.bwd_data(dZ2, W2, m2, a2, in_mask=m1)
    dZ1 = dA1 * (fw["Z1"] > 0.0)
    dW1 = gemm.bwd_weight(X, dZ1, m1, a1)
    dX = gemm.bwd_data(dZ1, W1, m1, a1)
    return {"dW3": dW3, "dA2": dA2, "dZ2": dZ2, "dW2": dW2, "dA1": dA1,
            "dZ1": dZ1, "dW1": dW1, "dX": dX}
