"""Pins for oracle/lstm.py: library LSTM (dp = 1 and the kept sub-network) and finite differences."""
import numpy as np
import torch

from oracle import lstm as L
from oracle import pattern as P


def _torch_lstm(W, bias, I, H):
    """torch.nn.LSTM (gate order i, f, g, o) loaded with W[(I+H) x 4H] in math orientation."""
    net = torch.nn.LSTM(I, H, num_layers=1, bias=True).double()
    with torch.no_grad():
        net.weight_ih_l0.copy_(torch.from_numpy(W[:I].T.copy()))
        net.weight_hh_l0.copy_(torch.from_numpy(W[I:].T.copy()))
        net.bias_ih_l0.copy_(torch.from_numpy(bias))
        net.bias_hh_l0.zero_()
    return net


def test_dense_case_equals_library_lstm_forward_and_gradients():
    rng = np.random.default_rng(0)
    T, B, I, H = 5, 3, 4, 6
    W = rng.uniform(-0.5, 0.5, (I + H, 4 * H))
    bias = rng.uniform(-0.2, 0.2, 4 * H)
    X = rng.standard_normal((T, B, I))
    dHs = rng.standard_normal((T, B, H))
    dcT = rng.standard_normal((B, H))
    h0 = rng.standard_normal((B, H)) * 0.3
    c0 = rng.standard_normal((B, H)) * 0.3
    m = np.ones(H)
    fw = L.fwd(X, W, bias, m, 1.0, h0, c0)
    bw = L.bwd(fw, W, m, 1.0, dHs, None, dcT)

    net = _torch_lstm(W, bias, I, H)
    xt = torch.from_numpy(X).requires_grad_(True)
    h0t = torch.from_numpy(h0[None]).requires_grad_(True)
    c0t = torch.from_numpy(c0[None]).requires_grad_(True)
    out, (hT, cT) = net(xt, (h0t, c0t))
    np.testing.assert_allclose(fw["Hs"], out.detach().numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(fw["cT"], cT[0].detach().numpy(), rtol=1e-12, atol=1e-13)
    loss = (out * torch.from_numpy(dHs)).sum() + (cT[0] * torch.from_numpy(dcT)).sum()
    loss.backward()
    np.testing.assert_allclose(bw["dX"], xt.grad.numpy(), rtol=1e-10, atol=1e-12)
    dW_t = np.concatenate([net.weight_ih_l0.grad.numpy().T, net.weight_hh_l0.grad.numpy().T], axis=0)
    np.testing.assert_allclose(bw["dW"], dW_t, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(bw["dbias"], net.bias_ih_l0.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(bw["dh0"], h0t.grad[0].numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(bw["dc0"], c0t.grad[0].numpy(), rtol=1e-10, atol=1e-12)


def test_masked_case_equals_library_lstm_on_kept_subnetwork():
    """With hidden units dropped, the kept units form a textbook LSTM of size n_k whose
    recurrent weights see h scaled by alpha: h~ = h/alpha obeys the plain recursion with
    W_hh scaled by alpha."""
    rng = np.random.default_rng(1)
    T, B, I, H = 6, 2, 5, 9
    dp, b, alpha = 3, 2, 1.0 / (1.0 - 0.6)
    W = rng.uniform(-0.4, 0.4, (I + H, 4 * H))
    bias = rng.uniform(-0.2, 0.2, 4 * H)
    X = rng.standard_normal((T, B, I))
    dHs = rng.standard_normal((T, B, H))
    m = P.row_mask(H, dp, b)
    keep = P.row_keep(H, dp, b)
    nk = len(keep)
    fw = L.fwd(X, W, bias, m, alpha)
    bw = L.bwd(fw, W, m, alpha, dHs)
    assert np.all(fw["Hs"][:, :, m == 0] == 0) and np.all(fw["cT"][:, m == 0] == 0)

    gate_cols = np.concatenate([g * H + keep for g in range(4)])
    rows = np.concatenate([np.arange(I), I + keep])
    Wsub = W[np.ix_(rows, gate_cols)].copy()
    Wsub[I:] *= alpha
    net = _torch_lstm(Wsub, bias[gate_cols], I, nk)
    xt = torch.from_numpy(X).requires_grad_(True)
    out, (hT, cT) = net(xt)
    np.testing.assert_allclose(fw["Hs"][:, :, keep], alpha * out.detach().numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(fw["cT"][:, keep], cT[0].detach().numpy(), rtol=1e-12, atol=1e-13)
    loss = (alpha * out * torch.from_numpy(dHs[:, :, keep])).sum()
    loss.backward()
    np.testing.assert_allclose(bw["dX"], xt.grad.numpy(), rtol=1e-10, atol=1e-12)
    dWsub = np.concatenate([net.weight_ih_l0.grad.numpy().T, alpha * net.weight_hh_l0.grad.numpy().T], axis=0)
    np.testing.assert_allclose(bw["dW"][np.ix_(rows, gate_cols)], dWsub, rtol=1e-10, atol=1e-12)
    # gate columns and recurrent rows of dropped units receive exactly zero gradient
    dropped_cols = np.setdiff1d(np.arange(4 * H), gate_cols)
    assert np.all(bw["dW"][:, dropped_cols] == 0)
    assert np.all(bw["dW"][I + np.where(m == 0)[0], :] == 0)
    assert np.all(bw["dbias"][dropped_cols] == 0)


def test_bptt_by_finite_differences_with_initial_state():
    rng = np.random.default_rng(2)
    T, B, I, H = 3, 2, 3, 4
    alpha = 2.0
    m = P.row_mask(H, 2, 1)
    W = rng.uniform(-0.5, 0.5, (I + H, 4 * H))
    bias = rng.uniform(-0.2, 0.2, 4 * H)
    X = rng.standard_normal((T, B, I))
    h0 = rng.standard_normal((B, H)) * 0.5
    c0 = rng.standard_normal((B, H)) * 0.5
    dHs = rng.standard_normal((T, B, H))
    dhT = rng.standard_normal((B, H))
    dcT = rng.standard_normal((B, H))

    def loss(W_, X_, h0_, c0_, bias_):
        fw = L.fwd(X_, W_, bias_, m, alpha, h0_, c0_)
        return float(np.sum(fw["Hs"] * dHs) + np.sum(fw["Hs"][-1] * dhT) + np.sum(fw["cT"] * dcT))

    fw = L.fwd(X, W, bias, m, alpha, h0, c0)
    bw = L.bwd(fw, W, m, alpha, dHs, dhT, dcT)
    eps = 1e-6
    args = [W, X, h0, c0, bias]
    for idx, g in [(0, bw["dW"]), (1, bw["dX"]), (2, bw["dh0"]), (3, bw["dc0"]), (4, bw["dbias"])]:
        num = np.zeros_like(args[idx])
        for pos in np.ndindex(*args[idx].shape):
            ap = [a.copy() for a in args]
            am = [a.copy() for a in args]
            ap[idx][pos] += eps
            am[idx][pos] -= eps
            num[pos] = (loss(*ap) - loss(*am)) / (2 * eps)
        np.testing.assert_allclose(g, num, rtol=2e-6, atol=1e-8)
