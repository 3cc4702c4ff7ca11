"""Pins for oracle/lstm_stack.py (stacked LSTM, dropout on the layer outputs only).

The paper prints no LSTM equations, so the pins are a library LSTM in fp64 (torch.nn.LSTM, one module per layer,
the mask applied between the modules by hand), its autograd gradients, central finite differences, and the two
properties the compact-matrix GPU path relies on: a dropped unit's fan-in row in the next layer receives no
gradient and its value is never needed.
"""
import numpy as np
import torch

from oracle import lstm_stack as S
from oracle import pattern as OP


def _setup(seed, T=5, B=3, dims=(4, 6, 5), dps=((3, 2), (2, 1))):
    rng = np.random.default_rng(seed)
    Ws = [rng.uniform(-0.4, 0.4, size=(dims[l] + dims[l + 1], 4 * dims[l + 1])) for l in range(len(dims) - 1)]
    bs = [rng.uniform(-0.2, 0.2, size=4 * dims[l + 1]) for l in range(len(dims) - 1)]
    masks = [OP.row_mask(dims[l + 1], *dps[l]) for l in range(len(dims) - 1)]
    alphas = [1.5, 2.0][:len(dims) - 1]
    X = rng.standard_normal((T, B, dims[0]))
    dY = rng.standard_normal((T, B, dims[-1]))
    return X, Ws, bs, masks, alphas, dY


def _torch_stack(X, Ws, bs, masks, alphas):
    """The same network from library modules: gate order i|f|g|o is torch's; weights are stored transposed there."""
    inp = torch.tensor(X, dtype=torch.float64, requires_grad=True)
    mods, y = [], inp
    for l, W in enumerate(Ws):
        H = W.shape[1] // 4
        I = W.shape[0] - H
        m = torch.nn.LSTM(I, H, num_layers=1, bias=True).double()
        with torch.no_grad():
            m.weight_ih_l0.copy_(torch.tensor(W[:I].T))
            m.weight_hh_l0.copy_(torch.tensor(W[I:].T))
            m.bias_ih_l0.copy_(torch.tensor(bs[l]))
            m.bias_hh_l0.zero_()
        h, _ = m(y)
        y = alphas[l] * torch.tensor(masks[l])[None, None, :] * h
        mods.append(m)
    return inp, mods, y


def test_one_layer_is_a_library_lstm_followed_by_a_column_mask():
    X, Ws, bs, masks, alphas, _ = _setup(1, dims=(4, 6), dps=((3, 2),))
    fw = S.fwd(X, Ws, bs, masks, alphas)
    _, _, y = _torch_stack(X, Ws, bs, masks, alphas)
    np.testing.assert_allclose(fw["Ys"][0], y.detach().numpy(), rtol=1e-11, atol=1e-13)
    assert np.all(fw["Ys"][0][:, :, masks[0] == 0] == 0)
    # the recurrent path is not masked: the hidden state of a dropped unit is what a plain LSTM computes
    plain = _torch_stack(X, Ws, bs, [np.ones(6)], [1.0])[2].detach().numpy()
    np.testing.assert_allclose(fw["layers"][0]["Hs"], plain, rtol=1e-11, atol=1e-13)


def test_two_layers_forward_and_gradients_against_autograd():
    X, Ws, bs, masks, alphas, dY = _setup(2)
    fw = S.fwd(X, Ws, bs, masks, alphas)
    bw = S.bwd(fw, Ws, masks, alphas, dY)
    inp, mods, y = _torch_stack(X, Ws, bs, masks, alphas)
    np.testing.assert_allclose(fw["Ys"][1], y.detach().numpy(), rtol=1e-11, atol=1e-13)
    y.backward(torch.tensor(dY))
    np.testing.assert_allclose(bw["dX"], inp.grad.numpy(), rtol=1e-10, atol=1e-12)
    for l, m in enumerate(mods):
        I = Ws[l].shape[0] - Ws[l].shape[1] // 4
        np.testing.assert_allclose(bw["dW"][l][:I], m.weight_ih_l0.grad.numpy().T, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(bw["dW"][l][I:], m.weight_hh_l0.grad.numpy().T, rtol=1e-10, atol=1e-12)
        np.testing.assert_allclose(bw["dbias"][l], m.bias_ih_l0.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_gradients_against_central_differences():
    X, Ws, bs, masks, alphas, dY = _setup(3, T=4, B=2, dims=(3, 4, 3), dps=((2, 2), (3, 1)))
    bw = S.bwd(S.fwd(X, Ws, bs, masks, alphas), Ws, masks, alphas, dY)
    loss = lambda Xv, Wv: float((S.fwd(Xv, Wv, bs, masks, alphas)["Ys"][-1] * dY).sum())
    rng = np.random.default_rng(0)
    eps = 1e-6
    for _ in range(12):
        l = int(rng.integers(0, 2))
        r, c = int(rng.integers(0, Ws[l].shape[0])), int(rng.integers(0, Ws[l].shape[1]))
        Wp = [w.copy() for w in Ws]; Wm = [w.copy() for w in Ws]
        Wp[l][r, c] += eps; Wm[l][r, c] -= eps
        fd = (loss(X, Wp) - loss(X, Wm)) / (2 * eps)
        assert abs(fd - bw["dW"][l][r, c]) <= 1e-6 * max(1.0, abs(fd)), (l, r, c)
    for _ in range(6):
        t, b, i = int(rng.integers(0, 4)), int(rng.integers(0, 2)), int(rng.integers(0, 3))
        Xp, Xm = X.copy(), X.copy()
        Xp[t, b, i] += eps; Xm[t, b, i] -= eps
        fd = (loss(Xp, Ws) - loss(Xm, Ws)) / (2 * eps)
        assert abs(fd - bw["dX"][t, b, i]) <= 1e-6 * max(1.0, abs(fd))


def test_dropped_outputs_cost_the_consumer_nothing():
    """What lets the consumer contract over kept units only: the fan-in rows of layer 1's weight that belong to
    dropped units of layer 0 get zero gradient, and changing them changes nothing."""
    X, Ws, bs, masks, alphas, dY = _setup(4)
    fw = S.fwd(X, Ws, bs, masks, alphas)
    bw = S.bwd(fw, Ws, masks, alphas, dY)
    dropped = np.where(masks[0] == 0)[0]
    assert len(dropped) > 0 and np.all(bw["dW"][1][dropped, :] == 0)
    W2 = [w.copy() for w in Ws]
    W2[1][dropped, :] += 7.0
    np.testing.assert_array_equal(S.fwd(X, W2, bs, masks, alphas)["Ys"][1], fw["Ys"][1])
    # and the top layer's dropped outputs are exact zeros whatever the weights
    assert np.all(fw["Ys"][1][:, :, masks[1] == 0] == 0)
