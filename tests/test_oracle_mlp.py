"""Pins for oracle/mlp.py (fused layer step: product -> bias -> ReLU -> dropout mask, Sec. 3.1 / 3.2).

What fixes the oracle from outside: torch autograd in fp64 on the same network written with library
ops (forward values and every gradient), central differences, the three-layer chain of
oracle/mlp_chain.py (no bias), and the equality of the masked full-width form with the form on compact
matrices that Sec. 3.1 describes.
"""
import numpy as np
import pytest
import torch

from oracle import mlp as M
from oracle import mlp_chain as C
from oracle import pattern as P


def _net(seed, dims, B, pats):
    rng = np.random.default_rng(seed)
    Ws = [rng.standard_normal((dims[l], dims[l + 1])) / np.sqrt(dims[l]) for l in range(len(dims) - 1)]
    bs = [rng.uniform(-0.3, 0.3, dims[l + 1]) for l in range(len(dims) - 1)]
    X = rng.standard_normal((B, dims[0]))
    masks = [P.row_mask(dims[l + 1], *pats[l]) for l in range(len(dims) - 2)] + [np.ones(dims[-1])]
    alphas = [1.0 / (1.0 - 0.4)] * (len(dims) - 2) + [1.0]
    dOut = rng.standard_normal((B, dims[-1]))
    return X, Ws, bs, masks, alphas, dOut


@pytest.mark.parametrize("pats", [[(1, 1), (1, 1)], [(2, 1), (3, 2)], [(5, 5), (2, 2)]])
def test_against_torch_autograd(pats):
    dims = [13, 24, 17, 5]
    X, Ws, bs, masks, alphas, dOut = _net(3, dims, 9, pats)
    fw = M.fwd(X, Ws, bs, masks, alphas)
    bw = M.bwd(fw, Ws, masks, alphas, dOut)
    tX = torch.tensor(X, dtype=torch.float64, requires_grad=True)
    tW = [torch.tensor(w, dtype=torch.float64, requires_grad=True) for w in Ws]
    tb = [torch.tensor(b, dtype=torch.float64, requires_grad=True) for b in bs]
    a = tX
    for l in range(3):
        z = torch.nn.functional.linear(a, tW[l].T, tb[l])
        a = alphas[l] * torch.relu(z) * torch.tensor(masks[l]) if l < 2 else z
    np.testing.assert_allclose(fw["A"][-1], a.detach().numpy(), rtol=1e-12, atol=1e-12)
    (a * torch.tensor(dOut)).sum().backward()
    np.testing.assert_allclose(bw["dX"], tX.grad.numpy(), rtol=1e-11, atol=1e-12)
    for l in range(3):
        np.testing.assert_allclose(bw["dW"][l], tW[l].grad.numpy(), rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(bw["db"][l], tb[l].grad.numpy(), rtol=1e-11, atol=1e-12)
        if l < 2:  # nothing flows through a dropped neuron
            assert np.all(bw["dW"][l][:, masks[l] == 0] == 0) and np.all(bw["db"][l][masks[l] == 0] == 0)


def test_central_differences():
    dims = [6, 10, 8, 3]
    X, Ws, bs, masks, alphas, dOut = _net(5, dims, 4, [(2, 2), (3, 1)])
    fw = M.fwd(X, Ws, bs, masks, alphas)
    bw = M.bwd(fw, Ws, masks, alphas, dOut)

    def loss():
        return float((M.fwd(X, Ws, bs, masks, alphas)["A"][-1] * dOut).sum())

    rng = np.random.default_rng(0)
    eps = 1e-6
    for arr, grad in [(Ws[0], bw["dW"][0]), (Ws[1], bw["dW"][1]), (Ws[2], bw["dW"][2]), (bs[0], bw["db"][0]),
                      (bs[1], bw["db"][1]), (bs[2], bw["db"][2]), (X, bw["dX"])]:
        for _ in range(6):
            i = tuple(rng.integers(0, s) for s in arr.shape)
            old = arr[i]
            arr[i] = old + eps
            lp = loss()
            arr[i] = old - eps
            lm = loss()
            arr[i] = old
            assert abs((lp - lm) / (2 * eps) - grad[i]) <= 1e-6 * max(1.0, abs(grad[i]))


def test_without_bias_it_is_the_three_layer_chain():
    dims = [20, 32, 16, 4]
    X, Ws, _, masks, alphas, dOut = _net(7, dims, 5, [(3, 2), (2, 1)])
    fw = M.fwd(X, Ws, None, masks, alphas)
    bw = M.bwd(fw, Ws, masks, alphas, dOut)
    cf = C.fwd(X, Ws[0], Ws[1], Ws[2], masks[0], masks[1], alphas[0], alphas[1])
    cb = C.bwd(X, Ws[0], Ws[1], Ws[2], masks[0], masks[1], alphas[0], alphas[1], cf, dOut)
    np.testing.assert_allclose(fw["A"][1], cf["A1"], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(fw["A"][3], cf["Z3"], rtol=1e-12, atol=1e-13)
    for l, k in enumerate(["dW1", "dW2", "dW3"]):
        np.testing.assert_allclose(bw["dW"][l], cb[k], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(bw["dX"], cb["dX"], rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("pin,pout", [((1, 1), (2, 1)), ((3, 2), (1, 1)), ((2, 2), (5, 3)), ((7, 7), (7, 1))])
def test_compact_matrices_give_the_masked_full_width_result(pin, pout):
    """Sec. 3.1: dropping a neuron removes its column of this layer's output AND its row of the next
    layer's weight; the product of the two compact matrices equals the masked full-width product."""
    B, K, N = 6, 23, 31
    rng = np.random.default_rng(11)
    m_in, keep_in = P.row_mask(K, *pin), P.row_keep(K, *pin)
    m, keep = P.row_mask(N, *pout), P.row_keep(N, *pout)
    A_prev = rng.standard_normal((B, K)) * m_in[None, :]     # output of a layer under pattern `pin`
    W = rng.standard_normal((K, N))
    bias = rng.standard_normal(N)
    Z, A = M.layer_fwd(A_prev, W, bias, m, 1.7)
    Ac = M.layer_fwd_compact(A_prev[:, keep_in], keep_in, W, bias, keep, 1.7)
    np.testing.assert_allclose(A[:, keep], Ac, rtol=1e-12, atol=1e-13)
    assert np.all(A[:, m == 0] == 0)
    dA = rng.standard_normal((B, N))
    dZ, dW, db, dA_prev = M.layer_bwd(A_prev, W, m, 1.7, Z, dA)
    dWc, dbc, dAc_prev = M.layer_bwd_compact(A_prev[:, keep_in], keep_in, W, keep, dZ[:, keep])
    np.testing.assert_allclose(dW[np.ix_(keep_in, keep)], dWc, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(db[keep], dbc, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dA_prev[:, keep_in], dAc_prev, rtol=1e-12, atol=1e-13)
    # what the compact form never computes is zero in the full-width form, or is never used:
    assert np.all(dW[:, m == 0] == 0) and np.all(dW[m_in == 0, :] == 0)


def test_relu_subgradient_at_zero_is_zero():
    Z, A = M.layer_fwd(np.zeros((1, 2)), np.zeros((2, 3)), np.array([0.0, 1.0, -1.0]), np.ones(3), 2.0)
    dZ, _, db, _ = M.layer_bwd(np.zeros((1, 2)), np.zeros((2, 3)), np.ones(3), 2.0, Z, np.ones((1, 3)))
    assert A.tolist() == [[0.0, 2.0, 0.0]] and dZ.tolist() == [[0.0, 2.0, 0.0]] and db.tolist() == [0.0, 2.0, 0.0]
