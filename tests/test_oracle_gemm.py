"""Pins for oracle/gemm.py and oracle/mlp_chain.py."""
import numpy as np
import pytest

from oracle import gemm as G
from oracle import mlp_chain as C
from oracle import pattern as P


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def test_bruteforce_row_all_patterns():
    B, K, N = 5, 7, 10
    X, W, dY = _rand((B, K), 1), _rand((K, N), 2), _rand((B, N), 3)
    for dp in range(1, N + 1):
        for b in range(1, dp + 1):
            m = P.row_mask(N, dp, b)
            kept = lambda k, n: (n + 1 - b) % dp == 0    # Eq. 1 on 1-based index
            a = 1.7
            np.testing.assert_allclose(G.fwd(X, W, m, a), G.fwd_bruteforce(X, W, kept, a), rtol=1e-13, atol=1e-13)
            np.testing.assert_allclose(G.bwd_data(dY, W, m, a), G.bwd_data_bruteforce(dY, W, kept, a), rtol=1e-13, atol=1e-13)
            np.testing.assert_allclose(G.bwd_weight(X, dY, m, a), G.bwd_weight_bruteforce(X, dY, kept, a), rtol=1e-13, atol=1e-13)
            # dropped outputs are exactly zero
            assert np.all(G.fwd(X, W, m, a)[:, m == 0] == 0.0)
            assert np.all(G.bwd_weight(X, dY, m, a)[:, m == 0] == 0.0)


def test_bruteforce_tile_all_patterns():
    B, K, N, ts = 3, 8, 12, 2
    Tc = N // ts
    X, W, dY = _rand((B, K), 4), _rand((K, N), 5), _rand((B, N), 6)
    for dp in range(1, 9):
        for b in range(1, dp + 1):
            M = P.tile_mask(K, N, ts, dp, b)
            kept = lambda k, n: (((k // ts) * Tc + n // ts + 1) - b) % dp == 0
            np.testing.assert_allclose(G.fwd(X, W, M, 2.0), G.fwd_bruteforce(X, W, kept, 2.0), rtol=1e-13, atol=1e-13)
            np.testing.assert_allclose(G.bwd_data(dY, W, M, 2.0), G.bwd_data_bruteforce(dY, W, kept, 2.0), rtol=1e-13, atol=1e-13)
            np.testing.assert_allclose(G.bwd_weight(X, dY, M, 2.0), G.bwd_weight_bruteforce(X, dY, kept, 2.0), rtol=1e-13, atol=1e-13)


def test_dense_special_case_is_plain_matmul():
    X, W, dY = _rand((9, 11), 7), _rand((11, 13), 8), _rand((9, 13), 9)
    ones = np.ones(13)
    np.testing.assert_allclose(G.fwd(X, W, ones), np.matmul(X, W), rtol=1e-14)
    np.testing.assert_allclose(G.bwd_data(dY, W, ones), np.matmul(dY, W.T), rtol=1e-14)
    np.testing.assert_allclose(G.bwd_weight(X, dY, ones), np.matmul(X.T, dY), rtol=1e-14)


@pytest.mark.parametrize("kind", ["row", "tile"])
def test_adjoint_identity(kind):
    """<dY, Y> = <dX, X> = <dW, W> for the masked linear map."""
    B, K, N = 6, 8, 12
    X, W, dY = _rand((B, K), 10), _rand((K, N), 11), _rand((B, N), 12)
    m = P.row_mask(N, 3, 2) if kind == "row" else P.tile_mask(K, N, 4, 3, 2)
    a = 1.0 / (1.0 - 0.5)
    s1 = np.sum(dY * G.fwd(X, W, m, a))
    s2 = np.sum(G.bwd_data(dY, W, m, a) * X)
    s3 = np.sum(G.bwd_weight(X, dY, m, a) * W)
    assert abs(s1 - s2) < 1e-10 * abs(s1) and abs(s1 - s3) < 1e-10 * abs(s1)


def test_input_side_mask():
    B, K, N = 4, 6, 9
    X, W, dY = _rand((B, K), 13), _rand((K, N), 14), _rand((B, N), 15)
    m, mi = P.row_mask(N, 2, 1), P.row_mask(K, 3, 2)
    Xm = X * mi[None, :]
    np.testing.assert_allclose(G.fwd(X, W, m, 1.5, in_mask=mi), G.fwd(Xm, W, m, 1.5))
    assert np.all(G.bwd_data(dY, W, m, 1.5, in_mask=mi)[:, mi == 0] == 0)
    assert np.all(G.bwd_weight(X, dY, m, 1.5, in_mask=mi)[mi == 0, :] == 0)


def test_sampled_forms_agree_with_full():
    B, K, N = 10, 8, 12
    X, W, dY = _rand((B, K), 16), _rand((K, N), 17), _rand((B, N), 18)
    m = P.row_mask(N, 4, 3)
    rows = [0, 3, 9]
    cols = [2, 6, 7]
    np.testing.assert_array_equal(G.fwd_rows(X, W, m, 2.0, rows), G.fwd(X, W, m, 2.0)[rows])
    np.testing.assert_array_equal(G.bwd_data_rows(dY, W, m, 2.0, rows), G.bwd_data(dY, W, m, 2.0)[rows])
    np.testing.assert_allclose(G.bwd_weight_cols(X, dY, m, 2.0, cols), G.bwd_weight(X, dY, m, 2.0)[:, cols], rtol=1e-14)


def test_chain_gradients_by_finite_differences():
    rng = np.random.default_rng(3)
    B, d0, d1, d2, d3 = 4, 5, 8, 6, 3
    X = rng.random((B, d0))
    W1, W2, W3 = (rng.standard_normal(s) * 0.7 for s in [(d0, d1), (d1, d2), (d2, d3)])
    m1, m2 = P.row_mask(d1, 2, 2), P.row_mask(d2, 3, 1)
    a1, a2 = 1 / 0.5, 1 / 0.7
    dZ3 = rng.standard_normal((B, d3))
    fw = C.fwd(X, W1, W2, W3, m1, m2, a1, a2)
    bw = C.bwd(X, W1, W2, W3, m1, m2, a1, a2, fw, dZ3)
    assert np.all(fw["A1"][:, m1 == 0] == 0) and np.all(fw["A2"][:, m2 == 0] == 0)

    def loss(X_, W1_, W2_, W3_):
        return float(np.sum(dZ3 * C.fwd(X_, W1_, W2_, W3_, m1, m2, a1, a2)["Z3"]))

    eps = 1e-6
    for name, idx, grad in [("W1", 1, bw["dW1"]), ("W2", 2, bw["dW2"]), ("W3", 3, bw["dW3"]), ("X", 0, bw["dX"])]:
        args = [X, W1, W2, W3]
        num = np.zeros_like(args[idx])
        for pos in np.ndindex(*args[idx].shape):
            ap = [a.copy() for a in args]
            am = [a.copy() for a in args]
            ap[idx][pos] += eps
            am[idx][pos] -= eps
            num[pos] = (loss(*ap) - loss(*am)) / (2 * eps)
        np.testing.assert_allclose(grad, num, rtol=1e-5, atol=1e-7, err_msg=name)
