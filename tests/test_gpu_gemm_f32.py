"""fp32 path (CUDA cores) vs the oracle: config 1 over every (dp, b), sampled iterations, tile patterns."""
import numpy as np
import pytest

from oracle import pattern as OP
from paper_2203_05705_b200 import ard, inputs
from gpu_helpers import Ctx, run_three_gemms, assert_ok, TOL
from distributions import max_entropy_K

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = Ctx(0)
    yield c
    c.close()


def test_config1_all_patterns(ctx):
    c1 = inputs.config1()
    X, W, dY = c1["X"], c1["W"], c1["dY"]
    pat = ctx.pattern(ard.ARD_ROW, 784, 256)
    alpha = 1.0 / (1.0 - c1["p"])
    for dp in range(1, c1["n_dp"] + 1):
        for b in range(1, dp + 1):
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            res = run_three_gemms(ctx, pat, ard.ARD_ROW, ard.ARD_F32, X, W, dY, dp, b, alpha)
            assert_ok(res, TOL[ard.ARD_F32], (dp, b))


def test_config1_sampled_iterations(ctx):
    c1 = inputs.config1()
    K = max_entropy_K(c1["p"], c1["n_dp"])
    cdf = OP.quantise_K(K)
    ard.ard_set_distribution(ctx.h, 0, K)
    pat = ctx.pattern(ard.ARD_ROW, 784, 256)
    alpha = 1.0 / (1.0 - c1["p"])
    for it in range(100):
        ard.ard_sample_pattern(ctx.h, pat, 0, inputs.BASE_SEED, it, 0)
        dp, b = OP.draw(cdf, inputs.BASE_SEED, it, 0)
        res = run_three_gemms(ctx, pat, ard.ARD_ROW, ard.ARD_F32, c1["X"], c1["W"], c1["dY"], dp, b, alpha,
                              compact=(it % 2 == 1), zero_fill=(it % 3 != 0))
        assert_ok(res, TOL[ard.ARD_F32], (it, dp, b))


@pytest.mark.parametrize("B,K,N,lds", [(37, 50, 77, None), (5, 33, 9, {"x": 40, "w": 35, "y": 12}), (1, 1, 1, None)])
def test_row_ragged_shapes(ctx, B, K, N, lds):
    rng = np.random.default_rng(B * 1000 + N)
    X = rng.standard_normal((B, K)).astype(np.float32)
    W = rng.standard_normal((K, N)).astype(np.float32)
    dY = rng.standard_normal((B, N)).astype(np.float32)
    pat = ctx.pattern(ard.ARD_ROW, K, N)
    for dp in sorted(d for d in {1, 2, 3, min(N, 7), N} if d <= N):
        for b in sorted({1, dp}):
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            for compact in (False, True):
                res = run_three_gemms(ctx, pat, ard.ARD_ROW, ard.ARD_F32, X, W, dY, dp, b, 1.25, lds=lds,
                                      compact=compact)
                assert_ok(res, TOL[ard.ARD_F32], (dp, b, compact))


def test_tile_patterns_f32(ctx):
    B, K, N, ts = 45, 96, 160, 32
    rng = np.random.default_rng(5)
    X = rng.standard_normal((B, K)).astype(np.float32)
    W = rng.standard_normal((K, N)).astype(np.float32)
    dY = rng.standard_normal((B, N)).astype(np.float32)
    pat = ctx.pattern(ard.ARD_TILE, K, N, ts)
    for dp, b in [(1, 1), (2, 1), (2, 2), (3, 1), (4, 3), (5, 5), (15, 7)]:
        ard.ard_pattern_set(ctx.h, pat, dp, b)
        for zf in (True, False):
            res = run_three_gemms(ctx, pat, ard.ARD_TILE, ard.ARD_F32, X, W, dY, dp, b, 2.0, ts=ts, zero_fill=zf)
            assert_ok(res, TOL[ard.ARD_F32], (dp, b, zf))


def test_empty_batch(ctx):
    import torch
    pat = ctx.pattern(ard.ARD_ROW, 16, 8)
    ard.ard_pattern_set(ctx.h, pat, 2, 1)
    x = torch.zeros((1, 16), device="cuda")
    w = torch.zeros((8, 16), device="cuda")
    y = torch.full((1, 8), 3.0, device="cuda")
    dw = torch.full((8, 16), float("nan"), device="cuda")
    ard.ard_fwd(ctx.h, pat, ard.ARD_F32, 0, 16, 8, 1.0, x, 16, w, 16, y, 8, 1)
    ard.ard_bwd_weight(ctx.h, pat, ard.ARD_F32, ard.ARD_F32, 0, 16, 8, 1.0, x, 16, y, 8, 0, dw, 16, 1)
    torch.cuda.synchronize()
    assert float(y.sum()) == 24.0 and float(dw.abs().sum()) == 0.0
