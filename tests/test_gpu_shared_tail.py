"""Row-pattern tensor-core GEMMs whose left-over output tiles are shared along the contraction.

When the tiles do not fill a whole number of waves over the SMs (or SM pairs), the left-over tiles are
cut along the contraction; their partial sums come from several workers and are added in contraction
order by whichever share arrives last.  The result must (1) match the oracle like any other product,
(2) be bit-identical from launch to launch and (3) leave the arrival counters ready for the next
launch.  The shapes have more tiles than a B200 has SM pairs (otherwise nothing is shared) and are
still small enough for the fp64 oracle; the thresholds are lowered so that short contractions are cut
into many shares.
"""
import numpy as np
import pytest
import torch

from paper_2203_05705_b200 import ard, inputs
from gpu_helpers import Ctx, run_three_gemms, assert_ok, TOL

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


def _layer(B, K, N, seed, wscale=0.05):
    rng = np.random.default_rng(seed)
    X = inputs.bf16_round(rng.standard_normal((B, K)).astype(np.float32))
    W = inputs.bf16_round((rng.standard_normal((K, N)) * wscale).astype(np.float32))
    dY = inputs.bf16_round(rng.standard_normal((B, N)).astype(np.float32))
    return X, W, dY


@pytest.mark.parametrize("B,K,N,min_blocks,bns,patterns", [
    # SM pairs (256-row tiles), every product has more tiles than workers for these periods
    (2048, 2048, 4096, 2, (0, 128), [(1, 1), (2, 2), (3, 1)]),
    # SM pairs, ragged in every dimension; the forward and the weight gradient have left-over tiles
    (300, 1000, 12000, 1, (128,), [(1, 1), (2, 1), (3, 3)]),
    # single-SM tiles (one 128-row tile): more than 148 tiles of 64 columns
    (100, 520, 9728, 1, (64,), [(1, 1)]),
])
def test_shared_tiles_match_the_oracle(B, K, N, min_blocks, bns, patterns):
    X, W, dY = _layer(B, K, N, 11, 0.03)
    ctx = Ctx(2 * B * N + 4096)
    try:
        ard.ard_set_path(ctx.h, ard.ARD_PATH_TENSOR_CORE)
        ard.ard_set_shared_tail(ctx.h, 1, min_blocks, 1)
        pat = ctx.pattern(ard.ARD_ROW, K, N)
        for i, (dp, b) in enumerate(patterns):
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            for bn in bns:
                ard.ard_set_tile_n(ctx.h, bn)
                res = run_three_gemms(ctx, pat, ard.ARD_ROW, ard.ARD_BF16, X, W, dY, dp, b, 2.0,
                                      compact=(i % 2 == 1), zero_fill=(i % 3 != 2),
                                      dw_dtype=ard.ARD_F32 if i % 2 else ard.ARD_BF16)
                assert_ok(res, TOL[ard.ARD_BF16], (B, K, N, dp, b, bn))
    finally:
        ctx.close()


def _three(ctx, pat, B, K, N, Xd, Wd, dYd, flags=0):
    Y = torch.full((B, N), float("nan"), dtype=BF, device="cuda")
    dX = torch.full((B, K), float("nan"), dtype=torch.float32 if flags & ard.ARD_FLAG_OUT_F32 else BF, device="cuda")
    dW = torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda")
    ard.ard_fwd(ctx.h, pat, ard.ARD_BF16, B, K, N, 2.0, Xd, K, Wd, K, Y, N, ard.ARD_OUT_SCATTER_ZEROFILL)
    ard.ard_bwd_data(ctx.h, pat, ard.ARD_BF16, B, K, N, 2.0, dYd, N, flags, Wd, K, dX, K)
    ard.ard_bwd_weight(ctx.h, pat, ard.ARD_BF16, ard.ARD_F32, B, K, N, 2.0, Xd, K, dYd, N, 0, dW, K, 1)
    return Y, dX, dW


def test_shared_tiles_are_reproducible_and_close_to_the_unshared_result():
    """Larger than the oracle cases: compares the two schedules of the same kernels with each other."""
    B, K, N = 2048, 2048, 8192
    g = torch.Generator(device="cuda").manual_seed(5)
    Xd = torch.randn((B, K), device="cuda", generator=g).to(BF)
    Wd = (torch.randn((N, K), device="cuda", generator=g) / 45).to(BF)
    dYd = torch.randn((B, N), device="cuda", generator=g).to(BF)
    ctx = Ctx(2 * B * N + 4096)
    try:
        pat = ctx.pattern(ard.ARD_ROW, K, N)
        for dp, b in [(1, 1), (2, 1), (3, 2)]:
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            ard.ard_set_shared_tail(ctx.h, 0)
            ref = _three(ctx, pat, B, K, N, Xd, Wd, dYd, ard.ARD_FLAG_OUT_F32)
            ard.ard_set_shared_tail(ctx.h, 1, 4, 1)
            runs = [_three(ctx, pat, B, K, N, Xd, Wd, dYd, ard.ARD_FLAG_OUT_F32) for _ in range(4)]
            assert ard.ard_last_device_status(ctx.h) == 0
            for r in runs[1:]:
                for a, c in zip(runs[0], r):
                    assert torch.equal(a, c), (dp, b)            # same bits every launch
            for a, c in zip(runs[0], ref):
                assert bool(torch.isfinite(a).all())
                err = float((a.double() - c.double()).norm() / c.double().norm())
                assert err <= 2e-3, (dp, b, err)                   # only the fp32 summation order differs
            # the fp32 outputs differ in a few last bits exactly when some tile was shared
            assert not torch.equal(runs[0][2], ref[2]), (dp, b)
    finally:
        ctx.close()


def test_accumulate_flag_with_shared_tiles():
    B, K, N = 2048, 2048, 1024
    X, W, dY = _layer(B, K, N, 12)
    from oracle import gemm as OG
    from oracle import pattern as OP
    ctx = Ctx(64 << 20)
    try:
        ard.ard_set_shared_tail(ctx.h, 1, 2, 1)
        pat = ctx.pattern(ard.ARD_ROW, K, N)
        dp, b = 3, 2
        ard.ard_pattern_set(ctx.h, pat, dp, b)
        ard.ard_set_tile_n(ctx.h, 128)          # 8 x 16 tiles of 256 x 128: one wave and 54 left-over tiles
        Wd = torch.from_numpy(np.ascontiguousarray(W.T)).to(BF).cuda()
        dYd = torch.from_numpy(dY).to(BF).cuda()
        base = np.random.default_rng(3).standard_normal((B, K)).astype(np.float32)
        dX = torch.from_numpy(base).cuda()
        ard.ard_bwd_data(ctx.h, pat, ard.ARD_BF16, B, K, N, 2.0, dYd, N,
                         ard.ARD_FLAG_OUT_F32 | ard.ARD_FLAG_ACCUMULATE, Wd, K, dX, K)
        assert ard.ard_last_device_status(ctx.h) == 0
        ref = base.astype(np.float64) + OG.bwd_data(dY, W, OP.row_mask(N, dp, b), 2.0)
        assert OG.rel_fro(dX.double().cpu().numpy(), ref) <= TOL[ard.ARD_BF16]
    finally:
        ctx.close()
