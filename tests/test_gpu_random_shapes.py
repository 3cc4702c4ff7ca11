"""Seeded sweep over random shapes, leading dimensions, patterns and options: the three products (row and
tile patterns, both kernel families chosen by the library itself) and the fused layer step against the oracle.

The parametrised parity tests pin chosen shapes; this sweep is there for the combinations nobody thought of
(ragged tails in all three dimensions at once, padded leading dimensions, periods close to the unit count,
a single kept unit).  Sizes are small enough for the fp64 oracle: 128 + 48 cases in under half a minute.
"""
import numpy as np
import pytest
import torch

from oracle import gemm as OG
from oracle import mlp as OM
from oracle import pattern as OP
from paper_2203_05705_b200 import ard, inputs
from gpu_helpers import Ctx, host, run_three_gemms, assert_ok, tdtype, TOL

pytestmark = pytest.mark.gpu


def _case(rng):
    kind = ard.ARD_ROW if rng.random() < 0.6 else ard.ARD_TILE
    dtype = ard.ARD_BF16 if rng.random() < 0.75 else ard.ARD_F32
    if kind == ard.ARD_TILE:
        ts = int(rng.choice([32, 64, 128]))
        K = ts * int(rng.integers(1, 7))
        N = ts * int(rng.integers(1, 7))
        units = (K // ts) * (N // ts)
    else:
        ts = 0
        mult = 8 if rng.random() < 0.8 else 1                      # a fifth of the cases miss the 16-byte alignment
        K = mult * int(rng.integers(1, 90 if mult == 8 else 300))
        N = mult * int(rng.integers(1, 90 if mult == 8 else 300))
        units = N
    B = int(rng.integers(1, 400))
    dp = int(min(units, rng.choice([1, 1, 2, 2, 3, 4, 5, 7, 8, 13, 16, 31])))
    if rng.random() < 0.1:
        dp = int(min(units, 32))
    b = int(rng.integers(1, dp + 1))
    pad = lambda v: v + 8 * int(rng.integers(0, 3)) if rng.random() < 0.3 else v
    lds = {"x": pad(K), "w": pad(K), "y": pad(N)}
    return dict(kind=kind, dtype=dtype, ts=ts, B=B, K=K, N=N, dp=dp, b=b, lds=lds,
                compact=bool(rng.random() < 0.4), zero_fill=bool(rng.random() < 0.6),
                dw_f32=bool(rng.random() < 0.5))


@pytest.mark.parametrize("seed", range(16))
def test_three_products_on_random_cases(seed):
    rng = np.random.default_rng(1000 + seed)
    ctx = Ctx(8 << 20)
    try:
        for i in range(8):
            c = _case(rng)
            X = rng.standard_normal((c["B"], c["K"])).astype(np.float32)
            W = (rng.standard_normal((c["K"], c["N"])) / np.sqrt(c["K"])).astype(np.float32)
            dY = rng.standard_normal((c["B"], c["N"])).astype(np.float32)
            if c["dtype"] == ard.ARD_BF16:
                X, W, dY = inputs.bf16_round(X), inputs.bf16_round(W), inputs.bf16_round(dY)
            pat = ctx.pattern(c["kind"], c["K"], c["N"], c["ts"])
            ard.ard_pattern_set(ctx.h, pat, c["dp"], c["b"])
            dw = ard.ARD_F32 if (c["dw_f32"] or c["dtype"] == ard.ARD_F32) else ard.ARD_BF16
            res = run_three_gemms(ctx, pat, c["kind"], c["dtype"], X, W, dY, c["dp"], c["b"], 1.7, ts=c["ts"],
                                  lds=c["lds"], dw_dtype=dw, compact=c["compact"] and c["kind"] == ard.ARD_ROW,
                                  zero_fill=c["zero_fill"])
            assert_ok(res, TOL[c["dtype"]], (seed, i, c))
    finally:
        ctx.close()


@pytest.mark.parametrize("seed", range(8))
def test_layer_step_on_random_cases(seed):
    """Compact input and weight under a random feeding pattern, bias, ReLU, ReLU adjoint; whichever kernel
    family the library picks for the shape."""
    rng = np.random.default_rng(2000 + seed)
    ctx = Ctx(8 << 20)
    try:
        for i in range(6):
            dtype = ard.ARD_BF16 if rng.random() < 0.8 else ard.ARD_F32
            mult = 8 if rng.random() < 0.8 else 1
            B = int(rng.integers(1, 300))
            K = mult * int(rng.integers(2, 80 if mult == 8 else 200))
            N = mult * int(rng.integers(2, 80 if mult == 8 else 200))
            if rng.random() < 0.2:
                N = int(rng.integers(1, 17))                          # an output layer
            dpi = int(min(K, rng.choice([1, 2, 3, 5, 16])))
            dpo = int(min(N, rng.choice([1, 2, 3, 4, 9])))
            pin, pout = (dpi, int(rng.integers(1, dpi + 1))), (dpo, int(rng.integers(1, dpo + 1)))
            tag = (seed, i, dtype, B, K, N, pin, pout)
            rnd = lambda shape, s=1.0: (inputs.bf16_round((rng.standard_normal(shape) * s).astype(np.float32))
                                        if dtype == ard.ARD_BF16 else (rng.standard_normal(shape) * s).astype(np.float32))
            W = rnd((K, N), 1.0 / np.sqrt(K))
            bias = rng.uniform(-0.5, 0.5, N).astype(np.float32)
            pat = ctx.pattern(ard.ARD_ROW, K, N)
            in_pat = ctx.pattern(ard.ARD_ROW, 8, K)
            ard.ard_pattern_set(ctx.h, in_pat, *pin)
            ard.ard_pattern_set(ctx.h, pat, *pout)
            keep_in, keep = OP.row_keep(K, *pin), OP.row_keep(N, *pout)
            n_in, n = len(keep_in), len(keep)
            td = tdtype(dtype)

            def devm(a, ld):
                t = torch.full((a.shape[0], ld), float("nan"), dtype=td, device="cuda")
                t[:, :a.shape[1]] = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(td)
                return t

            Wd = devm(W.T, K)
            Wk = torch.full((N, K), float("nan"), dtype=td, device="cuda")
            ard.ard_compact_weight_cols(ctx.h, pat, in_pat, dtype, K, N, Wd, K, Wk, K)
            Xc, dZc, act = rnd((B, n_in)), rnd((B, n)), rnd((B, n_in))
            Xd, dZd, actd = devm(Xc, K), devm(dZc, N), devm(act, K)
            A = torch.full((B, N), float("nan"), dtype=td, device="cuda")
            ard.ard_layer_fwd(ctx.h, pat, in_pat, dtype, B, K, N, 1.3, Xd, K, Wk, K, torch.from_numpy(bias).cuda(), A, N,
                              ard.ARD_OUT_SCATTER_ZEROFILL | ard.ARD_FLAG_RELU)
            ref = OM.layer_fwd_compact(Xc, keep_in, W, bias, keep, 1.3)
            Ah = host(A)
            assert OG.rel_fro(Ah[:, keep], ref) <= TOL[dtype], tag
            assert np.all(np.delete(Ah, keep, axis=1) == 0), tag
            dX = torch.full((B, K), float("nan"), dtype=td, device="cuda")
            ard.ard_layer_bwd_data(ctx.h, pat, in_pat, dtype, B, K, N, 1.3, dZd, N, 1, Wk, K, actd, K, dX, K)
            dWc, db, dAp = OM.layer_bwd_compact(Xc, keep_in, W, keep, dZc)
            assert OG.rel_fro(host(dX)[:, :n_in], 1.3 * dAp * (act > 0)) <= TOL[dtype], tag
            dWk = torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda")
            ard.ard_layer_bwd_weight(ctx.h, pat, in_pat, dtype, ard.ARD_F32, B, K, N, 1.0, Xd, K, dZd, N, 1, dWk, K, 0)
            assert OG.rel_fro(host(dWk)[:n, :n_in], dWc.T) <= TOL[dtype], tag
            dbd = torch.full((N,), float("nan"), dtype=torch.float32, device="cuda")
            ard.ard_bias_grad(ctx.h, pat, dtype, B, N, dZd, N, 1, dbd, 1)
            assert np.abs(host(dbd)[keep] - db).max() <= TOL[dtype] * max(1.0, np.abs(db).max()), tag
            assert ard.ard_last_device_status(ctx.h) == 0, tag
    finally:
        ctx.close()
