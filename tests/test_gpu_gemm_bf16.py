"""bf16 paths vs the oracle: tcgen05 kernels (every N tile) and the CUDA-core family, row and tile patterns.

Sizes span several output tiles, several 64-wide contraction blocks and ragged tails in every
dimension, and stay small enough for the fp64 oracle to finish in seconds.
"""
import numpy as np
import pytest

from paper_2203_05705_b200 import ard, inputs
from gpu_helpers import Ctx, run_three_gemms, assert_ok, TOL
from distributions import max_entropy_K

pytestmark = pytest.mark.gpu

ROW_PATTERNS = [(1, 1), (2, 1), (2, 2), (3, 2), (5, 5), (7, 1), (16, 4), (16, 16)]


@pytest.fixture(scope="module")
def ctx():
    c = Ctx(64 << 20)
    yield c
    c.close()


def _layer(B, K, N, seed, wscale):
    rng = np.random.default_rng(seed)
    X = inputs.bf16_round(rng.standard_normal((B, K)).astype(np.float32))
    W = inputs.bf16_round((rng.standard_normal((K, N)) * wscale).astype(np.float32))
    dY = inputs.bf16_round(rng.standard_normal((B, N)).astype(np.float32))
    return X, W, dY


@pytest.mark.parametrize("bn", [128, 256, 64, 224, 192, 160, 96])
def test_row_tensor_core(ctx, bn):
    B, K, N = 300, 520, 1000
    X, W, dY = _layer(B, K, N, 1, 0.05)
    ard.ard_set_path(ctx.h, ard.ARD_PATH_TENSOR_CORE)
    ard.ard_set_tile_n(ctx.h, bn)
    pat = ctx.pattern(ard.ARD_ROW, K, N)
    try:
        for i, (dp, b) in enumerate(ROW_PATTERNS):
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            res = run_three_gemms(ctx, pat, ard.ARD_ROW, ard.ARD_BF16, X, W, dY, dp, b, 1.0 / (1.0 - 0.5),
                                  compact=(i % 2 == 1), zero_fill=(i % 3 != 2),
                                  dw_dtype=ard.ARD_F32 if i % 2 else ard.ARD_BF16)
            assert_ok(res, TOL[ard.ARD_BF16], (bn, dp, b))
    finally:
        ard.ard_set_path(ctx.h, ard.ARD_PATH_AUTO)
        ard.ard_set_tile_n(ctx.h, 0)


def test_row_tensor_core_padded_leading_dimensions(ctx):
    B, K, N = 130, 200, 264
    X, W, dY = _layer(B, K, N, 2, 0.05)
    ard.ard_set_path(ctx.h, ard.ARD_PATH_TENSOR_CORE)
    pat = ctx.pattern(ard.ARD_ROW, K, N)
    try:
        for dp, b in [(1, 1), (3, 3), (4, 2)]:
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            for compact in (False, True):
                res = run_three_gemms(ctx, pat, ard.ARD_ROW, ard.ARD_BF16, X, W, dY, dp, b, 2.0,
                                      lds={"x": 208, "w": 216, "y": 272}, compact=compact)
                assert_ok(res, TOL[ard.ARD_BF16], (dp, b, compact))
    finally:
        ard.ard_set_path(ctx.h, ard.ARD_PATH_AUTO)


def test_row_sampled_patterns_auto_path(ctx):
    from oracle import pattern as OP
    B, K, N = 128, 784, 2048                         # first hidden layer of the 784-2048-2048-10 MLP
    X, W, dY = _layer(B, K, N, 3, np.sqrt(2.0 / K))
    Kd = max_entropy_K(0.5, 16)
    cdf = OP.quantise_K(Kd)
    ard.ard_set_distribution(ctx.h, 0, Kd)
    pat = ctx.pattern(ard.ARD_ROW, K, N)
    for it in range(12):
        ard.ard_sample_pattern(ctx.h, pat, 0, inputs.BASE_SEED, it, 1)
        dp, b = OP.draw(cdf, inputs.BASE_SEED, it, 1)
        res = run_three_gemms(ctx, pat, ard.ARD_ROW, ard.ARD_BF16, X, W, dY, dp, b, 2.0)
        assert_ok(res, TOL[ard.ARD_BF16], (it, dp, b))


def test_row_cuda_core_family_bf16(ctx):
    B, K, N = 70, 100, 90                            # K, N not multiples of 8: the TMA path cannot take these
    X, W, dY = _layer(B, K, N, 4, 0.1)
    pat = ctx.pattern(ard.ARD_ROW, K, N)
    for dp, b in [(1, 1), (2, 2), (9, 4)]:
        ard.ard_pattern_set(ctx.h, pat, dp, b)
        for compact in (False, True):
            res = run_three_gemms(ctx, pat, ard.ARD_ROW, ard.ARD_BF16, X, W, dY, dp, b, 1.5, compact=compact)
            assert_ok(res, TOL[ard.ARD_BF16], (dp, b, compact))
    ard.ard_set_path(ctx.h, ard.ARD_PATH_TENSOR_CORE)
    try:
        with pytest.raises(ard.ArdError) as e:
            run_three_gemms(ctx, pat, ard.ARD_ROW, ard.ARD_BF16, X, W, dY, 9, 4, 1.5)
        assert e.value.status == ard.ARD_ERR_ALIGNMENT
    finally:
        ard.ard_set_path(ctx.h, ard.ARD_PATH_AUTO)


@pytest.mark.parametrize("ts,bn", [(64, 0), (128, 0), (128, 64), (256, 0)])
def test_tile_tensor_core(ctx, ts, bn):
    B, K, N = 200, 3 * ts, 5 * ts
    X, W, dY = _layer(B, K, N, 5 + ts, 0.05)
    ard.ard_set_path(ctx.h, ard.ARD_PATH_TENSOR_CORE)
    ard.ard_set_tile_n(ctx.h, bn)
    pat = ctx.pattern(ard.ARD_TILE, K, N, ts)
    try:
        for i, (dp, b) in enumerate([(1, 1), (2, 1), (3, 3), (4, 2), (5, 1), (15, 8)]):
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            res = run_three_gemms(ctx, pat, ard.ARD_TILE, ard.ARD_BF16, X, W, dY, dp, b, 2.0, ts=ts,
                                  zero_fill=(i % 2 == 0), dw_dtype=ard.ARD_F32 if i % 2 else ard.ARD_BF16)
            assert_ok(res, TOL[ard.ARD_BF16], (ts, dp, b))
    finally:
        ard.ard_set_path(ctx.h, ard.ARD_PATH_AUTO)
        ard.ard_set_tile_n(ctx.h, 0)


def test_tile_cuda_core_family_bf16(ctx):
    B, K, N, ts = 50, 64, 96, 32
    X, W, dY = _layer(B, K, N, 9, 0.1)
    pat = ctx.pattern(ard.ARD_TILE, K, N, ts)
    for dp, b in [(1, 1), (2, 1), (3, 2), (6, 6)]:
        ard.ard_pattern_set(ctx.h, pat, dp, b)
        res = run_three_gemms(ctx, pat, ard.ARD_TILE, ard.ARD_BF16, X, W, dY, dp, b, 2.0, ts=ts)
        assert_ok(res, TOL[ard.ARD_BF16], (dp, b))


def test_small_workspace_is_reported(ctx):
    c2 = Ctx(1024)
    try:
        B, K, N = 128, 128, 128
        X, W, dY = _layer(B, K, N, 10, 0.1)
        pat = c2.pattern(ard.ARD_ROW, K, N)
        ard.ard_set_path(c2.h, ard.ARD_PATH_TENSOR_CORE)
        with pytest.raises(ard.ArdError) as e:
            run_three_gemms(c2, pat, ard.ARD_ROW, ard.ARD_BF16, X, W, dY, 1, 1, 1.0)
        assert e.value.status == ard.ARD_ERR_NOMEM
        ard.ard_set_path(c2.h, ard.ARD_PATH_AUTO)         # falls back to the CUDA-core family
        res = run_three_gemms(c2, pat, ard.ARD_ROW, ard.ARD_BF16, X, W, dY, 1, 1, 1.0)
        assert_ok(res, TOL[ard.ARD_BF16])
    finally:
        c2.close()


def test_compact_reuse_option(ctx):
    """With reuse enabled bwd-weight consumes the copy bwd-data compacted; results stay within tolerance
    across pattern changes (every new sample invalidates the copy)."""
    B, K, N = 256, 256, 1024
    ard.ard_set_path(ctx.h, ard.ARD_PATH_TENSOR_CORE)
    ard.ard_set_compact_reuse(ctx.h, 1)
    pat = ctx.pattern(ard.ARD_ROW, K, N)
    try:
        for i, (dp, b) in enumerate([(2, 1), (2, 2), (1, 1), (7, 3), (7, 3)]):
            X, W, dY = _layer(B, K, N, 100 + i, 0.05)
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            n0 = ard.ard_launch_count(ctx.h)
            res = run_three_gemms(ctx, pat, ard.ARD_ROW, ard.ARD_BF16, X, W, dY, dp, b, 2.0)
            assert_ok(res, TOL[ard.ARD_BF16], (dp, b))
            assert ard.ard_launch_count(ctx.h) - n0 == 4          # fwd, gather, bwd-data, bwd-weight
    finally:
        ard.ard_set_compact_reuse(ctx.h, 0)
        ard.ard_set_path(ctx.h, ard.ARD_PATH_AUTO)


def test_output_flags_fp32_and_accumulate(ctx):
    """ARD_FLAG_OUT_F32 / ARD_FLAG_ACCUMULATE on the tensor-core path (CTA pairs: more than 128 rows) and on the
    CUDA-core family."""
    import torch
    from oracle import gemm as OG
    from oracle import pattern as OP
    B, K, N, dp, b = 300, 264, 520, 3, 2
    X, W, dY = _layer(B, K, N, 21, 0.05)
    keep = OP.row_keep(N, dp, b)
    m = OP.row_mask(N, dp, b)
    pat = ctx.pattern(ard.ARD_ROW, K, N)
    ard.ard_pattern_set(ctx.h, pat, dp, b)
    bf = torch.bfloat16
    Xd = torch.from_numpy(X).to(bf).cuda()
    Wd = torch.from_numpy(np.ascontiguousarray(W.T)).to(bf).cuda()
    ldc = (len(keep) + 7) // 8 * 8                                        # 16-byte aligned rows for the TMA path
    dYc = torch.full((B, ldc), float("nan"), dtype=bf, device="cuda")
    dYc[:, :len(keep)] = torch.from_numpy(np.ascontiguousarray(dY[:, keep])).to(bf)
    Yref = OG.fwd(X, W, m, 2.0)[:, keep]
    dXref = OG.bwd_data(dY, W, m, 2.0)
    for path in (ard.ARD_PATH_TENSOR_CORE, ard.ARD_PATH_CUDA_CORE):
        ard.ard_set_path(ctx.h, path)
        try:
            Y = torch.full((B, N), 1.0, dtype=torch.float32, device="cuda")
            ard.ard_fwd(ctx.h, pat, ard.ARD_BF16, B, K, N, 2.0, Xd, K, Wd, K, Y, N,
                        ard.ARD_OUT_COMPACT | ard.ARD_FLAG_OUT_F32 | ard.ARD_FLAG_ACCUMULATE)
            got = Y.double().cpu().numpy()
            assert OG.rel_fro(got[:, :len(keep)] - 1.0, Yref) <= TOL[ard.ARD_BF16]
            assert np.all(got[:, len(keep):] == 1.0)                       # columns beyond n_keep untouched
            dX = torch.full((B, K), 0.5, dtype=torch.float32, device="cuda")
            ard.ard_bwd_data(ctx.h, pat, ard.ARD_BF16, B, K, N, 2.0, dYc, ldc, 1 | ard.ARD_FLAG_OUT_F32, Wd, K,
                             dX, K)
            assert OG.rel_fro(dX.double().cpu().numpy(), dXref) <= TOL[ard.ARD_BF16]
            ard.ard_bwd_data(ctx.h, pat, ard.ARD_BF16, B, K, N, 2.0, dYc, ldc,
                             1 | ard.ARD_FLAG_OUT_F32 | ard.ARD_FLAG_ACCUMULATE, Wd, K, dX, K)
            assert OG.rel_fro(dX.double().cpu().numpy(), 2.0 * dXref) <= TOL[ard.ARD_BF16]
            with pytest.raises(ard.ArdError):                              # accumulate cannot be combined with zero fill
                ard.ard_fwd(ctx.h, pat, ard.ARD_BF16, B, K, N, 2.0, Xd, K, Wd, K, Y, N,
                            ard.ARD_OUT_SCATTER_ZEROFILL | ard.ARD_FLAG_ACCUMULATE)
        finally:
            ard.ard_set_path(ctx.h, ard.ARD_PATH_AUTO)
    assert ard.ard_last_device_status(ctx.h) == 0


def test_lstm_gate_products_against_per_gate_calls(ctx):
    """ard_lstm_gate_gemm(_bwd): tensor-core single launch and the four-call fall-back agree with the oracle."""
    import torch
    from oracle import gemm as OG
    from oracle import pattern as OP
    B, I, H, dp, b = 40, 64, 136, 3, 1
    KH = I + H
    rng = np.random.default_rng(5)
    XH = inputs.bf16_round(rng.standard_normal((B, KH)).astype(np.float32))
    W = inputs.bf16_round((rng.standard_normal((KH, 4 * H)) * 0.1).astype(np.float32))     # math orientation
    keep = OP.row_keep(H, dp, b)
    n = len(keep)
    dZ = inputs.bf16_round(rng.standard_normal((B, 4 * n)).astype(np.float32))
    pat = ctx.pattern(ard.ARD_ROW, KH, H)
    ard.ard_pattern_set(ctx.h, pat, dp, b)
    bf = torch.bfloat16
    XHd = torch.from_numpy(XH).to(bf).cuda()
    Wd = torch.from_numpy(np.ascontiguousarray(W.T)).to(bf).cuda()
    gcols = np.concatenate([g * H + keep for g in range(4)])
    Zref = XH.astype(np.float64) @ W.astype(np.float64)[:, gcols]
    dref = dZ.astype(np.float64) @ W.astype(np.float64)[:, gcols].T
    for path in (ard.ARD_PATH_AUTO, ard.ARD_PATH_CUDA_CORE):
        ard.ard_set_path(ctx.h, path)
        try:
            Z = torch.full((B, 4 * H), float("nan"), dtype=torch.float32, device="cuda")
            ard.ard_lstm_gate_gemm(ctx.h, pat, B, KH, H, XHd, KH, Wd, KH, Z, H)
            Zh = Z.double().cpu().numpy()
            got = np.concatenate([Zh[:, g * H:g * H + n] for g in range(4)], axis=1)
            assert OG.rel_fro(got, Zref) <= TOL[ard.ARD_BF16]
            assert all(np.all(np.isnan(Zh[:, g * H + n:(g + 1) * H])) for g in range(4))
            dZd = torch.zeros((B, 4 * H), dtype=bf, device="cuda")
            for g in range(4):
                dZd[:, g * H:g * H + n] = torch.from_numpy(dZ[:, g * n:(g + 1) * n]).to(bf)
                dZd[:, g * H + n:(g + 1) * H] = float("nan")               # beyond n_keep: must not be read
            D = torch.full((B, KH), 0.25, dtype=torch.float32, device="cuda")
            ard.ard_lstm_gate_gemm_bwd(ctx.h, pat, B, KH, H, dZd, H, Wd, KH, D, KH, 1)
            assert OG.rel_fro(D.double().cpu().numpy() - 0.25, dref) <= TOL[ard.ARD_BF16]
        finally:
            ard.ard_set_path(ctx.h, ard.ARD_PATH_AUTO)
    assert ard.ard_last_device_status(ctx.h) == 0


@pytest.mark.parametrize("kind,ts,shape", [("row", 0, (300, 520, 1000)), ("tile", 64, (200, 192, 320)),
                                            ("row", 0, (70, 100, 90))])
def test_three_products_side_by_side(ctx, kind, ts, shape):
    """ard_layer_products: the forward and the two backward products of a layer enqueued on the context's own
    streams and joined again; against the oracle, eagerly and replayed from a CUDA graph (outputs start as
    NaN, so a product that was not joined before the read shows)."""
    import torch
    from oracle import gemm as OG
    from gpu_helpers import dev, host, nan_buf, oracle_mask
    B, K, N = shape
    X, W, dY = _layer(B, K, N, 21, 0.05)
    akind = ard.ARD_ROW if kind == "row" else ard.ARD_TILE
    pat = ctx.pattern(akind, K, N, ts)
    Xd, Wd, dYd = dev(X, ard.ARD_BF16, K), dev(W.T, ard.ARD_BF16, K), dev(dY, ard.ARD_BF16, N)
    bf = torch.bfloat16
    for dp, b in [(1, 1), (2, 2), (3, 1), (8, 5)]:
        ard.ard_pattern_set(ctx.h, pat, dp, b)
        mask = oracle_mask(akind, K, N, ts, dp, b)
        want = (OG.fwd(X, W, mask, 1.5), OG.bwd_data(dY, W, mask, 1.5), OG.bwd_weight(X, dY, mask, 1.5).T)

        def call(stream=None):
            ard.ard_layer_products(ctx.h, pat, ard.ARD_BF16, ard.ARD_BF16, B, K, N, 1.5, Xd, K, Wd, K, dYd, N, Y, N,
                                   ard.ARD_OUT_SCATTER_ZEROFILL, dX, K, dW, K, 1, stream)

        for mode in ("eager", "graph"):
            Y, dX, dW = nan_buf(B, N, bf), nan_buf(B, K, bf), nan_buf(N, K, bf)
            if mode == "eager":
                call()
            else:
                s = torch.cuda.Stream()
                with torch.cuda.stream(s):
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=s):
                        call(s.cuda_stream)
                    g.replay()
            torch.cuda.synchronize()
            assert ard.ard_last_device_status(ctx.h) == 0
            for got, w, name in zip((Y, dX, dW), want, ("fwd", "bwd_data", "bwd_weight")):
                assert OG.rel_fro(host(got), w) <= TOL[ard.ARD_BF16], (kind, dp, b, mode, name)
