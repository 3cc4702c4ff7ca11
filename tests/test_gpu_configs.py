"""Parity at the sizes and value distributions of the five benchmark configurations.

Config 1 (fp32) lives in test_gpu_gemm_f32.py.  Here: the 784-2048-2048-10 MLP chain graded per GEMM on
the operands the GPU consumed (config 2), the 4096x4096 tile-pattern layer in full (config 3), the LSTM
layer composed from the C-ABI calls (config 4) and the 8192x8192 layer on sampled rows / neurons in the
launch configuration the benchmark times (config 5).
"""
import numpy as np
import pytest
import torch

from oracle import gemm as OG
from oracle import lstm as OL
from oracle import pattern as OP
from paper_2203_05705_b200 import ard, inputs
from gpu_helpers import Ctx, host, run_three_gemms, assert_ok, tile_rel_fro, TOL
from distributions import max_entropy_K

pytestmark = pytest.mark.gpu
BF = torch.bfloat16
TOL_BF16 = TOL[ard.ARD_BF16]


def _bf(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(BF).cuda()


# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("p", [0.3, 0.5, 0.7])
def test_config2_mlp_chain_per_gemm(p):
    """Three layers, row patterns on both hidden layers drawn on the device, ReLU between them (applied
    with torch: the activation is not part of the graded products).  Every one of the 9 GEMMs of a
    step is compared with the oracle's product of the very operands the GPU kernel read."""
    Ws = inputs.config2_weights()
    dims = [784, 2048, 2048, 10]
    Kd = max_entropy_K(p, 16)
    cdf = OP.quantise_K(Kd)
    ctx = Ctx(2 * 128 * 2048 + 4096)
    try:
        ard.ard_set_distribution(ctx.h, 0, Kd)
        pats = [ctx.pattern(ard.ARD_ROW, dims[l], dims[l + 1]) for l in range(3)]
        Wd = [_bf(Ws[l].T) for l in range(3)]
        alpha = [1.0 / (1.0 - p), 1.0 / (1.0 - p), 1.0]
        B = 128
        worst = 0.0
        for step in range(8):
            X, dZ3 = inputs.config2_step(step)
            masks = []
            for l in range(2):
                ard.ard_sample_pattern(ctx.h, pats[l], 0, inputs.BASE_SEED, step, l + 1)
                dp, b = OP.draw(cdf, inputs.BASE_SEED, step, l + 1)
                gdp, gb, _, _ = ard.ard_pattern_to_host(pats[l], 0)
                assert (gdp, gb) == (dp, b)
                masks.append(OP.row_mask(dims[l + 1], dp, b))
            masks.append(np.ones(10))
            acts = [_bf(X)]
            zs = []
            for l in range(3):                                   # forward
                Z = torch.full((B, dims[l + 1]), float("nan"), dtype=BF, device="cuda")
                ard.ard_fwd(ctx.h, pats[l], ard.ARD_BF16, B, dims[l], dims[l + 1], alpha[l], acts[l], dims[l],
                            Wd[l], dims[l], Z, dims[l + 1], ard.ARD_OUT_SCATTER_ZEROFILL)
                ref = OG.fwd(host(acts[l]), Ws[l], masks[l], alpha[l])
                worst = max(worst, OG.rel_fro(host(Z), ref))
                assert bool(torch.all(Z[:, torch.from_numpy(masks[l] == 0).cuda()] == 0))
                zs.append(Z)
                acts.append(torch.relu(Z))
            dZ = _bf(dZ3)
            for l in (2, 1, 0):                                  # backward
                dW = torch.full((dims[l + 1], dims[l]), float("nan"), dtype=BF, device="cuda")
                dA = torch.full((B, dims[l]), float("nan"), dtype=BF, device="cuda")
                ard.ard_bwd_weight(ctx.h, pats[l], ard.ARD_BF16, ard.ARD_BF16, B, dims[l], dims[l + 1], alpha[l],
                                   acts[l], dims[l], dZ, dims[l + 1], 0, dW, dims[l], 1)
                ard.ard_bwd_data(ctx.h, pats[l], ard.ARD_BF16, B, dims[l], dims[l + 1], alpha[l], dZ, dims[l + 1], 0,
                                 Wd[l], dims[l], dA, dims[l])
                refW = OG.bwd_weight(host(acts[l]), host(dZ), masks[l], alpha[l]).T
                refA = OG.bwd_data(host(dZ), Ws[l], masks[l], alpha[l])
                worst = max(worst, OG.rel_fro(host(dW), refW), OG.rel_fro(host(dA), refA))
                if l > 0:
                    dZ = (dA * (zs[l - 1] > 0)).to(BF)            # ReLU' with relu'(0) = 0
        assert ard.ard_last_device_status(ctx.h) == 0
        assert worst <= TOL_BF16, worst
    finally:
        ctx.close()


# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("p", [0.3, 0.5, 0.7])
def test_config3_tile_layer_full_size(p):
    """The 4096 x 4096 layer with 64 x 64 tiles, batch 1024, in full against the oracle: the first four distinct
    periods the device sampler draws for this dropout rate."""
    c3 = inputs.config3()
    ctx = Ctx(0)
    try:
        Kd = max_entropy_K(p, c3["n_dp"])
        cdf = OP.quantise_K(Kd)
        ard.ard_set_distribution(ctx.h, 0, Kd)
        pat = ctx.pattern(ard.ARD_TILE, 4096, 4096, 64)
        done = set()
        for it in range(200):
            dp, b = OP.draw(cdf, inputs.BASE_SEED, it, 0)
            if dp in done:
                continue
            done.add(dp)
            ard.ard_sample_pattern(ctx.h, pat, 0, inputs.BASE_SEED, it, 0)
            gdp, gb, _, _ = ard.ard_pattern_to_host(pat, 0)
            assert (gdp, gb) == (dp, b)
            res = run_three_gemms(ctx, pat, ard.ARD_TILE, ard.ARD_BF16, c3["X"], c3["W"], c3["dY"], dp, b,
                                  1.0 / (1.0 - p), ts=64, zero_fill=(it % 2 == 0))
            assert_ok(res, TOL_BF16, (p, it, dp, b))
            if len(done) >= 4:
                break
        assert len(done) >= 4
    finally:
        ctx.close()


@pytest.mark.parametrize("dp,b", [(2, 1), (4, 3), (8, 8), (16, 5), (3, 2), (6, 1), (12, 7), (15, 15), (13, 4)])
def test_config3_tile_layer_every_kind_of_period(dp, b):
    """Same layer, forced periods: the even ones divide the 64 tile-columns, so the rule keeps whole tile-columns
    (every kept forward tile falls into 1/dp of the output columns); 3, 6, 12, 15 share a factor with neither or
    only part of it; 13 is coprime."""
    c3 = inputs.config3()
    ctx = Ctx(0)
    try:
        pat = ctx.pattern(ard.ARD_TILE, 4096, 4096, 64)
        ard.ard_pattern_set(ctx.h, pat, dp, b)
        res = run_three_gemms(ctx, pat, ard.ARD_TILE, ard.ARD_BF16, c3["X"], c3["W"], c3["dY"], dp, b, 1.7, ts=64,
                              zero_fill=(dp % 3 != 0))
        assert_ok(res, TOL_BF16, (dp, b))
    finally:
        ctx.close()


# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("kind,ts", [("row", 0), ("tile", 128)])
def test_config5_sampled_outputs(kind, ts):
    """Full 8192x8192 layer, batch 4096, default (benchmark) launch configuration; the oracle recomputes
    128 batch rows of Y and dX and 128 neurons of dW."""
    c5 = inputs.config5()
    X, W, dY = c5["X"], c5["W"], c5["dY"]
    B, K = X.shape
    N = W.shape[1]
    akind = ard.ARD_ROW if kind == "row" else ard.ARD_TILE
    ctx = Ctx(2 * B * N + 4096)
    try:
        ard.ard_set_compact_reuse(ctx.h, 1)
        pat = ctx.pattern(akind, K, N, ts)
        dXd, dWd, dYd = _bf(X), _bf(W.T), _bf(dY)
        Y = torch.empty((B, N), dtype=BF, device="cuda")
        dX = torch.empty((B, K), dtype=BF, device="cuda")
        dW = torch.empty((N, K), dtype=BF, device="cuda")
        rows = np.arange(7, B, B // 128)[:128]
        cols = np.arange(3, N, N // 128)[:128]
        # every period of the benchmark's distribution (3, 5, 7, 12 make the forward product pick output tiles 224,
        # 192, 160, 192 columns wide), the offset varied with it
        for dp, b in [(1, 1), (2, 2), (3, 1), (4, 4), (5, 3), (6, 1), (7, 2), (8, 5), (9, 9), (10, 3), (11, 6), (12, 5),
                      (13, 1), (14, 14), (15, 8), (16, 7)]:
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            Y.fill_(float("nan")); dX.fill_(float("nan")); dW.fill_(float("nan"))
            ard.ard_fwd(ctx.h, pat, ard.ARD_BF16, B, K, N, 2.0, dXd, K, dWd, K, Y, N, ard.ARD_OUT_SCATTER_ZEROFILL)
            ard.ard_bwd_data(ctx.h, pat, ard.ARD_BF16, B, K, N, 2.0, dYd, N, 0, dWd, K, dX, K)
            ard.ard_bwd_weight(ctx.h, pat, ard.ARD_BF16, ard.ARD_BF16, B, K, N, 2.0, dXd, K, dYd, N, 0, dW, K, 1)
            assert ard.ard_last_device_status(ctx.h) == 0
            mask = OP.row_mask(N, dp, b) if kind == "row" else OP.tile_mask(K, N, ts, dp, b)
            ri, ci = torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()
            got = (host(Y[ri]), host(dX[ri]), host(dW[ci]))
            want = (OG.fwd_rows(X, W, mask, 2.0, rows), OG.bwd_data_rows(dY, W, mask, 2.0, rows),
                    OG.bwd_weight_cols(X, dY, mask, 2.0, cols).T)
            errs = [OG.rel_fro(g, w) for g, w in zip(got, want)]
            assert max(errs) <= TOL_BF16, (kind, dp, b, errs)
            # the same bound for every 256-column piece of the 8 sampled rows of every 256-row output tile
            # (dW: 8 sampled neurons of every 512-neuron band), so that one misplaced column group shows
            terrs = [tile_rel_fro(g, w, 256, 8) for g, w in zip(got, want)]
            assert max(terrs) <= TOL_BF16, (kind, dp, b, terrs)
            # properties that hold for the whole output: finite everywhere, dropped part exactly zero
            assert bool(torch.isfinite(Y).all()) and bool(torch.isfinite(dX).all()) and bool(torch.isfinite(dW).all())
            if kind == "row":
                dropped = torch.from_numpy(mask == 0).cuda()
                assert bool(torch.all(Y[:, dropped] == 0)) and bool(torch.all(dW[dropped, :] == 0))
    finally:
        ctx.close()


# --------------------------------------------------------------------------------------------------
def _lstm_gpu(ctx, pat, Wnm, X, dH, I, H, alpha):
    """LSTM layer forward + BPTT through the C ABI (buffers and call order: paper_2203_05705_b200/lstm.py)."""
    from paper_2203_05705_b200.lstm import LstmLayer
    T, B, _ = X.shape
    layer = LstmLayer(ctx.h, pat, T, B, I, H, Wnm)
    layer.load_inputs(X)
    Hs = layer.forward(alpha).float()
    dX, dW = layer.backward(alpha, dH)
    torch.cuda.synchronize()
    return Hs, layer.C[T], dX, dW


@pytest.mark.parametrize("p,seq", [(0.5, 0), (0.7, 1), (0.3, 2)])
def test_config4_lstm_layer(p, seq):
    T, B, I, H = 35, 64, 1024, 1024
    c4 = inputs.config4(T, B, I, H, seq)
    W, X, dH = c4["W"], c4["X"], c4["dH"]
    Kd = max_entropy_K(p, c4["n_dp"])
    cdf = OP.quantise_K(Kd)
    alpha = 1.0 / (1.0 - p)
    ctx = Ctx(2 * T * B * 4 * H + 4096)
    try:
        ard.ard_set_distribution(ctx.h, 0, Kd)
        pat = ctx.pattern(ard.ARD_ROW, I + H, H)
        it = 0
        while OP.draw(cdf, inputs.BASE_SEED, it, 4)[0] == 1:      # skip to the first non-dense draw
            it += 1
        ard.ard_sample_pattern(ctx.h, pat, 0, inputs.BASE_SEED, it, 4)   # one pattern for the whole sequence
        dp, b = OP.draw(cdf, inputs.BASE_SEED, it, 4)
        m = OP.row_mask(H, dp, b)
        Hs, cT, dX, dW = _lstm_gpu(ctx, pat, _bf(W.T), _bf(X), torch.from_numpy(dH).cuda(), I, H, alpha)
        assert ard.ard_last_device_status(ctx.h) == 0
        fw = OL.fwd(X, W, None, m, alpha)
        bw = OL.bwd(fw, W, m, alpha, dH)
        keep = OP.row_keep(H, dp, b)
        errs = {"H": OG.rel_fro(host(Hs), fw["Hs"]), "cT": OG.rel_fro(host(cT)[:, :len(keep)], fw["cT"][:, keep]),
                "dX": OG.rel_fro(host(dX), bw["dX"]), "dW": OG.rel_fro(host(dW), bw["dW"].T)}
        assert bool(torch.all(Hs[:, :, torch.from_numpy(m == 0).cuda()] == 0))
        gate_dropped = np.concatenate([g * H + np.where(m == 0)[0] for g in range(4)])
        assert bool(torch.all(dW[torch.from_numpy(gate_dropped).cuda(), :] == 0))
        assert bool(torch.all(dW[:, torch.from_numpy(I + np.where(m == 0)[0]).cuda()] == 0))
        assert max(errs.values()) <= TOL_BF16, (dp, b, errs)
    finally:
        ctx.close()


def test_lstm_cell_kernels_teacher_forced():
    """ard_lstm_gates / ard_lstm_gates_bwd alone (fp32 in, fp32 out) against the oracle's cell."""
    B, H, dp, b, alpha = 37, 200, 3, 2, 1.6
    rng = np.random.default_rng(4)
    m = OP.row_mask(H, dp, b)
    keep = OP.row_keep(H, dp, b)
    n = len(keep)
    Zf = rng.standard_normal((B, 4 * H))
    bias = rng.standard_normal(4 * H) * 0.1
    c_prev = rng.standard_normal((B, H)) * m
    dh = rng.standard_normal((B, H))
    dc_in = rng.standard_normal((B, H)) * m
    i, f, g, o, c, h = OL.cell_fwd(Zf + bias[None, :], c_prev, m, alpha)
    dZ_o, dcp_o = OL.cell_bwd(i, f, g, o, c_prev, c, m, alpha, dh, dc_in)
    ctx = Ctx(0)
    try:
        pat = ctx.pattern(ard.ARD_ROW, 8, H)
        ard.ard_pattern_set(ctx.h, pat, dp, b)
        gcols = np.concatenate([q * H + keep for q in range(4)])
        f32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
        Zc = f32(Zf[:, gcols])                                   # compact [B][4n], block width n
        cp = f32(c_prev[:, keep])
        cn = torch.full((B, n), float("nan"), device="cuda")
        hs = torch.full((B, H), float("nan"), device="cuda")
        hc = torch.full((B, n), float("nan"), device="cuda")
        gs = torch.full((B, 4 * n), float("nan"), device="cuda")
        ard.ard_lstm_gates(ctx.h, pat, ard.ARD_F32, B, H, alpha, Zc, n, f32(bias), cp, n, cn, hs, H, 1, gs)
        ard.ard_lstm_gates(ctx.h, pat, ard.ARD_F32, B, H, alpha, Zc, n, f32(bias), cp, n, cn, hc, n, 0, gs)
        assert OG.rel_fro(host(hs), h) <= 1e-5 and OG.rel_fro(host(hc), h[:, keep]) <= 1e-5
        assert OG.rel_fro(host(cn), c[:, keep]) <= 1e-5
        assert bool(torch.all(hs[:, torch.from_numpy(m == 0).cuda()] == 0))
        dc = f32(dc_in[:, keep])
        dZ = torch.full((B, 4 * n), float("nan"), device="cuda")
        ard.ard_lstm_gates_bwd(ctx.h, pat, ard.ARD_F32, B, H, alpha, gs, cp, cn, n, f32(dh), H, 1, dc, dZ, n)
        assert OG.rel_fro(host(dZ), dZ_o[:, gcols]) <= 1e-5
        assert OG.rel_fro(host(dc), dcp_o[:, keep]) <= 1e-5
    finally:
        ctx.close()
