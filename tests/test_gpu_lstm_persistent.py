"""Whole-sequence LSTM forward in one cooperative kernel vs the oracle and vs the per-step path.

Small layers with ragged sizes (batch not a multiple of 32, kept units not a multiple of the 8 units a
CTA owns, a bias, non-zero initial state), every h buffer pre-filled with NaN so that the zeros at
dropped units have to be written by the kernel.
"""
import numpy as np
import pytest
import torch

from oracle import gemm as OG
from oracle import lstm as OL
from oracle import pattern as OP
from paper_2203_05705_b200 import ard, inputs
from gpu_helpers import Ctx, host, TOL

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


def _run(ctx, pat, T, B, I, H, Wnm, X, bias, h0, c0, keep, alpha, persistent):
    KH = I + H
    n = len(keep)
    XH = torch.full((T + 1, B, KH), float("nan"), dtype=BF, device="cuda")
    XH[:T, :, :I] = torch.from_numpy(X).to(BF).cuda()
    XH[0, :, I:] = torch.from_numpy(h0).to(BF).cuda()
    C = torch.full((T + 1, B, H), float("nan"), dtype=torch.float32, device="cuda")
    C[0].zero_()
    C[0, :, :n] = torch.from_numpy(c0[:, keep].astype(np.float32)).cuda()
    G = torch.full((T, B, 4 * H), float("nan"), dtype=torch.float32, device="cuda")
    Z = torch.zeros((B, 4 * H), dtype=torch.float32, device="cuda")
    bias_d = None if bias is None else torch.from_numpy(bias.astype(np.float32)).cuda()
    ard.ard_set_lstm_persistent(ctx.h, persistent)
    launches = ard.ard_launch_count(ctx.h)
    ard.ard_lstm_forward(ctx.h, pat, T, B, I, H, alpha, XH, Wnm, KH, bias_d, C, G, Z)
    torch.cuda.synchronize()
    launches = ard.ard_launch_count(ctx.h) - launches
    assert ard.ard_last_device_status(ctx.h) == 0
    return XH[1:, :, I:].float(), C, G, launches


@pytest.mark.parametrize("T,B,I,H", [(6, 33, 128, 264), (4, 128, 192, 64), (3, 1, 64, 1024), (1, 5, 64, 128)])
def test_persistent_forward_matches_the_oracle_and_the_per_step_path(T, B, I, H):
    rng = np.random.default_rng(T * 1000 + B)
    W = inputs.bf16_round(rng.uniform(-0.08, 0.08, size=(I + H, 4 * H)).astype(np.float32))
    X = inputs.bf16_round(rng.standard_normal((T, B, I)).astype(np.float32))
    bias = rng.uniform(-0.5, 0.5, size=4 * H).astype(np.float32)
    Wnm = torch.from_numpy(np.ascontiguousarray(W.T)).to(BF).cuda()
    ctx = Ctx(1 << 20)
    try:
        pat = ctx.pattern(ard.ARD_ROW, I + H, H)
        for dp, b in [(1, 1), (2, 2), (3, 1), (5, 4), (16, 7)]:
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            m = OP.row_mask(H, dp, b)
            keep = OP.row_keep(H, dp, b)
            h0 = inputs.bf16_round((rng.uniform(-1, 1, size=(B, H)) * m[None, :]).astype(np.float32))
            c0 = (rng.uniform(-1, 1, size=(B, H)) * m[None, :]).astype(np.float32)
            alpha = 1.7
            Hp, Cp, Gp, lp = _run(ctx, pat, T, B, I, H, Wnm, X, bias, h0, c0, keep, alpha, 1)
            Hs, Cs, Gs, ls = _run(ctx, pat, T, B, I, H, Wnm, X, bias, h0, c0, keep, alpha, 0)
            assert lp == 2 and ls == 2 * T, (lp, ls)          # input-half product + recurrence against two per step
            fw = OL.fwd(X, W, bias, m, alpha, h0=h0, c0=c0)
            n = len(keep)
            for name, Hg, Cg in (("persistent", Hp, Cp), ("per-step", Hs, Cs)):
                assert OG.rel_fro(host(Hg), fw["Hs"]) <= TOL[ard.ARD_BF16], (name, dp, b)
                assert OG.rel_fro(host(Cg[T])[:, :n], fw["cT"][:, keep]) <= TOL[ard.ARD_BF16], (name, dp, b)
                assert bool(torch.all(Hg[:, :, torch.from_numpy(m == 0).cuda()] == 0)), (name, dp, b)
            # saved gate activations and cell states feed BPTT: same layout, same values up to rounding
            for t in range(T):
                i_, f_, g_, o_ = fw["saved"][t][1:5]
                ref = np.concatenate([i_[:, keep], f_[:, keep], g_[:, keep], o_[:, keep]], axis=1)
                got = torch.cat([Gp[t, :, g * H:g * H + n] for g in range(4)], dim=1)
                assert OG.rel_fro(host(got), ref) <= TOL[ard.ARD_BF16], (dp, b, t)
            assert float((Hp - Hs).abs().max()) <= 0.05
            assert float((Cp[1:, :, :n] - Cs[1:, :, :n]).abs().max()) <= 0.05
    finally:
        ctx.close()


def test_compact_recurrence_and_full_width_recurrence_agree():
    """Under a pattern the one-kernel forward contracts over the kept units of h alone (a compact copy of h in
    context scratch, the weight's kept fan-in columns gathered by the kernel); with the option off it contracts over
    all H columns, the dropped ones being zero.  Both against the oracle, at kept counts that leave a ragged last
    block and a ragged last CTA, with a batch of more than one row box, a larger kept set run first (its values stay
    in the scratch beyond the smaller set's columns) and h_0 non-zero."""
    T, B, I, H = 5, 97, 64, 520
    rng = np.random.default_rng(99)
    W = inputs.bf16_round(rng.uniform(-0.08, 0.08, size=(I + H, 4 * H)).astype(np.float32))
    X = inputs.bf16_round(rng.standard_normal((T, B, I)).astype(np.float32))
    bias = rng.uniform(-0.5, 0.5, size=4 * H).astype(np.float32)
    Wnm = torch.from_numpy(np.ascontiguousarray(W.T)).to(BF).cuda()
    ctx = Ctx(1 << 20)
    try:
        pat = ctx.pattern(ard.ARD_ROW, I + H, H)
        for dp, b in [(2, 1), (7, 3), (3, 3), (13, 13)]:
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            m = OP.row_mask(H, dp, b)
            keep = OP.row_keep(H, dp, b)
            n = len(keep)
            h0 = inputs.bf16_round((rng.uniform(-1, 1, size=(B, H)) * m[None, :]).astype(np.float32))
            c0 = (rng.uniform(-1, 1, size=(B, H)) * m[None, :]).astype(np.float32)
            fw = OL.fwd(X, W, bias, m, 1.3, h0=h0, c0=c0)
            out = {}
            for compact in (1, 0):
                ard.ard_set_option(ctx.h, ard.ARD_OPT_LSTM_COMPACT_H, compact)
                Hg, Cg, Gg, launches = _run(ctx, pat, T, B, I, H, Wnm, X, bias, h0, c0, keep, 1.3, 1)
                assert launches == 2
                assert OG.rel_fro(host(Hg), fw["Hs"]) <= TOL[ard.ARD_BF16], (compact, dp, b)
                assert OG.rel_fro(host(Cg[T])[:, :n], fw["cT"][:, keep]) <= TOL[ard.ARD_BF16], (compact, dp, b)
                assert bool(torch.all(Hg[:, :, torch.from_numpy(m == 0).cuda()] == 0)), (compact, dp, b)
                out[compact] = (Hg, Cg[1:, :, :n].clone())
            # the same products in another order of fp32 additions
            assert float((out[1][0] - out[0][0]).abs().max()) <= 0.02, (dp, b)
            assert float((out[1][1] - out[0][1]).abs().max()) <= 0.02, (dp, b)
        ard.ard_set_option(ctx.h, ard.ARD_OPT_LSTM_COMPACT_H, 1)
    finally:
        ctx.close()


def test_layers_that_do_not_fit_use_the_per_step_path():
    """Batch above 128 rows: the same call enqueues the per-step kernels."""
    T, B, I, H = 2, 130, 64, 64
    rng = np.random.default_rng(1)
    W = inputs.bf16_round(rng.uniform(-0.08, 0.08, size=(I + H, 4 * H)).astype(np.float32))
    X = inputs.bf16_round(rng.standard_normal((T, B, I)).astype(np.float32))
    Wnm = torch.from_numpy(np.ascontiguousarray(W.T)).to(BF).cuda()
    ctx = Ctx(1 << 20)
    try:
        pat = ctx.pattern(ard.ARD_ROW, I + H, H)
        ard.ard_pattern_set(ctx.h, pat, 2, 1)
        m, keep = OP.row_mask(H, 2, 1), OP.row_keep(H, 2, 1)
        z = np.zeros((B, H), np.float32)
        Hg, Cg, _, launches = _run(ctx, pat, T, B, I, H, Wnm, X, None, z, z, keep, 2.0, 1)
        assert launches == 2 * T
        fw = OL.fwd(X, W, None, m, 2.0)
        assert OG.rel_fro(host(Hg), fw["Hs"]) <= TOL[ard.ARD_BF16]
    finally:
        ctx.close()


@pytest.mark.parametrize("T,B,I,H", [(5, 33, 128, 264), (3, 128, 64, 128), (4, 7, 192, 1024), (1, 5, 64, 128)])
def test_persistent_bptt_matches_the_oracle_and_the_per_step_path(T, B, I, H):
    """Whole-sequence BPTT kernel: dX, dW, dh_0, dc_0 against the oracle and against the per-step path."""
    from paper_2203_05705_b200.lstm import LstmLayer
    rng = np.random.default_rng(T * 100 + B)
    W = inputs.bf16_round(rng.uniform(-0.08, 0.08, size=(I + H, 4 * H)).astype(np.float32))
    X = inputs.bf16_round(rng.standard_normal((T, B, I)).astype(np.float32))
    dH = (rng.standard_normal((T, B, H)) / 8).astype(np.float32)
    Wnm = torch.from_numpy(np.ascontiguousarray(W.T)).to(BF).cuda()
    ctx = Ctx(1 << 20)
    try:
        pat = ctx.pattern(ard.ARD_ROW, I + H, H)
        for dp, b in [(1, 1), (2, 1), (3, 3), (16, 5)]:
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            m = OP.row_mask(H, dp, b)
            keep = OP.row_keep(H, dp, b)
            alpha = 1.5
            fw = OL.fwd(X, W, None, m, alpha)
            bw = OL.bwd(fw, W, m, alpha, dH)
            got = {}
            for mode in (1, 0):
                ard.ard_set_lstm_persistent(ctx.h, mode)
                layer = LstmLayer(ctx.h, pat, T, B, I, H, Wnm)
                layer.load_inputs(torch.from_numpy(X).to(BF).cuda())
                layer.forward(alpha)
                n0 = ard.ard_launch_count(ctx.h)
                dX, dW = layer.backward(alpha, torch.from_numpy(dH).cuda())
                torch.cuda.synchronize()
                launches = ard.ard_launch_count(ctx.h) - n0
                assert ard.ard_last_device_status(ctx.h) == 0
                # recurrence + input-half adjoint (or two kernels per step) + the four-gate weight gradient
                assert launches == (2 + 1 if mode else 2 * T + 1), (mode, launches)
                got[mode] = (dX.clone(), dW.clone(), layer.D[0, :, I:].clone(), layer.dc.clone())
                assert OG.rel_fro(host(dX), bw["dX"]) <= TOL[ard.ARD_BF16], (mode, dp, b)
                assert OG.rel_fro(host(dW), bw["dW"].T) <= TOL[ard.ARD_BF16], (mode, dp, b)
                dropped = torch.from_numpy(np.concatenate([g * H + np.where(m == 0)[0] for g in range(4)])).cuda()
                assert bool(torch.all(dW[dropped, :] == 0))
                kidx = torch.from_numpy(keep).cuda()
                assert OG.rel_fro(host(layer.D[0, :, I:][:, kidx]), bw["dh0"][:, keep]) <= TOL[ard.ARD_BF16], (mode, dp, b)
                assert OG.rel_fro(host(layer.dc[:, :len(keep)]), bw["dc0"][:, keep]) <= TOL[ard.ARD_BF16], (mode, dp, b)
            kept = torch.from_numpy(keep).cuda()
            n = len(keep)
            # gradient of h_0 (kept units) and of c_0: both paths agree closely
            a, c = got[1][2][:, kept], got[0][2][:, kept]
            assert float((a - c).abs().max()) <= 2e-2 * max(1.0, float(c.abs().max())), (dp, b)
            a, c = got[1][3][:, :n], got[0][3][:, :n]
            assert float((a - c).abs().max()) <= 2e-2 * max(1.0, float(c.abs().max())), (dp, b)
    finally:
        ctx.close()


@pytest.mark.parametrize("T,B,I,H,periods", [(4, 70, 64, 520, [(2, 2), (5, 1), (9, 4)]), (3, 64, 128, 1024, [(4, 3), (7, 7)])])
def test_both_forms_of_the_bptt_recurrence_match_the_oracle(T, B, I, H, periods):
    """With few kept units the BPTT kernel drops the cut along the contraction (a CTA owns 8 kept units and contracts
    all of dz itself; one grid-wide barrier per step); ARD_OPT_LSTM_COMPACT_H = 0 keeps the form with partial sums.
    The choice is made on the device from the drawn pattern: here both sides of the limit, a batch of two row boxes,
    kept counts with a ragged last block and a ragged last CTA."""
    from paper_2203_05705_b200.lstm import LstmLayer
    rng = np.random.default_rng(T * 31 + B)
    W = inputs.bf16_round(rng.uniform(-0.08, 0.08, size=(I + H, 4 * H)).astype(np.float32))
    X = inputs.bf16_round(rng.standard_normal((T, B, I)).astype(np.float32))
    dH = (rng.standard_normal((T, B, H)) / 8).astype(np.float32)
    Wnm = torch.from_numpy(np.ascontiguousarray(W.T)).to(BF).cuda()
    ctx = Ctx(1 << 20)
    try:
        pat = ctx.pattern(ard.ARD_ROW, I + H, H)
        for dp, b in periods:
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            m = OP.row_mask(H, dp, b)
            keep = OP.row_keep(H, dp, b)
            n = len(keep)
            fw = OL.fwd(X, W, None, m, 1.5)
            bw = OL.bwd(fw, W, m, 1.5, dH)
            got = {}
            for compact in (1, 0):
                ard.ard_set_option(ctx.h, ard.ARD_OPT_LSTM_COMPACT_H, compact)
                layer = LstmLayer(ctx.h, pat, T, B, I, H, Wnm)
                layer.load_inputs(torch.from_numpy(X).to(BF).cuda())
                layer.forward(1.5)
                n0 = ard.ard_launch_count(ctx.h)
                dX, dW = layer.backward(1.5, torch.from_numpy(dH).cuda())
                torch.cuda.synchronize()
                assert ard.ard_launch_count(ctx.h) - n0 == 3
                assert ard.ard_last_device_status(ctx.h) == 0
                assert OG.rel_fro(host(dX), bw["dX"]) <= TOL[ard.ARD_BF16], (compact, dp, b)
                assert OG.rel_fro(host(dW), bw["dW"].T) <= TOL[ard.ARD_BF16], (compact, dp, b)
                kidx = torch.from_numpy(keep).cuda()
                assert OG.rel_fro(host(layer.D[0, :, I:][:, kidx]), bw["dh0"][:, keep]) <= TOL[ard.ARD_BF16], (compact, dp, b)
                assert OG.rel_fro(host(layer.dc[:, :n]), bw["dc0"][:, keep]) <= TOL[ard.ARD_BF16], (compact, dp, b)
                got[compact] = (dX.clone(), layer.dc[:, :n].clone())
            assert float((got[1][0] - got[0][0]).abs().max()) <= 2e-2 * max(1.0, float(got[0][0].abs().max())), (dp, b)
            assert float((got[1][1] - got[0][1]).abs().max()) <= 2e-2 * max(1.0, float(got[0][1].abs().max())), (dp, b)
        ard.ard_set_option(ctx.h, ard.ARD_OPT_LSTM_COMPACT_H, 1)
    finally:
        ctx.close()


def test_a_sequence_replays_from_a_cuda_graph_with_a_new_pattern_each_time():
    """Sampler (device-resident iteration counter), whole-sequence forward and whole-sequence BPTT captured once into
    a CUDA graph: every replay draws the next pattern, and the kernels choose their form on the device from it
    (full contraction at a period of 1, compact h and partial sums at 2 - 3, compact h and one barrier per step
    from 4 on at this size).  Outputs against the oracle for the oracle's draw of the same iteration."""
    from distributions import max_entropy_K
    T, B, I, H = 3, 8, 64, 1024
    KH = I + H
    rng = np.random.default_rng(2024)
    W = inputs.bf16_round(rng.uniform(-0.05, 0.05, size=(KH, 4 * H)).astype(np.float32))
    X = inputs.bf16_round(rng.standard_normal((T, B, I)).astype(np.float32))
    dH = (rng.standard_normal((T, B, H)) / 8).astype(np.float32)
    ctx = Ctx(1 << 20)
    try:
        Kd = max_entropy_K(0.6, 8)
        cdf = ard.ard_quantise_distribution(Kd)
        ard.ard_set_distribution(ctx.h, 0, Kd)
        pat = ctx.pattern(ard.ARD_ROW, KH, H)
        counter = torch.zeros(1, dtype=torch.int64, device="cuda")
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            Wnm = torch.from_numpy(np.ascontiguousarray(W.T)).to(BF).cuda()
            XH = torch.zeros((T + 1, B, KH), dtype=BF, device="cuda")
            XH[:T, :, :I] = torch.from_numpy(X).to(BF).cuda()
            C = torch.zeros((T + 1, B, H), dtype=torch.float32, device="cuda")
            G = torch.zeros((T, B, 4 * H), dtype=torch.float32, device="cuda")
            Z = torch.zeros((B, 4 * H), dtype=torch.float32, device="cuda")
            DZ = torch.zeros((T, B, 4 * H), dtype=BF, device="cuda")
            D = torch.zeros((T, B, KH), dtype=torch.float32, device="cuda")
            D0 = torch.zeros((T, B, KH), dtype=torch.float32, device="cuda")
            D0[1:, :, I:] = torch.from_numpy(dH[:-1]).cuda()
            dc = torch.zeros((B, H), dtype=torch.float32, device="cuda")
            dW = torch.zeros((4 * H, KH), dtype=torch.float32, device="cuda")
            dh_last = torch.from_numpy(dH[T - 1]).cuda().contiguous()
            alpha = 1.0 / (1.0 - 0.6)

            def seq(cs):
                ard.ard_sample_pattern_counter(ctx.h, pat, 0, 31, 900, counter, 1, 5, cs)
                C[1:].zero_()
                D.copy_(D0)
                dc.zero_()
                ard.ard_lstm_forward(ctx.h, pat, T, B, I, H, alpha, XH, Wnm, KH, None, C, G, Z, cs)
                ard.ard_lstm_backward(ctx.h, pat, T, B, I, H, alpha, XH, Wnm, KH, C, G, dh_last, D, dc, DZ, dW, cs)

            seq(s.cuda_stream)  # one ordinary call first (iteration 900)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                seq(s.cuda_stream)
            seen = set()
            for it in range(1, 9):
                g.replay()
                torch.cuda.synchronize()
                assert int(counter.item()) == it + 1
                dp, b = OP.draw(cdf, 31, 900 + it, 5)
                seen.add(1 if dp == 1 else (2 if dp <= 3 else 3))
                m = OP.row_mask(H, dp, b)
                keep = OP.row_keep(H, dp, b)
                fw = OL.fwd(X, W, None, m, alpha)
                bw = OL.bwd(fw, W, m, alpha, dH)
                assert OG.rel_fro(host(XH[1:, :, I:].float()), fw["Hs"]) <= TOL[ard.ARD_BF16], (it, dp, b)
                assert OG.rel_fro(host(D[:, :, :I]), bw["dX"]) <= TOL[ard.ARD_BF16], (it, dp, b)
                assert OG.rel_fro(host(dW), bw["dW"].T) <= TOL[ard.ARD_BF16], (it, dp, b)
                assert OG.rel_fro(host(dc[:, :len(keep)]), bw["dc0"][:, keep]) <= TOL[ard.ARD_BF16], (it, dp, b)
            assert len(seen) >= 2, seen
        assert ard.ard_last_device_status(ctx.h) == 0
    finally:
        ctx.close()
