"""Row-based sensitivity-aware dropout (Sec. 5.1, 5.2.1) on the device against the oracle.

Region decisions, per-region probabilities and the kept-row list are integer work: bit-exact.  The three
products over the kept rows follow the floating-point tolerance of the other bf16 products.
"""
import numpy as np
import pytest
import torch

from oracle import cnn as OC
from oracle import gemm as OG
from paper_2203_05705_b200 import ard, inputs
from gpu_helpers import Ctx, host, TOL

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


def _input_matrix(rng, M, Kc, x):
    """Post-ReLU-like input matrix: non-negative, about half zeros, with quiet and busy regions of x rows."""
    A = np.maximum(rng.standard_normal((M, Kc)), 0.0).astype(np.float32)
    level = rng.choice([0.1, 1.0, 4.0], size=(M + x - 1) // x)
    A *= np.repeat(level, x)[:M, None].astype(np.float32)
    return inputs.bf16_round(A)


@pytest.mark.parametrize("M,Kc,x,dtype", [(777, 200, 1, ard.ARD_BF16), (1030, 96, 4, ard.ARD_BF16), (64, 33, 7, ard.ARD_F32)])
def test_prediction_and_row_list_are_bit_exact(M, Kc, x, dtype):
    rng = np.random.default_rng(M)
    A = _input_matrix(rng, M, Kc, x)
    td = BF if dtype == ard.ARD_BF16 else torch.float32
    Ad = torch.full((M, Kc + 8), float("nan"), dtype=td, device="cuda")
    Ad[:, :Kc] = torch.from_numpy(A).to(td)
    ctx = Ctx(4096)
    rows = ard.ard_rows_create(ctx.h, M, x)
    try:
        regions = (M + x - 1) // x
        # run length 1 (every value drawn on its own: the statement of Sec. 5.1) and the opt-in run form
        cases = [(0.3, 0.3, 0.5, 0.2, 0.8, 1), (0.05, 0.25, 0.1, 0.0, 1.0, 1), (1.0, 0.4, 0.3, 0.35, 0.65, 1),
                 (0.3, 0.3, 0.5, 0.2, 0.8, OC.transaction_run(Kc)), (0.05, 0.1, 0.1, 0.0, 1.0, OC.transaction_run(Kc))]
        for it, (k, t, thr, mp, npb, rl) in enumerate(cases):
            ard.ard_sensitivity_predict(ctx.h, rows, dtype, Ad, Kc + 8, Kc, k, rl, t, thr, mp, npb, 99, it, 5)
            ard.ard_rows_sample(ctx.h, rows, 99, it, 5)
            n_keep, idx, P = ard.ard_rows_to_host(rows, M, regions)
            Po, sens = OC.sensitivity_mask(A, x, k, t, thr, mp, npb, 99, it, 5, run_len=rl)
            assert np.array_equal(P.astype(np.uint64), Po), (it, int((P.astype(np.uint64) != Po).sum()))
            assert 0 < sens.sum() < regions                      # the input has both kinds of region
            keep = OC.draw_rows(Po, x, M, 99, it, 5)
            assert n_keep == len(keep) and np.array_equal(idx, keep), it
        ard.ard_rows_set_probability(ctx.h, rows, 0.0)
        ard.ard_rows_sample(ctx.h, rows, 1, 2, 3)
        n_keep, idx, _ = ard.ard_rows_to_host(rows, M)
        assert n_keep == M and np.array_equal(idx, np.arange(M))
        ard.ard_rows_set_probability(ctx.h, rows, 0.5)
        ard.ard_rows_sample(ctx.h, rows, 1, 2, 3)
        n_keep, idx, _ = ard.ard_rows_to_host(rows, M)
        Pq = np.full(regions, OC.quantise_probability(0.5), dtype=np.uint64)
        assert np.array_equal(idx, OC.draw_rows(Pq, x, M, 1, 2, 3))
    finally:
        torch.cuda.synchronize()
        ard.ard_rows_destroy(rows)
        ctx.close()


@pytest.mark.parametrize("M,K,N", [(300, 328, 520), (1000, 64, 72), (130, 1160, 264), (64, 72, 8)])
def test_products_over_the_kept_rows_match_the_oracle(M, K, N):
    """Forward, backward-data and backward-weight over the drawn rows; NaN wherever the kernels must write
    (so a row left out shows) and in the rows of the operands that must not be read."""
    rng = np.random.default_rng(M + K)
    A = inputs.bf16_round(rng.standard_normal((M, K)).astype(np.float32))
    W = inputs.bf16_round((rng.standard_normal((K, N)) / np.sqrt(K)).astype(np.float32))      # math orientation
    dY = inputs.bf16_round(rng.standard_normal((M, N)).astype(np.float32))
    ctx = Ctx(4096)
    rows = ard.ard_rows_create(ctx.h, M, 3)
    try:
        Wd = torch.from_numpy(np.ascontiguousarray(W.T)).to(BF).cuda()
        tol = TOL[ard.ARD_BF16]
        for it, p in enumerate([0.0, 0.3, 0.5, 0.9, 0.999]):
            ard.ard_rows_set_probability(ctx.h, rows, p)
            ard.ard_rows_sample(ctx.h, rows, 7, it, 1)
            n_keep, keep, _ = ard.ard_rows_to_host(rows, M)
            Pq = np.full((M + 2) // 3, OC.quantise_probability(p), dtype=np.uint64)
            assert np.array_equal(keep, OC.draw_rows(Pq, 3, M, 7, it, 1))
            dropped = np.setdiff1d(np.arange(M), keep)
            # operands: dropped rows hold NaN -- they must never be fetched
            Ad = torch.from_numpy(A).to(BF).cuda()
            dYd = torch.from_numpy(dY).to(BF).cuda()
            if len(dropped):
                Ad[torch.from_numpy(dropped).cuda()] = float("nan")
                dYd[torch.from_numpy(dropped).cuda()] = float("nan")
            Y = torch.full((M, N), float("nan"), dtype=BF, device="cuda")
            dA = torch.full((M, K), float("nan"), dtype=BF, device="cuda")
            dW = torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda")
            ard.ard_rows_fwd(ctx.h, rows, M, K, N, 1.5, Ad, K, Wd, K, Y, N)
            ard.ard_rows_bwd_data(ctx.h, rows, M, K, N, 1.5, dYd, N, Wd, K, dA, K)
            ard.ard_rows_bwd_weight(ctx.h, rows, ard.ARD_F32, M, K, N, 1.5, Ad, K, dYd, N, dW, K)
            torch.cuda.synchronize()
            assert ard.ard_last_device_status(ctx.h) == 0
            tag = (M, K, N, p, n_keep)
            Yh, dAh, dWh = host(Y), host(dA), host(dW)
            assert np.all(Yh[dropped] == 0) and np.all(dAh[dropped] == 0), tag
            if n_keep:
                assert OG.rel_fro(Yh, OC.fwd(A, W, keep, 1.5)) <= tol, tag
                assert OG.rel_fro(dAh, OC.bwd_data(dY, W, keep, 1.5)) <= tol, tag
                assert OG.rel_fro(dWh, OC.bwd_weight(A, dY, keep, 1.5).T) <= tol, tag
            else:
                assert np.all(Yh == 0) and np.all(dAh == 0) and np.all(dWh == 0), tag
    finally:
        torch.cuda.synchronize()
        ard.ard_rows_destroy(rows)
        ctx.close()


@pytest.mark.parametrize("M,K,N", [(300, 328, 520), (1000, 64, 72), (130, 1160, 264), (64, 72, 8), (2100, 520, 384)])
def test_products_on_gathered_rows_match_the_oracle(M, K, N):
    """The same three products through the dense small matrices of Sec. 5.2.1: gather the kept rows, multiply,
    fill back.  The compact buffers start as NaN, so rows the gather must write (kept rows and the zero rows up
    to the next multiple of 64) show if they are missing, and nothing past them may be read into a result."""
    rng = np.random.default_rng(M + K + 1)
    A = inputs.bf16_round(rng.standard_normal((M, K)).astype(np.float32))
    W = inputs.bf16_round((rng.standard_normal((K, N)) / np.sqrt(K)).astype(np.float32))      # math orientation
    dY = inputs.bf16_round(rng.standard_normal((M, N)).astype(np.float32))
    ctx = Ctx(4096)
    rows = ard.ard_rows_create(ctx.h, M, 3)
    cap = (M + 63) // 64 * 64
    try:
        Wd = torch.from_numpy(np.ascontiguousarray(W.T)).to(BF).cuda()
        Ad = torch.from_numpy(A).to(BF).cuda()
        dYd = torch.from_numpy(dY).to(BF).cuda()
        tol = TOL[ard.ARD_BF16]
        for it, p in enumerate([0.0, 0.3, 0.5, 0.9, 0.999]):
            ard.ard_rows_set_probability(ctx.h, rows, p)
            ard.ard_rows_sample(ctx.h, rows, 11, it, 2)
            n_keep, keep, _ = ard.ard_rows_to_host(rows, M)
            dropped = np.setdiff1d(np.arange(M), keep)
            Ak = torch.full((cap, K), float("nan"), dtype=BF, device="cuda")
            dYk = torch.full((cap, N), float("nan"), dtype=BF, device="cuda")
            ard.ard_rows_gather(ctx.h, rows, M, K, Ad, K, Ak, K)
            ard.ard_rows_gather(ctx.h, rows, M, N, dYd, N, dYk, N)
            torch.cuda.synchronize()
            pad = (n_keep + 63) // 64 * 64
            assert torch.equal(Ak[:n_keep], Ad[torch.from_numpy(keep).long().cuda()])          # bit-exact copy
            assert bool(torch.all(Ak[n_keep:pad] == 0)) and bool(torch.all(dYk[n_keep:pad] == 0))
            assert bool(torch.isnan(Ak[pad:]).all())                                           # nothing else written
            Y = torch.full((M, N), float("nan"), dtype=BF, device="cuda")
            dA = torch.full((M, K), float("nan"), dtype=BF, device="cuda")
            dW = torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda")
            dWb = torch.full((N, K), float("nan"), dtype=BF, device="cuda")
            ard.ard_rows_fwd_compact(ctx.h, rows, M, K, N, 1.5, Ak, K, Wd, K, Y, N)
            ard.ard_rows_bwd_data_compact(ctx.h, rows, M, K, N, 1.5, dYk, N, Wd, K, dA, K)
            ard.ard_rows_bwd_weight_compact(ctx.h, rows, ard.ARD_F32, M, K, N, 1.5, Ak, K, dYk, N, dW, K)
            ard.ard_rows_bwd_weight_compact(ctx.h, rows, ard.ARD_BF16, M, K, N, 1.5, Ak, K, dYk, N, dWb, K)
            torch.cuda.synchronize()
            assert ard.ard_last_device_status(ctx.h) == 0
            tag = (M, K, N, p, n_keep)
            Yh, dAh, dWh, dWbh = host(Y), host(dA), host(dW), host(dWb)
            assert np.all(Yh[dropped] == 0) and np.all(dAh[dropped] == 0), tag
            if n_keep:
                assert OG.rel_fro(Yh, OC.fwd_compact(A, W, keep, 1.5)) <= tol, tag
                assert OG.rel_fro(dAh, OC.bwd_data(dY, W, keep, 1.5)) <= tol, tag
                assert OG.rel_fro(dWh, OC.bwd_weight(A, dY, keep, 1.5).T) <= tol, tag
                assert OG.rel_fro(dWbh, OC.bwd_weight(A, dY, keep, 1.5).T) <= tol, tag
            else:
                assert np.all(Yh == 0) and np.all(dAh == 0) and np.all(dWh == 0) and np.all(dWbh == 0), tag
            # both gathers and the three products behind one call (two streams inside): the same bits
            Ak2 = torch.full((cap, K), float("nan"), dtype=BF, device="cuda")
            dYk2 = torch.full((cap, N), float("nan"), dtype=BF, device="cuda")
            Y2 = torch.full((M, N), float("nan"), dtype=BF, device="cuda")
            dA2 = torch.full((M, K), float("nan"), dtype=BF, device="cuda")
            dW2 = torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda")
            ard.ard_rows_products(ctx.h, rows, ard.ARD_F32, M, K, N, 1.5, Ad, K, Wd, K, dYd, N, Ak2, K, dYk2, N, Y2, N,
                                  dA2, K, dW2, K)
            torch.cuda.synchronize()
            assert ard.ard_last_device_status(ctx.h) == 0
            assert torch.equal(Y2, Y) and torch.equal(dA2, dA) and torch.equal(dW2, dW), tag
    finally:
        torch.cuda.synchronize()
        ard.ard_rows_destroy(rows)
        ctx.close()


def test_shared_weight_gradient_on_gathered_rows_is_reproducible():
    """A long list and few output tiles: the weight gradient's tiles are cut along the contraction and shared by
    all SMs; the partial sums are added in a fixed order, so every launch gives the same bits."""
    M, K, N = 20000, 576, 512
    rng = np.random.default_rng(9)
    A = torch.from_numpy(inputs.bf16_round(rng.standard_normal((M, K)).astype(np.float32))).to(BF).cuda()
    dY = torch.from_numpy(inputs.bf16_round(rng.standard_normal((M, N)).astype(np.float32))).to(BF).cuda()
    ctx = Ctx(4096)
    rows = ard.ard_rows_create(ctx.h, M, 1)
    cap = (M + 63) // 64 * 64
    try:
        ard.ard_rows_set_probability(ctx.h, rows, 0.45)
        ard.ard_rows_sample(ctx.h, rows, 3, 0, 0)
        n_keep, keep, _ = ard.ard_rows_to_host(rows, M)
        Ak = torch.zeros((cap, K), dtype=BF, device="cuda")
        dYk = torch.zeros((cap, N), dtype=BF, device="cuda")
        ard.ard_rows_gather(ctx.h, rows, M, K, A, K, Ak, K)
        ard.ard_rows_gather(ctx.h, rows, M, N, dY, N, dYk, N)
        ref = None
        for rep in range(10):
            dW = torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda")
            ard.ard_rows_bwd_weight_compact(ctx.h, rows, ard.ARD_F32, M, K, N, 1.0, Ak, K, dYk, N, dW, K)
            torch.cuda.synchronize()
            if ref is None:
                ref = dW
                kk = torch.from_numpy(keep).long().cuda()
                want = dY[kk].double().T @ A[kk].double()                      # library matmul in fp64 on the same bits
                err = float((dW.double() - want).norm() / want.norm())
                assert err <= 1e-5, err                                        # fp32 accumulation of exact bf16 products
            else:
                assert torch.equal(dW, ref), rep
        assert ard.ard_last_device_status(ctx.h) == 0
    finally:
        torch.cuda.synchronize()
        ard.ard_rows_destroy(rows)
        ctx.close()


def test_benchmark_layer_on_sampled_outputs():
    """The convolution layer the benchmark times (3 x 3, 256 -> 512 channels, 32768 output positions, regions of 8
    rows), in its launch configuration: gathered operands, CTA pairs, shared weight-gradient tiles.  The oracle
    recomputes the sensitivity decision of sampled regions, the whole kept-row list, sampled rows of Y and dA
    and sampled channels of dW; the zero rows and finiteness are checked over the whole outputs."""
    M, K, N, x = 32768, 2304, 512, 8
    kf, tf, thr, mp, npb = 0.05, 0.3, 0.5, 0.2, 0.8
    rng = np.random.default_rng(2025)
    A = _input_matrix(rng, M, K, x)
    W = inputs.bf16_round((rng.standard_normal((K, N)) / np.sqrt(K)).astype(np.float32))      # math orientation
    dY = inputs.bf16_round(rng.standard_normal((M, N)).astype(np.float32))
    ctx = Ctx(4096)
    rows = ard.ard_rows_create(ctx.h, M, x)
    cap = (M + 63) // 64 * 64
    try:
        Ad = torch.from_numpy(A).to(BF).cuda()
        dYd = torch.from_numpy(dY).to(BF).cuda()
        Wd = torch.from_numpy(np.ascontiguousarray(W.T)).to(BF).cuda()
        # Sec. 5.1 on sampled regions (integer decisions: exact)
        Pm, Pn = OC.quantise_probability(mp), OC.quantise_probability(npb)
        for rl in (1, OC.transaction_run(K)):
            ard.ard_sensitivity_predict(ctx.h, rows, ard.ARD_BF16, Ad, K, K, kf, rl, tf, thr, mp, npb, 5, 3, 1)
            _, _, P = ard.ard_rows_to_host(rows, M, M // x)
            for g in range(5, M // x, (M // x) // 40):
                sens, _, _ = OC.region_sensitive(A, g, x, kf, tf, thr, 5, 3, 1, run_len=rl)
                assert int(P[g]) == (Pm if sens else Pn), (g, rl)
            assert 0 < int(np.sum(P == Pm)) < M // x                     # both kinds of region occur
        # Sec. 5.2.1 with one probability for every region: the whole list against the oracle
        ard.ard_rows_set_probability(ctx.h, rows, 0.46)
        ard.ard_rows_sample(ctx.h, rows, 5, 3, 1)
        n_keep, keep, _ = ard.ard_rows_to_host(rows, M)
        Pq = np.full(M // x, OC.quantise_probability(0.46), dtype=np.uint64)
        assert np.array_equal(keep, OC.draw_rows(Pq, x, M, 5, 3, 1))
        dropped = np.setdiff1d(np.arange(M), keep)
        Ak = torch.full((cap, K), float("nan"), dtype=BF, device="cuda")
        dYk = torch.full((cap, N), float("nan"), dtype=BF, device="cuda")
        Y = torch.full((M, N), float("nan"), dtype=BF, device="cuda")
        dA = torch.full((M, K), float("nan"), dtype=BF, device="cuda")
        dW = torch.full((N, K), float("nan"), dtype=BF, device="cuda")
        ard.ard_rows_gather(ctx.h, rows, M, K, Ad, K, Ak, K)
        ard.ard_rows_fwd_compact(ctx.h, rows, M, K, N, 1.25, Ak, K, Wd, K, Y, N)
        ard.ard_rows_gather(ctx.h, rows, M, N, dYd, N, dYk, N)
        ard.ard_rows_bwd_data_compact(ctx.h, rows, M, K, N, 1.25, dYk, N, Wd, K, dA, K)
        ard.ard_rows_bwd_weight_compact(ctx.h, rows, ard.ARD_BF16, M, K, N, 1.25, Ak, K, dYk, N, dW, K)
        torch.cuda.synchronize()
        assert ard.ard_last_device_status(ctx.h) == 0
        # whole outputs: finite, dropped rows exactly zero
        assert bool(torch.isfinite(Y).all()) and bool(torch.isfinite(dA).all()) and bool(torch.isfinite(dW).all())
        dd = torch.from_numpy(dropped).long().cuda()
        assert bool(torch.all(Y[dd] == 0)) and bool(torch.all(dA[dd] == 0))
        # sampled rows (kept and dropped) of Y and dA
        sel = np.concatenate([keep[:: max(1, len(keep) // 96)][:96], dropped[:: max(1, len(dropped) // 32)][:32]])
        local_keep = np.flatnonzero(np.isin(sel, keep))
        sd = torch.from_numpy(sel).long().cuda()
        tol = TOL[ard.ARD_BF16]
        assert OG.rel_fro(host(Y[sd]), OC.fwd(A[sel], W, local_keep, 1.25)) <= tol
        assert OG.rel_fro(host(dA[sd]), OC.bwd_data(dY[sel], W, local_keep, 1.25)) <= tol
        # sampled channels of dW: the contraction runs over every kept row
        cols = np.arange(3, N, N // 48)[:48]
        want = OC.bwd_weight(A[keep], dY[keep][:, cols], np.arange(len(keep)), 1.25).T       # [48][K]
        assert OG.rel_fro(host(dW[torch.from_numpy(cols).long().cuda()]), want) <= tol
    finally:
        torch.cuda.synchronize()
        ard.ard_rows_destroy(rows)
        ctx.close()


def test_repeated_launches_give_the_same_bits():
    """The gathered operand reaches the tensor cores through ordinary asynchronous copies; a missing ordering
    between those writes and the MMA reads would show as run-to-run differences."""
    M, K, N = 2048, 1152, 256
    rng = np.random.default_rng(5)
    A = torch.from_numpy(inputs.bf16_round(rng.standard_normal((M, K)).astype(np.float32))).to(BF).cuda()
    W = torch.from_numpy(inputs.bf16_round((rng.standard_normal((N, K)) / 34).astype(np.float32))).to(BF).cuda()
    dY = torch.from_numpy(inputs.bf16_round(rng.standard_normal((M, N)).astype(np.float32))).to(BF).cuda()
    ctx = Ctx(4096)
    rows = ard.ard_rows_create(ctx.h, M, 1)
    try:
        ard.ard_rows_set_probability(ctx.h, rows, 0.4)
        ard.ard_rows_sample(ctx.h, rows, 3, 0, 0)
        ref = None
        for rep in range(20):
            Y = torch.zeros((M, N), dtype=BF, device="cuda")
            dA = torch.zeros((M, K), dtype=BF, device="cuda")
            dW = torch.zeros((N, K), dtype=torch.float32, device="cuda")
            ard.ard_rows_fwd(ctx.h, rows, M, K, N, 1.0, A, K, W, K, Y, N)
            ard.ard_rows_bwd_data(ctx.h, rows, M, K, N, 1.0, dY, N, W, K, dA, K)
            ard.ard_rows_bwd_weight(ctx.h, rows, ard.ARD_F32, M, K, N, 1.0, A, K, dY, N, dW, K)
            torch.cuda.synchronize()
            cur = (Y, dA, dW)
            if ref is None:
                ref = cur
            else:
                for a, c in zip(cur, ref):
                    assert torch.equal(a, c), rep
        assert ard.ard_last_device_status(ctx.h) == 0
    finally:
        torch.cuda.synchronize()
        ard.ard_rows_destroy(rows)
        ctx.close()
