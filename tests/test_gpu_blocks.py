"""Block-based sensitivity-aware dropout (Sec. 5.1, 5.2.2) on the device against the oracle.

Counts, labels, kept flags and the index lists are integer work: bit-exact.  The three products over the kept
blocks follow the floating-point tolerance of the other bf16 products.
"""
import numpy as np
import pytest
import torch

from oracle import cnn_blocks as OB
from oracle import gemm as OG
from paper_2203_05705_b200 import ard, inputs
from gpu_helpers import Ctx, host, TOL

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


def _input_matrix(rng, M, Kc, ts):
    """Post-ReLU-like input matrix: non-negative, about half zeros, quiet and busy blocks."""
    A = np.maximum(rng.standard_normal((M, Kc)), 0.0).astype(np.float32)
    level = rng.choice([0.1, 1.0, 4.0], size=(M // ts, Kc // ts))
    A *= np.kron(level, np.ones((ts, ts))).astype(np.float32)
    return inputs.bf16_round(A)


@pytest.mark.parametrize("M,Kc,ts,dtype", [(192, 320, 64, ard.ARD_BF16), (96, 40, 8, ard.ARD_F32),
                                           (2304, 128, 64, ard.ARD_BF16), (128, 4224, 128, ard.ARD_BF16)])
def test_counts_labels_draws_and_lists_are_bit_exact(M, Kc, ts, dtype):
    rng = np.random.default_rng(M + Kc)
    A = _input_matrix(rng, M, Kc, ts)
    td = BF if dtype == ard.ARD_BF16 else torch.float32
    Ad = torch.full((M, Kc + 8), float("nan"), dtype=td, device="cuda")
    Ad[:, :Kc] = torch.from_numpy(A).to(td)
    G, Q = M // ts, Kc // ts
    ctx = Ctx(4096)
    blocks = ard.ard_blocks_create(ctx.h, M, Kc, ts)
    try:
        pat = ard.ard_blocks_pattern(blocks)
        cases = [(0.02, 0.3, 0.5, max(1, Q // 2), 0.2, 0.8), (0.05, 0.25, 0.1, 1, 0.0, 1.0), (0.03, 0.4, 0.3, Q, 0.35, 0.65),
                 (0.02, 0.3, 0.5, 0, 0.1, 0.5)]
        # every case with run length 1 (each value drawn on its own: the statement of Sec. 5.1) and in the run form
        cases = [c + (rl,) for rl in (1, OB.transaction_run(ts)) for c in cases]
        for it, (k, t, thr, cap, mp, npb, rl) in enumerate(cases):
            ard.ard_blocks_predict(ctx.h, blocks, dtype, Ad, Kc + 8, k, rl, t, thr, cap, 99, it, 5)
            ard.ard_blocks_sample(ctx.h, blocks, mp, npb, 99, it, 5)
            counts, sens, keep = ard.ard_blocks_to_host(blocks, G * Q)
            co, so = OB.predict(A, ts, k, t, thr, cap, 99, it, 5, run_len=rl)
            assert np.array_equal(counts.reshape(G, Q), co), it
            assert np.array_equal(sens.reshape(G, Q).astype(bool), so), it
            if 0 < cap < Q:
                assert so.any() and not so.all()
            ko = OB.draw_blocks(so, mp, npb, 99, it, 5)
            assert np.array_equal(keep.reshape(G, Q).astype(bool), ko), it
            idx, col_ptr, col_idx, row_ptr, row_idx = OB.block_lists(ko)
            dp, b, n_keep, didx = ard.ard_pattern_to_host(pat, G * Q)
            assert n_keep == len(idx) and np.array_equal(didx, idx), it
            cp, ci, rp, ri = ard.ard_pattern_tile_lists_to_host(pat, Q, G)
            assert np.array_equal(cp, col_ptr) and np.array_equal(ci, col_idx), it
            assert np.array_equal(rp, row_ptr) and np.array_equal(ri, row_idx), it
        ard.ard_blocks_set_label(ctx.h, blocks, 1)
        ard.ard_blocks_sample(ctx.h, blocks, 0.0, 1.0, 1, 2, 3)
        _, sens, keep = ard.ard_blocks_to_host(blocks, G * Q)
        assert sens.all() and keep.all()
        ard.ard_blocks_set_label(ctx.h, blocks, 0)
        ard.ard_blocks_sample(ctx.h, blocks, 0.0, 0.5, 1, 2, 3)
        _, sens, keep = ard.ard_blocks_to_host(blocks, G * Q)
        assert np.array_equal(keep.reshape(G, Q).astype(bool), OB.draw_blocks(np.zeros((G, Q), bool), 0.0, 0.5, 1, 2, 3))
    finally:
        torch.cuda.synchronize()
        ard.ard_blocks_destroy(blocks)
        ctx.close()


@pytest.mark.parametrize("M,Kc,N,ts", [(384, 320, 72, 64), (256, 576, 136, 64), (512, 256, 264, 128), (1152, 64, 8, 64)])
def test_products_over_the_kept_blocks_match_the_oracle(M, Kc, N, ts):
    """Forward, weight gradient and input gradient over the drawn blocks.  Dropped blocks of A hold NaN (they
    must never be fetched), outputs start as NaN (so anything left unwritten shows)."""
    rng = np.random.default_rng(M + Kc + N)
    A = inputs.bf16_round(rng.standard_normal((M, Kc)).astype(np.float32))
    W = inputs.bf16_round((rng.standard_normal((Kc, N)) / np.sqrt(Kc)).astype(np.float32))   # math orientation
    dY = inputs.bf16_round(rng.standard_normal((M, N)).astype(np.float32))
    G, Q = M // ts, Kc // ts
    ldy = (M + 7) // 8 * 8
    ctx = Ctx(4096)
    blocks = ard.ard_blocks_create(ctx.h, M, Kc, ts)
    try:
        Wd = torch.from_numpy(np.ascontiguousarray(W.T)).to(BF).cuda()          # [N][Kc]
        dYt = torch.from_numpy(np.ascontiguousarray(dY.T)).to(BF).cuda()        # [N][M]
        tol = TOL[ard.ARD_BF16]
        ard.ard_blocks_set_label(ctx.h, blocks, 0)
        for it, p in enumerate([0.0, 0.3, 0.5, 0.9, 1.0]):
            ard.ard_blocks_sample(ctx.h, blocks, 0.0, p, 7, it, 1)
            _, _, keep = ard.ard_blocks_to_host(blocks, G * Q)
            keep = keep.reshape(G, Q).astype(bool)
            assert np.array_equal(keep, OB.draw_blocks(np.zeros((G, Q), bool), 0.0, p, 7, it, 1))
            mask = OB.block_mask(keep, ts).astype(bool)
            Ah = A.copy()
            Ah[~mask] = np.nan
            Ad = torch.from_numpy(Ah).to(BF).cuda()
            Yt = torch.full((N, ldy), float("nan"), dtype=BF, device="cuda")
            dW = torch.full((N, Kc), float("nan"), dtype=BF, device="cuda")
            dA = torch.full((M, Kc), float("nan"), dtype=torch.float32, device="cuda")
            dA2 = torch.full((M, Kc), float("nan"), dtype=BF, device="cuda")
            ard.ard_blocks_fwd(ctx.h, blocks, N, 1.5, Ad, Kc, Wd, Kc, Yt, ldy)
            ard.ard_blocks_bwd_weight(ctx.h, blocks, N, 1.5, Ad, Kc, dYt, M, dW, Kc)
            ard.ard_blocks_bwd_input(ctx.h, blocks, ard.ARD_F32, N, 1.5, dYt, M, Wd, Kc, dA, Kc, 1)
            ard.ard_blocks_bwd_input(ctx.h, blocks, ard.ARD_BF16, N, 1.5, dYt, M, Wd, Kc, dA2, Kc, 0)
            # the same through the one-call form
            Yt3 = torch.full((N, ldy), float("nan"), dtype=BF, device="cuda")
            dW3 = torch.full((N, Kc), float("nan"), dtype=BF, device="cuda")
            dA3 = torch.full((M, Kc), float("nan"), dtype=torch.float32, device="cuda")
            ard.ard_blocks_products(ctx.h, blocks, ard.ARD_F32, N, 1.5, Ad, Kc, Wd, Kc, dYt, M, Yt3, ldy, dW3, Kc, dA3, Kc, 1)
            torch.cuda.synchronize()
            assert ard.ard_last_device_status(ctx.h) == 0
            assert torch.equal(Yt3[:, :M], Yt[:, :M]) and torch.equal(dW3, dW) and torch.equal(dA3, dA)
            tag = (M, Kc, N, ts, p, int(keep.sum()))
            Yh, dWh, dAh, dA2h = host(Yt)[:, :M].T, host(dW).T, host(dA), host(dA2)
            assert np.all(dAh[~mask] == 0), tag
            assert np.all(np.isnan(dA2h[~mask])), tag                 # left untouched without the zero fill
            if keep.any():
                assert OG.rel_fro(Yh, OB.fwd(A, W, keep, ts, 1.5)) <= tol, tag
                assert OG.rel_fro(dWh, OB.bwd_weight(A, dY, keep, ts, 1.5)) <= tol, tag
                assert OG.rel_fro(dAh, OB.bwd_input(dY, W, keep, ts, 1.5)) <= tol, tag
                assert OG.rel_fro(np.where(mask, dA2h, 0.0), OB.bwd_input(dY, W, keep, ts, 1.5)) <= 2 * tol, tag
                # groups without a kept block: their rows of the output are exact zeros
                empty = np.repeat(~keep.any(axis=1), ts)
                assert np.all(Yh[empty] == 0), tag
            else:
                assert np.all(Yh == 0) and np.all(dWh == 0) and np.all(dAh == 0), tag
    finally:
        torch.cuda.synchronize()
        ard.ard_blocks_destroy(blocks)
        ctx.close()


@pytest.mark.parametrize("G,Q", [(200, 256), (280, 256), (3, 1), (1, 40)])
def test_draws_and_lists_on_other_grid_sizes(G, Q):
    """Block counts beyond what the list kernel keeps in shared memory (51200) and beyond what it draws itself
    (71680), and degenerate grids: the same flags and lists as the oracle."""
    ts = 8
    ctx = Ctx(4096)
    blocks = ard.ard_blocks_create(ctx.h, G * ts, Q * ts, ts)
    try:
        pat = ard.ard_blocks_pattern(blocks)
        ard.ard_blocks_set_label(ctx.h, blocks, 0)
        for it, p in enumerate([0.5, 0.97]):
            ard.ard_blocks_sample(ctx.h, blocks, 0.0, p, 21, it, 9)
            _, _, keep = ard.ard_blocks_to_host(blocks, G * Q)
            ko = OB.draw_blocks(np.zeros((G, Q), bool), 0.0, p, 21, it, 9)
            assert np.array_equal(keep.reshape(G, Q).astype(bool), ko)
            idx, col_ptr, col_idx, row_ptr, row_idx = OB.block_lists(ko)
            _, _, n_keep, didx = ard.ard_pattern_to_host(pat, G * Q)
            assert n_keep == len(idx) and np.array_equal(didx, idx)
            cp, ci, rp, ri = ard.ard_pattern_tile_lists_to_host(pat, Q, G)
            assert np.array_equal(cp, col_ptr) and np.array_equal(ci, col_idx)
            assert np.array_equal(rp, row_ptr) and np.array_equal(ri, row_idx)
    finally:
        torch.cuda.synchronize()
        ard.ard_blocks_destroy(blocks)
        ctx.close()


def test_benchmark_layer_on_sampled_outputs():
    """The convolution layer the benchmark times (3 x 3, 256 -> 512 channels, 32768 output positions, 128 x 128
    blocks, at most 6 sensitive blocks per group), in its launch configuration (ard_blocks_products).  The oracle
    recomputes counts and labels of sampled groups, every draw and the whole lists, the output rows and the
    input-gradient rows of sampled groups and sampled channels of the weight gradient; finiteness and the zero
    blocks are checked over the whole outputs."""
    M, K, N, ts, cap = 32768, 2304, 512, 128, 6
    kf, tf, thr, mp, npb = 0.05, 0.3, 0.5, 0.2, 0.8
    G, Q = M // ts, K // ts
    rng = np.random.default_rng(2026)
    A = _input_matrix(rng, M, K, ts)
    W = inputs.bf16_round((rng.standard_normal((K, N)) / np.sqrt(K)).astype(np.float32))      # math orientation
    dY = inputs.bf16_round(rng.standard_normal((M, N)).astype(np.float32))
    ctx = Ctx(4096)
    blocks = ard.ard_blocks_create(ctx.h, M, K, ts)
    try:
        Ad = torch.from_numpy(A).to(BF).cuda()
        Wd = torch.from_numpy(np.ascontiguousarray(W.T)).to(BF).cuda()
        dYt = torch.from_numpy(np.ascontiguousarray(dY.T)).to(BF).cuda()
        ard.ard_blocks_predict(ctx.h, blocks, ard.ARD_BF16, Ad, K, kf, 1, tf, thr, cap, 5, 3, 1)
        ard.ard_blocks_sample(ctx.h, blocks, mp, npb, 5, 3, 1)
        counts, sens, keep = ard.ard_blocks_to_host(blocks, G * Q)
        counts, sens, keep = counts.reshape(G, Q), sens.reshape(G, Q).astype(bool), keep.reshape(G, Q).astype(bool)
        need = OB.needed(tf, OB.n_samples(kf, ts))
        groups = list(range(3, G, G // 24))
        for g in groups:
            co = [OB.block_count(A, g, j, ts, kf, thr, 5, 3, 1) for j in range(Q)]
            assert counts[g].tolist() == co, g
            assert np.array_equal(sens[g], OB.label_group(co, need, cap)), g
        assert (sens.sum(1) <= cap).all() and 0 < sens.sum() < G * Q
        # every draw and the whole lists, from the device's labels
        ko = OB.draw_blocks(sens, mp, npb, 5, 3, 1)
        assert np.array_equal(keep, ko)
        idx, col_ptr, col_idx, row_ptr, row_idx = OB.block_lists(ko)
        pat = ard.ard_blocks_pattern(blocks)
        _, _, n_keep, didx = ard.ard_pattern_to_host(pat, G * Q)
        assert n_keep == len(idx) and np.array_equal(didx, idx)
        cp, ci, rp, ri = ard.ard_pattern_tile_lists_to_host(pat, Q, G)
        assert np.array_equal(cp, col_ptr) and np.array_equal(ci, col_idx)
        assert np.array_equal(rp, row_ptr) and np.array_equal(ri, row_idx)
        # products: dropped blocks of A hold NaN, outputs start as NaN
        mask_t = torch.from_numpy(ko).cuda().repeat_interleave(ts, 0).repeat_interleave(ts, 1)
        Ad[~mask_t] = float("nan")
        Yt = torch.full((N, M), float("nan"), dtype=BF, device="cuda")
        dW = torch.full((N, K), float("nan"), dtype=BF, device="cuda")
        dA = torch.full((M, K), float("nan"), dtype=BF, device="cuda")
        ard.ard_blocks_products(ctx.h, blocks, ard.ARD_BF16, N, 1.25, Ad, K, Wd, K, dYt, M, Yt, M, dW, K, dA, K, 1)
        torch.cuda.synchronize()
        assert ard.ard_last_device_status(ctx.h) == 0
        assert bool(torch.isfinite(Yt).all()) and bool(torch.isfinite(dW).all()) and bool(torch.isfinite(dA).all())
        assert bool(torch.all(dA[~mask_t] == 0))
        tol = TOL[ard.ARD_BF16]
        for g in groups[::3]:
            rs = slice(g * ts, (g + 1) * ts)
            kg = ko[g:g + 1]
            assert OG.rel_fro(host(Yt[:, rs]).T, OB.fwd(A[rs], W, kg, ts, 1.25)) <= tol, g
            assert OG.rel_fro(host(dA[rs]), OB.bwd_input(dY[rs], W, kg, ts, 1.25)) <= tol, g
        # sampled channels of dW: the contraction runs over every group
        cols = np.arange(3, N, N // 32)[:32]
        want = np.zeros((K, len(cols)))
        for g in range(G):
            rs = slice(g * ts, (g + 1) * ts)
            want += OB.bwd_weight(A[rs], dY[rs][:, cols], ko[g:g + 1], ts, 1.25)
        assert OG.rel_fro(host(dW[torch.from_numpy(cols).long().cuda()]).T, want) <= tol
    finally:
        torch.cuda.synchronize()
        ard.ard_blocks_destroy(blocks)
        ctx.close()


def test_argument_checks():
    ctx = Ctx(4096)
    try:
        with pytest.raises(ard.ArdError):
            ard.ard_blocks_create(ctx.h, 100, 64, 64)              # ts does not divide M
        blocks = ard.ard_blocks_create(ctx.h, 128, 128, 64)
        A = torch.zeros((128, 128), dtype=BF, device="cuda")
        with pytest.raises(ard.ArdError):
            ard.ard_blocks_predict(ctx.h, blocks, ard.ARD_BF16, A, 64, 0.1, 1, 0.5, 0.5, 1, 0, 0, 0)      # lda < Kc
        with pytest.raises(ard.ArdError):
            ard.ard_blocks_predict(ctx.h, blocks, ard.ARD_BF16, A, 128, 0.1, 1, 0.5, 0.5, 1, 0, 0, 1 << 16)
        with pytest.raises(ard.ArdError):
            ard.ard_blocks_predict(ctx.h, blocks, ard.ARD_BF16, A, 128, 0.1, 48, 0.5, 0.5, 1, 0, 0, 0)    # 48 does not divide 64
        with pytest.raises(ard.ArdError):
            ard.ard_blocks_predict(ctx.h, blocks, ard.ARD_BF16, A, 128, 0.1, 0, 0.5, 0.5, 1, 0, 0, 0)
        with pytest.raises(ard.ArdError):
            ard.ard_blocks_sample(ctx.h, blocks, 0.2, 1.5, 0, 0, 0)
        ard.ard_blocks_destroy(blocks)
    finally:
        ctx.close()
