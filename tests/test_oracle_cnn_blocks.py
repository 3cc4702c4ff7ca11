"""Pins for oracle/cnn_blocks.py (block-based sensitivity-aware dropout, Sec. 5.1 / 5.2.2).

The paper fixes no numbers for this part; the pins are what the mathematics fixes: decisions that do not depend
on the sample, that the sampled runs are whole, lie inside their block and are drawn uniformly, the binomial law of a
block's count over runs, the bound on sensitive blocks per group and which blocks it
picks, the drop rates of the two labels, brute-force loops over kept blocks, the all-kept case against a
plain matrix product, and the adjoint identities.
"""
import numpy as np

from oracle import cnn_blocks as C


def test_counts_that_do_not_depend_on_the_sample():
    ts = 4
    A = np.zeros((8, 12))
    A[0:4, 4:8] = 1.0                  # block (0, 1): every value above the threshold
    for it in range(4):
        counts, sens = C.predict(A, ts, 0.5, 0.5, 0.5, 3, 7, it, 2)
        assert counts[0, 1] == C.n_samples(0.5, ts) == 8      # eight single values
        assert counts.sum() == 8
        assert sens[0, 1] and sens.sum() == 1


def test_default_draws_every_value_on_its_own():
    """With the default run length the sampled positions of a block are independent single values: over a block
    whose values above the threshold are one row, the count is binomial over single values (not a multiple of
    the row length, variance of independent draws)."""
    ts = 8
    B = np.zeros((ts, ts))
    B[3, :] = 1.0
    s = C.n_samples(0.5, ts)
    assert s == C.n_runs(0.5, ts) == 32
    c = np.array([C.block_count(B, 0, 0, ts, 0.5, 0.5, 2, it, 0) for it in range(1500)])
    f = 1 / ts
    assert np.any(c % 8 != 0)
    assert abs(c.mean() - s * f) < 4 * np.sqrt(s * f * (1 - f) / 1500)
    assert abs(c.var() - s * f * (1 - f)) < 0.2 * s * f * (1 - f)      # runs of 8: eight times this
    assert C.needed(0.3, 10) == 3 and C.needed(0.1, 10) == 2 and C.needed(0.5, 7) == 4 and C.needed(0.0, 5) == 1


def test_runs_are_whole_and_inside_the_block():
    # values encode their own position: a count over a block whose ONLY large values sit in one run of another
    # block, or straddle a run boundary, must never see part of a run
    ts = 8                                   # run length gcd(8, 32) = 8: a run is a whole row of the block
    assert (C.transaction_run(ts) == 8 and C.transaction_run(64) == 32 and C.transaction_run(48) == 16
            and C.transaction_run(7) == 1)
    A = np.zeros((ts, 2 * ts))
    A[:, :ts] = 1.0                          # block 0 all above, block 1 all below
    for it in range(20):
        assert C.block_count(A, 0, 0, ts, 0.5, 0.5, 1, it, 0, run_len=8) == C.n_samples(0.5, ts, 8) == 32
        assert C.block_count(A, 0, 1, ts, 0.5, 0.5, 1, it, 0, run_len=8) == 0
    B = np.zeros((ts, ts))
    B[3, :] = 1.0                            # exactly one run above: every draw contributes 0 or 8
    counts = {C.block_count(B, 0, 0, ts, 0.5, 0.5, 2, it, 0, run_len=8) for it in range(200)}
    assert all(c % 8 == 0 for c in counts) and len(counts) > 1


def test_runs_are_drawn_uniformly():
    # one run of the block above the threshold: it is hit with probability 1/Cn per draw
    ts = 8
    B = np.zeros((ts, ts))
    n_c = C.n_runs(1.0, ts, 8)               # 8 draws per count
    hits = np.zeros(ts)
    for r in range(ts):
        B[:] = 0.0
        B[r, :] = 1.0
        hits[r] = sum(C.block_count(B, 0, 0, ts, 1.0, 0.5, 5, it, 1, run_len=8) for it in range(300)) / 8
    expect = 300 * n_c / ts
    assert np.all(np.abs(hits - expect) < 4.5 * np.sqrt(expect))


def test_count_follows_the_binomial_law_over_runs():
    rng = np.random.default_rng(0)
    ts = 8
    A = np.zeros((ts, 2 * ts))
    above = rng.random(ts) < 0.4             # whole runs (rows of block 1) above the threshold
    A[above, ts:] = 1.0
    frac = above.mean()
    n_c = C.n_runs(0.5, ts, 8)
    c = np.array([C.block_count(A, 0, 1, ts, 0.5, 0.5, 3, it, 0, run_len=8) for it in range(800)]) / 8
    assert abs(c.mean() - n_c * frac) < 4 * np.sqrt(n_c * frac * (1 - frac) / 800)
    assert abs(c.var() - n_c * frac * (1 - frac)) < 0.25 * n_c * frac * (1 - frac)


def test_bound_on_sensitive_blocks_picks_the_highest_counts():
    sens = C.label_group([5, 9, 9, 2, 7, 0], need=3, cap=3)
    assert sens.tolist() == [False, True, True, False, True, False]
    sens = C.label_group([5, 9, 9, 2, 7, 0], need=3, cap=1)
    assert sens.tolist() == [False, True, False, False, False, False]      # tie: lower index
    sens = C.label_group([5, 9, 9, 2, 7, 0], need=8, cap=4)
    assert sens.tolist() == [False, True, True, False, False, False]       # only two pass
    assert not C.label_group([1, 1], need=2, cap=2).any()
    assert not C.label_group([4, 4], need=2, cap=0).any()


def test_every_group_gets_at_most_cap_sensitive_blocks():
    rng = np.random.default_rng(2)
    ts, G, Q = 4, 6, 8
    A = rng.random((G * ts, Q * ts)) + np.linspace(0, 0.5, G)[:, None].repeat(ts, 0)   # lower groups brighter
    counts, sens = C.predict(A, ts, 1.0, 0.5, 0.6, 3, 1, 0, 0)
    need = C.needed(0.5, C.n_samples(1.0, ts))
    assert (sens.sum(1) <= 3).all()
    for g in range(G):
        assert sens[g].sum() == min(3, int((counts[g] >= need).sum()))
        if sens[g].any() and (~sens[g]).any():
            passing_out = counts[g][~sens[g] & (counts[g] >= need)]
            if len(passing_out):
                assert counts[g][sens[g]].min() >= passing_out.max()


def test_drop_rates_of_the_two_labels():
    G, Q = 40, 50
    sens = np.zeros((G, Q), dtype=bool)
    sens[:, ::2] = True
    keep = C.draw_blocks(sens, 0.2, 0.7, 5, 9, 2)
    n = G * Q / 2
    assert abs((1 - keep[sens].mean()) - 0.2) < 4 * np.sqrt(0.2 * 0.8 / n)
    assert abs((1 - keep[~sens].mean()) - 0.7) < 4 * np.sqrt(0.7 * 0.3 / n)
    assert C.draw_blocks(sens, 0.0, 0.0, 5, 9, 2).all()
    # different iterations and stream ids give different draws
    assert (C.draw_blocks(sens, 0.2, 0.7, 5, 10, 2) != keep).any()
    assert (C.draw_blocks(sens, 0.2, 0.7, 5, 9, 3) != keep).any()


def test_lists_describe_the_same_set():
    rng = np.random.default_rng(3)
    G, Q = 5, 7
    keep = rng.random((G, Q)) < 0.5
    idx, col_ptr, col_idx, row_ptr, row_idx = C.block_lists(keep)
    assert len(idx) == keep.sum() and (np.diff(idx) > 0).all()
    assert {(int(i) % G, int(i) // G) for i in idx} == {(g, j) for g in range(G) for j in range(Q) if keep[g, j]}
    for g in range(G):
        assert col_idx[col_ptr[g]:col_ptr[g + 1]].tolist() == np.nonzero(keep[g])[0].tolist()
    for j in range(Q):
        assert row_idx[row_ptr[j]:row_ptr[j + 1]].tolist() == np.nonzero(keep[:, j])[0].tolist()


def _case(seed=4, ts=3, G=4, Q=5, N=6):
    rng = np.random.default_rng(seed)
    A = rng.standard_normal((G * ts, Q * ts))
    W = rng.standard_normal((Q * ts, N))
    dY = rng.standard_normal((G * ts, N))
    keep = rng.random((G, Q)) < 0.6
    return A, W, dY, keep, ts


def test_products_against_loops_over_kept_blocks():
    A, W, dY, keep, ts = _case()
    G, Q = keep.shape
    Y = np.zeros((G * ts, W.shape[1]))
    dA = np.zeros_like(A)
    dW = np.zeros_like(W)
    for g in range(G):
        for j in range(Q):
            if not keep[g, j]:
                continue
            rs, cs = slice(g * ts, (g + 1) * ts), slice(j * ts, (j + 1) * ts)
            for a in range(rs.start, rs.stop):
                for k in range(cs.start, cs.stop):
                    for n in range(W.shape[1]):
                        Y[a, n] += 1.5 * A[a, k] * W[k, n]
                        dA[a, k] += 1.5 * dY[a, n] * W[k, n]
                        dW[k, n] += 1.5 * A[a, k] * dY[a, n]
    assert np.allclose(C.fwd(A, W, keep, ts, 1.5), Y, rtol=1e-12, atol=1e-12)
    assert np.allclose(C.bwd_input(dY, W, keep, ts, 1.5), dA, rtol=1e-12, atol=1e-12)
    assert np.allclose(C.bwd_weight(A, dY, keep, ts, 1.5), dW, rtol=1e-12, atol=1e-12)


def test_all_kept_is_the_plain_product_and_none_kept_is_zero():
    A, W, dY, keep, ts = _case(5)
    allk = np.ones_like(keep)
    assert np.allclose(C.fwd(A, W, allk, ts), A @ W)
    assert np.allclose(C.bwd_input(dY, W, allk, ts), dY @ W.T)
    assert np.allclose(C.bwd_weight(A, dY, allk, ts), A.T @ dY)
    none = np.zeros_like(keep)
    assert not C.fwd(A, W, none, ts).any() and not C.bwd_input(dY, W, none, ts).any()
    assert not C.bwd_weight(A, dY, none, ts).any()


def test_adjoint_identities():
    A, W, dY, keep, ts = _case(6)
    lhs = np.sum(C.fwd(A, W, keep, ts, 0.7) * dY)
    assert np.isclose(lhs, np.sum(A * C.bwd_input(dY, W, keep, ts, 0.7)))
    assert np.isclose(lhs, np.sum(W * C.bwd_weight(A, dY, keep, ts, 0.7)))
