"""Pins for oracle/cnn.py (sensitivity prediction and row-based sensitivity-aware dropout, Sec. 5.1 / 5.2.1).

The paper fixes no numbers for this part, so the pins are what the mathematics fixes: the decision rule on
regions whose answer does not depend on the sample (all values above / below the threshold), the binomial law
of the decision for a region with a known fraction above the threshold, the drop rate of the row sampler, the
worked row example of Sec. 5.2.1, the equality of the masked product with the product of the dense small
matrix, brute-force loops and the adjoint identities.
"""
import numpy as np
import pytest
from scipy import stats

from oracle import cnn as C


def test_regions_that_do_not_depend_on_the_sample():
    A = np.zeros((12, 40))
    A[0:4] = 1.0                       # region 0 (x = 4): every value above the threshold
    A[8:12, ::2] = 1.0                 # region 2: exactly half of the values above
    for it in range(5):
        s0, c0, n0 = C.region_sensitive(A, 0, 4, 0.3, 0.5, 0.5, 7, it, 3)
        s1, c1, n1 = C.region_sensitive(A, 1, 4, 0.3, 0.5, 0.5, 7, it, 3)
        assert s0 and c0 == n0 == C.n_samples(0.3, 4, 40) == 48
        assert (not s1) and c1 == 0
    P, sens = C.sensitivity_mask(A, 4, 0.3, 0.5, 0.5, 0.2, 0.8, 7, 0, 3)
    assert sens[0] and not sens[1]
    assert P[0] == C.quantise_probability(0.2) and P[1] == C.quantise_probability(0.8)


def test_ragged_last_region_counts_missing_rows_as_below():
    A = np.ones((5, 16))               # x = 4: region 1 has one real row of four
    fr = []
    for it in range(200):
        _, c, s = C.region_sensitive(A, 1, 4, 0.5, 0.5, 0.5, 1, it, 0)
        fr.append(c / s)
    assert abs(np.mean(fr) - 0.25) < 0.02          # a quarter of the positions exist


def test_default_draws_every_value_on_its_own():
    """Sec. 5.1, step 2 says a random k% of the VALUES: with the default run length the sampled positions are
    independent, so over a region whose values above the threshold sit side by side the count is binomial over
    single values -- not a multiple of a run length, and with the variance of independent draws (a sample taken in
    runs of c neighbours has c times that variance)."""
    x, Kc = 4, 64
    A = np.zeros((x, Kc))
    A[1, 0:32] = 1.0                               # one aligned piece of 32 neighbouring values above
    A[3, 32:64] = 1.0                              # and another
    s = C.n_samples(0.25, x, Kc)
    assert s == C.n_runs(0.25, x, Kc) == 64        # run_len = 1: a run is one value
    f = 64 / (x * Kc)
    res = np.array([C.region_sensitive(A, 0, x, 0.25, 0.5, 0.5, 3, it, 0)[1] for it in range(1200)])
    assert np.any(res % 2 == 1) and len(set(res.tolist())) > 8
    assert abs(res.mean() - s * f) < 4 * np.sqrt(s * f * (1 - f) / 1200)
    assert abs(res.var() - s * f * (1 - f)) < 0.2 * s * f * (1 - f)
    # two neighbouring positions are hit independently: P(both looked at) = P(one)^2 for single draws
    B = np.zeros((x, Kc))
    B[2, 10] = B[2, 11] = 1.0
    one = 1 - (1 - 1 / (x * Kc)) ** s              # a given position is looked at at least once
    both = 1 - 2 * (1 - 1 / (x * Kc)) ** s + (1 - 2 / (x * Kc)) ** s
    cnt = np.array([C.region_sensitive(B, 0, x, 0.25, 0.5, 0.5, 9, it, 1)[1] for it in range(3000)])
    B[2, 11] = 0.0
    cnt_one = np.array([C.region_sensitive(B, 0, x, 0.25, 0.5, 0.5, 9, it, 1)[1] for it in range(3000)])
    B[2, 10], B[2, 11] = 0.0, 1.0
    cnt_other = np.array([C.region_sensitive(B, 0, x, 0.25, 0.5, 0.5, 9, it, 1)[1] for it in range(3000)])
    p_both = np.mean((cnt_one > 0) & (cnt_other > 0))
    assert abs(np.mean(cnt_one > 0) - one) < 4 * np.sqrt(one * (1 - one) / 3000)
    assert abs(p_both - both) < 4 * np.sqrt(both * (1 - both) / 3000) + 2e-3   # runs of neighbours: p_both = one
    assert np.array_equal(cnt, cnt_one + cnt_other)                              # same positions, whatever A holds


def test_threshold_count_is_exact():
    # ceil(t * s) with the product taken exactly: 0.3 (a little below 3/10 as a double) of 10 samples needs 3,
    # 0.1 (a little above 1/10) of 10 needs 2, a half of 7 needs 4, and at least one value is always needed
    assert C.needed(0.3, 10) == 3 and C.needed(0.1, 10) == 2 and C.needed(0.5, 7) == 4 and C.needed(0.5, 8) == 4
    assert C.needed(0.0, 100) == 1 and C.needed(1.0, 100) == 100 and C.needed(0.25, 1 << 30) == 1 << 28


def test_decision_follows_the_binomial_law_over_runs():
    # the opt-in run form: whole runs (32 neighbouring values of a row) above or below the threshold: the count is
    # 32 times a binomial variable over the drawn runs
    rng = np.random.default_rng(0)
    x, Kc = 8, 64
    assert C.transaction_run(Kc) == 32 and C.transaction_run(200) == 8 and C.transaction_run(33) == 1
    above = np.zeros(16, dtype=bool)
    above[rng.choice(16, 6, replace=False)] = True
    A = np.repeat(above.reshape(x, 2), 32, axis=1).astype(np.float64)
    n_c = C.n_runs(0.5, x, Kc, 32)
    s = C.n_samples(0.5, x, Kc, 32)
    assert n_c == 8 and s == 256
    need_runs = -(-C.needed(0.5, s) // 32)
    res = [C.region_sensitive(A, 0, x, 0.5, 0.5, 0.5, 11, it, 0, run_len=32) for it in range(1500)]
    assert all(c % 32 == 0 and n == s for _, c, n in res)
    hits = sum(r[0] for r in res)
    p_theory = stats.binom.sf(need_runs - 1, n_c, 6 / 16)
    sd = np.sqrt(p_theory * (1 - p_theory) / 1500)
    assert abs(hits / 1500 - p_theory) < 4 * sd + 1e-3
    mean_runs = np.mean([c for _, c, _ in res]) / 32
    assert abs(mean_runs - n_c * 6 / 16) < 4 * np.sqrt(n_c * (6 / 16) * (10 / 16) / 1500)


def test_runs_are_drawn_uniformly_and_stay_in_their_region():
    x, Kc = 2, 16                                  # runs of 16: a run is a whole row; region 1 = rows 2, 3
    n_c = C.n_runs(1.0, x, Kc, 16)
    assert n_c == 2
    hits = np.zeros(6)
    for r in range(6):
        A = np.zeros((6, Kc))
        A[r] = 1.0
        hits[r] = sum(C.region_sensitive(A, 1, x, 1.0, 0.5, 0.5, 5, it, 1, run_len=16)[1] for it in range(400)) / 16
    assert hits[0] == hits[1] == hits[4] == hits[5] == 0          # other regions' rows are never looked at
    expect = 400 * n_c / 2
    assert np.all(np.abs(hits[2:4] - expect) < 4.5 * np.sqrt(expect / 2))


def test_row_sampler_rates_and_extremes():
    M, x = 4000, 8
    P = np.array([C.quantise_probability(0.2), C.quantise_probability(0.8)] * (M // x // 2), dtype=np.uint64)
    keep = C.draw_rows(P, x, M, 5, 9, 2)
    m = C.row_mask(M, keep).reshape(-1, x)
    low, high = 1 - m[0::2].mean(), 1 - m[1::2].mean()
    assert abs(low - 0.2) < 4 * np.sqrt(0.2 * 0.8 / (M / 2)) and abs(high - 0.8) < 4 * np.sqrt(0.2 * 0.8 / (M / 2))
    assert np.all(np.diff(keep) > 0)
    assert len(C.draw_rows(np.zeros(M // x, dtype=np.uint64), x, M, 5, 9, 2)) == M      # probability 0: nothing dropped
    assert len(C.draw_rows(np.full(M // x, C.quantise_probability(1.0), dtype=np.uint64), x, M, 5, 9, 2)) <= 1
    # a pure function of (seed, iteration, stream): same draw twice, different draw for another iteration
    assert np.array_equal(keep, C.draw_rows(P, x, M, 5, 9, 2))
    assert not np.array_equal(keep, C.draw_rows(P, x, M, 5, 10, 2))


def test_worked_row_example_and_the_dense_small_matrix():
    """Sec. 5.2.1: six rows, the second, fifth and sixth dropped; the kept rows fill the same rows of Y."""
    rng = np.random.default_rng(3)
    A, W = rng.standard_normal((6, 9)), rng.standard_normal((9, 4))
    keep = np.array([0, 2, 3])
    Y = C.fwd(A, W, keep, 1.5)
    assert np.all(Y[[1, 4, 5]] == 0)
    np.testing.assert_allclose(Y[keep], 1.5 * A[keep] @ W, rtol=1e-13)
    np.testing.assert_allclose(Y, C.fwd_compact(A, W, keep, 1.5), rtol=1e-13, atol=1e-15)
    # brute force
    for r in range(6):
        for n in range(4):
            ref = 1.5 * sum(A[r, k] * W[k, n] for k in range(9)) if r in keep else 0.0
            assert abs(Y[r, n] - ref) < 1e-12


def test_backward_products_are_the_adjoints():
    rng = np.random.default_rng(4)
    M, Kc, N = 17, 11, 7
    A, W, dY = rng.standard_normal((M, Kc)), rng.standard_normal((Kc, N)), rng.standard_normal((M, N))
    keep = np.array([1, 2, 5, 9, 16])
    lhs = float((C.fwd(A, W, keep, 1.3) * dY).sum())
    assert abs(lhs - float((A * C.bwd_data(dY, W, keep, 1.3)).sum())) < 1e-10
    assert abs(lhs - float((W * C.bwd_weight(A, dY, keep, 1.3)).sum())) < 1e-10
    dropped = np.setdiff1d(np.arange(M), keep)
    assert np.all(C.bwd_data(dY, W, keep)[dropped] == 0)
    np.testing.assert_allclose(C.bwd_weight(A, dY, keep, 1.0), A[keep].T @ dY[keep], rtol=1e-12, atol=1e-13)
