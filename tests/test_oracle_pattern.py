"""Pins for oracle/pattern.py against what the paper and the mathematics fix."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import pattern as P
from paper_2203_05705_b200 import inputs
from distributions import max_entropy_K

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_philox_known_answers():
    with open(os.path.join(GOLD, "philox4x32_10_kat.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        ctr = [int(x, 16) for x in r[0:4]]
        key = [int(x, 16) for x in r[4:6]]
        out = [int(x, 16) for x in r[6:10]]
        assert list(P.philox4x32_10(ctr, key)) == out


def _paper_examples():
    """tests/golden/paper_examples.txt: the kept units the paper's worked examples name."""
    out = []
    with open(os.path.join(GOLD, "paper_examples.txt")) as f:
        for line in f:
            if not line.strip() or line.startswith("#"):
                continue
            head, tail = line.split("->")
            out.append((head.split(), tail))
    return out


def test_paper_worked_examples():
    seen = set()
    for head, tail in _paper_examples():
        kind = head[0]
        seen.add(kind)
        if kind == "row":        # Sec. 3.1: dp = 3, b = 1 keeps rows 1, 4, 7 (1-based)
            dp, b, units = int(head[1]), int(head[2]), int(head[3])
            assert (P.row_keep(units, dp, b) + 1).tolist() == [int(x) for x in tail.split()]
            assert (np.flatnonzero(P.row_mask(units, dp, b)) + 1).tolist() == [int(x) for x in tail.split()]
        elif kind == "tile":     # Sec. 3.2: dp = 4, b = 1 keeps tiles 1, 5, 9, 13 of a grid numbered row-major from 1
            dp, b, units = int(head[1]), int(head[2]), int(head[3])
            g = int(round(units ** 0.5))
            kept = P.tile_keep(g * 2, g * 2, 2, dp, b)          # g x g grid of 2 x 2 tiles
            assert (kept[:, 0] * g + kept[:, 1] + 1).tolist() == [int(x) for x in tail.split()]
            M = P.tile_mask(g * 2, g * 2, 2, dp, b)
            assert M.sum() == (g * 2) ** 2 / dp                  # a quarter of the synapses survive
            # the mask is 1 exactly on the kept tiles
            want = np.zeros((g, g))
            want[kept[:, 0], kept[:, 1]] = 1
            assert np.array_equal(M, np.kron(want, np.ones((2, 2))))
        elif kind == "mask":     # Sec. 6: the mask has 1 where a row is KEPT (six rows, rows 1, 3, 4 kept)
            units = int(head[1])
            bits, rows = tail.split(":")
            bits = [int(x) for x in bits.split()]
            rows = [int(x) for x in rows.split()]
            assert len(bits) == units and [i + 1 for i, v in enumerate(bits) if v == 1] == rows
            # the oracle's masks follow that convention: ones at the kept units, and only there
            for dp, b in [(2, 1), (3, 2), (6, 6)]:
                m = P.row_mask(units, dp, b)
                assert set(m.tolist()) <= {0.0, 1.0}
                assert (np.flatnonzero(m == 1)).tolist() == P.row_keep(units, dp, b).tolist()
    assert seen == {"row", "tile", "mask"}


@pytest.mark.parametrize("N", [12, 256, 257, 1000])
def test_row_keep_counts(N):
    for dp in range(1, min(N, 16) + 1):
        total = 0
        for b in range(1, dp + 1):
            keep = P.row_keep(N, dp, b)
            assert len(keep) == (N - b) // dp + 1
            assert keep[0] == b - 1 and np.all(np.diff(keep) == dp)
            assert P.row_mask(N, dp, b).sum() == len(keep)
            if N % dp == 0:
                assert len(keep) * dp == N                # kept fraction exactly 1/dp
            total += len(keep)
        assert total == N                                 # every unit kept for exactly one bias


def test_tile_keep_counts_and_lists():
    K_dim, N_dim, ts = 24, 40, 4                          # 6 x 10 grid
    for dp in range(1, 13):
        tot = np.zeros((K_dim, N_dim))
        for b in range(1, dp + 1):
            M = P.tile_mask(K_dim, N_dim, ts, dp, b)
            tot += M
            kept = P.tile_keep(K_dim, N_dim, ts, dp, b)
            assert len(kept) == (60 - b) // dp + 1
            cp, ci, rp, ri = P.tile_lists(K_dim, N_dim, ts, dp, b)
            assert cp[-1] == rp[-1] == len(kept)
            S = set(map(tuple, kept.tolist()))
            assert {(int(r), c) for c in range(10) for r in ci[cp[c]:cp[c + 1]]} == S
            assert {(r, int(c)) for r in range(6) for c in ri[rp[r]:rp[r + 1]]} == S
            # blocks are constant
            assert np.all(M.reshape(6, ts, 10, ts).std(axis=(1, 3)) == 0)
        assert np.all(tot == 1)


def test_reject_bad_parameters():
    with pytest.raises(ValueError):
        P.row_keep(10, 3, 4)
    with pytest.raises(ValueError):
        P.row_keep(4, 5, 1)                               # dp_max = M (Sec. 3.1)
    with pytest.raises(ValueError):
        P.tile_keep(10, 8, 4, 2, 1)
    with pytest.raises(ValueError):
        P.quantise_K([0.5, 0.4])
    with pytest.raises(ValueError):
        P.quantise_K([1.5, -0.5])


def test_quantise_sums_to_one_and_zero_entries_never_drawn():
    K = [0.25, 0.0, 0.5, 0.0, 0.25]
    cdf = P.quantise_K(K)
    q = P.quantised_probabilities(cdf)
    assert sum(q) == 1 << 32 and cdf[-1] == 1 << 32      # sum k_i = 1 (Sec. 3.3), exactly
    assert q[1] == 0 and q[3] == 0
    seen = {P.draw(cdf, 7, it, 0)[0] for it in range(3000)}
    assert seen == {1, 3, 5}
    for p, n in [(0.3, 16), (0.5, 16), (0.7, 16), (0.5, 8)]:
        k = max_entropy_K(p, n)
        q = P.quantised_probabilities(P.quantise_K(k))
        assert sum(q) == 1 << 32
        assert max(abs(qi / 2**32 - ki) for qi, ki in zip(q, k)) < 2**-31
        assert abs(P.global_dropout_rate([qi / 2**32 for qi in q]) - p) < 1e-6


def test_draw_extremes_of_the_cdf():
    # r0 < c_1 -> dp = 1; the comparison is strict and done in 64 bits
    cdf = P.quantise_K([0.5, 0.5])
    assert cdf == [1 << 31, 1 << 32]
    # cover both branches over many counters
    dps = [P.draw(cdf, 1, it, 3)[0] for it in range(2000)]
    assert set(dps) == {1, 2} and abs(dps.count(1) / 2000 - 0.5) < 0.06


def test_exact_per_unit_drop_probability_equals_global_rate():
    """Eq. 2-3 as an exact identity in rationals: for every unit i,
    sum_dp k_dp * #{b : unit dropped}/dp == sum_dp k_dp (dp-1)/dp, for any N."""
    for N in (10, 37):
        K = max_entropy_K(0.5, 8)
        q = P.quantised_probabilities(P.quantise_K(K))
        pg = sum(Fraction(qi, 1 << 32) * Fraction(dp - 1, dp) for dp, qi in enumerate(q, 1))
        for i in range(N):
            pn = Fraction(0)
            for dp, qi in enumerate(q, 1):
                dropped = sum(1 for b in range(1, dp + 1) if P.row_mask(N, dp, b)[i] == 0)
                pn += Fraction(qi, 1 << 32) * Fraction(dropped, dp)
            assert pn == pg


def test_monte_carlo_matches_bernoulli_rate():
    """Sampler end to end: empirical per-neuron drop rate -> target p; dp ~ K; b | dp uniform."""
    p, n_dp, N, S = 0.5, 8, 64, 20000
    K = max_entropy_K(p, n_dp)
    cdf = P.quantise_K(K)
    drops = np.zeros(N)
    hist = np.zeros(n_dp + 1)
    bh = {dp: np.zeros(dp) for dp in range(1, n_dp + 1)}
    for it in range(S):
        dp, b = P.draw(cdf, 20220305, it, 0)
        assert 1 <= b <= dp <= n_dp
        hist[dp] += 1
        bh[dp][b - 1] += 1
        drops += 1.0 - P.row_mask(N, dp, b)
    tol = 5.0 * np.sqrt(p * (1 - p) / S)
    assert np.max(np.abs(drops / S - p)) < tol
    expect = np.array(K) * S
    chi2 = float(((hist[1:] - expect) ** 2 / expect).sum())
    assert chi2 < 30.0                                   # 7 dof, p ~ 1e-4
    for dp in range(2, n_dp + 1):
        e = hist[dp] / dp
        assert float(((bh[dp] - e) ** 2 / e).sum()) < 12.0 + 3.5 * dp


def test_draw_is_a_pure_function_of_the_counter():
    cdf = P.quantise_K(max_entropy_K(0.3, 16))
    a = [P.draw(cdf, 5, it, 2) for it in range(50)]
    b = [P.draw(cdf, 5, it, 2) for it in reversed(range(50))][::-1]
    assert a == b
    assert [P.draw(cdf, 5, it, 3) for it in range(50)] != a
    assert [P.draw(cdf, 6, it, 2) for it in range(50)] != a


def test_golden_patterns_file_is_current():
    with open(os.path.join(GOLD, "oracle_patterns.txt")) as f:
        lines = f.read().splitlines()
    cdf = [int(x) for x in lines[1].split("=")[1].split()]
    for l in lines[3:]:
        lhs, rhs = l.split("->")
        seed, it, stream = (int(x) for x in lhs.split())
        assert P.draw(cdf, seed, it, stream) == tuple(int(x) for x in rhs.split())
