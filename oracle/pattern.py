"""Dropout-pattern oracle: distribution K -> (dp, b) -> kept units -> 0/1 mask.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  Pure Python integers and
numpy; every function names the passage of the paper it restates.
"""
from __future__ import annotations

import numpy as np

TWO32 = 1 << 32
MASK32 = TWO32 - 1

# ---------------------------------------------------------------------------
# Counter-based generator.  The paper (Sec. 3.4) does not name a generator;
# both sides of the parity test implement the published Philox4x32-10
# generator (Salmon et al., SC'11) so that draws can be compared bit for bit.
# ---------------------------------------------------------------------------
_PHILOX_M0 = 0xD2511F53
_PHILOX_M1 = 0xCD9E8D57
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85


def philox4x32_10(counter, key):
    """One block of Philox4x32 with 10 rounds.  counter: 4 words, key: 2 words."""
    c0, c1, c2, c3 = (int(x) & MASK32 for x in counter)
    k0, k1 = (int(x) & MASK32 for x in key)
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _PHILOX_W0) & MASK32
            k1 = (k1 + _PHILOX_W1) & MASK32
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> 32, p0 & MASK32
        hi1, lo1 = p1 >> 32, p1 & MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & MASK32, lo1, (hi0 ^ c3 ^ k1) & MASK32, lo0
    return c0, c1, c2, c3


# ---------------------------------------------------------------------------
# Sec. 3.3: K = {k_i}, i = 1..dp_max, sum k_i = 1.
# ---------------------------------------------------------------------------
def quantise_K(K):
    """Integer CDF of K on a 2^32 grid.

    The paper gives K as real probabilities summing to one (Sec. 3.3) and is
    silent on representation.  Reading: sequential fp64 prefix sums s_i, then
    c_i = floor(s_i * 2^32 + 1/2) clamped to [c_{i-1}, 2^32], c_last = 2^32.
    The quantised k_i = (c_i - c_{i-1}) / 2^32 sum to one exactly.
    """
    K = [float(k) for k in K]
    if len(K) == 0 or any((k < 0.0) or (k != k) for k in K):
        raise ValueError("K must be non-empty and non-negative")
    s = 0.0
    for k in K:
        s += k
    if abs(s - 1.0) > 1e-9:
        raise ValueError("K must sum to 1")
    cdf = []
    s = 0.0
    prev = 0
    for i, k in enumerate(K):
        s += k
        if i == len(K) - 1:
            c = TWO32
        else:
            c = int(np.floor(s * 4294967296.0 + 0.5))
            c = min(max(c, prev), TWO32)
        cdf.append(c)
        prev = c
    return cdf


def quantised_probabilities(cdf):
    """k_i actually realised by the integer CDF, as exact fractions of 2^32."""
    out, prev = [], 0
    for c in cdf:
        out.append(c - prev)
        prev = c
    return out


def draw(cdf, seed, iteration, stream_id):
    """Sec. 3.4: sample dp subject to K, then b uniformly from {1..dp}.

    Randomness: Philox4x32-10 with key = (seed low, seed high) and
    counter = (iteration low, iteration high, stream_id, 0).  Word 0 picks dp
    as the smallest i with r0 < c_i; word 1 picks b = 1 + floor(r1 * dp / 2^32).
    """
    seed = int(seed)
    iteration = int(iteration)
    r = philox4x32_10(
        (iteration & MASK32, (iteration >> 32) & MASK32, int(stream_id) & MASK32, 0),
        (seed & MASK32, (seed >> 32) & MASK32),
    )
    dp = 1
    for c in cdf:
        if r[0] < c:
            break
        dp += 1
    b = 1 + ((r[1] * dp) >> 32)
    return dp, b


# ---------------------------------------------------------------------------
# Sec. 3.1, Eq. 1: drop every row whose 1-based index i has (i - b) mod dp != 0.
# ---------------------------------------------------------------------------
def row_keep(n_units, dp, b):
    """Ascending 0-based indices of the kept units among n_units."""
    if not (1 <= b <= dp):
        raise ValueError("b must lie in 1..dp")
    if dp > n_units:
        raise ValueError("dp may not exceed the number of units (Sec. 3.1: dp_max = M)")
    return np.array([i - 1 for i in range(1, n_units + 1) if (i - b) % dp == 0], dtype=np.int32)


def row_mask(n_units, dp, b):
    """0/1 vector, 1 = keep (mask convention of Sec. 6)."""
    m = np.zeros(n_units, dtype=np.float64)
    m[row_keep(n_units, dp, b)] = 1.0
    return m


# ---------------------------------------------------------------------------
# Sec. 3.2: the same (dp, b) rule over weight tiles: out of each run of dp
# consecutive tiles only one survives.  The weight is taken in its math orientation
# W[K x N] (Y = X W); tile (r, c) covers rows r*ts.. and columns c*ts..; tiles
# are numbered row-major from 1: t = r*Tc + c + 1.
# ---------------------------------------------------------------------------
def tile_keep(K_dim, N_dim, ts, dp, b):
    """Kept tiles as an int32 array of (r, c) pairs in ascending t."""
    if ts <= 0 or K_dim % ts or N_dim % ts:
        raise ValueError("tile size must divide both weight dimensions")
    if not (1 <= b <= dp):
        raise ValueError("b must lie in 1..dp")
    Tr, Tc = K_dim // ts, N_dim // ts
    if dp > Tr * Tc:
        raise ValueError("dp may not exceed the number of tiles (Sec. 3.2: dp_max)")
    out = []
    for t in range(1, Tr * Tc + 1):
        if (t - b) % dp == 0:
            out.append(((t - 1) // Tc, (t - 1) % Tc))
    return np.array(out, dtype=np.int32).reshape(-1, 2)


def tile_mask(K_dim, N_dim, ts, dp, b):
    """Dense 0/1 mask [K x N] of the kept synapses."""
    M = np.zeros((K_dim, N_dim), dtype=np.float64)
    for r, c in tile_keep(K_dim, N_dim, ts, dp, b):
        M[r * ts:(r + 1) * ts, c * ts:(c + 1) * ts] = 1.0
    return M


def tile_lists(K_dim, N_dim, ts, dp, b):
    """The kept tiles grouped by tile-column (rows ascending) and by tile-row
    (columns ascending), in compressed pointer/index form."""
    Tr, Tc = K_dim // ts, N_dim // ts
    kept = tile_keep(K_dim, N_dim, ts, dp, b)
    col_ptr = np.zeros(Tc + 1, dtype=np.int32)
    row_ptr = np.zeros(Tr + 1, dtype=np.int32)
    by_col = [[] for _ in range(Tc)]
    by_row = [[] for _ in range(Tr)]
    for r, c in kept:
        by_col[c].append(int(r))
        by_row[r].append(int(c))
    col_idx, row_idx = [], []
    for c in range(Tc):
        col_idx += sorted(by_col[c])
        col_ptr[c + 1] = len(col_idx)
    for r in range(Tr):
        row_idx += sorted(by_row[r])
        row_ptr[r + 1] = len(row_idx)
    return (col_ptr, np.array(col_idx, dtype=np.int32),
            row_ptr, np.array(row_idx, dtype=np.int32))


# ---------------------------------------------------------------------------
# Sec. 3.4, Eq. 2-3: per-unit drop probability and global dropout rate of K.
# ---------------------------------------------------------------------------
def global_dropout_rate(K):
    """p_g = sum_i k_i (i-1)/i  (Eq. 3)."""
    return sum(float(k) * (i - 1) / i for i, k in enumerate(K, start=1))
