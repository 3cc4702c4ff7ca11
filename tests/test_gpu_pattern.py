"""Device sampler vs the oracle: bit-exact (dp, b), kept lists and tile lists."""
import numpy as np
import pytest
import torch

from oracle import pattern as OP
from paper_2203_05705_b200 import ard, inputs
from gpu_helpers import Ctx
from distributions import max_entropy_K

pytestmark = pytest.mark.gpu


@pytest.fixture()
def ctx():
    c = Ctx(0)
    yield c
    c.close()


def test_cdf_table_matches_oracle(ctx):
    for i, (p, n) in enumerate([(0.3, 16), (0.5, 16), (0.7, 16), (0.5, 8)]):
        K = max_entropy_K(p, n)
        ard.ard_set_distribution(ctx.h, i, K)
        assert ard.ard_get_distribution_cdf(ctx.h, i).tolist() == OP.quantise_K(K)
    K = [0.25, 0.0, 0.5, 0.0, 0.25]
    ard.ard_set_distribution(ctx.h, 5, K)
    assert ard.ard_get_distribution_cdf(ctx.h, 5).tolist() == OP.quantise_K(K)


@pytest.mark.parametrize("p,n_dp,N", [(0.5, 8, 256), (0.3, 16, 2048), (0.7, 16, 1000)])
def test_sampled_row_patterns_bit_exact(ctx, p, n_dp, N):
    K = max_entropy_K(p, n_dp)
    cdf = OP.quantise_K(K)
    ard.ard_set_distribution(ctx.h, 0, K)
    pat = ctx.pattern(ard.ARD_ROW, 64, N)
    seen = set()
    for seed, stream_id in [(20220305, 0), (7, 3), ((1 << 40) + 11, 1)]:
        for it in list(range(400)) + [(1 << 32) + 5, (1 << 63) + 1]:
            ard.ard_sample_pattern(ctx.h, pat, 0, seed, it, stream_id)
            dp, b, nk, idx = ard.ard_pattern_to_host(pat, N)
            assert (dp, b) == OP.draw(cdf, seed, it, stream_id)
            keep = OP.row_keep(N, dp, b)
            assert nk == len(keep) and np.array_equal(idx, keep)
            seen.add(dp)
    assert len(seen) >= n_dp // 2


def test_sampler_statistics_many_counters(ctx):
    """10^5 counters: the device histogram of (dp, b) equals the oracle's exactly."""
    p, n_dp, N = 0.5, 16, 64
    K = max_entropy_K(p, n_dp)
    cdf = OP.quantise_K(K)
    ard.ard_set_distribution(ctx.h, 1, K)
    pat = ctx.pattern(ard.ARD_ROW, 8, N)
    S = 3000
    for it in range(S):
        ard.ard_sample_pattern(ctx.h, pat, 1, 99, it, 0)
        dp, b, nk, _ = ard.ard_pattern_to_host(pat, 0)
        assert (dp, b) == OP.draw(cdf, 99, it, 0)


def test_counter_is_stateless(ctx):
    K = max_entropy_K(0.5, 8)
    ard.ard_set_distribution(ctx.h, 2, K)
    pat = ctx.pattern(ard.ARD_ROW, 8, 100)
    ard.ard_sample_pattern(ctx.h, pat, 2, 5, 17, 0)
    first = ard.ard_pattern_to_host(pat, 100)
    for it in (3, 9, 1):
        ard.ard_sample_pattern(ctx.h, pat, 2, 5, it, 0)
    ard.ard_sample_pattern(ctx.h, pat, 2, 5, 17, 0)
    again = ard.ard_pattern_to_host(pat, 100)
    assert first[:3] == again[:3] and np.array_equal(first[3], again[3])


@pytest.mark.parametrize("Kd,Nd,ts", [(24, 40, 4), (4096, 4096, 64), (8192, 8192, 128), (192, 320, 64)])
def test_tile_lists_bit_exact(ctx, Kd, Nd, ts):
    pat = ctx.pattern(ard.ARD_TILE, Kd, Nd, ts)
    Tr, Tc = Kd // ts, Nd // ts
    cases = [(1, 1), (2, 1), (2, 2), (3, 2), (4, 1), (5, 5), (7, 3), (16, 9), (16, 16)]
    for dp, b in cases:
        if dp > Tr * Tc:
            continue
        ard.ard_pattern_set(ctx.h, pat, dp, b)
        gdp, gb, nk, idx = ard.ard_pattern_to_host(pat, Tr * Tc)
        kept = OP.tile_keep(Kd, Nd, ts, dp, b)
        assert (gdp, gb, nk) == (dp, b, len(kept))
        assert np.array_equal(idx, kept[:, 0] * Tc + kept[:, 1])
        cp, ci, rp, ri = ard.ard_pattern_tile_lists_to_host(pat, Tr, Tc)
        ocp, oci, orp, ori = OP.tile_lists(Kd, Nd, ts, dp, b)
        assert np.array_equal(cp, ocp) and np.array_equal(ci, oci)
        assert np.array_equal(rp, orp) and np.array_equal(ri, ori)


def test_sampled_tile_pattern(ctx):
    K = max_entropy_K(0.5, 16)
    cdf = OP.quantise_K(K)
    ard.ard_set_distribution(ctx.h, 3, K)
    pat = ctx.pattern(ard.ARD_TILE, 512, 512, 64)
    for it in range(50):
        ard.ard_sample_pattern(ctx.h, pat, 3, 1, it, 2)
        dp, b, nk, idx = ard.ard_pattern_to_host(pat, 64)
        assert (dp, b) == OP.draw(cdf, 1, it, 2)
        kept = OP.tile_keep(512, 512, 64, dp, b)
        assert np.array_equal(idx, kept[:, 0] * 8 + kept[:, 1])


def test_host_side_rejections(ctx):
    h = ctx.h
    with pytest.raises(ard.ArdError) as e:
        ard.ard_set_distribution(h, 0, [0.5, 0.4])
    assert e.value.status == ard.ARD_ERR_DISTRIBUTION
    with pytest.raises(ard.ArdError):
        ard.ard_set_distribution(h, 0, [1.5, -0.5])
    with pytest.raises(ard.ArdError):
        ard.ard_set_distribution(h, 99, [1.0])
    with pytest.raises(ard.ArdError) as e:
        ard.ard_pattern_create(h, ard.ARD_TILE, 100, 64, 64)
    assert e.value.status == ard.ARD_ERR_SHAPE
    pat = ctx.pattern(ard.ARD_ROW, 8, 4)
    ard.ard_set_distribution(h, 4, max_entropy_K(0.5, 8))
    with pytest.raises(ard.ArdError) as e:                       # more periods than units (dp_max = M)
        ard.ard_sample_pattern(h, pat, 4, 0, 0, 0)
    assert e.value.status == ard.ARD_ERR_DISTRIBUTION
    with pytest.raises(ard.ArdError):
        ard.ard_pattern_set(h, pat, 3, 4)
    with pytest.raises(ard.ArdError) as e:                       # unset distribution
        ard.ard_sample_pattern(h, pat, 9, 0, 0, 0)
    assert e.value.status == ard.ARD_ERR_DISTRIBUTION
    x = torch.zeros((4, 8), device="cuda")
    w = torch.zeros((4, 8), device="cuda")
    y = torch.zeros((4, 4), device="cuda")
    with pytest.raises(ard.ArdError) as e:                       # shape does not match the pattern
        ard.ard_fwd(h, pat, ard.ARD_F32, 4, 16, 4, 1.0, x, 16, w, 16, y, 4, 1)
    assert e.value.status == ard.ARD_ERR_SHAPE
    with pytest.raises(ard.ArdError) as e:                       # ld < extent
        ard.ard_fwd(h, pat, ard.ARD_F32, 4, 8, 4, 1.0, x, 4, w, 8, y, 4, 1)
    assert e.value.status == ard.ARD_ERR_SHAPE
    with pytest.raises(ard.ArdError) as e:
        ard.ard_fwd(h, pat, ard.ARD_F32, 4, 8, 4, 1.0, None, 8, w, 8, y, 4, 1)
    assert e.value.status == ard.ARD_ERR_INVALID_ARG
    assert ard.ard_last_device_status(h) == 0
