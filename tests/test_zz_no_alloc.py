"""ard_bwd_data_static_scratch -- the entry point for callers that may not allocate device memory
(frozen memory plan, host application owns the allocator, no device-wide sync allowed) -- must give
what the definition gives (the oracle's masked fp64 product) and what ard_bwd_data gives.  Collected last so that
a failure here cannot hide another test's result.
"""
import numpy as np
import pytest
import torch

from oracle import gemm as OG
from oracle import pattern as OP
from paper_2203_05705_b200 import ard, inputs

pytestmark = pytest.mark.gpu

TOL_BF16 = 5e-3      # the same relative Frobenius bounds the other parity tests use
TOL_F32 = 1e-5


def _rel(a, b):
    a, b = a.double(), b.double()
    return float((a - b).norm() / b.norm())


@pytest.mark.parametrize("dtype", [ard.ARD_BF16, ard.ARD_F32])
@pytest.mark.parametrize("pads", [(0, 0), (8, 16)])
def test_calls_in_a_row_match_the_definition_and_the_allocating_entry_point(dtype, pads):
    B, K, N = 200, 264, 520
    lddy, lddx = N + pads[0], K + pads[1]           # also with rows that do not follow one another in memory
    td = torch.bfloat16 if dtype == ard.ARD_BF16 else torch.float32
    tol = TOL_BF16 if dtype == ard.ARD_BF16 else TOL_F32
    rng = np.random.default_rng(11)
    Wh = inputs.bf16_round((rng.standard_normal((N, K)) * 0.05).astype(np.float32))       # neuron-major
    W = torch.from_numpy(Wh).to(td).cuda()
    ctx = ard.ard_create(0, 2 * B * N + 4096)
    pat = ard.ard_pattern_create(ctx, ard.ARD_ROW, K, N, 0)
    try:
        # different patterns and gradients back to back: every call after the first starts with the previous
        # call's data still in the shared scratch array; (300, 7) keeps two neurons, (520, 520) only the last one
        for call, (dp, b) in enumerate([(3, 2), (1, 1), (5, 5), (300, 7), (520, 520)]):
            dYh = inputs.bf16_round(rng.standard_normal((B, N)).astype(np.float32))
            dY = torch.full((B, lddy), float("nan"), dtype=td, device="cuda")
            dY[:, :N] = torch.from_numpy(dYh).to(td)
            ard.ard_pattern_set(ctx, pat, dp, b)
            ref = torch.full((B, lddx), float("nan"), dtype=td, device="cuda")
            out = torch.full((B, lddx), float("nan"), dtype=td, device="cuda")
            ard.ard_bwd_data(ctx, pat, dtype, B, K, N, 2.0, dY, lddy, 0, W, K, ref, lddx)
            ard.ard_bwd_data_static_scratch(ctx, pat, dtype, B, K, N, 2.0, dY, lddy, W, K, out, lddx)
            torch.cuda.synchronize()
            assert bool(torch.isfinite(out[:, :K]).all()), (call, dp, b)
            assert bool(torch.isnan(out[:, K:]).all()), (call, dp, b)           # nothing written beyond the K columns
            want = OG.bwd_data(dYh, Wh.T, OP.row_mask(N, dp, b), 2.0)            # the definition: masked fp64 product
            err = OG.rel_fro(out[:, :K].double().cpu().numpy(), want)
            assert err <= tol, (call, dp, b, err)
            assert _rel(out[:, :K], ref[:, :K]) <= tol, (call, dp, b, _rel(out[:, :K], ref[:, :K]))
        assert ard.ard_last_device_status(ctx) == 0
    finally:
        torch.cuda.synchronize()
        ard.ard_pattern_destroy(pat)
        ard.ard_destroy(ctx)


def test_sizes_beyond_the_fixed_array_are_refused():
    B, K, N = 4096, 64, 2048                     # 4096 * 2048 * 2 bytes = 16 MiB > 8 MiB
    assert B * N * 2 > ard.ARD_STATIC_SCRATCH_BYTES
    ctx = ard.ard_create(0, 0)
    pat = ard.ard_pattern_create(ctx, ard.ARD_ROW, K, N, 0)
    try:
        dY = torch.zeros((B, N), dtype=torch.bfloat16, device="cuda")
        W = torch.zeros((N, K), dtype=torch.bfloat16, device="cuda")
        dX = torch.zeros((B, K), dtype=torch.bfloat16, device="cuda")
        n0 = ard.ard_launch_count(ctx)
        with pytest.raises(ard.ArdError) as e:
            ard.ard_bwd_data_static_scratch(ctx, pat, ard.ARD_BF16, B, K, N, 1.0, dY, N, W, K, dX, K)
        assert e.value.status == ard.ARD_ERR_NOMEM
        assert ard.ard_launch_count(ctx) == n0     # nothing was launched
        tpat = ard.ard_pattern_create(ctx, ard.ARD_TILE, 64, 2048, 64)
        with pytest.raises(ard.ArdError) as e:      # tile patterns are not covered by this variant
            ard.ard_bwd_data_static_scratch(ctx, tpat, ard.ARD_BF16, 8, K, N, 1.0, dY, N, W, K, dX, K)
        assert e.value.status == ard.ARD_ERR_UNSUPPORTED
        ard.ard_pattern_destroy(tpat)
    finally:
        torch.cuda.synchronize()
        ard.ard_pattern_destroy(pat)
        ard.ard_destroy(ctx)
