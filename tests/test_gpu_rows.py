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
        for it, (k, t, thr, mp, npb) in enumerate([(0.3, 0.3, 0.5, 0.2, 0.8), (0.05, 0.25, 0.1, 0.0, 1.0), (1.0, 0.4, 0.3, 0.35, 0.65)]):
            ard.ard_sensitivity_predict(ctx.h, rows, dtype, Ad, Kc + 8, Kc, k, t, thr, mp, npb, 99, it, 5)
            ard.ard_rows_sample(ctx.h, rows, 99, it, 5)
            n_keep, idx, P = ard.ard_rows_to_host(rows, M, regions)
            Po, sens = OC.sensitivity_mask(A, x, k, t, thr, mp, npb, 99, it, 5)
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
