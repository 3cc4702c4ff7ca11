"""Stacked LSTM with dropout on the layer outputs only (second reading of the LSTM experiment of Sec. 7): the
compact-matrix GPU path (kept outputs of a layer feed the next layer's input half over both compact operands)
against the oracle's masked full-width stack, end to end over the whole sequence and both layers."""
import numpy as np
import pytest
import torch

from oracle import gemm as OG
from oracle import lstm_stack as OS
from oracle import pattern as OP
from paper_2203_05705_b200 import ard, inputs
from paper_2203_05705_b200.lstm import LstmStack
from gpu_helpers import Ctx, host, TOL

pytestmark = pytest.mark.gpu
BF = torch.bfloat16
TOL_BF16 = TOL[ard.ARD_BF16]


def _bf(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(BF).cuda()


def _run(T, B, dims, dps, alphas, seed):
    rng = np.random.default_rng(seed)
    L = len(dims) - 1
    Ws = [inputs.bf16_round(rng.uniform(-0.03, 0.03, size=(dims[l] + dims[l + 1], 4 * dims[l + 1])).astype(np.float32))
          for l in range(L)]
    X = inputs.bf16_round(rng.standard_normal((T, B, dims[0])).astype(np.float32))
    masks = [OP.row_mask(dims[l + 1], *dps[l]) for l in range(L)]
    keeps = [OP.row_keep(dims[l + 1], *dps[l]) for l in range(L)]
    dY = inputs.bf16_round((rng.standard_normal((T, B, dims[-1])) / 64).astype(np.float32)) * masks[-1][None, None, :]
    ctx = Ctx(2 * T * B * 4 * max(dims) + 4096)
    try:
        stack = LstmStack(ctx.h, T, B, dims, [_bf(W.T) for W in Ws])
        for l in range(L):
            ard.ard_pattern_set(ctx.h, stack.out_pats[l], *dps[l])
        Yc = stack.forward(_bf(X), alphas)
        nk = len(keeps[-1])
        dYc = torch.zeros((T * B, dims[-1]), dtype=BF, device="cuda")
        dYc[:, :nk] = _bf(dY.reshape(T * B, -1)[:, keeps[-1]])
        dYc[:, nk:] = float("nan")                                   # beyond the kept count: must not be read
        dX, dWs = stack.backward(dYc, alphas)
        torch.cuda.synchronize()
        assert ard.ard_last_device_status(ctx.h) == 0
        fw = OS.fwd(X, Ws, None, masks, alphas)
        bw = OS.bwd(fw, Ws, masks, alphas, dY)
        errs = {}
        # the top layer's kept outputs (the GPU holds them unscaled)
        errs["Y"] = OG.rel_fro(alphas[-1] * host(Yc)[:, :nk], fw["Ys"][-1].reshape(T * B, -1)[:, keeps[-1]])
        for l in range(L):
            hs = host(stack.layers[l].XH[1:, :, dims[l]:])
            errs["H%d" % l] = OG.rel_fro(hs, fw["layers"][l]["Hs"])          # every unit is computed, none is masked
            errs["dW%d" % l] = OG.rel_fro(host(dWs[l]), bw["dW"][l].T)
            if l > 0:
                dropped = np.where(masks[l - 1] == 0)[0]
                assert bool(torch.all(dWs[l][:, torch.from_numpy(dropped).cuda()] == 0)), l   # fan-in of dropped units
        errs["dX"] = OG.rel_fro(host(dX), bw["dX"])
        stack.close()
        return errs
    finally:
        ctx.close()


@pytest.mark.parametrize("dps", [((2, 1), (3, 2)), ((5, 5), (1, 1)), ((1, 1), (16, 7))])
def test_two_layers_small(dps):
    errs = _run(6, 24, (64, 128, 128), dps, (1.5, 2.0), 3)
    assert max(errs.values()) <= TOL_BF16, errs


def test_three_layers_small():
    errs = _run(5, 16, (64, 128, 192, 128), ((3, 1), (2, 2), (4, 3)), (1.5, 2.0, 1.25), 4)
    assert max(errs.values()) <= TOL_BF16, errs


@pytest.mark.parametrize("dps,p", [(((2, 2), (4, 1)), 0.5), (((7, 3), (3, 3)), 0.7)])
def test_two_layers_of_1024_units_over_35_steps(dps, p):
    """The size of the paper's LSTM layers (config 4's layer, stacked twice): 2 x 1024 units, T = 35, batch 64."""
    a = 1.0 / (1.0 - p)
    errs = _run(35, 64, (1024, 1024, 1024), dps, (a, a), 5)
    assert max(errs.values()) <= TOL_BF16, errs
