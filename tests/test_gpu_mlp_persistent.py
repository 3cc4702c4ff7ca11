"""The whole iteration of a small stack in one cooperative kernel (ard_mlp_step, batch <= 128, narrow output layer).

Every stage is graded against the fp64 oracle (oracle/mlp.py) on the operands the GPU consumed, for stacks of one,
two and three hidden layers, ragged batches, forced patterns of every kind (dense, small and large periods, every
offset position), fp32 and bf16 gradients, with and without biases / ReLU / input gradient.  The call-by-call path
(ARD_OPT_MLP_PERSISTENT = 0) must draw the same patterns and give the same results up to bf16 rounding; calls the
kernel cannot take must fall back without a trace.
"""
import numpy as np
import pytest
import torch

from oracle import gemm as OG
from oracle import mlp as OM
from oracle import pattern as OP
from paper_2203_05705_b200 import ard, inputs
from gpu_helpers import Ctx, host, TOL
from distributions import max_entropy_K

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


def _stack(ctx, dims, B, rng, f32_grads=True, bias=True, relu=True, alpha=2.0, sample=0):
    L = len(dims) - 1
    Ws = [inputs.bf16_round((rng.standard_normal((dims[l], dims[l + 1])) * np.sqrt(2.0 / dims[l])).astype(np.float32))
          for l in range(L)]
    bs = [rng.uniform(-0.1, 0.1, dims[l + 1]).astype(np.float32) for l in range(L)]
    gd = torch.float32 if f32_grads else BF
    layers = []
    for l in range(L):
        K, N = dims[l], dims[l + 1]
        hidden = l < L - 1
        layers.append(dict(
            K=K, N=N, pat=ctx.pattern(ard.ARD_ROW, K, N), sample=sample if hidden else 0, relu=1 if (hidden and relu) else 0,
            compact_out=1 if hidden else 0, dW_is_f32=1 if f32_grads else 0, alpha=alpha if hidden else 1.0, ldw=K,
            W=torch.from_numpy(np.ascontiguousarray(Ws[l].T)).to(BF).cuda(),
            bias=torch.from_numpy(bs[l]).cuda() if bias else None,
            Wk=torch.full((N, K), float("nan"), dtype=BF, device="cuda"),
            A=torch.full((B, N), float("nan"), dtype=BF, device="cuda"),
            dZ=torch.full((B, N), float("nan"), dtype=BF, device="cuda"),
            dWk=torch.full((N, K), float("nan"), dtype=gd, device="cuda"),
            dW=torch.full((N, K), float("nan"), dtype=gd, device="cuda"),
            db=torch.full((N,), float("nan"), dtype=torch.float32, device="cuda")))
    ard.ard_pattern_set(ctx.h, layers[-1]["pat"], 1, 1)
    return layers, ard.mlp_layers(layers), Ws, (bs if bias else None)


def _check_against_oracle(layers, Ws, bs, pats, X, dOut, dX, B, relu, with_dx, tol):
    L = len(layers)
    dims = [layers[0]["K"]] + [d["N"] for d in layers]
    keeps = [OP.row_keep(dims[l + 1], *pats[l]) for l in range(L)]
    masks = [OP.row_mask(dims[l + 1], *pats[l]) for l in range(L)]
    alphas = [d["alpha"] for d in layers]

    def full(l, t):
        h = host(t)
        if not layers[l]["compact_out"]:
            return h
        out = np.zeros_like(h)
        out[:, keeps[l]] = h[:, :len(keeps[l])]
        return out

    a_prev = X.astype(np.float64)
    acts = [a_prev]
    for l in range(L):
        _, ref = OM.layer_fwd(a_prev, Ws[l], None if bs is None else bs[l], masks[l], alphas[l], relu=(relu and l < L - 1))
        got = full(l, layers[l]["A"])
        assert OG.rel_fro(got, ref) <= tol, ("fwd", l, pats)
        assert np.all(got[:, masks[l] == 0] == 0)
        a_prev = got
        acts.append(got)
    dz = dOut.astype(np.float64)
    for l in range(L - 1, -1, -1):
        dW_ref = acts[l].T @ dz
        dW = host(layers[l]["dW"])
        assert OG.rel_fro(dW, dW_ref.T) <= tol, ("dW", l, pats)
        assert np.all(dW[masks[l] == 0, :] == 0), ("dW rows of dropped neurons", l, pats)
        if l > 0:
            assert np.all(dW[:, masks[l - 1] == 0] == 0), ("dW columns of dropped inputs", l, pats)
        db_ref = dz.sum(axis=0)
        assert np.abs(host(layers[l]["db"]) - db_ref).max() <= tol * max(1.0, np.abs(db_ref).max()), ("db", l, pats)
        dA = dz @ Ws[l].T.astype(np.float64)
        if l > 0:
            gate = (acts[l] > 0) if relu else 1.0
            ref = alphas[l - 1] * dA * masks[l - 1][None, :] * gate
            got = full(l - 1, layers[l - 1]["dZ"])
            assert OG.rel_fro(got, ref) <= tol, ("dZ", l - 1, pats)
            dz = got
        elif with_dx:
            assert OG.rel_fro(host(dX), dA) <= tol, ("dX", pats)


CASES = [
    # dims, batch, patterns of the hidden layers, fp32 gradients, bias, relu, input gradient
    ([784, 2048, 2048, 10], 128, [(1, 1), (1, 1)], True, True, True, True),
    ([784, 2048, 2048, 10], 128, [(2, 2), (3, 1)], True, True, True, True),
    ([784, 2048, 2048, 10], 128, [(16, 16), (5, 3)], False, True, True, False),
    ([784, 2048, 2048, 10], 100, [(7, 4), (16, 1)], True, False, True, True),
    ([264, 512, 16], 77, [(3, 2)], True, True, True, True),             # one hidden layer, ragged batch
    ([264, 512, 16], 128, [(1, 1)], False, True, False, True),
    ([328, 1024, 512, 256, 10], 64, [(2, 1), (1, 1), (4, 4)], True, True, True, True),   # three hidden layers
    ([328, 1024, 512, 256, 10], 9, [(5, 5), (3, 1), (2, 2)], False, False, True, False),
    ([784, 4096, 1024, 10], 128, [(1, 1), (2, 1)], True, True, True, True),   # 32-wide forward tiles
    ([64, 64, 2], 1, [(1, 1)], True, True, True, True),                       # the smallest stack, one batch row
    ([72, 128, 64, 16], 128, [(16, 7), (13, 13)], False, True, True, True),   # a handful of kept neurons per layer
    ([1024, 4096, 4096, 8], 31, [(3, 3), (2, 2)], True, True, True, False),   # the widest layers the tile lists take
]


@pytest.mark.parametrize("dims,B,pats,f32,bias,relu,with_dx", CASES)
def test_forced_patterns_match_the_oracle_and_the_call_by_call_path(dims, B, pats, f32, bias, relu, with_dx):
    rng = np.random.default_rng(sum(dims) + B)
    tol = TOL[ard.ARD_BF16]
    L = len(dims) - 1
    X = inputs.bf16_round(rng.random((B, dims[0])).astype(np.float32))
    dOut = inputs.bf16_round((rng.standard_normal((B, dims[-1])) / B).astype(np.float32))
    results = []
    for persistent in (1, 0):
        ctx = Ctx(2 * B * max(dims) + 4096)
        try:
            ard.ard_set_option(ctx.h, ard.ARD_OPT_MLP_PERSISTENT, persistent)
            layers, arr, Ws, bs = _stack(ctx, dims, B, np.random.default_rng(5), f32_grads=f32, bias=bias, relu=relu)
            for l in range(L - 1):
                ard.ard_pattern_set(ctx.h, layers[l]["pat"], *pats[l])
            Xd, dOd = torch.from_numpy(X).to(BF).cuda(), torch.from_numpy(dOut).to(BF).cuda()
            dX = torch.full((B, dims[0]), float("nan"), dtype=BF, device="cuda") if with_dx else None
            counter = torch.zeros(1, dtype=torch.int64, device="cuda")
            n0 = ard.ard_launch_count(ctx.h)
            ard.ard_mlp_step(ctx.h, arr, L, B, Xd, dims[0], dOd, dims[-1], dX, dims[0], 0, inputs.BASE_SEED, 7, counter)
            torch.cuda.synchronize()
            assert ard.ard_last_device_status(ctx.h) == 0
            launches = ard.ard_launch_count(ctx.h) - n0
            assert (launches == 1) if persistent else (launches > 4), launches
            _check_against_oracle(layers, Ws, bs, pats + [(1, 1)], X, dOut, dX, B, relu, with_dx, tol)
            n_keep = [len(OP.row_keep(dims[l + 1], *pats[l])) for l in range(L - 1)]
            results.append(dict(
                A=[host(layers[l]["A"])[:, :n_keep[l]] for l in range(L - 1)] + [host(layers[-1]["A"])],
                dZ=[host(layers[l]["dZ"])[:, :n_keep[l]] for l in range(L - 1)],
                dW=[host(d["dW"]) for d in layers], db=[host(d["db"]) for d in layers],
                dX=host(dX) if with_dx else None))
        finally:
            ctx.close()
    one, many = results
    # same operands, fp32 accumulation in another order, bf16 activations in between: equal up to a few roundings
    for key in ("A", "dZ", "dW", "db"):
        for a, c in zip(one[key], many[key]):
            assert OG.rel_fro(a, c) <= 2e-2, key
    if with_dx:
        assert OG.rel_fro(one["dX"], many["dX"]) <= 2e-2


def test_sampled_patterns_follow_the_counter_and_leave_the_lists_of_the_sampler():
    """Patterns drawn inside the kernel: the oracle's draw for (seed, iteration, layer), headers and kept lists as
    the sampler kernel writes them, the counter advanced once per call, the same bits at every repetition."""
    dims, B, p = [784, 2048, 2048, 10], 128, 0.5
    rng = np.random.default_rng(3)
    Kd = max_entropy_K(p, 16)
    cdf = OP.quantise_K(Kd)
    ctx = Ctx(4096)
    try:
        ard.ard_set_distribution(ctx.h, 0, Kd)
        layers, arr, Ws, bs = _stack(ctx, dims, B, rng, sample=1)
        L = len(layers)
        X, dOut = inputs.config2_step(1)
        Xd, dOd = torch.from_numpy(X).to(BF).cuda(), torch.from_numpy(dOut).to(BF).cuda()
        dX = torch.zeros((B, dims[0]), dtype=BF, device="cuda")
        counter = torch.zeros(1, dtype=torch.int64, device="cuda")
        seen = set()
        for step in range(12):
            n0 = ard.ard_launch_count(ctx.h)
            ard.ard_mlp_step(ctx.h, arr, L, B, Xd, dims[0], dOd, dims[-1], dX, dims[0], 0, inputs.BASE_SEED, 300, counter)
            torch.cuda.synchronize()
            assert ard.ard_launch_count(ctx.h) - n0 == 1
            assert ard.ard_last_device_status(ctx.h) == 0
            assert int(counter.item()) == step + 1
            pats = [OP.draw(cdf, inputs.BASE_SEED, 300 + step, l + 1) for l in range(L - 1)]
            for l in range(L - 1):
                dp, b, nk, idx = ard.ard_pattern_to_host(layers[l]["pat"], dims[l + 1])
                assert (dp, b) == pats[l]
                assert np.array_equal(np.asarray(idx), OP.row_keep(dims[l + 1], dp, b))
            seen.add(tuple(pats))
            _check_against_oracle(layers, Ws, bs, pats + [(1, 1)], X, dOut, dX, B, True, True, TOL[ard.ARD_BF16])
        assert len(seen) > 3
        # the same iteration again (counter rewound): the same bits
        ref = [layers[l]["dW"].clone() for l in range(L)] + [dX.clone()]
        counter.fill_(11)
        for d in layers:
            d["dW"].fill_(float("nan"))
        ard.ard_mlp_step(ctx.h, arr, L, B, Xd, dims[0], dOd, dims[-1], dX, dims[0], 0, inputs.BASE_SEED, 300, counter)
        torch.cuda.synchronize()
        for a, c in zip([layers[l]["dW"] for l in range(L)] + [dX], ref):
            assert torch.equal(a, c)
    finally:
        ctx.close()


def test_many_iterations_in_a_row_keep_the_status_clean():
    """The kernel's stages hand over through barriers with bounded waits; a lost hand-over would show as a timeout
    status (and two seconds of stall).  Replays of a captured iteration, back to back."""
    dims, B = [784, 2048, 2048, 10], 128
    ctx = Ctx(4096)
    try:
        ard.ard_set_distribution(ctx.h, 0, max_entropy_K(0.5, 16))
        layers, arr, _, _ = _stack(ctx, dims, B, np.random.default_rng(1), f32_grads=False, sample=1)
        L = len(layers)
        X, dOut = inputs.config2_step(0)
        Xd, dOd = torch.from_numpy(X).to(BF).cuda(), torch.from_numpy(dOut).to(BF).cuda()
        counter = torch.zeros(1, dtype=torch.int64, device="cuda")

        def step():
            ard.ard_mlp_step(ctx.h, arr, L, B, Xd, dims[0], dOd, dims[-1], None, dims[0], 0, inputs.BASE_SEED, 0, counter)

        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            step()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(600):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        assert ard.ard_last_device_status(ctx.h) == 0
        assert int(counter.item()) == 601             # one eager call, 600 replays (the capture does not run)
        assert e0.elapsed_time(e1) < 600 * 1.0          # ms: far below one bounded wait (2 s) per replay
        assert bool(torch.isfinite(layers[0]["dW"].float()).all())
    finally:
        ctx.close()


def test_stacks_the_kernel_cannot_take_fall_back():
    """A wide output layer, full-width activations, a batch above 128: the call-by-call path runs (several
    launches), the results are the oracle's (covered elsewhere); here: the switch is silent and the status clean."""
    rng = np.random.default_rng(2)
    for dims, B, compact in [([264, 512, 64], 64, 1), ([264, 512, 10], 200, 1), ([264, 512, 10], 64, 0)]:
        ctx = Ctx(2 * B * max(dims) + 4096)
        try:
            layers, arr, _, _ = _stack(ctx, dims, B, rng)
            layers[0]["compact_out"] = compact
            arr = ard.mlp_layers(layers)
            ard.ard_pattern_set(ctx.h, layers[0]["pat"], 2, 1)
            Xd = torch.rand((B, dims[0]), device="cuda").to(BF)
            dOd = torch.randn((B, dims[-1]), device="cuda").to(BF)
            counter = torch.zeros(1, dtype=torch.int64, device="cuda")
            n0 = ard.ard_launch_count(ctx.h)
            ard.ard_mlp_step(ctx.h, arr, 2, B, Xd, dims[0], dOd, dims[-1], None, dims[0], 0, inputs.BASE_SEED, 0, counter)
            torch.cuda.synchronize()
            assert ard.ard_launch_count(ctx.h) - n0 > 1
            assert ard.ard_last_device_status(ctx.h) == 0
            assert bool(torch.isfinite(layers[0]["dW"]).all())
        finally:
            ctx.close()
