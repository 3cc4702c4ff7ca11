"""Fused layer step (product -> bias -> ReLU -> dropout) on compact input AND compact weight matrices.

Every call of the layer-step family is compared with the fp64 oracle (oracle/mlp.py) on the operands the
GPU consumed: weight compaction along the fan-in, forward with bias and ReLU (compact and full-width
output), backward-data with the ReLU adjoint of the feeding layer, backward-weight on compact operands,
expansion of the compact weight gradient, bias gradient; on the tensor-core path (bf16) and on the
CUDA-core path (bf16 and fp32).  Buffers are pre-filled with NaN wherever the library must not read or
must write, so that a wrong extent shows.
"""
import numpy as np
import pytest
import torch

from oracle import gemm as OG
from oracle import mlp as OM
from oracle import pattern as OP
from paper_2203_05705_b200 import ard, inputs
from gpu_helpers import Ctx, host, tdtype, TOL
from distributions import max_entropy_K

pytestmark = pytest.mark.gpu

PATTERNS = [((1, 1), (1, 1)), ((2, 1), (3, 2)), ((3, 3), (1, 1)), ((1, 1), (2, 2)), ((5, 2), (4, 4)), ((16, 9), (7, 1))]


def _rnd(rng, shape, dtype, scale=1.0):
    a = (rng.standard_normal(shape) * scale).astype(np.float32)
    return inputs.bf16_round(a) if dtype == ard.ARD_BF16 else a


def _dev(a, dtype, ld, fill=float("nan")):
    t = torch.full((a.shape[0], ld), fill, dtype=tdtype(dtype), device="cuda")
    t[:, :a.shape[1]] = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(tdtype(dtype))
    return t


@pytest.mark.parametrize("path,dtype,B,K,N", [
    (ard.ARD_PATH_TENSOR_CORE, ard.ARD_BF16, 300, 328, 520),     # two M tiles (CTA pairs), ragged everywhere
    (ard.ARD_PATH_TENSOR_CORE, ard.ARD_BF16, 100, 1024, 264),    # one M tile, several contraction blocks
    (ard.ARD_PATH_CUDA_CORE, ard.ARD_BF16, 37, 90, 70),
    (ard.ARD_PATH_CUDA_CORE, ard.ARD_F32, 37, 90, 70),
    (ard.ARD_PATH_AUTO, ard.ARD_BF16, 130, 1000, 10),            # an output layer: the kernels for <= 16 neurons
    (ard.ARD_PATH_AUTO, ard.ARD_F32, 33, 300, 16),
])
def test_every_layer_step_call_matches_the_oracle(path, dtype, B, K, N):
    rng = np.random.default_rng(B * 7 + K)
    tol = TOL[dtype]
    W = _rnd(rng, (K, N), dtype, 1.0 / np.sqrt(K))               # math orientation
    bias = rng.uniform(-0.5, 0.5, N).astype(np.float32)
    ctx = Ctx(2 * B * (N + 8) + 4096)
    try:
        ard.ard_set_path(ctx.h, path)
        pat = ctx.pattern(ard.ARD_ROW, K, N)
        in_pat = ctx.pattern(ard.ARD_ROW, 8, K)                    # the feeding layer: K neurons
        Wd = _dev(W.T, dtype, K)
        bias_d = torch.from_numpy(bias).cuda()
        for (pin, pout) in PATTERNS:
            ard.ard_pattern_set(ctx.h, in_pat, *pin)
            ard.ard_pattern_set(ctx.h, pat, *pout)
            keep_in, keep = OP.row_keep(K, *pin), OP.row_keep(N, *pout)
            n_in, n = len(keep_in), len(keep)
            alpha = 1.6
            tag = (pin, pout)

            # ---- weight compaction along the fan-in ----
            Wk = torch.full((N, K), float("nan"), dtype=tdtype(dtype), device="cuda")
            ard.ard_compact_weight_cols(ctx.h, pat, in_pat, dtype, K, N, Wd, K, Wk, K)
            Wkh = host(Wk)                                         # packed in both dimensions
            assert np.array_equal(Wkh[:n, :n_in], W.T.astype(np.float64)[np.ix_(keep, keep_in)]), tag
            pad, pad_rows = min(K, (n_in + 63) // 64 * 64), min(N, (n + 63) // 64 * 64)
            assert np.all(Wkh[:n, n_in:pad] == 0) and np.all(Wkh[n:pad_rows, :pad] == 0), tag
            assert np.all(np.isnan(Wkh[pad_rows:])) and np.all(np.isnan(Wkh[:, pad:])), tag   # nothing else is touched
            dropped = np.setdiff1d(np.arange(N), keep)

            # ---- forward: compact input, bias, ReLU; compact and full-width output ----
            Xc = _rnd(rng, (B, n_in), dtype)
            Xd = _dev(Xc, dtype, K)                                # columns >= n_in hold NaN
            ref = OM.layer_fwd_compact(Xc, keep_in, W, bias, keep, alpha)
            A = torch.full((B, N), float("nan"), dtype=tdtype(dtype), device="cuda")
            ard.ard_layer_fwd(ctx.h, pat, in_pat, dtype, B, K, N, alpha, Xd, K, Wk, K, bias_d, A, N,
                              ard.ARD_OUT_COMPACT | ard.ARD_FLAG_RELU)
            Ah = host(A)
            assert OG.rel_fro(Ah[:, :n], ref) <= tol, tag
            assert np.all(Ah[:, :n] >= 0), tag
            A2 = torch.full((B, N), float("nan"), dtype=tdtype(dtype), device="cuda")
            ard.ard_layer_fwd(ctx.h, pat, in_pat, dtype, B, K, N, alpha, Xd, K, Wk, K, bias_d, A2, N,
                              ard.ARD_OUT_SCATTER_ZEROFILL | ard.ARD_FLAG_RELU)
            A2h = host(A2)
            assert OG.rel_fro(A2h[:, keep], ref) <= tol, tag
            assert np.all(A2h[:, dropped] == 0), tag
            # no activation, no bias: the plain compact product
            A3 = torch.full((B, N), float("nan"), dtype=tdtype(dtype), device="cuda")
            ard.ard_layer_fwd(ctx.h, pat, in_pat, dtype, B, K, N, alpha, Xd, K, Wk, K, None, A3, N, ard.ARD_OUT_COMPACT)
            assert OG.rel_fro(host(A3)[:, :n], OM.layer_fwd_compact(Xc, keep_in, W, None, keep, alpha, relu=False)) <= tol, tag

            # ---- backward-data with the ReLU adjoint of the feeding layer ----
            dZc = _rnd(rng, (B, n), dtype)
            act = _rnd(rng, (B, n_in), dtype)
            act[rng.random((B, n_in)) < 0.2] = 0.0                 # exact zeros: relu'(0) = 0
            dZd, actd = _dev(dZc, dtype, N), _dev(act, dtype, K)
            _, _, dA_prev = OM.layer_bwd_compact(Xc, keep_in, W, keep, dZc)
            refdx = alpha * dA_prev * (act > 0)
            dX = torch.full((B, K), float("nan"), dtype=tdtype(dtype), device="cuda")
            ard.ard_layer_bwd_data(ctx.h, pat, in_pat, dtype, B, K, N, alpha, dZd, N, 1, Wk, K, actd, K, dX, K)
            dXh = host(dX)
            assert OG.rel_fro(dXh[:, :n_in], refdx) <= tol, tag
            assert np.all(dXh[:, :n_in][act <= 0] == 0), tag
            assert np.all(np.isnan(dXh[:, n_in:])), tag

            # ---- backward-weight on compact operands, expansion, bias gradient ----
            dWc_ref, db_ref, _ = OM.layer_bwd_compact(Xc, keep_in, W, keep, dZc)       # [n_in x n], [n]
            dWk = torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda")
            ard.ard_layer_bwd_weight(ctx.h, pat, in_pat, dtype, ard.ARD_F32, B, K, N, 1.0, Xd, K, dZd, N, 1, dWk, K, 0)
            dWkh = host(dWk)                                       # packed like Wk
            assert OG.rel_fro(dWkh[:n, :n_in], dWc_ref.T) <= tol, tag
            assert np.all(np.isnan(dWkh[n:])) and np.all(np.isnan(dWkh[:, n_in:])), tag
            dW = torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda")
            ard.ard_expand_weight_grad_cols(ctx.h, pat, in_pat, ard.ARD_F32, K, N, dWk, K, dW, K, 1)
            dWh = host(dW)
            full = np.zeros((N, K))
            full[np.ix_(keep, keep_in)] = dWkh[:n, :n_in]
            assert np.array_equal(dWh, full), tag
            db = torch.full((N,), float("nan"), dtype=torch.float32, device="cuda")
            ard.ard_bias_grad(ctx.h, pat, dtype, B, N, dZd, N, 1, db, 1)
            dbh = host(db)
            assert np.abs(dbh[keep] - db_ref).max() <= tol * max(1.0, np.abs(db_ref).max()), tag
            assert np.all(dbh[dropped] == 0), tag
            # the same from a full-width gradient whose dropped columns hold NaN (never read as values)
            dZfull = torch.full((B, N), float("nan"), dtype=tdtype(dtype), device="cuda")
            dZfull[:, torch.from_numpy(keep).cuda()] = dZd[:, :n]
            db2 = torch.full((N,), float("nan"), dtype=torch.float32, device="cuda")
            ard.ard_bias_grad(ctx.h, pat, dtype, B, N, dZfull, N, 0, db2, 1)
            assert torch.equal(db2, db), tag
            assert ard.ard_last_device_status(ctx.h) == 0
    finally:
        ctx.close()


def test_full_width_input_with_fused_epilogues():
    """in_pat = NULL: the first hidden layer (full-width input), bias + ReLU fused, and the ReLU adjoint on a
    full-width gradient."""
    B, K, N = 260, 392, 1032
    dtype = ard.ARD_BF16
    rng = np.random.default_rng(2)
    W = _rnd(rng, (K, N), dtype, 1.0 / np.sqrt(K))
    X = _rnd(rng, (B, K), dtype)
    bias = rng.uniform(-0.5, 0.5, N).astype(np.float32)
    ctx = Ctx(2 * B * (N + 8) + 4096)
    try:
        ard.ard_set_path(ctx.h, ard.ARD_PATH_TENSOR_CORE)
        pat = ctx.pattern(ard.ARD_ROW, K, N)
        Wd, Xd, bias_d = _dev(W.T, dtype, K), _dev(X, dtype, K), torch.from_numpy(bias).cuda()
        for dp, b in [(1, 1), (2, 2), (3, 1), (9, 4)]:
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            m, keep = OP.row_mask(N, dp, b), OP.row_keep(N, dp, b)
            Z, Aref = OM.layer_fwd(X, W, bias, m, 2.0)
            A = torch.full((B, N), float("nan"), dtype=torch.bfloat16, device="cuda")
            ard.ard_layer_fwd(ctx.h, pat, None, dtype, B, K, N, 2.0, Xd, K, Wd, K, bias_d, A, N,
                              ard.ARD_OUT_SCATTER_ZEROFILL | ard.ARD_FLAG_RELU)
            assert OG.rel_fro(host(A), Aref) <= TOL[dtype], (dp, b)
            dZ = _rnd(rng, (B, N), dtype)
            act = _rnd(rng, (B, K), dtype)
            dX = torch.full((B, K), float("nan"), dtype=torch.bfloat16, device="cuda")
            ard.ard_layer_bwd_data(ctx.h, pat, None, dtype, B, K, N, 1.5, _dev(dZ, dtype, N), N, 0, Wd, K,
                                   _dev(act, dtype, K), K, dX, K)
            ref = OG.bwd_data(dZ, W, m, 1.5) * (act > 0)
            assert OG.rel_fro(host(dX), ref) <= TOL[dtype], (dp, b)
        assert ard.ard_last_device_status(ctx.h) == 0
    finally:
        ctx.close()


def test_rejections():
    ctx = Ctx(1 << 20)
    try:
        pat = ctx.pattern(ard.ARD_ROW, 64, 128)
        wrong = ctx.pattern(ard.ARD_ROW, 8, 72)                    # N_dim != this layer's K
        tile = ctx.pattern(ard.ARD_TILE, 64, 128, 32)
        t = torch.zeros((128, 128), dtype=torch.bfloat16, device="cuda")
        with pytest.raises(ard.ArdError) as e:
            ard.ard_layer_fwd(ctx.h, pat, wrong, ard.ARD_BF16, 16, 64, 128, 1.0, t, 64, t, 64, None, t, 128, 0)
        assert e.value.status == ard.ARD_ERR_SHAPE
        with pytest.raises(ard.ArdError) as e:
            ard.ard_layer_fwd(ctx.h, tile, None, ard.ARD_BF16, 16, 64, 128, 1.0, t, 64, t, 64, None, t, 128, 0)
        assert e.value.status == ard.ARD_ERR_INVALID_ARG
        with pytest.raises(ard.ArdError) as e:                       # ReLU is not an ard_fwd flag
            ard.ard_fwd(ctx.h, pat, ard.ARD_BF16, 16, 64, 128, 1.0, t, 64, t, 64, t, 128, ard.ARD_FLAG_RELU)
        assert e.value.status == ard.ARD_ERR_INVALID_ARG
        with pytest.raises(ard.ArdError) as e:
            ard.ard_compact_weight_cols(ctx.h, pat, None, ard.ARD_BF16, 64, 128, t, 64, t, 64)
        assert e.value.status == ard.ARD_ERR_INVALID_ARG
    finally:
        ctx.close()


def test_a_captured_step_draws_a_new_pattern_at_every_replay():
    """The iteration counter lives on the device: a CUDA graph of {sample, sample, layer forward} replays
    with iteration base + 0, 1, 2, ... and gives what the same calls give when issued one by one."""
    B, K, N = 128, 256, 512
    dtype = ard.ARD_BF16
    rng = np.random.default_rng(4)
    W = _rnd(rng, (K, N), dtype, 1.0 / np.sqrt(K))
    X = _rnd(rng, (B, K), dtype)
    Kd = max_entropy_K(0.5, 8)
    cdf = OP.quantise_K(Kd)
    ctx = Ctx(1 << 20)
    try:
        ard.ard_set_distribution(ctx.h, 0, Kd)
        pat = ctx.pattern(ard.ARD_ROW, K, N)
        in_pat = ctx.pattern(ard.ARD_ROW, 8, K)
        Wd, bias_d = _dev(W.T, dtype, K), torch.zeros(N, device="cuda")
        Xd = _dev(X, dtype, K)
        Wk = torch.zeros((N, K), dtype=torch.bfloat16, device="cuda")
        A = torch.zeros((B, N), dtype=torch.bfloat16, device="cuda")
        counter = torch.zeros(1, dtype=torch.int64, device="cuda")
        base = 1000

        def step():
            ard.ard_sample_pattern_counter(ctx.h, in_pat, 0, inputs.BASE_SEED, base, counter, 0, 1)
            ard.ard_sample_pattern_counter(ctx.h, pat, 0, inputs.BASE_SEED, base, counter, 1, 2)
            ard.ard_compact_weight_cols(ctx.h, pat, in_pat, dtype, K, N, Wd, K, Wk, K)
            ard.ard_layer_fwd(ctx.h, pat, in_pat, dtype, B, K, N, 2.0, Xd, K, Wk, K, bias_d, A, N,
                              ard.ARD_OUT_SCATTER_ZEROFILL | ard.ARD_FLAG_RELU)

        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            step()                                                  # the context creates its side streams outside the capture
        torch.cuda.synchronize()
        assert int(counter.item()) == 1
        counter.zero_()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        seen = set()
        for it in range(6):
            graph.replay()
            torch.cuda.synchronize()
            assert int(counter.item()) == it + 1
            got_in = ard.ard_pattern_to_host(in_pat, 0)[:2]
            got = ard.ard_pattern_to_host(pat, 0)[:2]
            assert tuple(got_in) == OP.draw(cdf, inputs.BASE_SEED, base + it, 1)
            assert tuple(got) == OP.draw(cdf, inputs.BASE_SEED, base + it, 2)
            seen.add((tuple(got_in), tuple(got)))
            keep_in, keep = OP.row_keep(K, *got_in), OP.row_keep(N, *got)
            ref = OM.layer_fwd_compact(X[:, :len(keep_in)], keep_in, W, None, keep, 2.0)
            Ah = host(A)
            assert OG.rel_fro(Ah[:, keep], ref) <= TOL[dtype], it
            assert np.all(np.delete(Ah, keep, axis=1) == 0)
        assert len(seen) > 1
        assert ard.ard_last_device_status(ctx.h) == 0
    finally:
        ctx.close()


def _stack(ctx, dims, B, p, compact, rng):
    """Buffers of a stack of layers for ard_mlp_step; returns (layer dicts, C array, numpy weights, biases)."""
    L = len(dims) - 1
    Ws = [inputs.bf16_round((rng.standard_normal((dims[l], dims[l + 1])) * np.sqrt(2.0 / dims[l])).astype(np.float32))
          for l in range(L)]
    bs = [rng.uniform(-0.1, 0.1, dims[l + 1]).astype(np.float32) for l in range(L)]
    bf = torch.bfloat16
    layers = []
    for l in range(L):
        K, N = dims[l], dims[l + 1]
        hidden = l < L - 1
        layers.append(dict(
            K=K, N=N, pat=ctx.pattern(ard.ARD_ROW, K, N), sample=1 if hidden else 0, relu=1 if hidden else 0,
            compact_out=1 if (hidden and compact) else 0, dW_is_f32=1, alpha=(1.0 / (1.0 - p)) if hidden else 1.0, ldw=K,
            W=torch.from_numpy(np.ascontiguousarray(Ws[l].T)).to(bf).cuda(), bias=torch.from_numpy(bs[l]).cuda(),
            Wk=torch.full((N, K), float("nan"), dtype=bf, device="cuda"),
            A=torch.full((B, N), float("nan"), dtype=bf, device="cuda"),
            dZ=torch.full((B, N), float("nan"), dtype=bf, device="cuda"),
            dWk=torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda"),
            dW=torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda"),
            db=torch.full((N,), float("nan"), dtype=torch.float32, device="cuda")))
    ard.ard_pattern_set(ctx.h, layers[-1]["pat"], 1, 1)             # the output layer is not dropped
    return layers, ard.mlp_layers(layers), Ws, bs


@pytest.mark.parametrize("compact", [1, 0])
@pytest.mark.parametrize("p", [0.3, 0.7])
def test_mlp_step_784_2048_2048_10(compact, p):
    """One native call per training iteration of the 784-2048-2048-10 network (batch 128): patterns drawn on
    the device, forward and backward chains; compact matrices between the hidden layers or full width.
    Every stage is graded against the oracle on the operands the GPU consumed, the whole step against the
    oracle's step on the same inputs with a tolerance for the bf16 activations in between."""
    dims, B = [784, 2048, 2048, 10], 128
    rng = np.random.default_rng(17)
    Kd = max_entropy_K(p, 16)
    cdf = OP.quantise_K(Kd)
    ctx = Ctx(2 * B * 2048 + 4096)
    try:
        ard.ard_set_distribution(ctx.h, 0, Kd)
        layers, arr, Ws, bs = _stack(ctx, dims, B, p, compact, rng)
        L = len(layers)
        counter = torch.zeros(1, dtype=torch.int64, device="cuda")
        tol = TOL[ard.ARD_BF16]
        for step in range(3):
            X, dOut = inputs.config2_step(step)
            Xd = torch.from_numpy(X).to(torch.bfloat16).cuda()
            dOd = torch.from_numpy(dOut).to(torch.bfloat16).cuda()
            dX = torch.full((B, dims[0]), float("nan"), dtype=torch.bfloat16, device="cuda")
            ard.ard_mlp_step(ctx.h, arr, L, B, Xd, dims[0], dOd, dims[-1], dX, dims[0], 0, inputs.BASE_SEED, 50, counter)
            torch.cuda.synchronize()
            assert ard.ard_last_device_status(ctx.h) == 0
            assert int(counter.item()) == step + 1
            pats = [OP.draw(cdf, inputs.BASE_SEED, 50 + step, l + 1) for l in range(L - 1)] + [(1, 1)]
            for l in range(L):
                assert tuple(ard.ard_pattern_to_host(layers[l]["pat"], 0)[:2]) == pats[l]
            keeps = [OP.row_keep(dims[l + 1], *pats[l]) for l in range(L)]
            masks = [OP.row_mask(dims[l + 1], *pats[l]) for l in range(L)]
            alphas = [layers[l]["alpha"] for l in range(L)]

            def full(l, t):
                """Activation / gradient buffer of layer l as a full-width fp64 matrix."""
                h = host(t)
                if not layers[l]["compact_out"]:
                    return h
                out = np.zeros_like(h)
                out[:, keeps[l]] = h[:, :len(keeps[l])]
                return out

            # ---- stage by stage, on the GPU's own inputs ----
            a_prev = X.astype(np.float64)
            acts = [a_prev]
            for l in range(L):
                _, ref = OM.layer_fwd(a_prev, Ws[l], bs[l], masks[l], alphas[l], relu=(l < L - 1))
                got = full(l, layers[l]["A"])
                assert OG.rel_fro(got, ref) <= tol, ("fwd", l, pats)
                assert np.all(got[:, masks[l] == 0] == 0)
                a_prev = got
                acts.append(got)
            dz = dOut.astype(np.float64)
            for l in range(L - 1, -1, -1):
                dW_ref = acts[l].T @ dz                               # [K x N]; dz is zero at dropped neurons
                assert OG.rel_fro(host(layers[l]["dW"]), dW_ref.T) <= tol, ("dW", l, pats)
                assert np.abs(host(layers[l]["db"]) - dz.sum(axis=0)).max() <= tol * max(1.0, np.abs(dz.sum(axis=0)).max())
                dA = dz @ Ws[l].T.astype(np.float64)
                if l > 0:
                    ref = alphas[l - 1] * dA * masks[l - 1][None, :] * (acts[l] > 0)
                    got = full(l - 1, layers[l - 1]["dZ"])
                    if not layers[l - 1]["compact_out"]:
                        got = got * masks[l - 1][None, :]             # full width: dropped columns are never read
                    assert OG.rel_fro(got, ref) <= tol, ("dZ", l - 1, pats)
                    dz = got
                else:
                    assert OG.rel_fro(host(dX), dA) <= tol, ("dX", pats)

            # ---- the whole step against the oracle's step: a wiring check (a misplaced rescale or a missing
            # ReLU adjoint is an error of order one).  The bf16 activations between the layers move
            # pre-activations next to zero across it, which flips their ReLU adjoint: a few entries in a
            # thousand are then off by their whole value, a few percent in the Frobenius norm. ----
            fw = OM.fwd(X, Ws, bs, masks, alphas)
            bw = OM.bwd(fw, Ws, masks, alphas, dOut)
            assert OG.rel_fro(host(layers[-1]["A"]), fw["A"][-1]) <= 2e-2
            for l in range(L):
                assert OG.rel_fro(host(layers[l]["dW"]), bw["dW"][l].T) <= 0.1, ("step dW", l)
                assert np.all(host(layers[l]["dW"])[masks[l] == 0, :] == 0)
                if l > 0:
                    assert np.all(host(layers[l]["dW"])[:, masks[l - 1] == 0] == 0)
            assert OG.rel_fro(host(dX), bw["dX"]) <= 0.1
    finally:
        ctx.close()


def test_full_size_layer_with_compact_matrices_on_sampled_outputs():
    """The second hidden layer of the 8192-wide stack the benchmark times (batch 4096, K = N = 8192, default
    launch configuration): compact input, compact weight, fused bias + ReLU and ReLU adjoint.  The oracle
    recomputes 128 batch rows of the activations and of the input gradient and 64 neurons of the weight
    gradient; finiteness and the zero pattern are checked on the whole outputs."""
    c5 = inputs.config5()
    X, W, dY = c5["X"], c5["W"], c5["dY"]
    B, K = X.shape
    N = W.shape[1]
    bf = torch.bfloat16
    rng = np.random.default_rng(8)
    bias = rng.uniform(-0.5, 0.5, N).astype(np.float32)
    ctx = Ctx(4096)
    try:
        pat = ctx.pattern(ard.ARD_ROW, K, N)
        in_pat = ctx.pattern(ard.ARD_ROW, 8, K)
        Wd = torch.from_numpy(np.ascontiguousarray(W.T)).to(bf).cuda()
        Xd = torch.from_numpy(X).to(bf).cuda()
        dZd = torch.from_numpy(dY).to(bf).cuda()
        act = inputs.bf16_round(rng.standard_normal((B, K)).astype(np.float32))
        actd = torch.from_numpy(act).to(bf).cuda()
        bias_d = torch.from_numpy(bias).cuda()
        Wk = torch.empty((N, K), dtype=bf, device="cuda")
        A = torch.empty((B, N), dtype=bf, device="cuda")
        dX = torch.empty((B, K), dtype=bf, device="cuda")
        dWk = torch.empty((N, K), dtype=bf, device="cuda")
        dW = torch.empty((N, K), dtype=bf, device="cuda")
        rows = np.arange(5, B, B // 128)[:128]
        tol = TOL[ard.ARD_BF16]
        for pin, pout in [((2, 1), (2, 2)), ((3, 2), (5, 1)), ((1, 1), (16, 7))]:
            ard.ard_pattern_set(ctx.h, in_pat, *pin)
            ard.ard_pattern_set(ctx.h, pat, *pout)
            keep_in, keep = OP.row_keep(K, *pin), OP.row_keep(N, *pout)
            n_in, n = len(keep_in), len(keep)
            for t in (Wk, A, dX, dWk, dW):
                t.fill_(float("nan"))
            ard.ard_compact_weight_cols(ctx.h, pat, in_pat, ard.ARD_BF16, K, N, Wd, K, Wk, K)
            ard.ard_layer_fwd(ctx.h, pat, in_pat, ard.ARD_BF16, B, K, N, 2.0, Xd, K, Wk, K, bias_d, A, N,
                              ard.ARD_OUT_COMPACT | ard.ARD_FLAG_RELU)
            ard.ard_layer_bwd_data(ctx.h, pat, in_pat, ard.ARD_BF16, B, K, N, 2.0, dZd, N, 1, Wk, K, actd, K, dX, K)
            ard.ard_layer_bwd_weight(ctx.h, pat, in_pat, ard.ARD_BF16, ard.ARD_BF16, B, K, N, 1.0, Xd, K, dZd, N, 1,
                                     dWk, K, 0)
            ard.ard_expand_weight_grad_cols(ctx.h, pat, in_pat, ard.ARD_BF16, K, N, dWk, K, dW, K, 1)
            torch.cuda.synchronize()
            assert ard.ard_last_device_status(ctx.h) == 0
            tag = (pin, pout)
            ridx = torch.from_numpy(rows).cuda()
            # forward: sampled batch rows (the compact input is the first n_in columns of X)
            ref = OM.layer_fwd_compact(X[rows][:, :n_in], keep_in, W, bias, keep, 2.0)
            assert OG.rel_fro(host(A[ridx])[:, :n], ref) <= tol, tag
            # input gradient with the ReLU adjoint: sampled batch rows
            _, _, dA_prev = OM.layer_bwd_compact(X[rows][:, :n_in], keep_in, W, keep, dY[rows][:, :n])
            refdx = 2.0 * dA_prev * (act[rows][:, :n_in] > 0)
            assert OG.rel_fro(host(dX[ridx])[:, :n_in], refdx) <= tol, tag
            # weight gradient: sampled kept neurons, through the expansion
            js = np.arange(1, n, max(1, n // 64))[:64]
            refw = dY[:, js].astype(np.float64).T @ X[:, :n_in].astype(np.float64)      # [64 x n_in]
            got = host(dW[torch.from_numpy(keep[js]).cuda()])
            assert OG.rel_fro(got[:, keep_in], refw) <= tol, tag
            # whole outputs: finite where written, zeros exactly where the pattern says
            assert bool(torch.isfinite(A[:, :n]).all()) and bool(torch.isfinite(dX[:, :n_in]).all())
            assert bool(torch.isfinite(dW).all())
            mrow = torch.from_numpy(OP.row_mask(N, *pout) == 0).cuda()
            mcol = torch.from_numpy(OP.row_mask(K, *pin) == 0).cuda()
            assert bool(torch.all(dW[mrow, :] == 0)) and bool(torch.all(dW[:, mcol] == 0)), tag
    finally:
        ctx.close()


def test_mlp_step_replayed_from_a_graph_equals_the_same_iterations_called_one_by_one():
    """The iteration forks its weight-side work onto a second stream; captured once and replayed, it must draw
    the next pattern every time and give the bits the one-by-one calls give."""
    dims, B, p = [784, 2048, 2048, 10], 128, 0.5
    rng = np.random.default_rng(23)
    ctx = Ctx(4096)
    try:
        ard.ard_set_distribution(ctx.h, 0, max_entropy_K(p, 16))
        layers, arr, _, _ = _stack(ctx, dims, B, p, 1, rng)
        L = len(layers)
        counter = torch.zeros(1, dtype=torch.int64, device="cuda")
        X, dOut = inputs.config2_step(0)
        Xd = torch.from_numpy(X).to(torch.bfloat16).cuda()
        dOd = torch.from_numpy(dOut).to(torch.bfloat16).cuda()
        dX = torch.zeros((B, dims[0]), dtype=torch.bfloat16, device="cuda")

        def step():
            ard.ard_mlp_step(ctx.h, arr, L, B, Xd, dims[0], dOd, dims[-1], dX, dims[0], 0, inputs.BASE_SEED, 900, counter)

        def snapshot():
            torch.cuda.synchronize()
            out = [dX.clone(), layers[-1]["A"].clone()]
            for d in layers:
                out += [d["dW"].clone(), d["db"].clone()]
            return out, [tuple(ard.ard_pattern_to_host(d["pat"], 0)[:2]) for d in layers]

        side = torch.cuda.Stream()
        ref = []
        with torch.cuda.stream(side):
            for _ in range(4):
                step()
                ref.append(snapshot())
        counter.zero_()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        for it in range(4):
            for d in layers:                                        # stale results must not pass for fresh ones
                d["dW"].fill_(float("nan"))
            graph.replay()
            got, pats = snapshot()
            assert int(counter.item()) == it + 1
            assert pats == ref[it][1], it
            for a, c in zip(got, ref[it][0]):
                assert torch.equal(a, c), it
        assert len({tuple(r[1]) for r in ref}) > 1                 # the patterns did change
        assert ard.ard_last_device_status(ctx.h) == 0
    finally:
        ctx.close()
