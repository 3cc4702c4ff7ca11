"""Behaviour at the boundary that the kernels' own parity tests do not reach: operands that move between calls,
a gradient buffer rewritten in place between two calls of ard_layer_products (eagerly and under graph replay),
and the shared-tail schedule together with products enqueued side by side."""
import numpy as np
import pytest
import torch

from oracle import gemm as OG
from oracle import pattern as OP
from paper_2203_05705_b200 import ard, inputs
from gpu_helpers import Ctx, dev, host, nan_buf, tile_rel_fro, TOL

pytestmark = pytest.mark.gpu
BF = torch.bfloat16
TOL_BF16 = TOL[ard.ARD_BF16]


def _layer(B, K, N, seed, wscale=0.05):
    rng = np.random.default_rng(seed)
    X = inputs.bf16_round(rng.standard_normal((B, K)).astype(np.float32))
    W = inputs.bf16_round((rng.standard_normal((K, N)) * wscale).astype(np.float32))
    dY = inputs.bf16_round(rng.standard_normal((B, N)).astype(np.float32))
    return X, W, dY


@pytest.mark.parametrize("kind,ts", [("row", 0), ("tile", 64)])
def test_operands_that_move_between_calls(kind, ts):
    """Every call gets freshly allocated operands and outputs (the earlier ones stay alive, so the addresses
    differ), as under a framework allocator; results against the oracle each time."""
    B, K, N = 300, 512, 1024
    akind = ard.ARD_ROW if kind == "row" else ard.ARD_TILE
    ctx = Ctx(2 * B * N + 4096)
    held = []
    try:
        ard.ard_set_path(ctx.h, ard.ARD_PATH_TENSOR_CORE)
        pat = ctx.pattern(akind, K, N, ts)
        seen = set()
        for call, (dp, b) in enumerate([(3, 2), (3, 2), (1, 1), (8, 5), (3, 2), (16, 9)]):
            X, W, dY = _layer(B, K, N, 100 + call)
            Xd, Wd, dYd = dev(X, ard.ARD_BF16), dev(W.T, ard.ARD_BF16), dev(dY, ard.ARD_BF16)
            Y, dX, dW = nan_buf(B, N, BF), nan_buf(B, K, BF), nan_buf(N, K, BF)
            held += [Xd, Wd, dYd, Y, dX, dW]
            assert Xd.data_ptr() not in seen
            seen.update(t.data_ptr() for t in (Xd, Wd, dYd))
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            ard.ard_fwd(ctx.h, pat, ard.ARD_BF16, B, K, N, 1.5, Xd, K, Wd, K, Y, N, ard.ARD_OUT_SCATTER_ZEROFILL)
            ard.ard_bwd_data(ctx.h, pat, ard.ARD_BF16, B, K, N, 1.5, dYd, N, 0, Wd, K, dX, K)
            ard.ard_bwd_weight(ctx.h, pat, ard.ARD_BF16, ard.ARD_BF16, B, K, N, 1.5, Xd, K, dYd, N, 0, dW, K, 1)
            mask = OP.row_mask(N, dp, b) if kind == "row" else OP.tile_mask(K, N, ts, dp, b)
            for got, want, name in ((Y, OG.fwd(X, W, mask, 1.5), "fwd"), (dX, OG.bwd_data(dY, W, mask, 1.5), "bwd_data"),
                                    (dW, OG.bwd_weight(X, dY, mask, 1.5).T, "bwd_weight")):
                assert OG.rel_fro(host(got), want) <= TOL_BF16, (call, dp, b, name)
                assert tile_rel_fro(host(got), want) <= TOL_BF16, (call, dp, b, name)
        assert ard.ard_last_device_status(ctx.h) == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("mode", ["eager", "graph"])
def test_layer_products_reads_the_gradient_it_is_given(mode):
    """Two calls of ard_layer_products with ONE pattern (set once, dp = 3) and new values written into the same
    dY buffer between them: the second call's input and weight gradients must come from the new values.  With a
    graph: captured after an eager warm-up, replayed after every rewrite."""
    B, K, N, dp, b = 300, 520, 1000, 3, 2
    X, W, dY0 = _layer(B, K, N, 31)
    ctx = Ctx(2 * B * N + 4096)
    try:
        pat = ctx.pattern(ard.ARD_ROW, K, N)
        ard.ard_pattern_set(ctx.h, pat, dp, b)
        mask = OP.row_mask(N, dp, b)
        Xd, Wd, dYd = dev(X, ard.ARD_BF16), dev(W.T, ard.ARD_BF16), dev(dY0, ard.ARD_BF16)
        Y, dX, dW = nan_buf(B, N, BF), nan_buf(B, K, BF), nan_buf(N, K, BF)

        def call(stream=None):
            ard.ard_layer_products(ctx.h, pat, ard.ARD_BF16, ard.ARD_BF16, B, K, N, 1.5, Xd, K, Wd, K, dYd, N, Y, N,
                                   ard.ARD_OUT_SCATTER_ZEROFILL, dX, K, dW, K, 1, stream)

        n0 = ard.ard_launch_count(ctx.h)
        call()
        torch.cuda.synchronize()
        per_call = ard.ard_launch_count(ctx.h) - n0
        assert per_call == 4            # three products and the compaction of dY
        run = call
        if mode == "graph":
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=s):
                    n1 = ard.ard_launch_count(ctx.h)
                    call(s.cuda_stream)
                    assert ard.ard_launch_count(ctx.h) - n1 == 4     # the capture holds the compaction too
            run = g.replay
        rng = np.random.default_rng(5)
        for rewrite in range(3):
            dY = inputs.bf16_round(rng.standard_normal((B, N)).astype(np.float32))
            dYd.copy_(torch.from_numpy(dY).to(BF))
            dX.fill_(float("nan")); dW.fill_(float("nan"))
            torch.cuda.synchronize()
            run()
            torch.cuda.synchronize()
            assert OG.rel_fro(host(dX), OG.bwd_data(dY, W, mask, 1.5)) <= TOL_BF16, (mode, rewrite)
            assert OG.rel_fro(host(dW), OG.bwd_weight(X, dY, mask, 1.5).T) <= TOL_BF16, (mode, rewrite)
        assert ard.ard_last_device_status(ctx.h) == 0
    finally:
        ctx.close()


def test_layer_products_with_the_shared_tail_enabled():
    """The shared-tail schedule keeps its partial sums in one scratch per context; ard_layer_products runs a row
    pattern's products on two streams and therefore launches them without it.  More tiles than SM pairs, so the
    schedule would engage if it were left on."""
    B, K, N = 2048, 1024, 4096
    X, W, dY = _layer(B, K, N, 41, 0.03)
    ctx = Ctx(2 * B * N + 4096)
    try:
        ard.ard_set_path(ctx.h, ard.ARD_PATH_TENSOR_CORE)
        ard.ard_set_shared_tail(ctx.h, 1, 2, 1)
        pat = ctx.pattern(ard.ARD_ROW, K, N)
        Xd, Wd, dYd = dev(X, ard.ARD_BF16), dev(W.T, ard.ARD_BF16), dev(dY, ard.ARD_BF16)
        for dp, b in [(1, 1), (3, 1)]:
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            mask = OP.row_mask(N, dp, b)
            want = (OG.fwd(X, W, mask, 2.0), OG.bwd_data(dY, W, mask, 2.0), OG.bwd_weight(X, dY, mask, 2.0).T)
            for rep in range(3):
                Y, dX, dW = nan_buf(B, N, BF), nan_buf(B, K, BF), nan_buf(N, K, BF)
                ard.ard_layer_products(ctx.h, pat, ard.ARD_BF16, ard.ARD_BF16, B, K, N, 2.0, Xd, K, Wd, K, dYd, N, Y, N,
                                       ard.ARD_OUT_SCATTER_ZEROFILL, dX, K, dW, K, 1)
                torch.cuda.synchronize()
                for got, w, name in zip((Y, dX, dW), want, ("fwd", "bwd_data", "bwd_weight")):
                    assert OG.rel_fro(host(got), w) <= TOL_BF16, (dp, b, rep, name)
                    assert tile_rel_fro(host(got), w) <= TOL_BF16, (dp, b, rep, name)
        assert ard.ard_last_device_status(ctx.h) == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("dtype", [ard.ARD_BF16, ard.ARD_F32])
def test_compact_and_expand_columns(dtype):
    """ard_compact_cols / ard_expand_cols: Eq. 1 applied to the columns of a matrix and its adjoint with a rescale,
    exact (copies and one multiplication) against the oracle's kept list."""
    rows_, N, ld = 77, 200, 208
    rng = np.random.default_rng(8)
    src = inputs.bf16_round(rng.standard_normal((rows_, N)).astype(np.float32))
    td = BF if dtype == ard.ARD_BF16 else torch.float32
    ctx = Ctx(4096)
    try:
        pat = ctx.pattern(ard.ARD_ROW, 8, N)
        S = torch.full((rows_, ld), float("nan"), dtype=td, device="cuda")
        S[:, :N] = torch.from_numpy(src).to(td)
        for dp, b in [(1, 1), (3, 2), (7, 7), (16, 9), (150, 30)]:
            ard.ard_pattern_set(ctx.h, pat, dp, b)
            keep = OP.row_keep(N, dp, b)
            C = torch.full((rows_, ld), float("nan"), dtype=td, device="cuda")
            ard.ard_compact_cols(ctx.h, pat, dtype, rows_, N, S, ld, C, ld)
            got = host(C)
            assert np.array_equal(got[:, :len(keep)], src[:, keep].astype(np.float64)), (dp, b)
            assert np.all(np.isnan(got[:, len(keep):])), (dp, b)                  # nothing written beyond n_keep
            E = torch.full((rows_, ld), float("nan"), dtype=torch.float32, device="cuda")
            ard.ard_expand_cols(ctx.h, pat, dtype, rows_, N, 1.5, C, ld, E, ld)
            want = np.zeros((rows_, N), dtype=np.float32)
            want[:, keep] = np.float32(1.5) * src[:, keep]
            got = host(E)
            assert np.array_equal(got[:, :N], want.astype(np.float64)), (dp, b)
            assert np.all(np.isnan(got[:, N:])), (dp, b)
        with pytest.raises(ard.ArdError):
            ard.ard_compact_cols(ctx.h, pat, dtype, rows_, N + 8, S, ld, C, ld)     # N differs from the pattern's
    finally:
        ctx.close()


def test_options_are_validated_and_do_not_change_results():
    B, K, N = 300, 512, 1024
    X, W, dY = _layer(B, K, N, 51)
    ctx = Ctx(2 * B * N + 4096)
    try:
        with pytest.raises(ard.ArdError):
            ard.ard_set_option(ctx.h, 99, 1)
        with pytest.raises(ard.ArdError):
            ard.ard_set_option(ctx.h, ard.ARD_OPT_PDL, -1)
        pat = ctx.pattern(ard.ARD_ROW, K, N)
        ard.ard_pattern_set(ctx.h, pat, 3, 1)
        mask = OP.row_mask(N, 3, 1)
        Xd, Wd, dYd = dev(X, ard.ARD_BF16), dev(W.T, ard.ARD_BF16), dev(dY, ard.ARD_BF16)
        want = (OG.fwd(X, W, mask, 2.0), OG.bwd_data(dY, W, mask, 2.0), OG.bwd_weight(X, dY, mask, 2.0).T)
        for opts in [{}, {ard.ARD_OPT_PDL: 0}, {ard.ARD_OPT_SIDE_STREAMS: 0}, {ard.ARD_OPT_CTA_PAIRS: 0}, {ard.ARD_OPT_BAND_ROWS: 2}]:
            for k, v in opts.items():
                ard.ard_set_option(ctx.h, k, v)
            Y, dX, dW = nan_buf(B, N, BF), nan_buf(B, K, BF), nan_buf(N, K, BF)
            ard.ard_layer_products(ctx.h, pat, ard.ARD_BF16, ard.ARD_BF16, B, K, N, 2.0, Xd, K, Wd, K, dYd, N, Y, N,
                                   ard.ARD_OUT_SCATTER_ZEROFILL, dX, K, dW, K, 1)
            torch.cuda.synchronize()
            for got, w, name in zip((Y, dX, dW), want, ("fwd", "bwd_data", "bwd_weight")):
                assert OG.rel_fro(host(got), w) <= TOL_BF16, (opts, name)
            for k in opts:
                ard.ard_set_option(ctx.h, k, 1 if k != ard.ARD_OPT_BAND_ROWS else 16)
        assert ard.ard_last_device_status(ctx.h) == 0
    finally:
        ctx.close()


@pytest.mark.parametrize("kind,ts", [("row", 0), ("tile", 128)])
def test_first_use_of_new_buffers_inside_a_stream_capture(kind, ts):
    """No product call allocates, copies or synchronises, so the very first call on buffers the library has never
    seen can be recorded into a CUDA graph (pattern drawn inside the graph from a device counter); the replays are
    compared with the oracle."""
    B, K, N = 384, 512, 1024
    X, W, dY = _layer(B, K, N, 61)
    akind = ard.ARD_ROW if kind == "row" else ard.ARD_TILE
    from distributions import max_entropy_K
    Kd = max_entropy_K(0.5, 8)
    cdf = OP.quantise_K(Kd)
    ctx = Ctx(2 * B * N + 4096)
    try:
        ard.ard_set_path(ctx.h, ard.ARD_PATH_TENSOR_CORE)
        ard.ard_set_distribution(ctx.h, 0, Kd)
        pat = ctx.pattern(akind, K, N, ts)
        counter = torch.zeros(1, dtype=torch.int64, device="cuda")
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            Xd, Wd, dYd = dev(X, ard.ARD_BF16), dev(W.T, ard.ARD_BF16), dev(dY, ard.ARD_BF16)
            Y, dX, dW = nan_buf(B, N, BF), nan_buf(B, K, BF), nan_buf(N, K, BF)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                cs = s.cuda_stream
                ard.ard_sample_pattern_counter(ctx.h, pat, 0, 77, 500, counter, 1, 3, cs)
                ard.ard_fwd(ctx.h, pat, ard.ARD_BF16, B, K, N, 2.0, Xd, K, Wd, K, Y, N, ard.ARD_OUT_SCATTER_ZEROFILL, cs)
                ard.ard_bwd_data(ctx.h, pat, ard.ARD_BF16, B, K, N, 2.0, dYd, N, 0, Wd, K, dX, K, cs)
                ard.ard_bwd_weight(ctx.h, pat, ard.ARD_BF16, ard.ARD_BF16, B, K, N, 2.0, Xd, K, dYd, N, 0, dW, K, 1, cs)
            seen = set()
            for it in range(6):
                g.replay()
                torch.cuda.synchronize()
                dp, b = OP.draw(cdf, 77, 500 + it, 3)
                seen.add(dp)
                mask = OP.row_mask(N, dp, b) if kind == "row" else OP.tile_mask(K, N, ts, dp, b)
                for got, want, name in ((Y, OG.fwd(X, W, mask, 2.0), "fwd"), (dX, OG.bwd_data(dY, W, mask, 2.0), "bwd_data"),
                                        (dW, OG.bwd_weight(X, dY, mask, 2.0).T, "bwd_weight")):
                    assert OG.rel_fro(host(got), want) <= TOL_BF16, (it, dp, b, name)
            assert len(seen) >= 2
        assert ard.ard_last_device_status(ctx.h) == 0
    finally:
        ctx.close()
