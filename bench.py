#!/usr/bin/env python
"""Benchmark of the ARD hot path on B200.

A "step" is one pass of the whole path over one batch: draw a fresh pattern from K on the device,
then the forward, backward-data and backward-weight GEMMs of the layer over the kept neurons only.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line (rank 0).  Workload `mlp8192_row` (the default) is the large MLP layer of the paper's
Table-1 sweep scaled to B200: W 8192x8192 bf16, batch 4096, row pattern, p = 0.5, K = the
maximum-entropy distribution over periods 1..16.  Other workloads (`--workload`): `mlp8192_tile`,
`mlp4096_tile`, `mlp2048_row` (single layers), `lstm1024` (a step is a whole sequence, forward + BPTT), `lstm1024x2_out` (two stacked
LSTM layers with dropout on the layer outputs only),
`mlp2048_step` / `mlp8192_step` (a step is a whole training iteration of a stack of layers, replayed from a
CUDA graph), `conv_rows` (a convolution layer as an im2col product with rows dropped by predicted sensitivity),
`conv_blocks` (the same layer with blocks of the input matrix dropped).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2203_05705_b200 import inputs  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum per launch of ard_gemm_tc_kernel, averaged over the three
# GEMMs of one step of the 8192 x 8192 layer at batch 4096, per period dp, from the ncu captures summarised
# under profiles/ (dp = 1: fwd 679.5 MB, bwd-data 674.4 MB, bwd-weight 390.3 MB; dp = 2, 4, 8, 16: the
# sparse-draw capture).  Periods in between are interpolated linearly in 1/dp, the kept share of the layer.
DRAM_TRAFFIC_BY_DP = {"row": {1: 581.0e6, 2: 257.0e6, 4: 130.8e6, 8: 71.3e6, 16: 60.5e6}, "tile": {}}

METRIC = "layer fwd+bwd kept TFLOP/s (row pattern, p=0.5)"
UNIT = "TFLOP/s"

WORKLOADS = {
    # name: (config, B, K, N, kind, ts, p, n_dp)
    "mlp8192_row": dict(config=5, B=4096, K=8192, N=8192, kind="row", ts=0, p=0.5, n_dp=16),
    "mlp8192_tile": dict(config=5, B=4096, K=8192, N=8192, kind="tile", ts=128, p=0.5, n_dp=16),
    "mlp4096_tile": dict(config=3, B=1024, K=4096, N=4096, kind="tile", ts=64, p=0.5, n_dp=16),
    "mlp2048_row": dict(config=2, B=128, K=2048, N=2048, kind="row", ts=0, p=0.5, n_dp=16),
    # whole training iteration of a stack of layers through ard_mlp_step (fused layer steps, compact matrices
    # between the hidden layers, one CUDA graph per iteration): the 784-2048-2048-10 network of config 2 and a
    # stack of large layers where the second hidden layer multiplies two compact matrices
    "mlp2048_step": dict(config=2, dims=[784, 2048, 2048, 10], B=128, kind="mlp_step", p=0.5, n_dp=16),
    "mlp8192_step": dict(config=5, dims=[8192, 8192, 8192, 1024], B=4096, kind="mlp_step", p=0.5, n_dp=16),
    # the other hidden sizes of the paper's MLP table (Sec. 7, Table 1: 1024 x 64, 1024 x 1024, 4096 x 4096; batch 128)
    "mlp1024x64_step": dict(config=2, dims=[784, 1024, 64, 10], B=128, kind="mlp_step", p=0.5, n_dp=16),
    "mlp1024_step": dict(config=2, dims=[784, 1024, 1024, 10], B=128, kind="mlp_step", p=0.5, n_dp=16),
    "mlp4096_step": dict(config=2, dims=[784, 4096, 4096, 10], B=128, kind="mlp_step", p=0.5, n_dp=16),
    # a convolution layer as the product of its im2col input matrix with the filters, rows of the input matrix
    # dropped by predicted sensitivity (Sec. 5.1, 5.2.1): 3x3 filters, 256 -> 512 channels, 32768 output positions
    # run_len = 32: the sampled values of the sensitivity prediction are taken in runs of 32 neighbours, a departure
    # from Sec. 5.1 (which samples single values: --conv-run-len 1) chosen for its memory traffic
    "conv_rows": dict(config=5, M=32768, K=2304, N=512, kind="conv_rows", region_rows=8, k_frac=0.05, run_len=32,
                      t_frac=0.3, threshold=0.5, m_prob=0.2, n_prob=0.8),
    # the same layer with blocks of the input matrix as the dropout granularity (Sec. 5.2.2)
    "conv_blocks": dict(config=5, M=32768, K=2304, N=512, kind="conv_blocks", ts=128, k_frac=0.05, run_len=32,
                        t_frac=0.3, threshold=0.5, cap=6, m_prob=0.2, n_prob=0.8),
    # LSTM layer (config 4): a step is one sequence, forward + BPTT, one fresh pattern per sequence
    "lstm1024": dict(config=4, T=35, B=64, I=1024, H=1024, kind="lstm", p=0.5, n_dp=16),
    # two stacked LSTM layers of that size with dropout on the layer outputs only (the non-recurrent connections):
    # the second layer's input half contracts over the kept outputs of the first
    "lstm1024x2_out": dict(config=4, T=35, B=64, dims=[1024, 1024, 1024], kind="lstm_stack", p=0.5, n_dp=16),
}

def max_entropy_K(p, n_dp):
    """K of every benchmark workload: over the periods dp = 1..n_dp, the distribution of greatest entropy whose
    global dropout rate sum_i k_i (i-1)/i (Eq. 2-3) is p, i.e. k_i proportional to exp(beta (i-1)/i) with beta by
    bisection.  It stands in for the output of the search of Sec. 3.3 (whose constants are not printed): K is an
    input of the hot path, this is the workload recipe's choice of it."""
    pu = np.array([(i - 1) / i for i in range(1, n_dp + 1)])
    if n_dp < 2 or not (0.0 < p < pu[-1]):
        raise ValueError("need n_dp >= 2 and 0 < p < (n_dp-1)/n_dp")
    lo, hi = -200.0, 200.0
    for _ in range(200):
        beta = 0.5 * (lo + hi)
        w = np.exp(beta * (pu - pu[-1])) if beta > 0 else np.exp(beta * pu)
        k = w / w.sum()
        if float(k @ pu) < p:
            lo = beta
        else:
            hi = beta
    return k / k.sum()


# Measured peaks of this machine's B200s (generated file), else the documented fallback.
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def kept_count(units, dp, b):
    return (units - b) // dp + 1


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "20"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    @staticmethod
    def _ts(s):
        import datetime
        try:
            return datetime.datetime.strptime(s, "%Y/%m/%d %H:%M:%S.%f").timestamp()
        except ValueError:
            return None

    def stop(self, t_begin=None, t_end=None):
        """Median SM clock over the samples taken inside [t_begin, t_end] (wall clock), else over the
        busier half of all samples."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons, inside, rec = [], [], set(), [], []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                clk = float(parts[1])
                mx.append(float(parts[2]))
            except ValueError:
                continue
            sm.append(clk)
            ts = self._ts(parts[0])
            rec.append((ts, clk, [nm for nm, val in zip(names, parts[4:8]) if val.lower().startswith("active")]))
        self.f.close()
        os.unlink(self.f.name)
        window = "whole run"
        if t_begin is not None:
            # samples inside the timed region; the region is short, so widen to +-0.3 s if fewer than 3 fall in it
            for margin, label in ((0.02, "timed region"), (0.3, "timed region +-0.3 s")):
                pick = [r for r in rec if r[0] is not None and t_begin - margin <= r[0] <= t_end + margin]
                if len(pick) >= 3 or margin == 0.3:
                    break
            if pick:
                inside = [r[1] for r in pick]
                window = label
                for r in pick:
                    reasons.update(r[2])
        if not inside:
            inside = sorted(sm)[len(sm) // 2:]
            for r in rec:
                reasons.update(r[2])
        if sm:
            out.update(sm_mhz=statistics.median(inside), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(inside), window=window)
        return out


def aggregate_over_ranks(ms, kept_flops, dense_flops, device="cpu"):
    """Whole-job figures from per-rank ones: the slowest rank's time, the sum of the work.  Uses the
    default process group (NCCL on the GPUs, gloo in the CPU test); identity for a single process."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms, kept_flops, dense_flops
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    f = torch.tensor([kept_flops, dense_flops], device=device, dtype=torch.float64)
    dist.all_reduce(f, op=dist.ReduceOp.SUM)
    return float(t.item()), float(f[0].item()), float(f[1].item())


def oracle_sample_seconds(wl, d, rows=256):
    """Times the fp64 oracle, as it stands, on a bounded sample of one step: `rows` batch rows of the
    forward and backward-data products and `rows` neuron columns of the backward-weight product,
    with the full weight and the dense mask.  Returns (seconds, kept flops of the sample, threads)."""
    from oracle import gemm as OG
    from oracle import pattern as OP
    K, N, B = wl["K"], wl["N"], wl["B"]
    dp, b = 2, 1
    mask = OP.row_mask(N, dp, b) if wl["kind"] == "row" else OP.tile_mask(K, N, wl["ts"], dp, b)
    alpha = 1.0 / (1.0 - wl["p"])
    sel = np.arange(0, B, max(1, B // rows))[:rows]
    cols = np.arange(0, N, max(1, N // rows))[:rows]
    t0 = time.perf_counter()
    OG.fwd_rows(d["X"], d["W"], mask, alpha, sel)
    OG.bwd_data_rows(d["dY"], d["W"], mask, alpha, sel)
    OG.bwd_weight_cols(d["X"], d["dY"], mask, alpha, cols)
    dt = time.perf_counter() - t0
    kept_frac = float(np.mean(mask))
    flops = 2.0 * len(sel) * K * N * kept_frac * 2 + 2.0 * B * K * len(cols) * float(np.mean(mask[..., cols]))
    try:
        from threadpoolctl import threadpool_info
        threads = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    return dt, flops, threads, f"{len(sel)} of {B} batch rows (fwd, bwd-data) + {len(cols)} of {N} neurons (bwd-weight), dp=2"


def run_reference(args, wl):
    """--impl reference: the CPU oracle on the host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    if wl["kind"] not in ("row", "tile"):
        print(json.dumps({"impl": "reference", "unavailable": "the reference arm covers the single-layer workloads; "
                          "for this one the oracle is timed in the cpu_baseline field of the ordinary run"}))
        return
    d = inputs.dense_layer(wl["config"], wl["B"], wl["K"], wl["N"], 1.0 / 90.0)
    rows = 64
    for _ in range(args.warmup):
        oracle_sample_seconds(wl, d, rows)
    tot_t, tot_f = 0.0, 0.0
    for _ in range(args.steps):
        dt, fl, threads, sample = oracle_sample_seconds(wl, d, rows)
        tot_t += dt
        tot_f += fl
    val = tot_f / tot_t / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": layer_config(args, wl, 1),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_lstm(args, wl):
    """LSTM workload: every step is one sequence (T time steps forward, then BPTT and the weight gradient)."""
    import torch
    from paper_2203_05705_b200 import ard
    from paper_2203_05705_b200.lstm import LstmLayer
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    clocks = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    T, B, I, H, p, n_dp = wl["T"], wl["B"], wl["I"], wl["H"], wl["p"], wl["n_dp"]
    c4 = inputs.config4(T, B, I, H, 0)
    bf = torch.bfloat16
    W = torch.from_numpy(np.ascontiguousarray(c4["W"].T)).to(bf).cuda()
    hX = torch.from_numpy(c4["X"]).to(bf).pin_memory()
    hdH = torch.from_numpy(c4["dH"]).pin_memory()
    X, dH = hX.cuda(), hdH.cuda()
    hH = torch.empty((T, B, H), dtype=bf).pin_memory()
    ctx = ard.ard_create(0, 2 * T * B * 4 * H + 4096)
    apply_options(ctx, args)
    ard.ard_set_distribution(ctx, 0, max_entropy_K(p, n_dp))
    pat = ard.ard_pattern_create(ctx, ard.ARD_ROW, I + H, H, 0)
    layer = LstmLayer(ctx, pat, T, B, I, H, W)
    alpha = 1.0 / (1.0 - p)

    def seq(it, dense=False, host=False, dist=0, scale=None, forced=None):
        if dense:
            ard.ard_pattern_set(ctx, pat, 1, 1)
        elif forced is not None:
            ard.ard_pattern_set(ctx, pat, forced, 1)
        else:
            ard.ard_sample_pattern(ctx, pat, dist, inputs.BASE_SEED, it, 4)
        if host:
            X.copy_(hX, non_blocking=True)
            dH.copy_(hdH, non_blocking=True)
        layer.load_inputs(X)
        Hs = layer.forward(alpha if scale is None else scale)
        layer.backward(alpha if scale is None else scale, dH)
        if host:
            hH.copy_(Hs, non_blocking=True)

    def timed(n, first, **kw):
        for w in range(args.warmup):
            seq(first + w, **kw)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record()
        for i in range(n):
            seq(first + args.warmup + i, **kw)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1), t0, time.time()

    steps = args.steps
    l0 = ard.ard_launch_count(ctx)
    ms, t0, t1 = timed(steps, 0)
    launches = (ard.ard_launch_count(ctx) - l0) * steps // (steps + args.warmup)
    clk = clocks.stop(t0, t1)
    status = ard.ard_last_device_status(ctx)
    nks = []
    for i in range(steps):
        ard.ard_sample_pattern(ctx, pat, 0, inputs.BASE_SEED, args.warmup + i, 4)
        nks.append(ard.ard_pattern_to_host(pat, 0)[2])
    per_unit = 3 * 2.0 * T * B * (I + H) * 4            # FLOPs per kept hidden unit and sequence
    kept = sum(per_unit * nk for nk in nks)
    value = kept / (ms * 1e-3) / 1e12
    ms_dense, _, _ = timed(max(5, steps // 4), 100000, dense=True)
    ms_e, _, _ = timed(max(5, steps // 4), 200000, host=True)
    ne = max(5, steps // 4)
    nks_e = []
    for i in range(ne):
        ard.ard_sample_pattern(ctx, pat, 0, inputs.BASE_SEED, 200000 + args.warmup + i, 4)
        nks_e.append(ard.ard_pattern_to_host(pat, 0)[2])
    # the other rates of the paper's LSTM experiment (Sec. 7), each with its own distribution over the periods, and
    # the sequence at a fixed period
    nsw = max(5, steps // 4)
    sweep, per_dp = {}, {}
    for di, rate in enumerate(() if args.quick else RATES):
        ard.ard_set_distribution(ctx, 1 + di, max_entropy_K(rate, n_dp))
        ms_r, _, _ = timed(nsw, 300000 + 1000 * di, dist=1 + di, scale=1.0 / (1.0 - rate))
        sweep["%.1f" % rate] = {"ms_per_step": ms_r / nsw}
    for dpf in () if args.quick else (1, 2, 3, 4, 6, 8, 12, 16):
        ms_f, _, _ = timed(nsw, 0, forced=dpf)
        per_dp[str(dpf)] = {"ms_per_step": ms_f / nsw}
    # dense library baseline for context: the same layer without dropout in torch.nn.LSTM (cuDNN), bf16
    ms_lib = None
    try:
        ref = torch.nn.LSTM(I, H, num_layers=1, bias=True).to(device="cuda", dtype=bf)
        ref.flatten_parameters()
        Xr = X.clone().requires_grad_(True)
        dHr = dH.to(bf)

        def lib_seq():
            for prm in ref.parameters():
                prm.grad = None
            Xr.grad = None
            out, _ = ref(Xr)
            out.backward(dHr)

        for _ in range(args.warmup):
            lib_seq()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        nl = max(5, steps // 4)
        e0.record()
        for _ in range(nl):
            lib_seq()
        e1.record()
        torch.cuda.synchronize()
        ms_lib = e0.elapsed_time(e1) / nl
    except Exception as ex:  # the library baseline is context only
        sys.stderr.write("torch.nn.LSTM baseline skipped: %r\n" % (ex,))
    peaks = load_peaks()
    cpu = None
    if not args.no_cpu_baseline:
        from oracle import lstm as OL
        from oracle import pattern as OP
        m = OP.row_mask(H, 2, 1)
        tc0 = time.perf_counter()
        fw = OL.fwd(c4["X"], c4["W"], None, m, alpha)
        OL.bwd(fw, c4["W"], m, alpha, c4["dH"])
        dt = time.perf_counter() - tc0
        try:
            from threadpoolctl import threadpool_info
            threads = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
        except Exception:
            threads = os.cpu_count() or 1
        cpu = {"value": per_unit * (H // 2) / dt / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": "one full sequence, dp=2", "seconds": dt}
    ms_own_dense = ms_dense / max(5, steps // 4)
    for v in list(sweep.values()) + list(per_dp.values()):
        v["speedup_vs_own_kernels_dp1"] = ms_own_dense / v["ms_per_step"]
        if ms_lib:
            v["speedup_vs_torch_nn_lstm"] = ms_lib / v["ms_per_step"]
    for k, v in sweep.items():
        v["ideal_speedup"] = 1.0 / (1.0 - float(k))
    line = {
        "metric": "LSTM layer fwd+BPTT kept TFLOP/s (row pattern on hidden units, p=0.5)", "value": value,
        "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": args.warmup, "ms_per_step": ms / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "T": T, "B": B, "I": I, "H": H, "p": p, "n_dp": n_dp,
                   "l2": "weights (16 MB) stay in L2 by design; a step is a whole sequence"},
        "dense_equiv_tflops": per_unit * H * steps / (ms * 1e-3) / 1e12, "clocks": clk,
        "e2e": {"value": sum(per_unit * nk for nk in nks_e) / (ms_e * 1e-3) / 1e12, "unit": UNIT,
                "h2d_bytes_per_step": hX.numel() * 2 + hdH.numel() * 4, "d2h_bytes_per_step": hH.numel() * 2,
                "ms_per_step": ms_e / ne},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "achieved": value, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": value / peaks["bf16_tflops"], "traffic": None,
                     "note": "35 dependent steps of a 64-row product: bound by per-step latency, not by the tensor pipe"},
        "cpu_baseline": cpu,
        "detail": {"dense_ms_per_step": {"own_kernels_dp1": ms_dense / max(5, steps // 4), "torch_nn_lstm": ms_lib},
                   "speedup_vs_dense": {str(p): min(ms_dense / max(5, steps // 4), ms_lib or 1e30) / (ms / steps)},
                   "kept_fraction": {str(p): float(np.mean(nks)) / H},
                   "rate_sweep": sweep, "per_dp": per_dp},
        "device_status": int(status),
    }
    print(json.dumps(line))
    ard.ard_pattern_destroy(pat)
    ard.ard_destroy(ctx)


def run_lstm_stack(args, wl):
    """A step is one sequence through the stack: a fresh pattern per layer, forward of all layers, BPTT of all layers."""
    import torch
    from paper_2203_05705_b200 import ard
    from paper_2203_05705_b200.lstm import LstmStack
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    clocks = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    T, B, dims, p, n_dp = wl["T"], wl["B"], wl["dims"], wl["p"], wl["n_dp"]
    L = len(dims) - 1
    bf = torch.bfloat16
    Ws, Xs = [], None
    for l in range(L):
        c4 = inputs.config4(T, B, dims[l], dims[l + 1], l)
        Ws.append(c4["W"])
        if l == 0:
            Xs = c4["X"]
    dY = inputs.config4(T, B, dims[-2], dims[-1], 0)["dH"]
    ctx = ard.ard_create(0, 2 * T * B * 4 * max(dims) + 4096)
    ard.ard_set_distribution(ctx, 0, max_entropy_K(p, n_dp))
    stack = LstmStack(ctx, T, B, dims, [torch.from_numpy(np.ascontiguousarray(W.T)).to(bf).cuda() for W in Ws])
    hX = torch.from_numpy(Xs).to(bf).pin_memory()
    hdY = torch.from_numpy(dY.reshape(T * B, -1)).to(bf).pin_memory()
    X, dYc = hX.cuda(), hdY.cuda()
    hY = torch.empty((T * B, dims[-1]), dtype=bf).pin_memory()
    alphas = [1.0 / (1.0 - p)] * L

    def seq(it, dense=False, host=False):
        for l in range(L):
            if dense:
                ard.ard_pattern_set(ctx, stack.out_pats[l], 1, 1)
            else:
                ard.ard_sample_pattern(ctx, stack.out_pats[l], 0, inputs.BASE_SEED, it, 10 + l)
        if host:
            X.copy_(hX, non_blocking=True)
            dYc.copy_(hdY, non_blocking=True)
        Yc = stack.forward(X, alphas)
        stack.backward(dYc, alphas)       # the first n_keep columns of dYc are read: a synthetic upstream gradient
        if host:
            hY.copy_(Yc, non_blocking=True)

    def timed(n, first, **kw):
        for w in range(args.warmup):
            seq(first + w, **kw)
        torch.cuda.synchronize()
        out = []
        for _ in range(3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0 = time.time()
            e0.record()
            for i in range(n):
                seq(first + args.warmup + i, **kw)
            e1.record()
            torch.cuda.synchronize()
            out.append((e0.elapsed_time(e1), t0, time.time()))
        out.sort()
        return out[1]

    def kept_flops(its):
        tot, fr = 0.0, []
        for it in its:
            n_in = []
            for l in range(L):
                ard.ard_sample_pattern(ctx, stack.out_pats[l], 0, inputs.BASE_SEED, it, 10 + l)
                n_in.append(ard.ard_pattern_to_host(stack.out_pats[l], 0)[2])
            for l in range(L):
                kin = dims[l] if l == 0 else n_in[l - 1]
                tot += 3 * 2.0 * T * B * (kin + dims[l + 1]) * 4 * dims[l + 1]
            fr.append([n_in[l] / dims[l + 1] for l in range(L)])
        return tot, fr

    steps = args.steps
    l0 = ard.ard_launch_count(ctx)
    ms, t0, t1 = timed(steps, 0)
    launches = (ard.ard_launch_count(ctx) - l0) * steps // (3 * steps + args.warmup)
    clk = clocks.stop(t0, t1)
    status = ard.ard_last_device_status(ctx)
    kept, fracs = kept_flops(range(args.warmup, args.warmup + steps))
    dense_flops = sum(3 * 2.0 * T * B * (dims[l] + dims[l + 1]) * 4 * dims[l + 1] for l in range(L))
    value = kept / (ms * 1e-3) / 1e12
    n2 = max(5, steps // 4)
    ms_dense = timed(n2, 100000, dense=True)[0] / n2
    ms_e = timed(n2, 200000, host=True)[0] / n2
    kept_e, _ = kept_flops(range(200000 + args.warmup, 200000 + args.warmup + n2))
    ms_lib = None
    try:
        ref = torch.nn.LSTM(dims[0], dims[1], num_layers=L, bias=True, dropout=p).to(device="cuda", dtype=bf)
        ref.train()
        ref.flatten_parameters()
        Xr = X.clone().requires_grad_(True)
        dHr = dYc.reshape(T, B, -1)

        def lib_seq():
            for prm in ref.parameters():
                prm.grad = None
            Xr.grad = None
            out, _ = ref(Xr)
            out.backward(dHr)

        for _ in range(args.warmup):
            lib_seq()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n2):
            lib_seq()
        e1.record()
        torch.cuda.synchronize()
        ms_lib = e0.elapsed_time(e1) / n2
    except Exception as ex:  # the library baseline is context only
        sys.stderr.write("torch.nn.LSTM baseline skipped: %r\n" % (ex,))
    peaks = load_peaks()
    cpu = None
    if not args.no_cpu_baseline:
        from oracle import lstm_stack as OS
        from oracle import pattern as OP
        masks = [OP.row_mask(dims[l + 1], 2, 1) for l in range(L)]
        tc0 = time.perf_counter()
        fw = OS.fwd(Xs, Ws, None, masks, alphas)
        OS.bwd(fw, Ws, masks, alphas, dY)
        dt = time.perf_counter() - tc0
        try:
            from threadpoolctl import threadpool_info
            threads = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
        except Exception:
            threads = os.cpu_count() or 1
        fl = sum(3 * 2.0 * T * B * ((dims[l] if l == 0 else dims[l] // 2) + dims[l + 1]) * 4 * dims[l + 1] for l in range(L))
        cpu = {"value": fl / dt / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": "one full sequence through the stack, dp=2 on every layer's output", "seconds": dt}
    best_dense = min(ms_dense, ms_lib or 1e30)
    line = {
        "metric": "stacked LSTM fwd+BPTT kept TFLOP/s (row pattern on every layer's outputs, p=%s)" % p, "value": value,
        "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": args.warmup, "ms_per_step": ms / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "T": T, "B": B, "dims": dims, "p": p, "n_dp": n_dp,
                   "l2": "weights (%d MB) stay in L2 by design; a step is a whole sequence" % (sum(w.size for w in Ws) * 2 // 2 ** 20)},
        "dense_equiv_tflops": dense_flops * steps / (ms * 1e-3) / 1e12, "clocks": clk,
        "e2e": {"value": kept_e / n2 / (ms_e * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": hX.numel() * 2 + hdY.numel() * 2,
                "d2h_bytes_per_step": hY.numel() * 2, "ms_per_step": ms_e},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "achieved": value, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": value / peaks["bf16_tflops"], "traffic": None,
                     "note": "35 dependent steps of a 64-row product per layer: bound by per-step latency, not by the tensor "
                             "pipe; only the input half of the upper layer shrinks with the pattern"},
        "cpu_baseline": cpu,
        "detail": {"dense_ms_per_step": {"own_kernels_dp1": ms_dense, "torch_nn_lstm_2_layers_dropout": ms_lib},
                   "speedup_vs_dense": {str(p): best_dense / (ms / steps)},
                   "kept_fraction_of_outputs": {str(p): [float(x) for x in np.mean(np.array(fracs), axis=0)]}},
        "device_status": int(status),
    }
    print(json.dumps(line))
    stack.close()
    ard.ard_destroy(ctx)


def apply_options(ctx, args):
    """--opt NAME=VALUE: tuning switches of the context (ard_set_option)."""
    from paper_2203_05705_b200 import ard
    for kv in getattr(args, "opt", []):
        name, val = kv.split("=")
        ard.ard_set_option(ctx, getattr(ard, "ARD_OPT_" + name.upper()), int(val))


def run_mlp_step(args, wl):
    """A step is one training iteration of the whole stack: patterns drawn on the device, forward chain,
    backward chain (weight, bias and input gradients), as ONE native call replayed from a CUDA graph."""
    import torch
    from paper_2203_05705_b200 import ard
    dev_index = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(dev_index)
    clocks = ClockSampler(dev_index)
    dims, B, p, n_dp = wl["dims"], wl["B"], wl["p"], wl["n_dp"]
    L = len(dims) - 1
    bf = torch.bfloat16
    alpha = 1.0 / (1.0 - p)
    ctx = ard.ard_create(0, 2 * B * max(dims) + 4096)
    apply_options(ctx, args)
    ard.ard_set_compact_reuse(ctx, 1)
    Kd = max_entropy_K(p, n_dp)
    ard.ard_set_distribution(ctx, 0, Kd)
    g = torch.Generator(device="cuda").manual_seed(inputs.BASE_SEED)
    hX = torch.rand((B, dims[0]), generator=torch.Generator().manual_seed(1)).to(bf).pin_memory()
    hdO = (torch.randn((B, dims[-1]), generator=torch.Generator().manual_seed(2)) / B).to(bf).pin_memory()
    hOut = torch.empty((B, dims[-1]), dtype=bf).pin_memory()
    X, dOut = hX.cuda(), hdO.cuda()

    def make_stack(compact):
        layers, keep = [], []
        for l in range(L):
            K, N = dims[l], dims[l + 1]
            hidden = l < L - 1
            d = dict(K=K, N=N, pat=ard.ard_pattern_create(ctx, ard.ARD_ROW, K, N, 0), sample=1 if hidden else 0,
                     relu=1 if hidden else 0, compact_out=1 if (hidden and compact) else 0, dW_is_f32=0,
                     alpha=alpha if hidden else 1.0, ldw=K,
                     W=(torch.randn((N, K), device="cuda", generator=g) * (2.0 / K) ** 0.5).to(bf),
                     bias=torch.zeros(N, device="cuda"), Wk=torch.zeros((N, K), dtype=bf, device="cuda"),
                     A=torch.zeros((B, N), dtype=bf, device="cuda"), dZ=torch.zeros((B, N), dtype=bf, device="cuda"),
                     dWk=torch.zeros((N, K), dtype=bf, device="cuda"), dW=torch.zeros((N, K), dtype=bf, device="cuda"),
                     db=torch.zeros(N, device="cuda"))
            layers.append(d)
        ard.ard_pattern_set(ctx, layers[-1]["pat"], 1, 1)
        return layers, ard.mlp_layers(layers)

    counter = torch.zeros(1, dtype=torch.int64, device="cuda")
    dX = torch.zeros((B, dims[0]), dtype=bf, device="cuda")
    base = 7000

    def eager(stack, sample=True):
        ard.ard_mlp_step(ctx, stack[1], L, B, X, dims[0], dOut, dims[-1], dX, dims[0], 0, inputs.BASE_SEED, base, counter)

    def graphed(stack):
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            eager(stack)                     # warm-up; the context creates its side streams outside the capture
        torch.cuda.synchronize()
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            eager(stack)
        return gr

    def timed(fn, n, warm):
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1), t0, time.time()

    compact = make_stack(1)
    gr = graphed(compact)
    steps, warm = args.steps, max(3, args.warmup)
    # headline: graph replays of the compact chain; the realised patterns are read back afterwards by
    # replaying the same iterations one call at a time
    counter.zero_()
    l0 = ard.ard_launch_count(ctx)
    eager(compact)
    torch.cuda.synchronize()
    launches_per_step = int(ard.ard_launch_count(ctx) - l0)
    counter.zero_()
    ms, t0, t1 = timed(gr.replay, steps, warm)
    clk = clocks.stop(t0, t1)
    status = ard.ard_last_device_status(ctx)
    # kept FLOPs of the timed iterations (iteration = base + warm + i; stream id = layer + 1)
    def kept_flops(it):
        n = [dims[0]]
        for l in range(L - 1):
            ard.ard_sample_pattern(ctx, compact[0][l]["pat"], 0, inputs.BASE_SEED, it, l + 1)
            n.append(ard.ard_pattern_to_host(compact[0][l]["pat"], 0)[2])
        n.append(dims[-1])
        fl = 0.0
        for l in range(L):
            fl += 2.0 * B * n[l] * n[l + 1] * 3            # forward, weight gradient, input gradient
        return fl, n
    kept = 0.0
    fracs = []
    for i in range(steps):
        f, n = kept_flops(base + warm + i)
        kept += f
        fracs.append([n[l + 1] / dims[l + 1] for l in range(L - 1)])
    dense_flops = sum(2.0 * B * dims[l] * dims[l + 1] * 3 for l in range(L))
    value = kept / (ms * 1e-3) / 1e12
    detail = {"ms_per_step": {"graph_compact": ms / steps}}
    if not args.quick:
        n2 = max(5, steps // 4)
        # cold L2: a 256 MB buffer is overwritten between the replays (the weights, 12 - 290 MB here, otherwise stay in
        # the 126 MB L2 from one iteration to the next); the cost of the overwriting alone is timed and subtracted
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

        def cold_step():
            flush.fill_(1)
            gr.replay()

        t_cold = timed(cold_step, n2, warm)[0] / n2
        t_flush = timed(lambda: flush.fill_(1), n2, warm)[0] / n2
        detail["ms_per_step"]["graph_compact_cold_l2"] = t_cold - t_flush
        detail["ms_per_step"]["graph_compact_warm_l2"] = ms / steps
        del flush
        detail["ms_per_step"]["eager_compact"] = timed(lambda: eager(compact), n2, warm)[0] / n2
        # the same iterations call by call (one launch per product, three streams) instead of the one-kernel form
        if launches_per_step == 1:
            ard.ard_set_option(ctx, ard.ARD_OPT_MLP_PERSISTENT, 0)
            gr_c = graphed(compact)
            detail["ms_per_step"]["graph_compact_call_by_call"] = timed(gr_c.replay, n2, warm)[0] / n2
            detail["ms_per_step"]["eager_compact_call_by_call"] = timed(lambda: eager(compact), n2, warm)[0] / n2
            ard.ard_set_option(ctx, ard.ARD_OPT_MLP_PERSISTENT, 1)
            del gr_c
        fullw = make_stack(0)
        gr_f = graphed(fullw)
        detail["ms_per_step"]["graph_full_width"] = timed(gr_f.replay, n2, warm)[0] / n2
        detail["ms_per_step"]["eager_full_width"] = timed(lambda: eager(fullw), n2, warm)[0] / n2
        # the same iteration at dp = 1 everywhere (nothing dropped), own kernels
        for d in compact[0][:-1]:
            d["sample"] = 0
            ard.ard_pattern_set(ctx, d["pat"], 1, 1)
        dense_stack = (compact[0], ard.mlp_layers(compact[0]))
        gr_d = graphed(dense_stack)
        detail["ms_per_step"]["graph_own_kernels_dp1"] = timed(gr_d.replay, n2, warm)[0] / n2
        # library baseline: the same network with conventional dropout in torch (bf16 autograd), eager and graphed
        Wt = [d["W"].clone().requires_grad_(True) for d in compact[0]]
        bt = [d["bias"].to(bf).clone().requires_grad_(True) for d in compact[0]]
        Xt = X.clone().requires_grad_(True)

        def torch_step():
            for t in Wt + bt + [Xt]:
                t.grad = None
            a = Xt
            for l in range(L):
                a = torch.nn.functional.linear(a, Wt[l], bt[l])
                if l < L - 1:
                    a = torch.nn.functional.dropout(torch.relu(a), p, True)
            a.backward(dOut)

        detail["ms_per_step"]["torch_eager_dropout"] = timed(torch_step, n2, warm)[0] / n2
        try:
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                for _ in range(3):
                    torch_step()
            torch.cuda.synchronize()
            gt = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gt):
                torch_step()
            detail["ms_per_step"]["torch_graph_dropout"] = timed(gt.replay, n2, warm)[0] / n2
        except Exception as ex:
            sys.stderr.write("torch graph baseline skipped: %r\n" % (ex,))
        best_dense = min(v for k, v in detail["ms_per_step"].items() if k.startswith("torch") or k.endswith("dp1"))
        detail["speedup_vs_dense"] = {str(p): best_dense / (ms / steps)}
        # the paper's sweep over the dropout rate on this network (Sec. 7, Table 1 reports conventional dropout /
        # ARD): graph replays of the iteration at p = 0.3, 0.5, 0.7 (maximum-entropy K for each rate, rescale 1/(1-p))
        # against torch's conventional dropout in a graph (whose time does not depend on p) and the own kernels
        # with nothing dropped
        sweep = {}
        for di, rate in enumerate(RATES):
            ard.ard_set_distribution(ctx, 1 + di, max_entropy_K(rate, n_dp))
            for d in compact[0][:-1]:
                d["sample"] = 1
                d["alpha"] = 1.0 / (1.0 - rate)
            st_r = (compact[0], ard.mlp_layers(compact[0]))

            def eager_r():
                ard.ard_mlp_step(ctx, st_r[1], L, B, X, dims[0], dOut, dims[-1], dX, dims[0], 1 + di, inputs.BASE_SEED,
                                 base, counter)

            sr = torch.cuda.Stream()
            with torch.cuda.stream(sr):
                eager_r()
            torch.cuda.synchronize()
            gr_r = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gr_r):
                eager_r()
            t_r = timed(gr_r.replay, max(20, steps), warm)[0] / max(20, steps)
            sweep[str(rate)] = {"ms_per_step": t_r, "ideal_speedup": 1.0 / (1.0 - rate),
                                "speedup_vs_own_kernels_dp1": detail["ms_per_step"]["graph_own_kernels_dp1"] / t_r}
            if "torch_graph_dropout" in detail["ms_per_step"]:
                sweep[str(rate)]["speedup_vs_torch_graph_dropout"] = detail["ms_per_step"]["torch_graph_dropout"] / t_r
            sweep[str(rate)]["speedup_vs_torch_eager_dropout"] = detail["ms_per_step"]["torch_eager_dropout"] / t_r
            del gr_r
        detail["rate_sweep"] = sweep
        for d in compact[0][:-1]:
            d["alpha"] = alpha
        # end to end: the input batch and the loss gradient come from pinned host memory and the network's
        # output goes back every iteration
        for d in compact[0][:-1]:
            d["sample"] = 1
        compact = (compact[0], ard.mlp_layers(compact[0]))

        def e2e_step():
            X.copy_(hX, non_blocking=True)
            dOut.copy_(hdO, non_blocking=True)
            eager(compact)
            hOut.copy_(compact[0][-1]["A"], non_blocking=True)

        counter.zero_()
        ms_e = timed(e2e_step, n2, warm)[0] / n2
        kept_e = sum(kept_flops(base + warm + i)[0] for i in range(n2))
        e2e = {"value": kept_e / n2 / (ms_e * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": hX.numel() * 2 + hdO.numel() * 2,
               "d2h_bytes_per_step": hOut.numel() * 2, "ms_per_step": ms_e}
    else:
        e2e = None
    peaks = load_peaks()
    cpu = None
    if not args.no_cpu_baseline and not args.quick:
        from oracle import mlp as OM
        from oracle import pattern as OP
        rows = min(B, 256)
        Ws = [d["W"].float().cpu().numpy().T.astype(np.float64) for d in compact[0]]
        masks = [OP.row_mask(dims[l + 1], 2, 1) for l in range(L - 1)] + [np.ones(dims[-1])]
        Xh = hX[:rows].float().numpy()
        tc0 = time.perf_counter()
        fw = OM.fwd(Xh, Ws, None, masks, [alpha] * (L - 1) + [1.0])
        OM.bwd(fw, Ws, masks, [alpha] * (L - 1) + [1.0], hdO[:rows].float().numpy())
        dt = time.perf_counter() - tc0
        try:
            from threadpoolctl import threadpool_info
            threads = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
        except Exception:
            threads = os.cpu_count() or 1
        n = [dims[0]] + [dims[l + 1] // 2 for l in range(L - 1)] + [dims[-1]]
        cpu = {"value": sum(2.0 * rows * n[l] * n[l + 1] * 3 for l in range(L)) / dt / 1e12, "unit": UNIT, "cores": threads,
               "kind": "oracle", "sample": "%d batch rows of one iteration, dp=2 on every hidden layer" % rows, "seconds": dt}
    line = {
        "metric": "MLP training iteration kept TFLOP/s (row patterns on the hidden layers, p=%s)" % p, "value": value,
        "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": warm, "ms_per_step": ms / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "dims": dims, "B": B, "p": p, "n_dp": n_dp,
                   "l2": "a fresh pattern every iteration; working set %.0f MB" % (sum(dims[l] * dims[l + 1] for l in range(L)) * 2 / 1e6)},
        "dense_equiv_tflops": dense_flops * steps / (ms * 1e-3) / 1e12, "clocks": clk, "e2e": e2e,
        "gpu_launches": launches_per_step * steps,
        "roofline": {"bound": "tensor", "achieved": value, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": value / peaks["bf16_tflops"], "traffic": None,
                     "note": "whole iteration incl. sampler, weight compaction, gradient expansion and bias gradients"},
        "cpu_baseline": cpu,
        "detail": dict(detail, kept_fraction_per_hidden_layer=[float(np.mean([f[l] for f in fracs])) for l in range(L - 1)],
                       launches_per_step=launches_per_step),
        "device_status": int(status),
    }
    print(json.dumps(line))


def run_conv_rows(args, wl):
    """A step = sensitivity prediction + row sampling + gathering the kept rows of the input matrix and of the output
    gradient + the three products on the gathered matrices (results filled back into the kept rows); gathers and
    products through one call, ard_rows_products."""
    import torch
    from paper_2203_05705_b200 import ard
    dev_index = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(dev_index)
    clocks = ClockSampler(dev_index)
    M, K, N, x = wl["M"], wl["K"], wl["N"], wl["region_rows"]
    bf = torch.bfloat16
    g = torch.Generator(device="cuda").manual_seed(inputs.BASE_SEED)
    # post-ReLU-like input matrix with quiet and busy regions, so that both kinds of region occur
    level = torch.tensor([0.1, 1.0, 4.0], device="cuda")[torch.randint(0, 3, (M // x,), device="cuda", generator=g)]
    A = (torch.relu(torch.randn((M, K), device="cuda", generator=g)) * level.repeat_interleave(x)[:, None]).to(bf)
    W = (torch.randn((N, K), device="cuda", generator=g) / K ** 0.5).to(bf)
    dY = torch.randn((M, N), device="cuda", generator=g).to(bf)
    Y = torch.empty((M, N), dtype=bf, device="cuda")
    dA = torch.empty((M, K), dtype=bf, device="cuda")
    dW = torch.empty((N, K), dtype=bf, device="cuda")
    hA, hdY = A.cpu().pin_memory(), dY.cpu().pin_memory()
    hY = torch.empty((M, N), dtype=bf).pin_memory()
    ctx = ard.ard_create(0, 4096)
    rows = ard.ard_rows_create(ctx, M, x)
    cap = (M + 63) // 64 * 64
    Ak = torch.zeros((cap, K), dtype=bf, device="cuda")    # the dense small matrices of Sec. 5.2.1
    dYk = torch.zeros((cap, N), dtype=bf, device="cuda")

    def step(it, dense=False, host=False, gathered=True):
        if host:
            A.copy_(hA, non_blocking=True)
            dY.copy_(hdY, non_blocking=True)
        if dense:
            ard.ard_rows_set_probability(ctx, rows, 0.0)
        else:
            ard.ard_sensitivity_predict(ctx, rows, ard.ARD_BF16, A, K, K, wl["k_frac"], wl["run_len"], wl["t_frac"], wl["threshold"],
                                        wl["m_prob"], wl["n_prob"], inputs.BASE_SEED, it, 0)
        ard.ard_rows_sample(ctx, rows, inputs.BASE_SEED, it, 0)
        if gathered:
            # gather the kept rows once per operand, multiply dense, fill back; the gathered input serves the
            # forward product and the weight gradient
            ard.ard_rows_gather(ctx, rows, M, K, A, K, Ak, K)
            ard.ard_rows_fwd_compact(ctx, rows, M, K, N, 1.0, Ak, K, W, K, Y, N)
            ard.ard_rows_gather(ctx, rows, M, N, dY, N, dYk, N)
            ard.ard_rows_bwd_data_compact(ctx, rows, M, K, N, 1.0, dYk, N, W, K, dA, K)
            ard.ard_rows_bwd_weight_compact(ctx, rows, ard.ARD_BF16, M, K, N, 1.0, Ak, K, dYk, N, dW, K)
        else:
            # the producer warps of the GEMM kernel follow the list themselves
            ard.ard_rows_fwd(ctx, rows, M, K, N, 1.0, A, K, W, K, Y, N)
            ard.ard_rows_bwd_data(ctx, rows, M, K, N, 1.0, dY, N, W, K, dA, K)
            ard.ard_rows_bwd_weight(ctx, rows, ard.ARD_BF16, M, K, N, 1.0, A, K, dY, N, dW, K)
        if host:
            hY.copy_(Y, non_blocking=True)

    def step_one_call(it, host=False):
        """The same work through ard_rows_products: both gathers and the three products in one call, the
        output-gradient half on the context's side stream beside the input half."""
        if host:
            A.copy_(hA, non_blocking=True)
            dY.copy_(hdY, non_blocking=True)
        ard.ard_sensitivity_predict(ctx, rows, ard.ARD_BF16, A, K, K, wl["k_frac"], wl["run_len"], wl["t_frac"], wl["threshold"],
                                    wl["m_prob"], wl["n_prob"], inputs.BASE_SEED, it, 0)
        ard.ard_rows_sample(ctx, rows, inputs.BASE_SEED, it, 0)
        ard.ard_rows_products(ctx, rows, ard.ARD_BF16, M, K, N, 1.0, A, K, W, K, dY, N, Ak, K, dYk, N, Y, N, dA, K, dW, K)
        if host:
            hY.copy_(Y, non_blocking=True)

    def timed(fn, n, warm):
        for w in range(warm):
            fn(w)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record()
        for i in range(n):
            fn(warm + i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1), t0, time.time()

    steps, warm = args.steps, max(3, args.warmup)
    l0 = ard.ard_launch_count(ctx)
    ms, t0, t1 = timed(step_one_call, steps, warm)
    launches = (ard.ard_launch_count(ctx) - l0) * steps // (steps + warm)
    clk = clocks.stop(t0, t1)
    status = ard.ard_last_device_status(ctx)
    kept_rows = []
    for i in range(steps):
        ard.ard_sensitivity_predict(ctx, rows, ard.ARD_BF16, A, K, K, wl["k_frac"], wl["run_len"], wl["t_frac"], wl["threshold"],
                                    wl["m_prob"], wl["n_prob"], inputs.BASE_SEED, warm + i, 0)
        ard.ard_rows_sample(ctx, rows, inputs.BASE_SEED, warm + i, 0)
        kept_rows.append(ard.ard_rows_to_host(rows, 0)[0])
    kept = sum(3 * 2.0 * nk * K * N for nk in kept_rows)
    value = kept / (ms * 1e-3) / 1e12
    detail = {"ms_per_step": {"ours": ms / steps}, "kept_row_fraction": float(np.mean(kept_rows)) / M}
    e2e = None
    if not args.quick:
        n2 = max(5, steps // 4)
        detail["ms_per_step"]["own_kernels_all_rows"] = timed(lambda it: step(it, dense=True), n2, warm)[0] / n2
        detail["ms_per_step"]["gather_inside_the_gemm_kernels"] = timed(lambda it: step(it, gathered=False), n2, warm)[0] / n2
        detail["ms_per_step"]["calls_in_sequence_on_one_stream"] = timed(step, n2, warm)[0] / n2
        # per stage, serialised (one stage per timed loop)
        stage = {}
        stage["sensitivity_predict"] = lambda it: ard.ard_sensitivity_predict(
            ctx, rows, ard.ARD_BF16, A, K, K, wl["k_frac"], wl["run_len"], wl["t_frac"], wl["threshold"], wl["m_prob"], wl["n_prob"],
            inputs.BASE_SEED, 1, 0)
        stage["sensitivity_predict_single_values"] = lambda it: ard.ard_sensitivity_predict(
            ctx, rows, ard.ARD_BF16, A, K, K, wl["k_frac"], 1, wl["t_frac"], wl["threshold"], wl["m_prob"], wl["n_prob"],
            inputs.BASE_SEED, 1, 0)
        stage["rows_sample"] = lambda it: ard.ard_rows_sample(ctx, rows, inputs.BASE_SEED, 1, 0)
        stage["gather_A"] = lambda it: ard.ard_rows_gather(ctx, rows, M, K, A, K, Ak, K)
        stage["gather_dY"] = lambda it: ard.ard_rows_gather(ctx, rows, M, N, dY, N, dYk, N)
        stage["fwd(+zero rows)"] = lambda it: ard.ard_rows_fwd_compact(ctx, rows, M, K, N, 1.0, Ak, K, W, K, Y, N)
        stage["bwd_data(+zero rows)"] = lambda it: ard.ard_rows_bwd_data_compact(ctx, rows, M, K, N, 1.0, dYk, N, W, K, dA, K)
        stage["bwd_weight"] = lambda it: ard.ard_rows_bwd_weight_compact(ctx, rows, ard.ARD_BF16, M, K, N, 1.0, Ak, K, dYk,
                                                                         N, dW, K)
        step(1)
        detail["us_per_stage"] = {k: round(timed(f, n2, warm)[0] / n2 * 1e3, 1) for k, f in stage.items()}

        def torch_step(it):
            torch.matmul(A, W.t(), out=Y)
            torch.matmul(dY, W, out=dA)
            torch.matmul(dY.t(), A, out=dW)

        detail["ms_per_step"]["torch_matmul_dense"] = timed(torch_step, n2, warm)[0] / n2
        detail["speedup_vs_dense"] = min(detail["ms_per_step"]["own_kernels_all_rows"],
                                         detail["ms_per_step"]["torch_matmul_dense"]) / (ms / steps)
        ms_e = timed(lambda it: step_one_call(it + 100000, host=True), n2, warm)[0] / n2
        e2e = {"value": float(np.mean(kept_rows)) * 3 * 2.0 * K * N / (ms_e * 1e-3) / 1e12, "unit": UNIT,
               "h2d_bytes_per_step": hA.numel() * 2 + hdY.numel() * 2, "d2h_bytes_per_step": hY.numel() * 2,
               "ms_per_step": ms_e}
    peaks = load_peaks()
    cpu = None
    if not args.no_cpu_baseline and not args.quick:
        from oracle import cnn as OC
        Mh = 2048
        Ah, Wh, dYh = A[:Mh].float().cpu().numpy(), W.float().cpu().numpy().T, dY[:Mh].float().cpu().numpy()
        keep = np.arange(0, Mh, 2)
        tc0 = time.perf_counter()
        OC.fwd(Ah, Wh, keep)
        OC.bwd_data(dYh, Wh, keep)
        OC.bwd_weight(Ah, dYh, keep)
        dt = time.perf_counter() - tc0
        try:
            from threadpoolctl import threadpool_info
            threads = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
        except Exception:
            threads = os.cpu_count() or 1
        cpu = {"value": 3 * 2.0 * len(keep) * K * N / dt / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": "%d of %d rows of the input matrix, every second one kept (the oracle multiplies the masked full matrix)" % (Mh, M),
               "seconds": dt}
    line = {
        "metric": "convolution layer (im2col product) fwd+bwd kept TFLOP/s, rows dropped by predicted sensitivity",
        "value": value, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": warm, "ms_per_step": ms / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, **{k: wl[k] for k in ("M", "K", "N", "region_rows", "k_frac", "run_len",
                                                                       "t_frac", "threshold", "m_prob", "n_prob")},
                   "sampling": ("single values, as Sec. 5.1 states" if wl["run_len"] == 1 else
                                "runs of %d neighbouring values: a departure from Sec. 5.1" % wl["run_len"]),
                   "l2": "working set %.0f MB per step" % ((2 * M * K + 2 * M * N + 2 * N * K) * 2 / 1e6)},
        "dense_equiv_tflops": 3 * 2.0 * M * K * N * steps / (ms * 1e-3) / 1e12, "clocks": clk, "e2e": e2e,
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "achieved": value, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": value / peaks["bf16_tflops"], "traffic": None,
                     "note": "whole step incl. sensitivity prediction, row sampling and zero fill of the dropped rows"},
        "cpu_baseline": cpu, "detail": detail, "device_status": int(status),
    }
    print(json.dumps(line))
    ard.ard_rows_destroy(rows)
    ard.ard_destroy(ctx)


def run_conv_blocks(args, wl):
    """A step = per-block sensitivity counts + labels (at most `cap` sensitive blocks per group) + block draws +
    index lists + the three products over the kept blocks of the input matrix, through ard_blocks_products."""
    import torch
    from paper_2203_05705_b200 import ard
    dev_index = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(dev_index)
    clocks = ClockSampler(dev_index)
    M, K, N, ts = wl["M"], wl["K"], wl["N"], wl["ts"]
    G, Q = M // ts, K // ts
    bf = torch.bfloat16
    g = torch.Generator(device="cuda").manual_seed(inputs.BASE_SEED)
    # post-ReLU-like input matrix with quiet and busy blocks, so that both labels occur
    level = torch.tensor([0.1, 1.0, 4.0], device="cuda")[torch.randint(0, 3, (G, Q), device="cuda", generator=g)]
    A = (torch.relu(torch.randn((M, K), device="cuda", generator=g))
         * level.repeat_interleave(ts, 0).repeat_interleave(ts, 1)).to(bf)
    W = (torch.randn((N, K), device="cuda", generator=g) / K ** 0.5).to(bf)
    dYt = torch.randn((N, M), device="cuda", generator=g).to(bf)       # output gradient, one row per channel
    Yt = torch.empty((N, M), dtype=bf, device="cuda")
    dA = torch.empty((M, K), dtype=bf, device="cuda")
    dW = torch.empty((N, K), dtype=bf, device="cuda")
    hA, hdY = A.cpu().pin_memory(), dYt.cpu().pin_memory()
    hY = torch.empty((N, M), dtype=bf).pin_memory()
    ctx = ard.ard_create(0, 4096)
    blocks = ard.ard_blocks_create(ctx, M, K, ts)

    def sample(it):
        ard.ard_blocks_predict(ctx, blocks, ard.ARD_BF16, A, K, wl["k_frac"], wl["run_len"], wl["t_frac"], wl["threshold"], wl["cap"],
                               inputs.BASE_SEED, it, 0)
        ard.ard_blocks_sample(ctx, blocks, wl["m_prob"], wl["n_prob"], inputs.BASE_SEED, it, 0)

    def products():
        ard.ard_blocks_products(ctx, blocks, ard.ARD_BF16, N, 1.0, A, K, W, K, dYt, M, Yt, M, dW, K, dA, K, 1)

    def step(it, host=False, dense=False):
        if host:
            A.copy_(hA, non_blocking=True)
            dYt.copy_(hdY, non_blocking=True)
        if dense:
            ard.ard_blocks_set_label(ctx, blocks, 1)
            ard.ard_blocks_sample(ctx, blocks, 0.0, 0.0, inputs.BASE_SEED, it, 0)
        else:
            sample(it)
        products()
        if host:
            hY.copy_(Yt, non_blocking=True)

    def timed(fn, n, warm):
        for w in range(warm):
            fn(w)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record()
        for i in range(n):
            fn(warm + i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1), t0, time.time()

    steps, warm = args.steps, max(3, args.warmup)
    l0 = ard.ard_launch_count(ctx)
    ms, t0, t1 = timed(step, steps, warm)
    launches = (ard.ard_launch_count(ctx) - l0) * steps // (steps + warm)
    clk = clocks.stop(t0, t1)
    status = ard.ard_last_device_status(ctx)
    kept_blocks = []
    for i in range(steps):
        sample(warm + i)
        kept_blocks.append(int(ard.ard_blocks_to_host(blocks, G * Q)[2].sum()))
    flops_per_block = 3 * 2.0 * ts * ts * N
    value = sum(kept_blocks) * flops_per_block / (ms * 1e-3) / 1e12
    detail = {"ms_per_step": {"ours": ms / steps}, "kept_block_fraction": float(np.mean(kept_blocks)) / (G * Q)}
    e2e = None
    if not args.quick:
        n2 = max(5, steps // 4)
        detail["ms_per_step"]["own_kernels_all_blocks"] = timed(lambda it: step(it, dense=True), n2, warm)[0] / n2
        detail["us_per_stage"] = {"predict+sample": round(timed(sample, n2, warm)[0] / n2 * 1e3, 1)}
        sample(1)
        detail["us_per_stage"]["products"] = round(timed(lambda it: products(), n2, warm)[0] / n2 * 1e3, 1)

        def torch_step(it):
            torch.matmul(W, A.t(), out=Yt)
            torch.matmul(dYt, A, out=dW)
            torch.matmul(dYt.t(), W, out=dA)

        detail["ms_per_step"]["torch_matmul_dense"] = timed(torch_step, n2, warm)[0] / n2
        detail["speedup_vs_dense"] = min(detail["ms_per_step"]["own_kernels_all_blocks"],
                                         detail["ms_per_step"]["torch_matmul_dense"]) / (ms / steps)
        ms_e = timed(lambda it: step(it + 100000, host=True), n2, warm)[0] / n2
        e2e = {"value": float(np.mean(kept_blocks)) * flops_per_block / (ms_e * 1e-3) / 1e12, "unit": UNIT,
               "h2d_bytes_per_step": hA.numel() * 2 + hdY.numel() * 2, "d2h_bytes_per_step": hY.numel() * 2,
               "ms_per_step": ms_e}
    peaks = load_peaks()
    cpu = None
    if not args.no_cpu_baseline and not args.quick:
        from oracle import cnn_blocks as OB
        Mh = 2048
        Ah, Wh, dYh = A[:Mh].float().cpu().numpy(), W.float().cpu().numpy().T, dYt[:, :Mh].float().cpu().numpy().T
        keep = (np.add.outer(np.arange(Mh // ts), np.arange(Q)) % 2 == 0)
        tc0 = time.perf_counter()
        OB.fwd(Ah, Wh, keep, ts)
        OB.bwd_input(dYh, Wh, keep, ts)
        OB.bwd_weight(Ah, dYh, keep, ts)
        dt = time.perf_counter() - tc0
        try:
            from threadpoolctl import threadpool_info
            threads = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
        except Exception:
            threads = os.cpu_count() or 1
        cpu = {"value": int(keep.sum()) * flops_per_block / dt / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": "%d of %d rows of the input matrix, every second block kept (the oracle multiplies the masked full matrix)" % (Mh, M),
               "seconds": dt}
    line = {
        "metric": "convolution layer (im2col product) fwd+bwd kept TFLOP/s, blocks dropped by predicted sensitivity",
        "value": value, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": warm, "ms_per_step": ms / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, **{k: wl[k] for k in ("M", "K", "N", "ts", "k_frac", "run_len", "t_frac",
                                                                       "threshold", "cap", "m_prob", "n_prob")},
                   "sampling": ("single values, as Sec. 5.1 states" if wl["run_len"] == 1 else
                                "runs of %d neighbouring values: a departure from Sec. 5.1" % wl["run_len"]),
                   "l2": "working set %.0f MB per step" % ((2 * M * K + 2 * M * N + 2 * N * K) * 2 / 1e6)},
        "dense_equiv_tflops": 3 * 2.0 * M * K * N * steps / (ms * 1e-3) / 1e12, "clocks": clk, "e2e": e2e,
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "achieved": value, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": value / peaks["bf16_tflops"], "traffic": 254e6,
                     "traffic_unit": "bytes per step, DRAM read + write summed over the step's kernels (ncu launch list)",
                     "note": "whole step incl. sensitivity counts, labels, block draws, lists and zero fill of the dropped blocks"},
        "cpu_baseline": cpu, "detail": detail, "device_status": int(status),
    }
    print(json.dumps(line))
    ard.ard_blocks_destroy(blocks)
    ard.ard_destroy(ctx)


RATES = (0.3, 0.4, 0.5, 0.6, 0.7)       # the dropout rates of the large-layer sweep
REPEATS = 5                              # timed regions per figure; the median is reported


def layer_config(args, wl, world):
    """The `config` object of a single-layer line; both arms (this library, the CPU reference) print the same."""
    return {"workload": args.workload, "B": wl["B"], "K": wl["K"], "N": wl["N"], "kind": wl["kind"], "ts": wl["ts"],
            "p": wl["p"], "n_dp": wl["n_dp"], "l2": "inputs larger than L2 (X, W, dY and outputs: ~0.5 GB per step)",
            "replicas": world}


class LayerBench:
    """One layer (X, W, dY resident on the device), one context, one pattern object; every timing helper of the
    single-layer workloads.  A step = draw a pattern on the device, then ard_layer_products: forward (full-width
    output, dropped columns written as zero), backward-data and backward-weight from the full-width dY (compacted
    once per step), enqueued side by side on the caller's stream and one stream of the context."""

    def __init__(self, torch, ard, args, wl, dev, rank, world, barrier, tensors=None):
        self.torch, self.ard, self.args, self.wl = torch, ard, args, wl
        self.rank, self.world, self.barrier = rank, world, barrier
        B, K, N = wl["B"], wl["K"], wl["N"]
        self.B, self.K, self.N, self.ts = B, K, N, wl["ts"]
        self.kind = ard.ARD_ROW if wl["kind"] == "row" else ard.ARD_TILE
        self.units = N if self.kind == ard.ARD_ROW else (K // wl["ts"]) * (N // wl["ts"])
        bf = torch.bfloat16
        if tensors is None:
            d = inputs.dense_layer(wl["config"], B, K, N, 1.0 / 90.0 if wl["config"] == 5 else 1.0 / 64.0)
            hX = torch.from_numpy(d["X"]).to(bf).pin_memory()
            hdY = torch.from_numpy(d["dY"]).to(bf).pin_memory()
            tensors = dict(host=d, hX=hX, hdY=hdY, X=hX.cuda(), dY=hdY.cuda(),
                           W=torch.from_numpy(np.ascontiguousarray(d["W"].T)).to(bf).cuda(),     # neuron-major [N][K]
                           Y=torch.empty((B, N), dtype=bf, device="cuda"), dX=torch.empty((B, K), dtype=bf, device="cuda"),
                           dW=torch.zeros((N, K), dtype=bf, device="cuda"), hY=torch.empty((B, N), dtype=bf).pin_memory())
        self.t = tensors
        self.ctx = ard.ard_create(dev, 2 * B * N + 4096)
        ard.ard_set_compact_reuse(self.ctx, 1)   # dY is not written between bwd-data and bwd-weight of a step
        apply_options(self.ctx, args)
        if args.shared_tail:
            ard.ard_set_shared_tail(self.ctx, 1, 0, 0)
        self.pat = ard.ard_pattern_create(self.ctx, self.kind, K, N, wl["ts"])
        self.dist_ids, self.khat = {}, {}
        for i, pp in enumerate(RATES):
            Kd = max_entropy_K(pp, wl["n_dp"])
            ard.ard_set_distribution(self.ctx, i, Kd)
            cdf = np.asarray(ard.ard_quantise_distribution(Kd), dtype=np.float64)
            self.dist_ids[pp] = i
            self.khat[pp] = np.diff(np.concatenate([[0.0], cdf])) / 2.0 ** 32      # the distribution the sampler realises
        self.seed = inputs.BASE_SEED
        self.cs = torch.cuda.current_stream().cuda_stream
        self.ptr = {k: tensors[k].data_ptr() for k in ("X", "W", "Y", "dY", "dX", "dW")}

    def close(self):
        self.ard.ard_pattern_destroy(self.pat)
        self.ard.ard_destroy(self.ctx)

    # ---- the calls of a step -----------------------------------------------------------------------
    def gemms(self, alpha, ev=None, ptr=None, zero_fill=0):
        ard, B, K, N, ctx, pat, cs = self.ard, self.B, self.K, self.N, self.ctx, self.pat, self.cs
        q = ptr or self.ptr
        if ev is not None:
            ev[0].record()
        ard.ard_fwd(ctx, pat, ard.ARD_BF16, B, K, N, alpha, q["X"], K, q["W"], K, q["Y"], N, ard.ARD_OUT_SCATTER_ZEROFILL, cs)
        if ev is not None:
            ev[1].record()
        ard.ard_bwd_data(ctx, pat, ard.ARD_BF16, B, K, N, alpha, q["dY"], N, 0, q["W"], K, q["dX"], K, cs)
        if ev is not None:
            ev[2].record()
        ard.ard_bwd_weight(ctx, pat, ard.ARD_BF16, ard.ARD_BF16, B, K, N, alpha, q["X"], K, q["dY"], N, 0, q["dW"], K,
                           zero_fill, cs)
        if ev is not None:
            ev[3].record()

    def products(self, alpha, ptr=None, stream=None):
        """The three products of the layer through the one call that enqueues them side by side.  The weight
        gradient writes the kept rows only (an optimiser that walks the kept rows needs no zeros) unless
        self.zero_fill_dW is set, which also writes zeros to the rows of dropped neurons."""
        ard, B, K, N = self.ard, self.B, self.K, self.N
        q = ptr or self.ptr
        ard.ard_layer_products(self.ctx, self.pat, ard.ARD_BF16, ard.ARD_BF16, B, K, N, alpha, q["X"], K, q["W"], K, q["dY"], N,
                               q["Y"], N, ard.ARD_OUT_SCATTER_ZEROFILL, q["dX"], K, q["dW"], K,
                               1 if getattr(self, "zero_fill_dW", False) else 0, self.cs if stream is None else stream)

    def step(self, pp, it, ev=None, ptr=None):
        """One step: draw the pattern on the device, then the layer's three products (ard_layer_products; with `ev`,
        one call per product in sequence so that each can be timed)."""
        self.ard.ard_sample_pattern(self.ctx, self.pat, self.dist_ids[pp], self.seed, it, self.rank, self.cs)
        if ev is not None:
            self.gemms(1.0 / (1.0 - pp), ev, ptr)
        else:
            self.products(1.0 / (1.0 - pp), ptr)

    def patterns_of(self, pp, its):
        """(dp, b, kept units) of the given iterations, read back from the device sampler outside any timed region."""
        out = []
        for it in its:
            self.ard.ard_sample_pattern(self.ctx, self.pat, self.dist_ids[pp], self.seed, it, self.rank)
            dp_, b_, nk, _ = self.ard.ard_pattern_to_host(self.pat, 0)
            out.append((dp_, b_, nk))
        return out

    def flops_per_unit(self):
        """FLOPs of ONE product per kept unit (a kept neuron, or a kept tile)."""
        return 2.0 * self.B * self.K if self.kind == self.ard.ARD_ROW else 2.0 * self.B * self.ts ** 2

    # ---- timed regions -----------------------------------------------------------------------------
    def timed_steps(self, pp, its, per_kernel=False, ptrs=None):
        """Times exactly len(its) steps between two barriers.  Returns (ms, per-kernel ms [steps][3] or None, wall)."""
        torch = self.torch
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in its] if per_kernel else None
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.barrier()
        w0 = time.time()
        e0.record()
        for i, it in enumerate(its):
            self.step(pp, it, evs[i] if per_kernel else None, None if ptrs is None else ptrs[i % len(ptrs)])
        e1.record()
        self.barrier()
        w1 = time.time()
        per = None
        if per_kernel:
            per = [[evs[i][j].elapsed_time(evs[i][j + 1]) for j in range(3)] for i in range(len(its))]
        return e0.elapsed_time(e1), per, (w0, w1)

    def repeated(self, pp, first_it, per_kernel=False):
        """Warm-up, then REPEATS timed regions over the SAME iterations (same patterns), so that the spread is the
        machine's and not the draw's."""
        a = self.args
        for w in range(a.warmup):
            self.step(pp, first_it + w)
        its = list(range(first_it + a.warmup, first_it + a.warmup + a.steps))
        runs = [self.timed_steps(pp, its, per_kernel) for _ in range(REPEATS)]
        return its, runs

    def time_fn(self, fn, n):
        torch = self.torch
        for _ in range(self.args.warmup):
            fn()
        out = []
        for _ in range(REPEATS):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            self.barrier()
            e0.record()
            for _ in range(n):
                fn()
            e1.record()
            self.barrier()
            out.append(e0.elapsed_time(e1) / n)
        return out

    def dense_baselines(self):
        """ms per dense step (median of REPEATS regions): this library's kernels at dp = 1, and torch.matmul."""
        torch, t = self.torch, self.t
        self.ard.ard_pattern_set(self.ctx, self.pat, 1, 1)
        n = max(5, self.args.steps // 4)
        own = self.time_fn(lambda: self.gemms(1.0), n)
        own_one = self.time_fn(lambda: self.products(1.0), n)
        X, dY, W = t["X"], t["dY"], t["W"]
        Wt = W.t()

        def lib():
            torch.matmul(X, Wt); torch.matmul(dY, W); torch.matmul(dY.t(), X)

        lib_ms = self.time_fn(lib, n)
        return {"own_kernels_dp1": min(statistics.median(own), statistics.median(own_one)),
                "torch_matmul": statistics.median(lib_ms), "own_kernels_dp1_in_sequence_all": own,
                "own_kernels_dp1_one_call_all": own_one, "torch_matmul_all": lib_ms}

    def algorithmic_bytes(self, op, kept_units):
        """Bytes a product has to move at least (bf16): operands read once, output written once (Sec. 3.1 / 3.2:
        only the kept part of the weight; the forward output is full width, the weight gradient's kept part)."""
        B, K, N = self.B, self.K, self.N
        if self.kind == self.ard.ARD_ROW:
            nk = kept_units
            return {"fwd": 2.0 * (B * K + nk * K + B * N), "bwd_data": 2.0 * (B * nk + nk * K + B * K),
                    "bwd_weight": 2.0 * (B * K + B * nk + nk * K),
                    "bwd_weight_zero_fill": 2.0 * (B * K + B * nk + N * K)}[op]
        w = 2.0 * self.ts ** 2 * kept_units
        return {"fwd": 2.0 * (B * K + B * N) + w, "bwd_data": 2.0 * (B * N + B * K) + w,
                "bwd_weight": 2.0 * (B * K + B * N) + w, "bwd_weight_zero_fill": 2.0 * (B * K + B * N + N * K)}[op]

    def per_dp_table(self, peak_burst):
        """Every (dp, b) of the distribution's support, forced with ard_pattern_set: per product and for the whole
        step the median over b and REPEATS of the CUDA-event time.  bwd_data includes the compaction of the
        full-width dY (once per step); bwd_weight reuses it; bwd_weight_zero_fill also writes the dropped rows."""
        torch, ard = self.torch, self.ard
        n_dp = self.wl["n_dp"]
        names = ["sampler", "fwd", "bwd_data", "bwd_weight", "bwd_weight_zero_fill"]
        table, step_by_dp, units_by_dp = {}, {}, {}
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
        self.dense_burst = {}
        for dp in range(1, n_dp + 1):
            ms = {nm: [] for nm in names}
            steps, kept, prods, onecall = [], [], [], []
            for b in range(1, dp + 1):
                ard.ard_pattern_set(self.ctx, self.pat, dp, b, self.cs)
                kept.append(self.ard.ard_pattern_to_host(self.pat, 0)[2])
                for rep in range(REPEATS + 1):                    # the first pass warms up
                    ev[0].record()
                    ard.ard_pattern_set(self.ctx, self.pat, dp, b, self.cs)      # the sampler kernel, pattern forced
                    self.gemms(2.0, ev[1:5])
                    q = self.ptr
                    ard.ard_bwd_weight(self.ctx, self.pat, ard.ARD_BF16, ard.ARD_BF16, self.B, self.K, self.N, 2.0, q["X"],
                                       self.K, q["dY"], self.N, 0, q["dW"], self.K, 1, self.cs)
                    ev[5].record()
                    torch.cuda.synchronize()
                    if rep == 0:
                        continue
                    for j, nm in enumerate(names):
                        ms[nm].append(ev[j].elapsed_time(ev[j + 1]))
                    steps.append(ev[0].elapsed_time(ev[4]))
                    prods.append(ev[1].elapsed_time(ev[4]))
                # the same step through ard_layer_products: the three products enqueued side by side
                t = self.t
                for rep in range(REPEATS + 1):
                    ev[0].record()
                    ard.ard_pattern_set(self.ctx, self.pat, dp, b, self.cs)
                    ard.ard_layer_products(self.ctx, self.pat, ard.ARD_BF16, ard.ARD_BF16, self.B, self.K, self.N, 2.0, t["X"],
                                           self.K, t["W"], self.K, t["dY"], self.N, t["Y"], self.N, ard.ARD_OUT_SCATTER_ZEROFILL,
                                           t["dX"], self.K, t["dW"], self.K, 0, self.cs)
                    ev[1].record()
                    torch.cuda.synchronize()
                    if rep:
                        onecall.append(ev[0].elapsed_time(ev[1]))
            if dp == 1:
                # the dense layer, timed the same way (one pass between two synchronisations): this library's three
                # products without a sampler, and torch.matmul
                X, dY, W = self.t["X"], self.t["dY"], self.t["W"]
                Wt = W.t()
                lib = []
                for rep in range(REPEATS + 1):
                    ev[0].record()
                    torch.matmul(X, Wt); torch.matmul(dY, W); torch.matmul(dY.t(), X)
                    ev[1].record()
                    torch.cuda.synchronize()
                    if rep:
                        lib.append(ev[0].elapsed_time(ev[1]))
                self.dense_burst = {"own_kernels_dp1": statistics.median(prods), "torch_matmul": statistics.median(lib)}
            fl = self.flops_per_unit() * float(np.mean(kept))
            row = {"kept_units_mean": float(np.mean(kept)), "step_ms": statistics.median(steps),
                   "step_one_call_ms": statistics.median(onecall)}
            for nm in names:
                m = statistics.median(ms[nm])
                row[nm + "_ms"] = m
                if nm != "sampler":
                    row[nm + "_tflops"] = fl / (m * 1e-3) / 1e12
                    row[nm + "_frac_of_burst"] = row[nm + "_tflops"] / peak_burst
                    # the roofline that binds this product: tensor time of its kept FLOPs or HBM time of its bytes
                    t_tc = fl / (peak_burst * 1e12) * 1e3
                    t_hbm = self.algorithmic_bytes(nm, float(np.mean(kept))) / (self.hbm_gbs * 1e9) * 1e3
                    row[nm + "_bound"] = "hbm" if t_hbm > t_tc else "tensor"
                    row[nm + "_frac_of_roofline"] = max(t_tc, t_hbm) / m
            table[str(dp)] = row
            step_by_dp[dp] = float(np.mean(steps))            # mean over b and repeats: what an expectation needs
            self.onecall_by_dp = getattr(self, "onecall_by_dp", {})
            self.onecall_by_dp[dp] = float(np.mean(onecall))
            if dp == 1:
                self.dense_burst["own_kernels_dp1_one_call"] = statistics.median(onecall)
            units_by_dp[dp] = float(np.mean(kept))
        return table, step_by_dp, units_by_dp

    def expectations(self, step_by_dp, units_by_dp, dense_ms):
        """What the sampled figures estimate, without the sampling: E[step time] = sum_dp k^_dp t(dp) under the
        quantised K of each rate, against the dense step; the ideal is 1/(1-p)."""
        out = {}
        for pp in RATES:
            k = self.khat[pp]
            t = sum(k[dp - 1] * step_by_dp[dp] for dp in step_by_dp)
            u = sum(k[dp - 1] * units_by_dp[dp] for dp in step_by_dp)
            out[str(pp)] = {"expected_ms_per_step": t, "expected_speedup": dense_ms / t, "ideal_speedup": 1.0 / (1.0 - pp),
                            "expected_speedup_vs_torch_matmul": self.dense_burst["torch_matmul"] / t,
                            "fraction_of_ideal": dense_ms / t * (1.0 - pp),
                            "expected_kept_tflops": 3 * self.flops_per_unit() * u / (t * 1e-3) / 1e12,
                            "expected_kept_fraction": u / self.units}
        return out

    def headline(self, peaks):
        """The timed regions the line's `value` comes from, and the roofline of the GEMM kernel inside them."""
        a, wl = self.args, self.wl
        p = wl["p"]
        launches0 = self.ard.ard_launch_count(self.ctx)
        its, runs = self.repeated(p, 0)
        launches = (self.ard.ard_launch_count(self.ctx) - launches0) * a.steps // (a.steps * REPEATS + a.warmup)
        # the same iterations once more with one call per product in sequence and an event between the calls: the
        # per-kernel durations the roofline needs cannot be separated while the products overlap
        seq_run = self.timed_steps(p, its, per_kernel=True)
        status = self.ard.ard_last_device_status(self.ctx)
        pats = self.patterns_of(p, its)
        kept = [3 * self.flops_per_unit() * nk for (_, _, nk) in pats]
        dense_flops = 3 * 2.0 * self.B * self.K * self.N * a.steps
        ms_all = [r[0] for r in runs]
        if self.world > 1:
            # whole job: slowest rank per region, work of all ranks
            agg = [aggregate_over_ranks(m, sum(kept), dense_flops, "cuda") for m in ms_all]
            ms_all = [x[0] for x in agg]
            kept_total, dense_total = agg[0][1], agg[0][2]
        else:
            kept_total, dense_total = sum(kept), dense_flops
        values = [kept_total / (m * 1e-3) / 1e12 for m in ms_all]
        order = sorted(range(REPEATS), key=lambda i: ms_all[i])
        mid = order[REPEATS // 2]
        per = np.array(seq_run[1])                       # [steps][3] ms, products in sequence
        gemm_ms = float(per.sum())
        achieved = sum(kept) / (gemm_ms * 1e-3) / 1e12
        per_op = {nm: {"ms_avg": float(per[:, j].mean()), "tflops": sum(kept) / 3.0 / (float(per[:, j].sum()) * 1e-3) / 1e12}
                  for j, nm in enumerate(["fwd", "bwd_data", "bwd_weight"])}
        wall = (runs[0][2][0], seq_run[2][1])
        return dict(its=its, pats=pats, ms=ms_all[mid], ms_all=ms_all, values=values, value=values[mid],
                    ms_sequential=seq_run[0],
                    dense_equiv=dense_total / (ms_all[mid] * 1e-3) / 1e12, launches=int(launches), status=int(status),
                    achieved=achieved, per_op=per_op, wall=wall, kept=kept)


def traffic_per_launch(lb, pats):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of ard_gemm_tc_kernel for the patterns of the timed
    region: the per-period figures of the ncu captures summarised under profiles/ (average of the three products),
    weighted by how often each period was drawn; None for a period that was not captured."""
    tab = DRAM_TRAFFIC_BY_DP.get(lb.wl["kind"], {})
    if not tab:
        return None
    xs = sorted(1.0 / dp for dp in tab)
    ys = [tab[round(1.0 / x)] for x in xs]
    tot, n = 0.0, 0
    for (dp, _, _) in pats:
        if 1.0 / dp < xs[0] or 1.0 / dp > xs[-1]:
            return None
        tot += float(np.interp(1.0 / dp, xs, ys))
        n += 1
    return tot / max(n, 1)


def roofline_of(h, peaks, clk, lb):
    # The timed regions are short (tens of ms each): if the SM clock stayed near its maximum the kernels ran in
    # the burst regime and are held against the burst cuBLAS figure, otherwise against the sustained one.
    burst = clk["sm_mhz"] is None or clk["sm_max_mhz"] is None or clk["sm_mhz"] >= 0.9 * clk["sm_max_mhz"]
    peak = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
    a = h["achieved"]
    return {"bound": "tensor", "achieved": a, "peak": peak, "unit": "TFLOP/s", "frac": a / peak,
            "traffic": traffic_per_launch(lb, h["pats"]),
            "traffic_unit": "bytes per launch, mean over the launches of the timed region (ncu captures at dp = 1, 2, 4, "
                            "8, 16, interpolated in 1/dp)",
            "peak_source": peaks["source"] + (" burst" if burst else " sustained") + " cuBLAS bf16 8192^3",
            "frac_of_burst": a / peaks["bf16_tflops"], "frac_of_sustained": a / peaks["bf16_tflops_sustained"],
            "frac_of_nominal_2250": a / 2250.0, "kernel": "ard_gemm_tc_kernel", "launches": 3 * lb.args.steps,
            "per_op": h["per_op"],
            "how": "CUDA events between the three product calls of the same iterations issued in sequence right after the "
                   "headline regions (in those the products overlap on two streams and have no separate durations); "
                   "%.4f ms per step in sequence" % (h["ms_sequential"] / lb.args.steps)}


def sweep_block(lb, peaks, dense):
    """Per-period table, expectations under every rate of the sweep, and the sampled figures beside them.  The
    expectations are held against the dense step timed like the table's entries (single passes); the sampled
    figures against the dense step timed like them (long loops, where the power cap lowers the clock)."""
    best_dense = min(dense["own_kernels_dp1"], dense["torch_matmul"])
    lb.hbm_gbs = peaks["hbm_gbs"]
    table, step_by_dp, units_by_dp = lb.per_dp_table(peaks["bf16_tflops"])
    exp = lb.expectations(step_by_dp, units_by_dp, min(lb.dense_burst.values()))
    exp_one = lb.expectations(lb.onecall_by_dp, units_by_dp, min(lb.dense_burst.values()))
    sampled = {}
    for pp in (0.3, 0.5, 0.7):
        its, runs = lb.repeated(pp, 10000 + int(pp * 100) * 1000)
        ms = statistics.median(r[0] for r in runs) / lb.args.steps
        pats = lb.patterns_of(pp, its)
        sampled[str(pp)] = {"ms_per_step": ms, "speedup_vs_dense": best_dense / ms,
                            "kept_fraction": float(np.mean([nk / lb.units for (_, _, nk) in pats]))}
    return {"per_dp": table, "dense_ms_single_pass": lb.dense_burst, "expected": exp,
            "per_dp_rooflines": "tensor: kept FLOPs / %.1f TFLOP/s; hbm: algorithmic bytes / %.1f GB/s (%s); a product's "
                                "bound is the longer of the two" % (peaks["bf16_tflops"], peaks["hbm_gbs"], peaks["source"]),
            "expected_products_in_one_call": exp_one, "sampled": sampled,
            "note": "per_dp: median over every offset b and %d repeats, pattern forced with ard_pattern_set; expected: "
                    "sum over dp of k^_dp x mean step time, k^ = the quantised distribution; sampled: %d device-drawn "
                    "steps per rate (a bimodal K makes these noisy; the expectations are the figures to read)"
                    % (REPEATS, lb.args.steps)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="mlp8192_row", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--quick", action="store_true", help="headline region only (for profiler captures)")
    ap.add_argument("--conv-run-len", type=int, default=0,
                    help="conv workloads: values per sampled run of the sensitivity prediction (1 = single values, "
                         "the statement of Sec. 5.1; default: the workload's 32)")
    ap.add_argument("--opt", action="append", default=[], metavar="NAME=VALUE",
                    help="tuning switch of the context, e.g. BAND_ROWS=8 (see ard_set_option); repeatable")
    ap.add_argument("--shared-tail", action="store_true", help="row products share their left-over tiles (ard_set_shared_tail)")
    ap.add_argument("--sweep-only", action="store_true", help="headline, dense baselines and the per-period table only")
    ap.add_argument("--force-dp", type=int, default=0, help="profiler captures: time steps of this period only (b = 1)")
    args = ap.parse_args()
    wl = dict(WORKLOADS[args.workload])
    if args.conv_run_len and "run_len" in wl:
        wl["run_len"] = args.conv_run_len
    if args.impl == "reference":
        return run_reference(args, wl)
    if wl["kind"] == "lstm":
        return run_lstm(args, wl)
    if wl["kind"] == "lstm_stack":
        return run_lstm_stack(args, wl)
    if wl["kind"] == "mlp_step":
        return run_mlp_step(args, wl)
    if wl["kind"] == "conv_rows":
        return run_conv_rows(args, wl)
    if wl["kind"] == "conv_blocks":
        return run_conv_blocks(args, wl)

    import torch
    import torch.distributed as dist
    from paper_2203_05705_b200 import ard

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    clocks = ClockSampler(local)          # started early: nvidia-smi needs a moment before its first sample
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    lb = LayerBench(torch, ard, args, wl, local, rank, world, barrier)
    B, K, N, p = wl["B"], wl["K"], wl["N"], wl["p"]
    peaks = load_peaks()

    if args.force_dp:
        # a handful of steps of one period, for a profiler capture of sparse draws
        ard.ard_pattern_set(lb.ctx, lb.pat, args.force_dp, 1)
        for _ in range(args.warmup + args.steps):
            lb.gemms(2.0)
        torch.cuda.synchronize()
        clocks.stop()            # ends the nvidia-smi child: a profiler waits for every child of the command
        if rank == 0:
            print(json.dumps({"forced_dp": args.force_dp, "steps": args.steps, "status": int(ard.ard_last_device_status(lb.ctx))}))
        lb.close()
        return

    # ---- the timed regions the headline value comes from (p = 0.5) ----
    h = lb.headline(peaks)
    clk = clocks.stop(*h["wall"])
    roofline = roofline_of(h, peaks, clk, lb)
    if args.quick:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": h["value"], "unit": UNIT, "quick": True,
                              "ms_per_step": h["ms"] / args.steps, "roofline": roofline, "clocks": clk}))
        lb.close()
        return

    # ---- dense baselines, the per-period table, expectations for the sweep's rates ----
    detail = {}
    dense = lb.dense_baselines()
    dense_flops_step = 3 * 2.0 * B * K * N
    detail["dense_ms_per_step"] = dense
    detail["dense_tflops"] = {k2: dense_flops_step / (dense[k2] * 1e-3) / 1e12 for k2 in ("own_kernels_dp1", "torch_matmul")}
    sw = sweep_block(lb, peaks, dense)
    detail.update(sw)
    detail["speedup_vs_dense"] = {k2: v["expected_speedup"] for k2, v in sw["expected_products_in_one_call"].items()}
    detail["ideal_speedup"] = {k2: v["ideal_speedup"] for k2, v in sw["expected"].items()}
    detail["repeats"] = {"n": REPEATS, "values": h["values"], "ms_per_step": [m / args.steps for m in h["ms_all"]],
                         "spread": (max(h["values"]) - min(h["values"])) / h["value"]}
    # the same iterations with the weight gradient also writing zeros to the rows of dropped neurons
    lb.zero_fill_dW = True
    zf = statistics.median(lb.timed_steps(p, h["its"])[0] for _ in range(3)) / args.steps
    lb.zero_fill_dW = False
    detail["ms_per_step_with_dW_zero_fill"] = zf

    if args.sweep_only:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": h["value"], "unit": UNIT, "sweep_only": True, "options": args.opt,
                              "ms_per_step": h["ms"] / args.steps, "roofline": roofline, "clocks": clk, "detail": detail}))
        lb.close()
        return

    # ---- the other half of the large-layer sweep: the same layer under the 128 x 128 tile pattern ----
    if args.workload == "mlp8192_row" and world == 1:
        twl = WORKLOADS["mlp8192_tile"]
        tb = LayerBench(torch, ard, args, twl, local, rank, world, barrier, tensors=lb.t)
        th = tb.headline(peaks)
        tdense = tb.dense_baselines()
        tsw = sweep_block(tb, peaks, tdense)
        detail["tile"] = {"workload": "mlp8192_tile", "ts": twl["ts"], "value": th["value"], "values": th["values"],
                          "ms_per_step": th["ms"] / args.steps, "roofline_frac_of_burst": th["achieved"] / peaks["bf16_tflops"],
                          "per_op": th["per_op"], "gpu_launches": th["launches"], "device_status": th["status"],
                          "dense_ms_per_step": {k2: tdense[k2] for k2 in ("own_kernels_dp1", "torch_matmul")}, **tsw}
        tb.close()

    # ---- operands that move: the same steps with three rotating buffer sets, and with never-seen addresses ----
    if world == 1:
        t = lb.t
        n_rot = max(8, min(args.steps, 48))
        sets = [lb.ptr]
        keep_alive = []
        for _ in range(2):
            extra = {k2: torch.empty_like(t[k2]) for k2 in ("X", "dY", "Y", "dX", "dW")}
            extra["X"].copy_(t["X"]); extra["dY"].copy_(t["dY"])
            keep_alive.append(extra)
            sets.append({**lb.ptr, **{k2: v.data_ptr() for k2, v in extra.items()}})
        its_r = list(range(40000, 40000 + n_rot))
        for s_ in sets:
            lb.step(p, 39999, None, s_)
        fixed = statistics.median(lb.timed_steps(p, its_r)[0] for _ in range(3)) / n_rot
        rot = statistics.median(lb.timed_steps(p, its_r, ptrs=sets)[0] for _ in range(3)) / n_rot
        # never-seen addresses: one pool per operand, the base sliding by 256 bytes per step
        pool = {k2: torch.empty(t[k2].numel() + 128 * (n_rot + 1), dtype=t[k2].dtype, device="cuda") for k2 in ("X", "dY")}
        slide = []
        for i in range(n_rot):
            q = dict(lb.ptr)
            for k2 in ("X", "dY"):
                view = pool[k2][128 * i:128 * i + t[k2].numel()]
                q[k2] = view.data_ptr()
            slide.append(q)
        pool["X"][:t["X"].numel()].copy_(t["X"].reshape(-1)); pool["dY"][:t["dY"].numel()].copy_(t["dY"].reshape(-1))
        fresh = lb.timed_steps(p, its_r, ptrs=slide)[0] / n_rot
        detail["moving_operands"] = {"ms_per_step_fixed_buffers": fixed, "ms_per_step_three_rotating_sets": rot,
                                     "ms_per_step_new_addresses_every_step": fresh, "steps": n_rot}
        del pool, keep_alive

    # ---- the same step as one CUDA graph: sampler on a device counter + ard_layer_products (the three products
    # enqueued side by side on the context's streams); the dense torch step replayed from a graph beside it ----
    if world == 1:
        X, W, dY, Y, dX, dW = (lb.t[k2] for k2 in ("X", "W", "dY", "Y", "dX", "dW"))
        gstream = torch.cuda.Stream()
        counter = torch.zeros(1, dtype=torch.int64, device="cuda")
        reps = 10

        def graph_ms(body, n_replays):
            with torch.cuda.stream(gstream):
                for _ in range(3):
                    body()
                torch.cuda.synchronize()
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr, stream=gstream):
                    for _ in range(reps):
                        body()
                for _ in range(3):
                    gr.replay()
                torch.cuda.synchronize()
                a, b2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                for _ in range(n_replays):
                    gr.replay()
                b2.record()
                torch.cuda.synchronize()
            return a.elapsed_time(b2) / (n_replays * reps)

        n_replays = max(2, args.steps // reps)
        side, side_kept = {}, {}
        for pp in (0.3, 0.5, 0.7):
            def body(pp=pp):
                gs = gstream.cuda_stream
                ard.ard_sample_pattern_counter(lb.ctx, lb.pat, lb.dist_ids[pp], lb.seed, 30000, counter, 1, rank, gs)
                ard.ard_layer_products(lb.ctx, lb.pat, ard.ARD_BF16, ard.ARD_BF16, B, K, N, 1.0 / (1.0 - pp), X, K, W, K, dY, N,
                                       Y, N, ard.ARD_OUT_SCATTER_ZEROFILL, dX, K, dW, K, 0, gs)
            counter.zero_()
            side[str(pp)] = graph_ms(body, n_replays)
            # iterations of the timed replays: 3 eager calls and 3 replays of `reps` steps came before them
            first = 30000 + 3 + 3 * reps
            pats_g = lb.patterns_of(pp, range(first, first + n_replays * reps))
            side_kept[str(pp)] = float(np.mean([nk / lb.units for (_, _, nk) in pats_g]))
        Wt_ = W.t()

        def torch_body():
            torch.matmul(X, Wt_, out=Y)
            torch.matmul(dY, W, out=dX)
            torch.matmul(dY.t(), X, out=dW)

        torch_graph = graph_ms(torch_body, n_replays)
        detail["graph_side_by_side"] = {"ms_per_step": side, "kept_fraction": side_kept,
                                        "torch_matmul_graph_ms": torch_graph,
                                        "speedup_vs_dense": {k2: torch_graph / v for k2, v in side.items()}}

    # ---- end to end through the C ABI with host buffers ----
    t = lb.t
    hX, hdY, hY = t["hX"], t["hdY"], t["hY"]
    h2d = hX.numel() * 2 + hdY.numel() * 2
    d2h = hY.numel() * 2
    e2e_steps = max(4, min(args.steps, 40))
    # Three streams and three sets of device buffers: the copy-in of step i+1 and the copy-out of step i-1
    # overlap the kernels of step i; every step still moves its own inputs and result over PCIe, and the operands
    # of consecutive steps sit at different addresses.
    s_in, s_cmp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    NB = 3
    Xb = [t["X"]] + [torch.empty_like(t["X"]) for _ in range(NB - 1)]
    dYb = [t["dY"]] + [torch.empty_like(t["dY"]) for _ in range(NB - 1)]
    Yb = [t["Y"]] + [torch.empty_like(t["Y"]) for _ in range(NB - 1)]
    al = 1.0 / (1.0 - p)
    dXt, dWt, Wt2 = t["dX"], t["dW"], t["W"]

    def e2e_run(its_list):
        in_done, cmp_done, out_done = {}, {}, {}
        for i, it in enumerate(its_list):
            k = i % NB
            with torch.cuda.stream(s_in):
                if i >= NB:
                    s_in.wait_event(cmp_done[i - NB])          # buffers k are free again
                Xb[k].copy_(hX, non_blocking=True)
                dYb[k].copy_(hdY, non_blocking=True)
                in_done[i] = s_in.record_event()
            with torch.cuda.stream(s_cmp):
                s_cmp.wait_event(in_done[i])
                if i >= NB:
                    s_cmp.wait_event(out_done[i - NB])         # Y[k] has been read out
                sc = s_cmp.cuda_stream
                ard.ard_sample_pattern(lb.ctx, lb.pat, lb.dist_ids[p], lb.seed, it, rank, sc)
                ard.ard_layer_products(lb.ctx, lb.pat, ard.ARD_BF16, ard.ARD_BF16, B, K, N, al, Xb[k], K, Wt2, K, dYb[k], N,
                                       Yb[k], N, ard.ARD_OUT_SCATTER_ZEROFILL, dXt, K, dWt, K, 0, sc)
                cmp_done[i] = s_cmp.record_event()
            with torch.cuda.stream(s_out):
                s_out.wait_event(cmp_done[i])
                hY.copy_(Yb[k], non_blocking=True)
                out_done[i] = s_out.record_event()

    e2e_run([20000, 20001, 20002])                            # warm-up
    barrier()
    its_e = list(range(20003, 20003 + e2e_steps))
    ms_e_all = []
    for _ in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for st in (s_in, s_cmp, s_out):
            st.wait_stream(torch.cuda.current_stream())
        e0.record(s_in)
        e2e_run(its_e)
        e1.record(s_out)
        barrier()
        ms_e_all.append(e0.elapsed_time(e1))
    ms_e = statistics.median(ms_e_all)
    pats_e = lb.patterns_of(p, its_e)
    fl_e = sum(3 * lb.flops_per_unit() * nk for (_, _, nk) in pats_e)
    e2e = {"value": fl_e / (ms_e * 1e-3) / 1e12 * world, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
           "ms_per_step": ms_e / e2e_steps, "steps": e2e_steps, "repeats": len(ms_e_all),
           "how": "C-ABI calls on a compute stream; pinned-host copies on two more streams, three buffer sets"}

    # ---- CPU baseline: the oracle on the host cores (rank 0, N = 1 only) ----
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        dt, fl, threads, sample = oracle_sample_seconds(wl, t["host"], max(wl["B"], wl["N"]))   # one full step
        cpu = {"value": fl / dt / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
               "seconds": dt}

    if rank == 0:
        line = {
            "metric": METRIC, "value": h["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": h["ms"] / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": layer_config(args, wl, world),
            "dense_equiv_tflops": h["dense_equiv"], "clocks": clk, "e2e": e2e, "gpu_launches": h["launches"],
            "roofline": roofline, "cpu_baseline": cpu, "detail": detail, "device_status": h["status"],
        }
        print(json.dumps(line))
    lb.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
