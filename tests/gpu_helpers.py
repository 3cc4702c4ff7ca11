"""Helpers for the GPU parity tests: device buffers via torch, comparison against the fp64 oracle."""
import numpy as np
import torch

from oracle import gemm as OG
from oracle import pattern as OP
from paper_2203_05705_b200 import ard

TOL = {ard.ARD_F32: 1e-5, ard.ARD_BF16: 5e-3}   # max relative Frobenius error (fp32 path / bf16 path)


def tile_rel_fro(G, O, T=256, Tr=None):
    """Worst relative Frobenius error over the T x T tiles of an output (tiles where the oracle is all zero are
    skipped: those are covered by the exact-zero checks).  A few mis-scattered columns inside one tile of a large
    output move the whole-tensor norm by far less than its tolerance; they cannot hide from this."""
    G = np.asarray(G, dtype=np.float64)
    O = np.asarray(O, dtype=np.float64)
    Tr = T if Tr is None else Tr      # rows per tile (fewer when only sampled rows of every tile are compared)
    R, C = O.shape
    pr, pc = (-R) % Tr, (-C) % T
    D2 = np.pad((G - O) ** 2, ((0, pr), (0, pc)))
    O2 = np.pad(O ** 2, ((0, pr), (0, pc)))
    d = D2.reshape((R + pr) // Tr, Tr, (C + pc) // T, T).sum(axis=(1, 3))
    o = O2.reshape((R + pr) // Tr, Tr, (C + pc) // T, T).sum(axis=(1, 3))
    nz = o > 0
    return float(np.sqrt((d[nz] / o[nz]).max())) if nz.any() else 0.0


def tdtype(dtype):
    return torch.float32 if dtype == ard.ARD_F32 else torch.bfloat16


def dev(a, dtype, ld=None, fill=None):
    """Upload a 2-D fp32 numpy array as a row-major device matrix with leading dimension ld."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    rows, cols = a.shape
    ld = cols if ld is None else ld
    t = torch.empty((rows, ld), dtype=tdtype(dtype), device="cuda")
    if fill is not None:
        t.fill_(fill)
    t[:, :cols] = torch.from_numpy(a).to(tdtype(dtype))
    return t


def nan_buf(rows, ld, torch_dtype):
    return torch.full((rows, ld), float("nan"), dtype=torch_dtype, device="cuda")


def host(t):
    return t.detach().to(torch.float64).cpu().numpy()


class Ctx:
    def __init__(self, workspace_bytes=64 << 20):
        self.h = ard.ard_create(0, workspace_bytes)
        self.pats = []

    def pattern(self, kind, K, N, ts=0):
        p = ard.ard_pattern_create(self.h, kind, K, N, ts)
        self.pats.append(p)
        return p

    def close(self):
        torch.cuda.synchronize()
        for p in self.pats:
            ard.ard_pattern_destroy(p)
        ard.ard_destroy(self.h)


def oracle_mask(kind, K, N, ts, dp, b):
    return OP.row_mask(N, dp, b) if kind == ard.ARD_ROW else OP.tile_mask(K, N, ts, dp, b)


def run_three_gemms(ctx, pat, kind, dtype, X, W, dY, dp, b, alpha, ts=0, lds=None, dw_dtype=None,
                    compact=False, zero_fill=True):
    """Runs fwd / bwd-data / bwd-weight through the C ABI on the pattern already set in `pat` and
    returns the relative Frobenius errors against the oracle plus exact-zero checks.
    X [B,K], W [K,N] (math orientation), dY [B,N] are fp32 numpy arrays (bf16-representable for bf16)."""
    B, K = X.shape
    N = W.shape[1]
    lds = lds or {}
    ldx, ldw, ldy = lds.get("x", K), lds.get("w", K), lds.get("y", N)
    dw_dtype = dtype if dw_dtype is None else dw_dtype
    mask = oracle_mask(kind, K, N, ts, dp, b)
    keep = OP.row_keep(N, dp, b) if kind == ard.ARD_ROW else None

    dX_ = dev(X, dtype, ldx)
    dW_ = dev(W.T, dtype, ldw)          # neuron-major
    out = {}

    # ---- forward ----
    Yo = OG.fwd(X, W, mask, alpha)
    if kind == ard.ARD_ROW and compact:
        Y = nan_buf(B, ldy, tdtype(dtype))
        ard.ard_fwd(ctx.h, pat, dtype, B, K, N, alpha, dX_, ldx, dW_, ldw, Y, ldy, ard.ARD_OUT_COMPACT)
        Yh = host(Y)
        out["fwd"] = OG.rel_fro(Yh[:, :len(keep)], Yo[:, keep])
        out["fwd_tile"] = tile_rel_fro(Yh[:, :len(keep)], Yo[:, keep])
        out["fwd_untouched"] = bool(np.all(np.isnan(Yh[:, len(keep):])))
    else:
        Y = nan_buf(B, ldy, tdtype(dtype))
        ard.ard_fwd(ctx.h, pat, dtype, B, K, N, alpha, dX_, ldx, dW_, ldw, Y, ldy, ard.ARD_OUT_SCATTER_ZEROFILL)
        Yh = host(Y)
        out["fwd"] = OG.rel_fro(Yh[:, :N], Yo)
        out["fwd_tile"] = tile_rel_fro(Yh[:, :N], Yo)
        out["fwd_zero"] = bool(np.all(Yh[:, :N][Yo == 0] == 0)) if kind == ard.ARD_ROW else True
        out["fwd_untouched"] = bool(np.all(np.isnan(Yh[:, N:])))

    # ---- backward data ----
    dXo = OG.bwd_data(dY, W, mask, alpha)
    if kind == ard.ARD_ROW and compact:
        dYc = dev(dY[:, keep] if len(keep) else np.zeros((B, 0), np.float32), dtype, ldy, fill=float("nan"))
        dyarg, is_c = dYc, 1
    else:
        dYd = dev(dY, dtype, ldy)
        if kind == ard.ARD_ROW:
            dYd[:, :N][:, torch.from_numpy(mask == 0).cuda()] = float("nan")   # dropped columns must not be read
        dyarg, is_c = dYd, 0
    dXb = nan_buf(B, ldx, tdtype(dtype))
    ard.ard_bwd_data(ctx.h, pat, dtype, B, K, N, alpha, dyarg, ldy, is_c, dW_, ldw, dXb, ldx)
    dXh = host(dXb)
    out["bwd_data"] = OG.rel_fro(dXh[:, :K], dXo)
    out["bwd_data_tile"] = tile_rel_fro(dXh[:, :K], dXo)
    out["bwd_data_untouched"] = bool(np.all(np.isnan(dXh[:, K:])))

    # ---- backward weight ----
    dWo = OG.bwd_weight(X, dY, mask, alpha).T          # neuron-major [N][K]
    dWb = nan_buf(N, ldw, tdtype(dw_dtype))
    ard.ard_bwd_weight(ctx.h, pat, dtype, dw_dtype, B, K, N, alpha, dX_, ldx, dyarg, ldy, is_c, dWb, ldw,
                       1 if zero_fill else 0)
    dWh = host(dWb)
    Mnm = (np.broadcast_to(mask[None, :], (K, N)) if mask.ndim == 1 else mask).T
    if zero_fill:
        out["bwd_weight"] = OG.rel_fro(dWh[:, :K], dWo)
        out["bwd_weight_tile"] = tile_rel_fro(dWh[:, :K], dWo)
        out["bwd_weight_zero"] = bool(np.all(dWh[:, :K][Mnm == 0] == 0))
    else:
        out["bwd_weight"] = OG.rel_fro(np.where(Mnm == 1, dWh[:, :K], 0.0), dWo)
        out["bwd_weight_tile"] = tile_rel_fro(np.where(Mnm == 1, dWh[:, :K], 0.0), dWo)
        out["bwd_weight_zero"] = bool(np.all(np.isnan(dWh[:, :K][Mnm == 0])))      # dropped part untouched
    out["bwd_weight_untouched"] = bool(np.all(np.isnan(dWh[:, K:])))
    st = ard.ard_last_device_status(ctx.h)
    out["status"] = st
    return out


def assert_ok(res, tol, what=""):
    assert res["status"] == 0, (what, res)
    for k, v in res.items():
        if k in ("fwd", "bwd_data", "bwd_weight") or k.endswith("_tile"):
            assert v <= tol, (what, k, v, res)      # whole tensor, and the worst 256 x 256 tile of it
        elif k != "status":
            assert v is True, (what, k, res)
