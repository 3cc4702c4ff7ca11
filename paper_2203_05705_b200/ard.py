"""Thin ctypes binding over libard.so: argument marshalling only.

Every function here has the name and the argument order of its C counterpart in
include/ard.h; tensors are torch CUDA tensors (used for device memory and
streams only) or raw integer device pointers.  All arithmetic runs in the
library's CUDA kernels.  If the library is missing or fails to load this module
raises -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libard.so")

ARD_OK = 0
ARD_ERR_INVALID_ARG, ARD_ERR_SHAPE, ARD_ERR_ALIGNMENT, ARD_ERR_DISTRIBUTION = 1, 2, 3, 4
ARD_ERR_UNSUPPORTED, ARD_ERR_CUDA, ARD_ERR_TIMEOUT, ARD_ERR_NOMEM = 5, 6, 7, 8
ARD_F32, ARD_BF16 = 0, 1
ARD_ROW, ARD_TILE = 0, 1
ARD_OUT_COMPACT, ARD_OUT_SCATTER_ZEROFILL = 0, 1
ARD_FLAG_OUT_F32, ARD_FLAG_ACCUMULATE = 0x10, 0x20
ARD_PATH_AUTO, ARD_PATH_CUDA_CORE, ARD_PATH_TENSOR_CORE = 0, 1, 2
ARD_STATIC_SCRATCH_BYTES = 8 << 20

EXPORTS = [
    "ard_create", "ard_destroy", "ard_set_path", "ard_set_tile_n", "ard_set_shared_tail", "ard_set_compact_reuse", "ard_set_distribution", "ard_quantise_distribution", "ard_search_distribution", "ard_get_distribution_cdf",
    "ard_pattern_create", "ard_pattern_destroy", "ard_sample_pattern", "ard_pattern_set",
    "ard_pattern_to_host", "ard_pattern_tile_lists_to_host", "ard_fwd", "ard_bwd_data", "ard_bwd_weight",
    "ard_bwd_data_static_scratch", "ard_lstm_gates", "ard_lstm_gates_bwd", "ard_lstm_gate_gemm", "ard_lstm_gate_gemm_bwd", "ard_set_lstm_persistent", "ard_lstm_forward", "ard_lstm_backward", "ard_last_device_status", "ard_status_string", "ard_launch_count",
]

_lib = None


class ArdError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        msg = lib().ard_status_string(self.status).decode()
        super().__init__(f"{where}: {msg} (status {self.status})")


def lib():
    """Loads libard.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2203_05705_b200.build`")
    L = C.CDLL(LIB_PATH)
    vp, i32, u32, u64, f32, sz = C.c_void_p, C.c_int, C.c_uint32, C.c_uint64, C.c_float, C.c_size_t
    P = C.POINTER
    sig = {
        "ard_create": [P(vp), i32, sz],
        "ard_destroy": [vp],
        "ard_set_path": [vp, i32],
        "ard_set_tile_n": [vp, i32],
        "ard_set_lstm_persistent": [vp, i32],
        "ard_set_shared_tail": [vp, i32, i32, i32],
        "ard_set_compact_reuse": [vp, i32],
        "ard_set_distribution": [vp, i32, P(C.c_double), i32],
        "ard_quantise_distribution": [P(C.c_double), i32, P(u64)],
        "ard_search_distribution": [C.c_double, i32, C.c_double, C.c_double, i32, C.c_double, P(C.c_double), P(i32)],
        "ard_get_distribution_cdf": [vp, i32, P(u64), i32, P(i32)],
        "ard_pattern_create": [vp, P(vp), i32, i32, i32, i32],
        "ard_pattern_destroy": [vp],
        "ard_sample_pattern": [vp, vp, i32, u64, u64, u32, vp],
        "ard_pattern_set": [vp, vp, i32, i32, vp],
        "ard_pattern_to_host": [vp, P(C.c_int32), P(C.c_int32), P(C.c_int32), P(C.c_int32), sz, vp],
        "ard_pattern_tile_lists_to_host": [vp, P(C.c_int32), P(C.c_int32), P(C.c_int32), P(C.c_int32), vp],
        "ard_fwd": [vp, vp, i32, i32, i32, i32, f32, vp, i32, vp, i32, vp, i32, i32, vp],
        "ard_bwd_data": [vp, vp, i32, i32, i32, i32, f32, vp, i32, i32, vp, i32, vp, i32, vp],
        "ard_bwd_data_static_scratch": [vp, vp, i32, i32, i32, i32, f32, vp, i32, vp, i32, vp, i32, vp],
        "ard_bwd_weight": [vp, vp, i32, i32, i32, i32, i32, f32, vp, i32, vp, i32, i32, vp, i32, i32, vp],
        "ard_lstm_gate_gemm": [vp, vp, i32, i32, i32, vp, i32, vp, i32, vp, i32, vp],
        "ard_lstm_gate_gemm_bwd": [vp, vp, i32, i32, i32, vp, i32, vp, i32, vp, i32, i32, vp],
        "ard_lstm_forward": [vp, vp, i32, i32, i32, i32, f32, vp, vp, i32, vp, vp, vp, vp, vp],
        "ard_lstm_backward": [vp, vp, i32, i32, i32, i32, f32, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp],
        "ard_lstm_gates": [vp, vp, i32, i32, i32, f32, vp, i32, vp, vp, i32, vp, vp, i32, i32, vp, vp],
        "ard_lstm_gates_bwd": [vp, vp, i32, i32, i32, f32, vp, vp, vp, i32, vp, i32, i32, vp, vp, i32, vp],
        "ard_last_device_status": [vp, vp],
        "ard_launch_count": [vp],
    }
    for name, args in sig.items():
        fn = getattr(L, name)
        fn.argtypes = args
        fn.restype = i32
    L.ard_launch_count.restype = u64
    L.ard_status_string.argtypes = [i32]
    L.ard_status_string.restype = C.c_char_p
    _lib = L
    return L


def _check(st, where):
    if st != ARD_OK:
        raise ArdError(st, where)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def ard_create(device=0, workspace_bytes=0):
    h = C.c_void_p()
    _check(lib().ard_create(C.byref(h), device, workspace_bytes), "ard_create")
    return h


def ard_destroy(ctx):
    _check(lib().ard_destroy(ctx), "ard_destroy")


def ard_set_path(ctx, path):
    _check(lib().ard_set_path(ctx, path), "ard_set_path")


def ard_set_compact_reuse(ctx, enable):
    _check(lib().ard_set_compact_reuse(ctx, 1 if enable else 0), "ard_set_compact_reuse")


def ard_set_tile_n(ctx, bn):
    _check(lib().ard_set_tile_n(ctx, bn), "ard_set_tile_n")


def ard_set_lstm_persistent(ctx, enable):
    _check(lib().ard_set_lstm_persistent(ctx, 1 if enable else 0), "ard_set_lstm_persistent")


def ard_set_shared_tail(ctx, enable, min_blocks=0, min_gain_blocks=0):
    _check(lib().ard_set_shared_tail(ctx, 1 if enable else 0, min_blocks, min_gain_blocks), "ard_set_shared_tail")


def ard_set_distribution(ctx, dist_id, K):
    K = np.ascontiguousarray(K, dtype=np.float64)
    _check(lib().ard_set_distribution(ctx, dist_id, K.ctypes.data_as(C.POINTER(C.c_double)), len(K)),
           "ard_set_distribution")


def ard_search_distribution(p, ndp, lam=1e-3, step=10.0, max_iter=200000, tol=1e-16):
    """Host-only: Algorithm 1.  Returns (K as a float64 array, iterations)."""
    K = np.zeros(max(int(ndp), 1), dtype=np.float64)
    it = C.c_int(0)
    _check(lib().ard_search_distribution(float(p), int(ndp), float(lam), float(step), int(max_iter), float(tol),
                                         K.ctypes.data_as(C.POINTER(C.c_double)), C.byref(it)),
           "ard_search_distribution")
    return K[:ndp], it.value


def ard_quantise_distribution(K):
    """Host-only: the integer cumulative table of K (no GPU needed)."""
    K = np.ascontiguousarray(K, dtype=np.float64)
    out = np.zeros(max(len(K), 1), dtype=np.uint64)
    _check(lib().ard_quantise_distribution(K.ctypes.data_as(C.POINTER(C.c_double)), len(K),
                                           out.ctypes.data_as(C.POINTER(C.c_uint64))), "ard_quantise_distribution")
    return out[:len(K)]


def ard_get_distribution_cdf(ctx, dist_id):
    n = C.c_int()
    _check(lib().ard_get_distribution_cdf(ctx, dist_id, None, 0, C.byref(n)), "ard_get_distribution_cdf")
    out = np.zeros(n.value, dtype=np.uint64)
    _check(lib().ard_get_distribution_cdf(ctx, dist_id, out.ctypes.data_as(C.POINTER(C.c_uint64)), n.value,
                                          C.byref(n)), "ard_get_distribution_cdf")
    return out


def ard_pattern_create(ctx, kind, K_dim, N_dim, tile=0):
    h = C.c_void_p()
    _check(lib().ard_pattern_create(ctx, C.byref(h), kind, K_dim, N_dim, tile), "ard_pattern_create")
    return h


def ard_pattern_destroy(pat):
    _check(lib().ard_pattern_destroy(pat), "ard_pattern_destroy")


def ard_sample_pattern(ctx, pat, dist_id, seed, iteration, stream_id, stream=None):
    _check(lib().ard_sample_pattern(ctx, pat, dist_id, seed, iteration, stream_id, _stream(stream)),
           "ard_sample_pattern")


def ard_pattern_set(ctx, pat, dp, b, stream=None):
    _check(lib().ard_pattern_set(ctx, pat, dp, b, _stream(stream)), "ard_pattern_set")


def ard_pattern_to_host(pat, capacity, stream=None):
    """Returns (dp, b, n_keep, idx[:n_keep])."""
    dp, b, nk = C.c_int32(), C.c_int32(), C.c_int32()
    idx = np.zeros(max(capacity, 1), dtype=np.int32)
    _check(lib().ard_pattern_to_host(pat, C.byref(dp), C.byref(b), C.byref(nk),
                                     idx.ctypes.data_as(C.POINTER(C.c_int32)), capacity, _stream(stream)),
           "ard_pattern_to_host")
    return dp.value, b.value, nk.value, idx[:min(nk.value, capacity)].copy()


def ard_pattern_tile_lists_to_host(pat, Tr, Tc, stream=None):
    col_ptr = np.zeros(Tc + 1, dtype=np.int32)
    row_ptr = np.zeros(Tr + 1, dtype=np.int32)
    col_idx = np.zeros(Tr * Tc, dtype=np.int32)
    row_idx = np.zeros(Tr * Tc, dtype=np.int32)
    ip = C.POINTER(C.c_int32)
    _check(lib().ard_pattern_tile_lists_to_host(pat, col_ptr.ctypes.data_as(ip), col_idx.ctypes.data_as(ip),
                                                row_ptr.ctypes.data_as(ip), row_idx.ctypes.data_as(ip),
                                                _stream(stream)), "ard_pattern_tile_lists_to_host")
    return col_ptr, col_idx[:col_ptr[-1]].copy(), row_ptr, row_idx[:row_ptr[-1]].copy()


def ard_fwd(ctx, pat, dtype, B, K, N, alpha, X, ldx, W, ldw, Y, ldy, outmode, stream=None):
    _check(lib().ard_fwd(ctx, pat, dtype, B, K, N, alpha, _ptr(X), ldx, _ptr(W), ldw, _ptr(Y), ldy, outmode,
                         _stream(stream)), "ard_fwd")


def ard_bwd_data(ctx, pat, dtype, B, K, N, alpha, dY, lddy, dy_is_compact, W, ldw, dX, lddx, stream=None):
    _check(lib().ard_bwd_data(ctx, pat, dtype, B, K, N, alpha, _ptr(dY), lddy, dy_is_compact, _ptr(W), ldw,
                              _ptr(dX), lddx, _stream(stream)), "ard_bwd_data")


def ard_bwd_data_static_scratch(ctx, pat, dtype, B, K, N, alpha, dY, lddy, W, ldw, dX, lddx, stream=None):
    """Backward-data for callers that must not allocate: same result as ard_bwd_data (row pattern,
    full-width dY), with the compacted dY kept in the library's fixed device array."""
    _check(lib().ard_bwd_data_static_scratch(ctx, pat, dtype, B, K, N, alpha, _ptr(dY), lddy, _ptr(W), ldw,
                                             _ptr(dX), lddx, _stream(stream)), "ard_bwd_data_static_scratch")


def ard_bwd_weight(ctx, pat, dtype, dW_dtype, B, K, N, alpha, X, ldx, dY, lddy, dy_is_compact, dW, lddw,
                   zero_fill_dropped, stream=None):
    _check(lib().ard_bwd_weight(ctx, pat, dtype, dW_dtype, B, K, N, alpha, _ptr(X), ldx, _ptr(dY), lddy,
                                dy_is_compact, _ptr(dW), lddw, zero_fill_dropped, _stream(stream)),
           "ard_bwd_weight")


def ard_lstm_gate_gemm(ctx, pat, B, KH, H, XH, ldxh, W, ldw, Z, ldz_gate, stream=None):
    _check(lib().ard_lstm_gate_gemm(ctx, pat, B, KH, H, _ptr(XH), ldxh, _ptr(W), ldw, _ptr(Z), ldz_gate,
                                    _stream(stream)), "ard_lstm_gate_gemm")


def ard_lstm_gate_gemm_bwd(ctx, pat, B, KH, H, dZ, ldz_gate, W, ldw, dXH, lddxh, accumulate, stream=None):
    _check(lib().ard_lstm_gate_gemm_bwd(ctx, pat, B, KH, H, _ptr(dZ), ldz_gate, _ptr(W), ldw, _ptr(dXH), lddxh,
                                        accumulate, _stream(stream)), "ard_lstm_gate_gemm_bwd")


def ard_lstm_forward(ctx, pat, T, B, I, H, alpha, XH, W, ldw, bias, C, G, Z, stream=None):
    _check(lib().ard_lstm_forward(ctx, pat, T, B, I, H, alpha, _ptr(XH), _ptr(W), ldw, _ptr(bias), _ptr(C), _ptr(G),
                                  _ptr(Z), _stream(stream)), "ard_lstm_forward")


def ard_lstm_backward(ctx, pat, T, B, I, H, alpha, XH, W, ldw, C, G, dH_last, D, dc, DZ, dW, stream=None):
    _check(lib().ard_lstm_backward(ctx, pat, T, B, I, H, alpha, _ptr(XH), _ptr(W), ldw, _ptr(C), _ptr(G),
                                   _ptr(dH_last), _ptr(D), _ptr(dc), _ptr(DZ), _ptr(dW), _stream(stream)),
           "ard_lstm_backward")


def ard_lstm_gates(ctx, pat, h_dtype, B, H, alpha, Z, ldz_gate, bias, c_prev, ldc, c, h, ldh, h_scatter,
                   gates_saved, stream=None):
    _check(lib().ard_lstm_gates(ctx, pat, h_dtype, B, H, alpha, _ptr(Z), ldz_gate, _ptr(bias), _ptr(c_prev), ldc,
                                _ptr(c), _ptr(h), ldh, h_scatter, _ptr(gates_saved), _stream(stream)),
           "ard_lstm_gates")


def ard_lstm_gates_bwd(ctx, pat, dz_dtype, B, H, alpha, gates_saved, c_prev, c, ldc, dh, lddh, dh_scatter,
                       dc_inout, dZ, ldz_gate, stream=None):
    _check(lib().ard_lstm_gates_bwd(ctx, pat, dz_dtype, B, H, alpha, _ptr(gates_saved), _ptr(c_prev), _ptr(c), ldc,
                                    _ptr(dh), lddh, dh_scatter, _ptr(dc_inout), _ptr(dZ), ldz_gate,
                                    _stream(stream)), "ard_lstm_gates_bwd")


def ard_last_device_status(ctx, stream=None):
    return lib().ard_last_device_status(ctx, _stream(stream))


def ard_status_string(status):
    return lib().ard_status_string(status).decode()


def ard_launch_count(ctx):
    return int(lib().ard_launch_count(ctx))
