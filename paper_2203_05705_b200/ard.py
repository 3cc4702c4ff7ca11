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
ARD_FLAG_OUT_F32, ARD_FLAG_ACCUMULATE, ARD_FLAG_RELU = 0x10, 0x20, 0x40
ARD_PATH_AUTO, ARD_PATH_CUDA_CORE, ARD_PATH_TENSOR_CORE = 0, 1, 2
(ARD_OPT_PDL, ARD_OPT_PDL_IN_CAPTURE, ARD_OPT_SIDE_STREAMS, ARD_OPT_CTA_PAIRS, ARD_OPT_BAND_ROWS,
 ARD_OPT_MLP_PERSISTENT, ARD_OPT_LSTM_COMPACT_H) = range(7)
ARD_STATIC_SCRATCH_BYTES = 8 << 20

EXPORTS = [
    "ard_create", "ard_destroy", "ard_set_path", "ard_set_option", "ard_set_tile_n", "ard_set_shared_tail", "ard_set_compact_reuse", "ard_set_distribution", "ard_quantise_distribution", "ard_search_distribution", "ard_get_distribution_cdf",
    "ard_pattern_create", "ard_pattern_destroy", "ard_sample_pattern", "ard_pattern_set",
    "ard_pattern_to_host", "ard_pattern_tile_lists_to_host", "ard_fwd", "ard_bwd_data", "ard_bwd_weight",
    "ard_bwd_data_static_scratch", "ard_lstm_gates", "ard_lstm_gates_bwd", "ard_lstm_gate_gemm", "ard_lstm_gate_gemm_bwd", "ard_set_lstm_persistent", "ard_lstm_forward", "ard_lstm_backward", "ard_lstm_forward_from_gates", "ard_lstm_backward_recurrent", "ard_compact_cols", "ard_expand_cols", "ard_last_device_status", "ard_status_string", "ard_launch_count",
    "ard_layer_fwd", "ard_layer_bwd_data", "ard_layer_bwd_weight", "ard_compact_weight_cols",
    "ard_expand_weight_grad_cols", "ard_bias_grad", "ard_sample_pattern_counter", "ard_mlp_step",
    "ard_rows_create", "ard_rows_destroy", "ard_sensitivity_predict", "ard_rows_set_probability", "ard_rows_sample",
    "ard_rows_to_host", "ard_rows_fwd", "ard_rows_bwd_data", "ard_rows_bwd_weight",
    "ard_layer_products", "ard_rows_products", "ard_rows_gather", "ard_rows_fwd_compact", "ard_rows_bwd_data_compact", "ard_rows_bwd_weight_compact",
    "ard_blocks_create", "ard_blocks_destroy", "ard_blocks_predict", "ard_blocks_set_label", "ard_blocks_sample",
    "ard_blocks_fwd", "ard_blocks_bwd_weight", "ard_blocks_bwd_input", "ard_blocks_to_host", "ard_blocks_pattern", "ard_dropout_schedule", "ard_blocks_products",
]

_lib = None


class MlpLayer(C.Structure):
    """struct ard_mlp_layer of include/ard.h (device pointers as integers)."""
    _fields_ = [("K", C.c_int), ("N", C.c_int), ("pat", C.c_void_p), ("sample", C.c_int), ("relu", C.c_int),
                ("compact_out", C.c_int), ("dW_is_f32", C.c_int), ("alpha", C.c_float), ("ldw", C.c_int),
                ("W", C.c_void_p), ("bias", C.c_void_p), ("Wk", C.c_void_p), ("A", C.c_void_p), ("dZ", C.c_void_p),
                ("dWk", C.c_void_p), ("dW", C.c_void_p), ("db", C.c_void_p)]


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
        "ard_set_option": [vp, i32, i32],
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
        "ard_lstm_forward_from_gates": [vp, vp, i32, i32, i32, i32, f32, vp, vp, i32, vp, vp, vp, vp],
        "ard_lstm_backward_recurrent": [vp, vp, i32, i32, i32, i32, f32, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp],
        "ard_compact_cols": [vp, vp, i32, i32, i32, vp, i32, vp, i32, vp],
        "ard_expand_cols": [vp, vp, i32, i32, i32, f32, vp, i32, vp, i32, vp],
        "ard_lstm_gates": [vp, vp, i32, i32, i32, f32, vp, i32, vp, vp, i32, vp, vp, i32, i32, vp, vp],
        "ard_lstm_gates_bwd": [vp, vp, i32, i32, i32, f32, vp, vp, vp, i32, vp, i32, i32, vp, vp, i32, vp],
        "ard_last_device_status": [vp, vp],
        "ard_launch_count": [vp],
        "ard_layer_fwd": [vp, vp, vp, i32, i32, i32, i32, f32, vp, i32, vp, i32, vp, vp, i32, i32, vp],
        "ard_layer_bwd_data": [vp, vp, vp, i32, i32, i32, i32, f32, vp, i32, i32, vp, i32, vp, i32, vp, i32, vp],
        "ard_layer_bwd_weight": [vp, vp, vp, i32, i32, i32, i32, i32, f32, vp, i32, vp, i32, i32, vp, i32, i32, vp],
        "ard_compact_weight_cols": [vp, vp, vp, i32, i32, i32, vp, i32, vp, i32, vp],
        "ard_expand_weight_grad_cols": [vp, vp, vp, i32, i32, i32, vp, i32, vp, i32, i32, vp],
        "ard_bias_grad": [vp, vp, i32, i32, i32, vp, i32, i32, vp, i32, vp],
        "ard_sample_pattern_counter": [vp, vp, i32, u64, u64, vp, i32, u32, vp],
        "ard_mlp_step": [vp, P(MlpLayer), i32, i32, vp, i32, vp, i32, vp, i32, i32, u64, u64, vp, vp],
        "ard_dropout_schedule": [i32, C.c_double, C.c_double, C.c_double, C.c_double, C.c_double, P(C.c_double)],
        "ard_blocks_create": [vp, P(vp), i32, i32, i32],
        "ard_blocks_destroy": [vp],
        "ard_blocks_predict": [vp, vp, i32, vp, i32, C.c_double, i32, C.c_double, f32, i32, u64, u64, u32, vp],
        "ard_blocks_set_label": [vp, vp, i32, vp],
        "ard_blocks_sample": [vp, vp, C.c_double, C.c_double, u64, u64, u32, vp],
        "ard_blocks_fwd": [vp, vp, i32, f32, vp, i32, vp, i32, vp, i32, vp],
        "ard_blocks_bwd_weight": [vp, vp, i32, f32, vp, i32, vp, i32, vp, i32, vp],
        "ard_blocks_bwd_input": [vp, vp, i32, i32, f32, vp, i32, vp, i32, vp, i32, i32, vp],
        "ard_blocks_products": [vp, vp, i32, i32, f32, vp, i32, vp, i32, vp, i32, vp, i32, vp, i32, vp, i32, i32, vp],
        "ard_blocks_to_host": [vp, P(C.c_int32), P(C.c_uint8), P(C.c_uint8), vp],
        "ard_rows_create": [vp, P(vp), i32, i32],
        "ard_rows_destroy": [vp],
        "ard_sensitivity_predict": [vp, vp, i32, vp, i32, i32, C.c_double, i32, C.c_double, f32, C.c_double, C.c_double, u64, u64,
                                    u32, vp],
        "ard_rows_set_probability": [vp, vp, C.c_double, vp],
        "ard_rows_sample": [vp, vp, u64, u64, u32, vp],
        "ard_rows_to_host": [vp, P(C.c_int32), P(C.c_int32), sz, P(C.c_uint32), vp],
        "ard_rows_fwd": [vp, vp, i32, i32, i32, f32, vp, i32, vp, i32, vp, i32, vp],
        "ard_rows_bwd_data": [vp, vp, i32, i32, i32, f32, vp, i32, vp, i32, vp, i32, vp],
        "ard_rows_bwd_weight": [vp, vp, i32, i32, i32, i32, f32, vp, i32, vp, i32, vp, i32, vp],
        "ard_layer_products": [vp, vp, i32, i32, i32, i32, i32, f32, vp, i32, vp, i32, vp, i32, vp, i32, i32, vp, i32, vp,
                               i32, i32, vp],
        "ard_rows_products": [vp, vp, i32, i32, i32, i32, f32, vp, i32, vp, i32, vp, i32, vp, i32, vp, i32, vp, i32, vp,
                              i32, vp, i32, vp],
        "ard_rows_gather": [vp, vp, i32, i32, vp, i32, vp, i32, vp],
        "ard_rows_fwd_compact": [vp, vp, i32, i32, i32, f32, vp, i32, vp, i32, vp, i32, vp],
        "ard_rows_bwd_data_compact": [vp, vp, i32, i32, i32, f32, vp, i32, vp, i32, vp, i32, vp],
        "ard_rows_bwd_weight_compact": [vp, vp, i32, i32, i32, i32, f32, vp, i32, vp, i32, vp, i32, vp],
    }
    for name, args in sig.items():
        fn = getattr(L, name)
        fn.argtypes = args
        fn.restype = i32
    L.ard_launch_count.restype = u64
    L.ard_blocks_pattern.argtypes = [vp]
    L.ard_blocks_pattern.restype = vp
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


def ard_set_option(ctx, option, value):
    _check(lib().ard_set_option(ctx, option, value), "ard_set_option")


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


def ard_layer_fwd(ctx, pat, in_pat, dtype, B, K, N, alpha, X, ldx, Wk, ldw, bias, A, lda, outmode_and_flags,
                  stream=None):
    _check(lib().ard_layer_fwd(ctx, pat, in_pat, dtype, B, K, N, alpha, _ptr(X), ldx, _ptr(Wk), ldw, _ptr(bias),
                               _ptr(A), lda, outmode_and_flags, _stream(stream)), "ard_layer_fwd")


def ard_layer_bwd_data(ctx, pat, in_pat, dtype, B, K, N, alpha, dZ, lddz, dz_is_compact_and_flags, Wk, ldw, act_prev,
                       ldact, dX, lddx, stream=None):
    _check(lib().ard_layer_bwd_data(ctx, pat, in_pat, dtype, B, K, N, alpha, _ptr(dZ), lddz, dz_is_compact_and_flags,
                                    _ptr(Wk), ldw, _ptr(act_prev), ldact, _ptr(dX), lddx, _stream(stream)),
           "ard_layer_bwd_data")


def ard_layer_bwd_weight(ctx, pat, in_pat, dtype, dW_dtype, B, K, N, alpha, X, ldx, dZ, lddz, dz_is_compact, dWk, lddw,
                         zero_fill_dropped, stream=None):
    _check(lib().ard_layer_bwd_weight(ctx, pat, in_pat, dtype, dW_dtype, B, K, N, alpha, _ptr(X), ldx, _ptr(dZ), lddz,
                                      dz_is_compact, _ptr(dWk), lddw, zero_fill_dropped, _stream(stream)),
           "ard_layer_bwd_weight")


def ard_compact_weight_cols(ctx, pat, in_pat, dtype, K, N, W, ldw, Wk, ldwk, stream=None):
    _check(lib().ard_compact_weight_cols(ctx, pat, in_pat, dtype, K, N, _ptr(W), ldw, _ptr(Wk), ldwk, _stream(stream)),
           "ard_compact_weight_cols")


def ard_expand_weight_grad_cols(ctx, pat, in_pat, dtype, K, N, dWk, lddwk, dW, lddw, zero_fill, stream=None):
    _check(lib().ard_expand_weight_grad_cols(ctx, pat, in_pat, dtype, K, N, _ptr(dWk), lddwk, _ptr(dW), lddw,
                                             zero_fill, _stream(stream)), "ard_expand_weight_grad_cols")


def ard_bias_grad(ctx, pat, dtype, B, N, dZ, lddz, dz_is_compact, db, zero_fill_dropped, stream=None):
    _check(lib().ard_bias_grad(ctx, pat, dtype, B, N, _ptr(dZ), lddz, dz_is_compact, _ptr(db), zero_fill_dropped,
                               _stream(stream)), "ard_bias_grad")


def ard_sample_pattern_counter(ctx, pat, dist_id, seed, iteration_base, iteration_counter, advance, stream_id,
                               stream=None):
    _check(lib().ard_sample_pattern_counter(ctx, pat, dist_id, seed, iteration_base, _ptr(iteration_counter),
                                            1 if advance else 0, stream_id, _stream(stream)),
           "ard_sample_pattern_counter")


def mlp_layers(layers):
    """Marshals a list of dicts (keys = the fields of struct ard_mlp_layer; tensors or None for the
    pointers) into a C array.  Keep the tensors alive while the array is in use."""
    arr = (MlpLayer * len(layers))()
    for i, d in enumerate(layers):
        for name, ctype in MlpLayer._fields_:
            v = d.get(name)
            if ctype is C.c_void_p:
                v = v.value if isinstance(v, C.c_void_p) else _ptr(v)
            elif v is None:
                v = 0
            setattr(arr[i], name, v)
    return arr


def ard_mlp_step(ctx, layers, n_layers, B, X, ldx, dOut, lddout, dX, lddx, dist_id, seed, iteration_base,
                 iteration_counter, stream=None):
    """`layers`: the array made by mlp_layers()."""
    _check(lib().ard_mlp_step(ctx, layers, n_layers, B, _ptr(X), ldx, _ptr(dOut), lddout, _ptr(dX), lddx, dist_id,
                              seed, iteration_base, _ptr(iteration_counter), _stream(stream)), "ard_mlp_step")


def ard_dropout_schedule(n_epochs, p_total, mean_epoch, var_epoch, lam, p_max=1.0):
    out = np.zeros(max(n_epochs, 1), dtype=np.float64)
    _check(lib().ard_dropout_schedule(n_epochs, p_total, mean_epoch, var_epoch, lam, p_max,
                                      out.ctypes.data_as(C.POINTER(C.c_double))), "ard_dropout_schedule")
    return out[:n_epochs]


def ard_blocks_create(ctx, M, Kc, ts):
    h = C.c_void_p()
    _check(lib().ard_blocks_create(ctx, C.byref(h), M, Kc, ts), "ard_blocks_create")
    return h


def ard_blocks_destroy(blocks):
    _check(lib().ard_blocks_destroy(blocks), "ard_blocks_destroy")


def ard_blocks_predict(ctx, blocks, dtype, A, lda, k_frac, run_len, t_frac, threshold, cap, seed, iteration, stream_id,
                       stream=None):
    _check(lib().ard_blocks_predict(ctx, blocks, dtype, _ptr(A), lda, k_frac, run_len, t_frac, threshold, cap, seed,
                                    iteration, stream_id, _stream(stream)), "ard_blocks_predict")


def ard_blocks_set_label(ctx, blocks, sensitive, stream=None):
    _check(lib().ard_blocks_set_label(ctx, blocks, sensitive, _stream(stream)), "ard_blocks_set_label")


def ard_blocks_sample(ctx, blocks, m_prob, n_prob, seed, iteration, stream_id, stream=None):
    _check(lib().ard_blocks_sample(ctx, blocks, m_prob, n_prob, seed, iteration, stream_id, _stream(stream)),
           "ard_blocks_sample")


def ard_blocks_fwd(ctx, blocks, N, alpha, A, lda, W, ldw, Yt, ldyt, stream=None):
    _check(lib().ard_blocks_fwd(ctx, blocks, N, alpha, _ptr(A), lda, _ptr(W), ldw, _ptr(Yt), ldyt, _stream(stream)),
           "ard_blocks_fwd")


def ard_blocks_bwd_weight(ctx, blocks, N, alpha, A, lda, dYt, lddyt, dW, lddw, stream=None):
    _check(lib().ard_blocks_bwd_weight(ctx, blocks, N, alpha, _ptr(A), lda, _ptr(dYt), lddyt, _ptr(dW), lddw,
                                       _stream(stream)), "ard_blocks_bwd_weight")


def ard_blocks_bwd_input(ctx, blocks, dA_dtype, N, alpha, dYt, lddyt, W, ldw, dA, ldda, zero_fill_dropped, stream=None):
    _check(lib().ard_blocks_bwd_input(ctx, blocks, dA_dtype, N, alpha, _ptr(dYt), lddyt, _ptr(W), ldw, _ptr(dA), ldda,
                                      zero_fill_dropped, _stream(stream)), "ard_blocks_bwd_input")


def ard_blocks_products(ctx, blocks, dA_dtype, N, alpha, A, lda, W, ldw, dYt, lddyt, Yt, ldyt, dW, lddw, dA, ldda,
                        zero_fill_dropped, stream=None):
    _check(lib().ard_blocks_products(ctx, blocks, dA_dtype, N, alpha, _ptr(A), lda, _ptr(W), ldw, _ptr(dYt), lddyt,
                                     _ptr(Yt), ldyt, _ptr(dW), lddw, _ptr(dA), ldda, zero_fill_dropped, _stream(stream)),
           "ard_blocks_products")


def ard_blocks_to_host(blocks, n_blocks, stream=None):
    """Returns (counts, sensitive, keep), one entry per block g*Q + j."""
    counts = np.zeros(n_blocks, dtype=np.int32)
    sens = np.zeros(n_blocks, dtype=np.uint8)
    keep = np.zeros(n_blocks, dtype=np.uint8)
    _check(lib().ard_blocks_to_host(blocks, counts.ctypes.data_as(C.POINTER(C.c_int32)),
                                    sens.ctypes.data_as(C.POINTER(C.c_uint8)), keep.ctypes.data_as(C.POINTER(C.c_uint8)),
                                    _stream(stream)), "ard_blocks_to_host")
    return counts, sens, keep


def ard_blocks_pattern(blocks):
    return C.c_void_p(lib().ard_blocks_pattern(blocks))


def ard_rows_create(ctx, M, region_rows):
    h = C.c_void_p()
    _check(lib().ard_rows_create(ctx, C.byref(h), M, region_rows), "ard_rows_create")
    return h


def ard_rows_destroy(rows):
    _check(lib().ard_rows_destroy(rows), "ard_rows_destroy")


def ard_sensitivity_predict(ctx, rows, dtype, A, lda, Kc, k_frac, run_len, t_frac, threshold, m_prob, n_prob, seed,
                            iteration, stream_id, stream=None):
    _check(lib().ard_sensitivity_predict(ctx, rows, dtype, _ptr(A), lda, Kc, k_frac, run_len, t_frac, threshold, m_prob,
                                         n_prob, seed, iteration, stream_id, _stream(stream)), "ard_sensitivity_predict")


def ard_rows_set_probability(ctx, rows, p, stream=None):
    _check(lib().ard_rows_set_probability(ctx, rows, p, _stream(stream)), "ard_rows_set_probability")


def ard_rows_sample(ctx, rows, seed, iteration, stream_id, stream=None):
    _check(lib().ard_rows_sample(ctx, rows, seed, iteration, stream_id, _stream(stream)), "ard_rows_sample")


def ard_rows_to_host(rows, M, regions=0, stream=None):
    """Returns (n_keep, kept rows, per-region integers or None)."""
    nk = C.c_int32()
    idx = np.zeros(max(M, 1), dtype=np.int32)
    P = np.zeros(regions, dtype=np.uint32) if regions else None
    _check(lib().ard_rows_to_host(rows, C.byref(nk), idx.ctypes.data_as(C.POINTER(C.c_int32)), M,
                                  P.ctypes.data_as(C.POINTER(C.c_uint32)) if regions else None, _stream(stream)),
           "ard_rows_to_host")
    return nk.value, idx[:nk.value].copy(), P


def ard_rows_fwd(ctx, rows, M, K, N, alpha, A, lda, W, ldw, Y, ldy, stream=None):
    _check(lib().ard_rows_fwd(ctx, rows, M, K, N, alpha, _ptr(A), lda, _ptr(W), ldw, _ptr(Y), ldy, _stream(stream)),
           "ard_rows_fwd")


def ard_rows_bwd_data(ctx, rows, M, K, N, alpha, dY, lddy, W, ldw, dA, ldda, stream=None):
    _check(lib().ard_rows_bwd_data(ctx, rows, M, K, N, alpha, _ptr(dY), lddy, _ptr(W), ldw, _ptr(dA), ldda,
                                   _stream(stream)), "ard_rows_bwd_data")


def ard_rows_bwd_weight(ctx, rows, dW_dtype, M, K, N, alpha, A, lda, dY, lddy, dW, lddw, stream=None):
    _check(lib().ard_rows_bwd_weight(ctx, rows, dW_dtype, M, K, N, alpha, _ptr(A), lda, _ptr(dY), lddy, _ptr(dW), lddw,
                                     _stream(stream)), "ard_rows_bwd_weight")


def ard_layer_products(ctx, pat, dtype, dW_dtype, B, K, N, alpha, X, ldx, W, ldw, dY, lddy, Y, ldy, outmode, dX, lddx,
                       dW, lddw, zero_fill_dropped, stream=None):
    _check(lib().ard_layer_products(ctx, pat, dtype, dW_dtype, B, K, N, alpha, _ptr(X), ldx, _ptr(W), ldw, _ptr(dY),
                                    lddy, _ptr(Y), ldy, outmode, _ptr(dX), lddx, _ptr(dW), lddw, zero_fill_dropped,
                                    _stream(stream)), "ard_layer_products")


def ard_rows_products(ctx, rows, dW_dtype, M, K, N, alpha, A, lda, W, ldw, dY, lddy, Ak, ldak, dYk, lddyk, Y, ldy, dA,
                      ldda, dW, lddw, stream=None):
    _check(lib().ard_rows_products(ctx, rows, dW_dtype, M, K, N, alpha, _ptr(A), lda, _ptr(W), ldw, _ptr(dY), lddy,
                                   _ptr(Ak), ldak, _ptr(dYk), lddyk, _ptr(Y), ldy, _ptr(dA), ldda, _ptr(dW), lddw,
                                   _stream(stream)), "ard_rows_products")


def ard_rows_gather(ctx, rows, M, width, src, ld_src, dst, ld_dst, stream=None):
    _check(lib().ard_rows_gather(ctx, rows, M, width, _ptr(src), ld_src, _ptr(dst), ld_dst, _stream(stream)),
           "ard_rows_gather")


def ard_rows_fwd_compact(ctx, rows, M, K, N, alpha, Ak, ldak, W, ldw, Y, ldy, stream=None):
    _check(lib().ard_rows_fwd_compact(ctx, rows, M, K, N, alpha, _ptr(Ak), ldak, _ptr(W), ldw, _ptr(Y), ldy,
                                      _stream(stream)), "ard_rows_fwd_compact")


def ard_rows_bwd_data_compact(ctx, rows, M, K, N, alpha, dYk, lddyk, W, ldw, dA, ldda, stream=None):
    _check(lib().ard_rows_bwd_data_compact(ctx, rows, M, K, N, alpha, _ptr(dYk), lddyk, _ptr(W), ldw, _ptr(dA), ldda,
                                           _stream(stream)), "ard_rows_bwd_data_compact")


def ard_rows_bwd_weight_compact(ctx, rows, dW_dtype, M, K, N, alpha, Ak, ldak, dYk, lddyk, dW, lddw, stream=None):
    _check(lib().ard_rows_bwd_weight_compact(ctx, rows, dW_dtype, M, K, N, alpha, _ptr(Ak), ldak, _ptr(dYk), lddyk,
                                             _ptr(dW), lddw, _stream(stream)), "ard_rows_bwd_weight_compact")


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


def ard_lstm_forward_from_gates(ctx, pat, T, B, I, H, alpha, XH, W, ldw, bias, C, G, stream=None):
    _check(lib().ard_lstm_forward_from_gates(ctx, pat, T, B, I, H, alpha, _ptr(XH), _ptr(W), ldw, _ptr(bias), _ptr(C),
                                             _ptr(G), _stream(stream)), "ard_lstm_forward_from_gates")


def ard_lstm_backward_recurrent(ctx, pat, T, B, I, H, alpha, XH, W, ldw, C, G, dH_last, D, dc, DZ, dW, stream=None):
    _check(lib().ard_lstm_backward_recurrent(ctx, pat, T, B, I, H, alpha, _ptr(XH), _ptr(W), ldw, _ptr(C), _ptr(G),
                                             _ptr(dH_last), _ptr(D), _ptr(dc), _ptr(DZ), _ptr(dW), _stream(stream)),
           "ard_lstm_backward_recurrent")


def ard_compact_cols(ctx, pat, dtype, rows, N, src, ld_src, dst, ld_dst, stream=None):
    _check(lib().ard_compact_cols(ctx, pat, dtype, rows, N, _ptr(src), ld_src, _ptr(dst), ld_dst, _stream(stream)),
           "ard_compact_cols")


def ard_expand_cols(ctx, pat, src_dtype, rows, N, alpha, src, ld_src, dst, ld_dst, stream=None):
    _check(lib().ard_expand_cols(ctx, pat, src_dtype, rows, N, alpha, _ptr(src), ld_src, _ptr(dst), ld_dst,
                                 _stream(stream)), "ard_expand_cols")


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
