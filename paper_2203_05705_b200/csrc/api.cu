// C-ABI entry points: argument validation, context / pattern lifetime, the TMA descriptor cache and
// the dispatch between the CUDA-core and tcgen05 kernel families.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "ard_internal.h"
#include <initializer_list>

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DeviceGuard {
  int prev = -1;
  bool ok;
  bool switched = false;
  explicit DeviceGuard(int dev) {
    ok = cudaGetDevice(&prev) == cudaSuccess;
    if (ok && prev != dev) {  // the usual case needs no switch at all
      ok = cudaSetDevice(dev) == cudaSuccess;
      switched = ok;
    }
  }
  ~DeviceGuard() {
    if (switched) cudaSetDevice(prev);
  }
};

// One bf16 descriptor: [rows][cols] with a row pitch of pitch_bytes, 128-byte swizzle, zero fill
// outside the extents (which is what drops the rows / columns beyond n_keep for free).
bool encode_map(ard_ctx* ctx, CUtensorMap* out, const void* base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes,
                uint32_t box_cols, uint32_t box_rows) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_fn)(
      out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// Fills `out` with the descriptor of the whole matrix [rows][cols] at `base` (pitch ld elements, bf16) and with
// what the kernel needs to specialise it to the sampled pattern (see TcMap).  Host work only: one encode, no
// device memory, no copy, nothing cached, so operands may sit at a new address in every call and a call may be
// captured into a CUDA graph like any other launch.  `units` and `dp_bound` describe the pattern the variant
// follows; they are implied by the pattern header on the device and only checked here.
ard_status get_maps(ard_ctx* ctx, const void* base, int rows, int cols, int ld, int units, int variant, int dp_bound,
                    int box_rows, int box_cols, TcMap* out, const void* dense_base = nullptr, int dense_ld = 0) {
  (void)dp_bound;
  if (variant == MAP_STRIDED_ROWS && units != rows) return ARD_ERR_INVALID_ARG;
  if (variant == MAP_COMPACT_COLS && units != cols) return ARD_ERR_INVALID_ARG;
  if (!encode_map(ctx, &out->tm, base, (uint64_t)cols, (uint64_t)rows, (uint64_t)ld * 2, (uint32_t)box_cols,
                  (uint32_t)box_rows))
    return ARD_ERR_CUDA;
  out->base = base;
  out->dense_base = dense_base;
  out->ld = ld;
  out->dense_ld = dense_ld;
  out->variant = variant;
  out->pad_ = 0;
  return ARD_OK;
}

ard_status check_common(ard_ctx* ctx, const ard_pattern* pat, int B, int K, int N) {
  if (!ctx || !pat) return ARD_ERR_INVALID_ARG;
  if (pat->ctx != ctx) return ARD_ERR_INVALID_ARG;
  if (B < 0 || K < 0 || N < 0) return ARD_ERR_INVALID_ARG;
  if (K != pat->K_dim || N != pat->N_dim) return ARD_ERR_SHAPE;
  if (B > 65535 * 32) return ARD_ERR_UNSUPPORTED;
  return ARD_OK;
}

void fill_common(GemmArgs& g, ard_ctx* ctx, const ard_pattern* pat, int B, int K, int N, float alpha) {
  g.hdr = pat->d_hdr;
  g.idx = pat->d_idx;
  g.col_ptr = pat->d_col_ptr;
  g.col_idx = pat->d_col_idx;
  g.row_ptr = pat->d_row_ptr;
  g.row_idx = pat->d_row_idx;
  g.B = B; g.K = K; g.N = N;
  g.alpha = alpha;
  g.flag0 = g.flag1 = 0;
  g.out_is_f32 = 0;
  g.accumulate = 0;
  g.status = ctx->d_status;
  g.hdr_in = nullptr;
  g.bias = nullptr;
  g.relu = 0;
  g.act = nullptr;
  g.ldact = 0;
}

// Can the tcgen05 path take this call?  (bf16 only; 16-byte aligned pointers and pitches; distributions of
// at most ARD_MAX_NDP_TC periods.)
ard_status tc_eligible(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, int B, int K, int N,
                       const void* p0, int ld0, const void* p1, int ld1, const void* po, int ldo, int out_es) {
  if (dtype != ARD_BF16) return ARD_ERR_UNSUPPORTED;
  if (ctx->encode_fn == nullptr) return ARD_ERR_UNSUPPORTED;
  if (B < 1 || K < 1 || N < 1) return ARD_ERR_UNSUPPORTED;
  if (pat->kind == ARD_ROW && pat->dp_bound > ARD_MAX_NDP_TC) return ARD_ERR_UNSUPPORTED;
  if (pat->kind == ARD_TILE && pat->ts % 64 != 0) return ARD_ERR_UNSUPPORTED;
  if (!aligned16(p0) || !aligned16(p1) || !aligned16(po)) return ARD_ERR_ALIGNMENT;
  if (ld0 % 8 || ld1 % 8 || ((size_t)ldo * out_es) % 16) return ARD_ERR_ALIGNMENT;
  if (K % 8 || N % 8) return ARD_ERR_ALIGNMENT;
  return ARD_OK;
}

}  // namespace

ard_status ard_encode_tcmap(ard_ctx* ctx, const void* base, int rows, int cols, int ld, int units, int variant,
                            int box_rows, int box_cols, TcMap* out) {
  return get_maps(ctx, base, rows, cols, ld, units, variant, 0, box_rows, box_cols, out);
}

bool ard_side_streams(ard_ctx* ctx, cudaStream_t main) {
  if (ctx->n_ev == ARD_MLP_EVENTS && ctx->side_stream && ctx->aux_stream) return true;
  if (ctx->n_ev != 0) return false;  // an earlier attempt failed half way
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(main, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) return false;
  DeviceGuard guard(ctx->device);
  if (cudaStreamCreateWithFlags(&ctx->side_stream, cudaStreamNonBlocking) != cudaSuccess) {
    ctx->side_stream = nullptr;
    return false;
  }
  if (cudaStreamCreateWithFlags(&ctx->aux_stream, cudaStreamNonBlocking) != cudaSuccess) {
    ctx->aux_stream = nullptr;
    return false;
  }
  for (int i = 0; i < ARD_MLP_EVENTS; ++i) {
    if (cudaEventCreateWithFlags(&ctx->ev[i], cudaEventDisableTiming) != cudaSuccess) return false;
    ctx->n_ev = i + 1;
  }
  return true;
}

extern "C" {

const char* ard_status_string(ard_status s) {
  switch (s) {
    case ARD_OK: return "ok";
    case ARD_ERR_INVALID_ARG: return "invalid argument";
    case ARD_ERR_SHAPE: return "shape mismatch";
    case ARD_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
    case ARD_ERR_DISTRIBUTION: return "invalid pattern distribution";
    case ARD_ERR_UNSUPPORTED: return "unsupported configuration";
    case ARD_ERR_CUDA: return "CUDA call failed";
    case ARD_ERR_TIMEOUT: return "bounded device wait expired";
    case ARD_ERR_NOMEM: return "out of memory or workspace too small";
  }
  return "unknown status";
}

ard_status ard_create(ard_ctx** out, int device, size_t workspace_bytes) {
  if (!out || device < 0) return ARD_ERR_INVALID_ARG;
  *out = nullptr;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || device >= ndev) return ARD_ERR_CUDA;
  DeviceGuard guard(device);
  if (!guard.ok) return ARD_ERR_CUDA;
  ard_ctx* ctx = new (std::nothrow) ard_ctx();
  if (!ctx) return ARD_ERR_NOMEM;
  ctx->device = device;
  ctx->path = ARD_PATH_AUTO;
  ctx->force_bn = 0;
  ctx->band_m = 16;
  ctx->use_pairs = 1;
  ctx->reuse_compact = 0;
  ctx->stream_k = 0;
  ctx->use_pdl = 1;
  ctx->lstm_persistent = 1;
  ctx->d_grid_bar = nullptr;
  ctx->d_lstm_partial = nullptr;
  ctx->d_lstm_hc = nullptr;
  ctx->lstm_compact_h = 1;
  ctx->pdl_in_capture = 1;
  ctx->mlp_two_streams = 1;
  ctx->mlp_persistent = 1;
  ctx->side_stream = nullptr;
  ctx->aux_stream = nullptr;
  ctx->n_ev = 0;
  ctx->sk_min_blocks = 16;
  ctx->sk_min_gain = 24;
  ctx->d_sk_ws = nullptr;
  ctx->d_sk_cnt = nullptr;
  ctx->last_gather = {nullptr, 0, 0, 0, nullptr, 0ull, nullptr};
  ctx->workspace_bytes = workspace_bytes;
  ctx->d_workspace = nullptr;
  ctx->d_status = nullptr;
  ctx->launches = 0;
  ctx->d_tm_slots = nullptr;
  ctx->encode_fn = nullptr;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete ctx; return ARD_ERR_CUDA; }
  ctx->sm_count = prop.multiProcessorCount;
  if (prop.major == 10) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      ctx->encode_fn = fn;
  }
  if (cudaMalloc(&ctx->d_status, sizeof(int)) != cudaSuccess) { delete ctx; return ARD_ERR_NOMEM; }
  cudaMemset(ctx->d_status, 0, sizeof(int));
  if (workspace_bytes > 0 && cudaMalloc(&ctx->d_workspace, workspace_bytes) != cudaSuccess) {
    cudaFree(ctx->d_status);
    delete ctx;
    return ARD_ERR_NOMEM;
  }
  if (ctx->encode_fn != nullptr) {
    // scratch of the tensor-core row kernels' shared tail
    const size_t ws_bytes = sk_ws_bytes(ctx->sm_count);
    const size_t cnt_bytes = sk_cnt_bytes(ctx->sm_count);
    if (cudaMalloc(&ctx->d_sk_ws, ws_bytes) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&ctx->d_sk_cnt), cnt_bytes) != cudaSuccess ||
        cudaMemset(ctx->d_sk_cnt, 0, cnt_bytes) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&ctx->d_tm_slots), tm_slots_bytes()) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&ctx->d_grid_bar), 256) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&ctx->d_lstm_partial), lstm_bwd_partial_bytes(ctx->sm_count)) != cudaSuccess ||
        cudaMalloc(&ctx->d_lstm_hc, lstm_hc_bytes()) != cudaSuccess ||
        cudaMemset(ctx->d_lstm_hc, 0, lstm_hc_bytes()) != cudaSuccess) {
      if (ctx->d_lstm_hc) cudaFree(ctx->d_lstm_hc);
      if (ctx->d_lstm_partial) cudaFree(ctx->d_lstm_partial);
      if (ctx->d_grid_bar) cudaFree(ctx->d_grid_bar);
      if (ctx->d_tm_slots) cudaFree(ctx->d_tm_slots);
      if (ctx->d_sk_ws) cudaFree(ctx->d_sk_ws);
      if (ctx->d_sk_cnt) cudaFree(ctx->d_sk_cnt);
      if (ctx->d_workspace) cudaFree(ctx->d_workspace);
      cudaFree(ctx->d_status);
      delete ctx;
      return ARD_ERR_NOMEM;
    }
  }
  *out = ctx;
  return ARD_OK;
}

ard_status ard_destroy(ard_ctx* ctx) {
  if (!ctx) return ARD_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  cudaDeviceSynchronize();
  if (ctx->d_tm_slots) cudaFree(ctx->d_tm_slots);
  for (int i = 0; i < ARD_MAX_DISTRIBUTIONS; ++i)
    if (ctx->dist[i].d_cdf) cudaFree(ctx->dist[i].d_cdf);
  if (ctx->d_workspace) cudaFree(ctx->d_workspace);
  if (ctx->d_sk_ws) cudaFree(ctx->d_sk_ws);
  if (ctx->d_sk_cnt) cudaFree(ctx->d_sk_cnt);
  if (ctx->d_grid_bar) cudaFree(ctx->d_grid_bar);
  if (ctx->d_lstm_partial) cudaFree(ctx->d_lstm_partial);
  if (ctx->d_lstm_hc) cudaFree(ctx->d_lstm_hc);
  if (ctx->d_status) cudaFree(ctx->d_status);
  for (int i = 0; i < ctx->n_ev; ++i) cudaEventDestroy(ctx->ev[i]);
  if (ctx->side_stream) cudaStreamDestroy(ctx->side_stream);
  if (ctx->aux_stream) cudaStreamDestroy(ctx->aux_stream);
  delete ctx;
  return ARD_OK;
}

ard_status ard_set_path(ard_ctx* ctx, ard_path path) {
  if (!ctx || path < ARD_PATH_AUTO || path > ARD_PATH_TENSOR_CORE) return ARD_ERR_INVALID_ARG;
  ctx->path = path;
  return ARD_OK;
}

ard_status ard_set_option(ard_ctx* ctx, ard_option option, int value) {
  if (!ctx || value < 0) return ARD_ERR_INVALID_ARG;
  switch (option) {
    case ARD_OPT_PDL: ctx->use_pdl = value ? 1 : 0; return ARD_OK;
    case ARD_OPT_PDL_IN_CAPTURE: ctx->pdl_in_capture = value ? 1 : 0; return ARD_OK;
    case ARD_OPT_SIDE_STREAMS: ctx->mlp_two_streams = value ? 1 : 0; return ARD_OK;
    case ARD_OPT_CTA_PAIRS: ctx->use_pairs = value ? 1 : 0; return ARD_OK;
    case ARD_OPT_BAND_ROWS: ctx->band_m = value; return ARD_OK;
    case ARD_OPT_MLP_PERSISTENT: ctx->mlp_persistent = value ? 1 : 0; return ARD_OK;
    case ARD_OPT_LSTM_COMPACT_H: ctx->lstm_compact_h = value ? 1 : 0; return ARD_OK;
  }
  return ARD_ERR_INVALID_ARG;
}

ard_status ard_set_compact_reuse(ard_ctx* ctx, int enable) {
  if (!ctx) return ARD_ERR_INVALID_ARG;
  ctx->reuse_compact = enable ? 1 : 0;
  ctx->last_gather.src = nullptr;
  return ARD_OK;
}

ard_status ard_set_shared_tail(ard_ctx* ctx, int enable, int min_blocks, int min_gain_blocks) {
  if (!ctx || min_blocks < 0 || min_gain_blocks < 0) return ARD_ERR_INVALID_ARG;
  ctx->stream_k = enable ? 1 : 0;
  if (min_blocks > 0) ctx->sk_min_blocks = min_blocks;
  if (min_gain_blocks > 0) ctx->sk_min_gain = min_gain_blocks;
  return ARD_OK;
}

ard_status ard_set_lstm_persistent(ard_ctx* ctx, int enable) {
  if (!ctx) return ARD_ERR_INVALID_ARG;
  ctx->lstm_persistent = enable ? 1 : 0;
  return ARD_OK;
}

ard_status ard_set_tile_n(ard_ctx* ctx, int bn) {
  if (!ctx || (bn != 0 && (bn < 64 || bn > 256 || bn % 32 != 0))) return ARD_ERR_INVALID_ARG;
  ctx->force_bn = bn;
  return ARD_OK;
}

// Host-only: validates K and writes its integer cumulative table (no context, no GPU needed).
ard_status ard_quantise_distribution(const double* K, int ndp, uint64_t* cdf_out) {
  if (!K || !cdf_out) return ARD_ERR_INVALID_ARG;
  if (ndp < 1 || ndp > ARD_MAX_NDP) return ARD_ERR_DISTRIBUTION;
  double sum = 0.0;
  for (int i = 0; i < ndp; ++i) {
    if (!(K[i] >= 0.0)) return ARD_ERR_DISTRIBUTION;  // also rejects NaN
    sum += K[i];
  }
  if (!(fabs(sum - 1.0) <= 1e-9)) return ARD_ERR_DISTRIBUTION;
  // Integer cumulative table on a 2^32 grid from sequential prefix sums.
  const unsigned long long TOP = 1ull << 32;
  double s = 0.0;
  unsigned long long prev = 0;
  for (int i = 0; i < ndp; ++i) {
    s += K[i];
    unsigned long long c;
    if (i == ndp - 1) c = TOP;
    else {
      double v = floor(s * 4294967296.0 + 0.5);
      c = v <= 0.0 ? 0ull : (v >= 4294967296.0 ? TOP : (unsigned long long)v);
      if (c < prev) c = prev;
      if (c > TOP) c = TOP;
    }
    cdf_out[i] = c;
    prev = c;
  }
  return ARD_OK;
}

ard_status ard_set_distribution(ard_ctx* ctx, int dist_id, const double* K, int ndp) {
  if (!ctx || !K) return ARD_ERR_INVALID_ARG;
  if (dist_id < 0 || dist_id >= ARD_MAX_DISTRIBUTIONS) return ARD_ERR_INVALID_ARG;
  if (ndp < 1 || ndp > ARD_MAX_NDP) return ARD_ERR_DISTRIBUTION;
  std::vector<unsigned long long> cdf(ndp);
  {
    std::vector<uint64_t> tmp(ndp);
    ard_status qs = ard_quantise_distribution(K, ndp, tmp.data());
    if (qs != ARD_OK) return qs;
    for (int i = 0; i < ndp; ++i) cdf[i] = tmp[i];
  }
  DeviceGuard guard(ctx->device);
  ArdDistribution& d = ctx->dist[dist_id];
  if (d.d_cdf) {
    cudaDeviceSynchronize();
    cudaFree(d.d_cdf);
    d.d_cdf = nullptr;
    d.ndp = 0;
  }
  if (cudaMalloc(&d.d_cdf, sizeof(unsigned long long) * ndp) != cudaSuccess) return ARD_ERR_NOMEM;
  ARD_CUDA_OK(cudaMemcpy(d.d_cdf, cdf.data(), sizeof(unsigned long long) * ndp, cudaMemcpyHostToDevice));
  d.h_cdf = cdf;
  d.ndp = ndp;
  return ARD_OK;
}

ard_status ard_get_distribution_cdf(ard_ctx* ctx, int dist_id, uint64_t* cdf_out, int capacity, int* ndp_out) {
  if (!ctx || !ndp_out || dist_id < 0 || dist_id >= ARD_MAX_DISTRIBUTIONS) return ARD_ERR_INVALID_ARG;
  const ArdDistribution& d = ctx->dist[dist_id];
  if (d.ndp == 0) return ARD_ERR_DISTRIBUTION;
  *ndp_out = d.ndp;
  if (cdf_out)
    for (int i = 0; i < d.ndp && i < capacity; ++i) cdf_out[i] = d.h_cdf[i];
  return ARD_OK;
}

ard_status ard_pattern_create(ard_ctx* ctx, ard_pattern** out, ard_kind kind, int K_dim, int N_dim, int tile) {
  if (!ctx || !out) return ARD_ERR_INVALID_ARG;
  *out = nullptr;
  if (kind != ARD_ROW && kind != ARD_TILE) return ARD_ERR_INVALID_ARG;
  if (K_dim < 1 || N_dim < 1) return ARD_ERR_SHAPE;
  if (kind == ARD_ROW && tile != 0) return ARD_ERR_SHAPE;
  if (kind == ARD_TILE && (tile < 1 || K_dim % tile || N_dim % tile)) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  ard_pattern* p = new (std::nothrow) ard_pattern();
  if (!p) return ARD_ERR_NOMEM;
  p->ctx = ctx;
  p->kind = kind;
  p->K_dim = K_dim;
  p->N_dim = N_dim;
  p->ts = tile;
  p->Tr = kind == ARD_TILE ? K_dim / tile : 0;
  p->Tc = kind == ARD_TILE ? N_dim / tile : 0;
  const long long units = kind == ARD_TILE ? (long long)p->Tr * p->Tc : N_dim;
  if (units > (1ll << 30)) { delete p; return ARD_ERR_UNSUPPORTED; }
  p->units = (int)units;
  p->dp_bound = 1;
  p->generation = 0;
  size_t words = HDR_WORDS + (size_t)p->units;
  if (kind == ARD_TILE) words += (size_t)(p->Tc + 1) + (size_t)(p->Tr + 1) + 2 * (size_t)p->units;
  int32_t* d = nullptr;
  if (cudaMalloc(&d, words * sizeof(int32_t)) != cudaSuccess) { delete p; return ARD_ERR_NOMEM; }
  cudaMemset(d, 0, words * sizeof(int32_t));
  p->d_hdr = d;
  p->d_idx = d + HDR_WORDS;
  if (kind == ARD_TILE) {
    p->d_col_ptr = p->d_idx + p->units;
    p->d_col_idx = p->d_col_ptr + (p->Tc + 1);
    p->d_row_ptr = p->d_col_idx + p->units;
    p->d_row_idx = p->d_row_ptr + (p->Tr + 1);
  } else {
    p->d_col_ptr = p->d_col_idx = p->d_row_ptr = p->d_row_idx = nullptr;
  }
  *out = p;
  // A fresh pattern is dense (dp = 1) until sampled.
  return ard_pattern_set(ctx, p, 1, 1, nullptr);
}

ard_status ard_pattern_destroy(ard_pattern* pat) {
  if (!pat) return ARD_ERR_INVALID_ARG;
  DeviceGuard guard(pat->ctx->device);
  cudaDeviceSynchronize();
  cudaFree(pat->d_hdr);
  delete pat;
  return ARD_OK;
}

ard_status ard_sample_pattern(ard_ctx* ctx, ard_pattern* pat, int dist_id, uint64_t seed, uint64_t iteration,
                              uint32_t stream_id, void* cuda_stream) {
  if (!ctx || !pat || pat->ctx != ctx) return ARD_ERR_INVALID_ARG;
  if (dist_id < 0 || dist_id >= ARD_MAX_DISTRIBUTIONS) return ARD_ERR_INVALID_ARG;
  const ArdDistribution& d = ctx->dist[dist_id];
  if (d.ndp == 0 || d.ndp > pat->units) return ARD_ERR_DISTRIBUTION;
  DeviceGuard guard(ctx->device);
  pat->dp_bound = d.ndp;
  pat->generation++;
  return launch_sampler(ctx, pat, d.d_cdf, d.ndp, seed, iteration, stream_id, 0, 0, (cudaStream_t)cuda_stream);
}

ard_status ard_pattern_set(ard_ctx* ctx, ard_pattern* pat, int dp, int b, void* cuda_stream) {
  if (!ctx || !pat || pat->ctx != ctx) return ARD_ERR_INVALID_ARG;
  if (dp < 1 || b < 1 || b > dp || dp > pat->units) return ARD_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  pat->dp_bound = dp;
  pat->generation++;
  return launch_sampler(ctx, pat, nullptr, 0, 0, 0, 0, dp, b, (cudaStream_t)cuda_stream);
}

ard_status ard_pattern_to_host(const ard_pattern* pat, int32_t* dp, int32_t* b, int32_t* n_keep, int32_t* idx,
                               size_t idx_capacity, void* cuda_stream) {
  if (!pat) return ARD_ERR_INVALID_ARG;
  DeviceGuard guard(pat->ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  int32_t hdr[HDR_WORDS];
  ARD_CUDA_OK(cudaMemcpyAsync(hdr, pat->d_hdr, sizeof(hdr), cudaMemcpyDeviceToHost, s));
  ARD_CUDA_OK(cudaStreamSynchronize(s));
  if (dp) *dp = hdr[HDR_DP];
  if (b) *b = hdr[HDR_B];
  if (n_keep) *n_keep = hdr[HDR_NKEEP];
  if (idx && idx_capacity > 0) {
    size_t n = (size_t)hdr[HDR_NKEEP] < idx_capacity ? (size_t)hdr[HDR_NKEEP] : idx_capacity;
    ARD_CUDA_OK(cudaMemcpyAsync(idx, pat->d_idx, n * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    ARD_CUDA_OK(cudaStreamSynchronize(s));
  }
  return ARD_OK;
}

ard_status ard_pattern_tile_lists_to_host(const ard_pattern* pat, int32_t* col_ptr, int32_t* col_idx,
                                          int32_t* row_ptr, int32_t* row_idx, void* cuda_stream) {
  if (!pat || !col_ptr || !col_idx || !row_ptr || !row_idx) return ARD_ERR_INVALID_ARG;
  if (pat->kind != ARD_TILE) return ARD_ERR_INVALID_ARG;
  DeviceGuard guard(pat->ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  ARD_CUDA_OK(cudaMemcpyAsync(col_ptr, pat->d_col_ptr, (pat->Tc + 1) * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  ARD_CUDA_OK(cudaMemcpyAsync(row_ptr, pat->d_row_ptr, (pat->Tr + 1) * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  ARD_CUDA_OK(cudaMemcpyAsync(col_idx, pat->d_col_idx, (size_t)pat->units * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  ARD_CUDA_OK(cudaMemcpyAsync(row_idx, pat->d_row_idx, (size_t)pat->units * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  ARD_CUDA_OK(cudaStreamSynchronize(s));
  return ARD_OK;
}

// ---------------------------------------------------------------------------------------------------

// Validates the pattern of the layer that feeds a fused layer step.
static ard_status check_in_pattern(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, int K) {
  if (in_pat == nullptr) return ARD_OK;
  if (in_pat->ctx != ctx || in_pat->kind != ARD_ROW || pat->kind != ARD_ROW) return ARD_ERR_INVALID_ARG;
  if (in_pat->N_dim != K) return ARD_ERR_SHAPE;
  return ARD_OK;
}

static ard_status fwd_impl(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, ard_dtype dtype, int B, int K,
                           int N, float alpha, const void* X, int ldx, const void* W, int ldw, const float* bias,
                           int relu, void* Y, int ldy, int outmode, void* cuda_stream) {
  ard_status st = check_common(ctx, pat, B, K, N);
  if (st != ARD_OK) return st;
  st = check_in_pattern(ctx, pat, in_pat, K);
  if (st != ARD_OK) return st;
  if ((bias != nullptr || relu) && pat->kind != ARD_ROW) return ARD_ERR_INVALID_ARG;
  if (!X || !W || !Y) return ARD_ERR_INVALID_ARG;
  if (dtype != ARD_F32 && dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  const int mode = outmode & 0xF;
  const bool out_f32 = dtype == ARD_F32 || (outmode & ARD_FLAG_OUT_F32);
  const bool accumulate = (outmode & ARD_FLAG_ACCUMULATE) != 0;
  if ((outmode & ~(0xF | ARD_FLAG_OUT_F32 | ARD_FLAG_ACCUMULATE)) != 0) return ARD_ERR_INVALID_ARG;
  if (mode != ARD_OUT_COMPACT && mode != ARD_OUT_SCATTER_ZEROFILL) return ARD_ERR_INVALID_ARG;
  if (accumulate && mode == ARD_OUT_SCATTER_ZEROFILL && pat->kind == ARD_ROW) return ARD_ERR_INVALID_ARG;
  if (ldx < K || ldw < K || ldy < N) return ARD_ERR_SHAPE;
  if (B == 0) return ARD_OK;
  DeviceGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int es = out_f32 ? 4 : 2;

  GemmArgs g = {};
  fill_common(g, ctx, pat, B, K, N, alpha);
  g.A0 = X; g.lda0 = ldx; g.A1 = W; g.lda1 = ldw; g.out = Y; g.ldo = ldy;
  g.flag0 = pat->kind == ARD_ROW ? mode : 0;
  g.out_is_f32 = out_f32;
  g.accumulate = accumulate;
  g.hdr_in = in_pat ? in_pat->d_hdr : nullptr;
  g.bias = bias;
  g.relu = relu ? 1 : 0;
  if (accumulate && (bias != nullptr || relu)) return ARD_ERR_INVALID_ARG;

  ard_status el = ctx->path == ARD_PATH_CUDA_CORE ? ARD_ERR_UNSUPPORTED
                                                  : tc_eligible(ctx, pat, dtype, B, K, N, X, ldx, W, ldw, Y, ldy, es);
  if (el == ARD_OK && in_pat && in_pat->dp_bound > ARD_MAX_NDP_TC) el = ARD_ERR_UNSUPPORTED;
  // the tensor-core scatter epilogue writes bf16 only
  if (el == ARD_OK && out_f32 && pat->kind == ARD_ROW && mode == ARD_OUT_SCATTER_ZEROFILL) el = ARD_ERR_UNSUPPORTED;
  if (el != ARD_OK) {
    if (ctx->path == ARD_PATH_TENSOR_CORE) return el;
    return launch_gemm_cc(ctx, pat->kind, OP_FWD, dtype, g, pat->ts, s);
  }
  TcArgs t = {};
  t.g = g;
  t.ts = pat->ts;
  t.bn = tc_pick_bn(ctx, pat->kind, OP_FWD, pat->dp_bound, pat->ts);
  // A = X, K-major boxes [128 rows][64 k];  B = kept neurons of W, K-major boxes [64 rows][64 k].
  if (in_pat) {
    // compact X: one descriptor per pattern of the feeding layer, whose extent ends at its kept count
    st = get_maps(ctx, X, B, K, ldx, K, MAP_COMPACT_COLS, in_pat->dp_bound, 128, 64, &t.mapA);
    t.mapA_indexed = 2;
  } else {
    st = get_maps(ctx, X, B, K, ldx, 0, MAP_PLAIN, 0, 128, 64, &t.mapA);
    t.mapA_indexed = 0;
  }
  if (st != ARD_OK) return st;
  if (pat->kind == ARD_ROW && !in_pat) {
    st = get_maps(ctx, W, N, K, ldw, N, MAP_STRIDED_ROWS, pat->dp_bound, 64, 64, &t.mapB);
    t.mapB_indexed = 1;
  } else {
    // tile patterns; or the weight packed by ard_compact_weight_cols: its kept rows are rows 0..n_keep-1
    st = get_maps(ctx, W, N, K, ldw, 0, MAP_PLAIN, 0, 64, 64, &t.mapB);
    t.mapB_indexed = 0;
  }
  if (st != ARD_OK) return st;
  return launch_gemm_tc(ctx, pat->kind, OP_FWD, t, s);
}

ard_status ard_fwd(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, int B, int K, int N, float alpha,
                   const void* X, int ldx, const void* W, int ldw, void* Y, int ldy, ard_outmode outmode,
                   void* cuda_stream) {
  if (((int)outmode & ARD_FLAG_RELU) != 0) return ARD_ERR_INVALID_ARG;
  return fwd_impl(ctx, pat, nullptr, dtype, B, K, N, alpha, X, ldx, W, ldw, nullptr, 0, Y, ldy, (int)outmode, cuda_stream);
}

ard_status ard_layer_fwd(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, ard_dtype dtype, int B, int K,
                         int N, float alpha, const void* X, int ldx, const void* W, int ldw, const float* bias, void* A,
                         int lda, int outmode, void* cuda_stream) {
  if (!pat || pat->kind != ARD_ROW) return ARD_ERR_INVALID_ARG;
  const int relu = (outmode & ARD_FLAG_RELU) ? 1 : 0;
  return fwd_impl(ctx, pat, in_pat, dtype, B, K, N, alpha, X, ldx, W, ldw, bias, relu, A, lda, outmode & ~ARD_FLAG_RELU,
                  cuda_stream);
}

// Produces the operand the tensor-core backward GEMMs read for dY: the caller's compact matrix, or
// a compacted copy of the full-width one in the context workspace (row patterns only).
static ard_status compact_dy(ard_ctx* ctx, const ard_pattern* pat, int B, int N, const void* dY, int lddy,
                             int dy_is_compact, const void** out_ptr, int* out_ld, const void** dense_ptr,
                             int* dense_ld, cudaStream_t s) {
  *dense_ptr = nullptr;
  *dense_ld = 0;
  if (dy_is_compact) {
    *out_ptr = dY;
    *out_ld = lddy;
    return ARD_OK;
  }
  // A dense pattern (dp = 1) is not copied: the descriptor of that case reads dY itself.
  *dense_ptr = dY;
  *dense_ld = lddy;
  const int ldc = (N + 7) / 8 * 8;
  if ((size_t)B * ldc * 2 > ctx->workspace_bytes) return ARD_ERR_NOMEM;
  *out_ptr = ctx->d_workspace;
  *out_ld = ldc;
  auto& lg = ctx->last_gather;
  if (ctx->reuse_compact && lg.src == dY && lg.ld == lddy && lg.B == B && lg.N == N && lg.pat == pat &&
      lg.gen == pat->generation && lg.stream == s)
    return ARD_OK;  // the previous backward call on this stream already compacted this dY for this pattern
  lg = {dY, lddy, B, N, pat, pat->generation, s};
  ard_status st = launch_gather_cols(ctx, pat->d_hdr, pat->d_idx, dY, lddy, ctx->d_workspace, ldc, B, 2, N, 1, s);
  *out_ptr = ctx->d_workspace;
  *out_ld = ldc;
  return st;
}

static ard_status bwd_data_impl(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, ard_dtype dtype, int B,
                                int K, int N, float alpha, const void* dY, int lddy, int dy_is_compact, const void* W,
                                int ldw, const void* act, int ldact, void* dX, int lddx, void* cuda_stream) {
  ard_status st = check_common(ctx, pat, B, K, N);
  if (st != ARD_OK) return st;
  st = check_in_pattern(ctx, pat, in_pat, K);
  if (st != ARD_OK) return st;
  if (act != nullptr && (pat->kind != ARD_ROW || ldact < 1)) return ARD_ERR_INVALID_ARG;
  if (!dY || !W || !dX) return ARD_ERR_INVALID_ARG;
  if (dtype != ARD_F32 && dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  const int flags = dy_is_compact;
  if ((flags & ~(1 | ARD_FLAG_OUT_F32 | ARD_FLAG_ACCUMULATE)) != 0) return ARD_ERR_INVALID_ARG;
  dy_is_compact = flags & 1;
  const bool out_f32 = dtype == ARD_F32 || (flags & ARD_FLAG_OUT_F32);
  if (dy_is_compact && pat->kind != ARD_ROW) return ARD_ERR_INVALID_ARG;
  if (lddy < (dy_is_compact ? 1 : N) || ldw < K || lddx < K) return ARD_ERR_SHAPE;
  if (B == 0) return ARD_OK;
  DeviceGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int es = out_f32 ? 4 : 2;

  GemmArgs g = {};
  fill_common(g, ctx, pat, B, K, N, alpha);
  g.A0 = dY; g.lda0 = lddy; g.A1 = W; g.lda1 = ldw; g.out = dX; g.ldo = lddx;
  g.flag0 = dy_is_compact ? 1 : 0;
  g.out_is_f32 = out_f32;
  g.accumulate = (flags & ARD_FLAG_ACCUMULATE) != 0;
  g.hdr_in = in_pat ? in_pat->d_hdr : nullptr;
  g.act = act;
  g.ldact = ldact;
  if (g.accumulate && act != nullptr) return ARD_ERR_INVALID_ARG;

  ard_status el = ctx->path == ARD_PATH_CUDA_CORE
                      ? ARD_ERR_UNSUPPORTED
                      : tc_eligible(ctx, pat, dtype, B, K, N, dY, lddy, W, ldw, dX, lddx, es);
  // the tensor-core epilogue reads the activations in 16-byte pieces
  if (el == ARD_OK && act != nullptr && (!aligned16(act) || ldact % 8 != 0)) el = ARD_ERR_ALIGNMENT;
  if (el == ARD_OK && pat->kind == ARD_ROW && !dy_is_compact &&
      (size_t)B * ((N + 7) / 8 * 8) * 2 > ctx->workspace_bytes)
    el = ARD_ERR_NOMEM;
  if (el != ARD_OK) {
    if (ctx->path == ARD_PATH_TENSOR_CORE) return el;
    return launch_gemm_cc(ctx, pat->kind, OP_BWD_DATA, dtype, g, pat->ts, s);
  }
  TcArgs t = {};
  t.ts = pat->ts;
  t.bn = tc_pick_bn(ctx, pat->kind, OP_BWD_DATA, pat->dp_bound, pat->ts);
  if (pat->kind == ARD_ROW) {
    const void *dyc, *dense;
    int ldc, dense_ld;
    st = compact_dy(ctx, pat, B, N, dY, lddy, dy_is_compact, &dyc, &ldc, &dense, &dense_ld, s);
    if (st != ARD_OK) return st;
    g.A0 = dyc; g.lda0 = ldc; g.flag0 = 1;
    // A = compact dY [B][n_keep], K-major;  B = kept neurons of W read MN-major: boxes [64 kept rows][64 k].
    st = get_maps(ctx, dyc, B, N, ldc, N, MAP_COMPACT_COLS, pat->dp_bound, 128, 64, &t.mapA, dense, dense_ld);
    if (st != ARD_OK) return st;
    t.mapA_indexed = 1;
    if (in_pat) {  // packed weight: rows 0..n_keep-1 (zero rows up to the next multiple of 64)
      st = get_maps(ctx, W, N, K, ldw, 0, MAP_PLAIN, 0, 64, 64, &t.mapB);
      t.mapB_indexed = 0;
    } else {
      st = get_maps(ctx, W, N, K, ldw, N, MAP_STRIDED_ROWS, pat->dp_bound, 64, 64, &t.mapB);
      t.mapB_indexed = 1;
    }
  } else {
    st = get_maps(ctx, dY, B, N, lddy, 0, MAP_PLAIN, 0, 128, 64, &t.mapA);
    if (st != ARD_OK) return st;
    t.mapA_indexed = 0;
    st = get_maps(ctx, W, N, K, ldw, 0, MAP_PLAIN, 0, 64, 64, &t.mapB);
    t.mapB_indexed = 0;
  }
  if (st != ARD_OK) return st;
  t.g = g;
  return launch_gemm_tc(ctx, pat->kind, OP_BWD_DATA, t, s);
}

ard_status ard_bwd_data(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, int B, int K, int N, float alpha,
                        const void* dY, int lddy, int dy_is_compact, const void* W, int ldw, void* dX, int lddx,
                        void* cuda_stream) {
  return bwd_data_impl(ctx, pat, nullptr, dtype, B, K, N, alpha, dY, lddy, dy_is_compact, W, ldw, nullptr, 0, dX, lddx,
                       cuda_stream);
}

ard_status ard_layer_bwd_data(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, ard_dtype dtype, int B,
                              int K, int N, float alpha, const void* dZ, int lddz, int flags, const void* W, int ldw,
                              const void* act, int ldact, void* dX, int lddx, void* cuda_stream) {
  if (!pat || pat->kind != ARD_ROW) return ARD_ERR_INVALID_ARG;
  return bwd_data_impl(ctx, pat, in_pat, dtype, B, K, N, alpha, dZ, lddz, flags, W, ldw, act, ldact, dX, lddx,
                       cuda_stream);
}

static ard_status bwd_weight_impl(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, ard_dtype dtype,
                                  ard_dtype dW_dtype, int B, int K, int N, float alpha, const void* X, int ldx,
                                  const void* dY, int lddy, int dy_is_compact, void* dW, int lddw,
                                  int zero_fill_dropped, void* cuda_stream) {
  ard_status st = check_common(ctx, pat, B, K, N);
  if (st != ARD_OK) return st;
  st = check_in_pattern(ctx, pat, in_pat, K);
  if (st != ARD_OK) return st;
  if (!X || !dY || !dW) return ARD_ERR_INVALID_ARG;
  if (dtype != ARD_F32 && dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (dW_dtype != ARD_F32 && dW_dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (dtype == ARD_F32 && dW_dtype != ARD_F32) return ARD_ERR_INVALID_ARG;
  if (dy_is_compact && pat->kind != ARD_ROW) return ARD_ERR_INVALID_ARG;
  if (ldx < K || lddy < (dy_is_compact ? 1 : N) || lddw < K) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int es_out = dW_dtype == ARD_F32 ? 4 : 2;

  GemmArgs g = {};
  fill_common(g, ctx, pat, B, K, N, alpha);
  g.A0 = dY; g.lda0 = lddy; g.A1 = X; g.lda1 = ldx; g.out = dW; g.ldo = lddw;
  g.flag0 = dy_is_compact ? 1 : 0;
  g.flag1 = zero_fill_dropped ? 1 : 0;
  g.out_is_f32 = dW_dtype == ARD_F32;
  g.hdr_in = in_pat ? in_pat->d_hdr : nullptr;
  if (in_pat && zero_fill_dropped) return ARD_ERR_INVALID_ARG;  // the packed gradient has no rows of dropped neurons
  // Empty batch: the gradient of every kept weight is zero; the CUDA-core kernel writes exactly that.
  if (B == 0) return launch_gemm_cc(ctx, pat->kind, OP_BWD_WEIGHT, dtype, g, pat->ts, s);

  ard_status el = ctx->path == ARD_PATH_CUDA_CORE
                      ? ARD_ERR_UNSUPPORTED
                      : tc_eligible(ctx, pat, dtype, B, K, N, dY, lddy, X, ldx, dW, lddw, es_out);
  if (el == ARD_OK && pat->kind == ARD_ROW && !dy_is_compact &&
      (size_t)B * ((N + 7) / 8 * 8) * 2 > ctx->workspace_bytes)
    el = ARD_ERR_NOMEM;
  if (el != ARD_OK) {
    if (ctx->path == ARD_PATH_TENSOR_CORE) return el;
    return launch_gemm_cc(ctx, pat->kind, OP_BWD_WEIGHT, dtype, g, pat->ts, s);
  }
  TcArgs t = {};
  t.ts = pat->ts;
  t.bn = tc_pick_bn(ctx, pat->kind, OP_BWD_WEIGHT, pat->dp_bound, pat->ts);
  if (pat->kind == ARD_ROW) {
    const void *dyc, *dense;
    int ldc, dense_ld;
    st = compact_dy(ctx, pat, B, N, dY, lddy, dy_is_compact, &dyc, &ldc, &dense, &dense_ld, s);
    if (st != ARD_OK) return st;
    g.A0 = dyc; g.lda0 = ldc; g.flag0 = 1;
    // A = compact dY read MN-major (boxes [64 batch rows][64 kept cols]);  B = X read MN-major.
    st = get_maps(ctx, dyc, B, N, ldc, N, MAP_COMPACT_COLS, pat->dp_bound, 64, 64, &t.mapA, dense, dense_ld);
    t.mapA_indexed = 1;
  } else {
    if (zero_fill_dropped) {
      st = launch_zero_dropped_tiles(ctx, pat, dW, lddw, es_out, s);
      if (st != ARD_OK) return st;
    }
    st = get_maps(ctx, dY, B, N, lddy, 0, MAP_PLAIN, 0, 64, 64, &t.mapA);
    t.mapA_indexed = 0;
  }
  if (st != ARD_OK) return st;
  st = get_maps(ctx, X, B, K, ldx, 0, MAP_PLAIN, 0, 64, 64, &t.mapB);
  t.mapB_indexed = 0;
  if (st != ARD_OK) return st;
  t.g = g;
  return launch_gemm_tc(ctx, pat->kind, OP_BWD_WEIGHT, t, s);
}

ard_status ard_bwd_weight(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, ard_dtype dW_dtype, int B, int K,
                          int N, float alpha, const void* X, int ldx, const void* dY, int lddy, int dy_is_compact,
                          void* dW, int lddw, int zero_fill_dropped, void* cuda_stream) {
  return bwd_weight_impl(ctx, pat, nullptr, dtype, dW_dtype, B, K, N, alpha, X, ldx, dY, lddy, dy_is_compact, dW, lddw,
                         zero_fill_dropped, cuda_stream);
}

// The three products of one layer and one iteration, which depend only on X, W, dY and the pattern, enqueued so
// that they can run side by side: on small layers a product occupies a fraction of the SMs (and a tile pattern
// whose period divides the tile-column count concentrates the forward product's work in 1/dp of its output
// tiles), so the other two fill the idle ones.
ard_status ard_layer_products(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, ard_dtype dW_dtype, int B, int K,
                              int N, float alpha, const void* X, int ldx, const void* W, int ldw, const void* dY,
                              int lddy, void* Y, int ldy, ard_outmode outmode, void* dX, int lddx, void* dW, int lddw,
                              int zero_fill_dropped, void* cuda_stream) {
  if (!ctx || !pat) return ARD_ERR_INVALID_ARG;
  if (((int)outmode & ARD_FLAG_RELU) != 0) return ARD_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const bool streams = ctx->mlp_two_streams && ard_side_streams(ctx, s);
  SharedTailOff tail_guard(ctx, streams);
  // The compact copy of dY is shared by this call's two backward products only: whatever an earlier call left in
  // the workspace is never taken for it (same buffer, new contents), and nothing is left for a later call.
  struct ForgetGather {
    ard_ctx* c;
    explicit ForgetGather(ard_ctx* c_) : c(c_) { c->last_gather.src = nullptr; }
    ~ForgetGather() { c->last_gather.src = nullptr; }
  } forget(ctx);
  if (!streams) {
    // one stream: the calls in order, the second backward product reusing the first one's compact dY
    const int reuse = ctx->reuse_compact;
    ctx->reuse_compact = 1;
    ard_status st = fwd_impl(ctx, pat, nullptr, dtype, B, K, N, alpha, X, ldx, W, ldw, nullptr, 0, Y, ldy, (int)outmode, s);
    if (st == ARD_OK)
      st = bwd_data_impl(ctx, pat, nullptr, dtype, B, K, N, alpha, dY, lddy, 0, W, ldw, nullptr, 0, dX, lddx, s);
    if (st == ARD_OK)
      st = bwd_weight_impl(ctx, pat, nullptr, dtype, dW_dtype, B, K, N, alpha, X, ldx, dY, lddy, 0, dW, lddw,
                           zero_fill_dropped, s);
    ctx->reuse_compact = reuse;
    return st;
  }
  DeviceGuard guard(ctx->device);
  cudaStream_t side = ctx->side_stream, aux = ctx->aux_stream;
  // A row pattern's backward products share the compact copy of dY in the context workspace, so they stay on
  // one stream; a tile pattern's three products are independent.
  const bool three = pat->kind == ARD_TILE;
  ARD_CUDA_OK(cudaEventRecord(ctx->ev[100], s));
  ARD_CUDA_OK(cudaStreamWaitEvent(side, ctx->ev[100], 0));
  if (three) ARD_CUDA_OK(cudaStreamWaitEvent(aux, ctx->ev[100], 0));
  ard_status st = fwd_impl(ctx, pat, nullptr, dtype, B, K, N, alpha, X, ldx, W, ldw, nullptr, 0, Y, ldy, (int)outmode, s);
  const int reuse = ctx->reuse_compact;
  ctx->reuse_compact = 1;
  ard_status st2 = bwd_data_impl(ctx, pat, nullptr, dtype, B, K, N, alpha, dY, lddy, 0, W, ldw, nullptr, 0, dX, lddx, side);
  ard_status st3 = bwd_weight_impl(ctx, pat, nullptr, dtype, dW_dtype, B, K, N, alpha, X, ldx, dY, lddy, 0, dW, lddw,
                                   zero_fill_dropped, three ? aux : side);
  ctx->reuse_compact = reuse;
  // join whatever was enqueued, also after an error, so that a capture is not left forked
  ARD_CUDA_OK(cudaEventRecord(ctx->ev[101], side));
  ARD_CUDA_OK(cudaStreamWaitEvent(s, ctx->ev[101], 0));
  if (three) {
    ARD_CUDA_OK(cudaEventRecord(ctx->ev[102], aux));
    ARD_CUDA_OK(cudaStreamWaitEvent(s, ctx->ev[102], 0));
  }
  return st != ARD_OK ? st : (st2 != ARD_OK ? st2 : st3);
}

ard_status ard_layer_bwd_weight(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, ard_dtype dtype,
                                ard_dtype dW_dtype, int B, int K, int N, float alpha, const void* X, int ldx,
                                const void* dZ, int lddz, int dz_is_compact, void* dW, int lddw, int zero_fill_dropped,
                                void* cuda_stream) {
  if (!pat || pat->kind != ARD_ROW) return ARD_ERR_INVALID_ARG;
  return bwd_weight_impl(ctx, pat, in_pat, dtype, dW_dtype, B, K, N, alpha, X, ldx, dZ, lddz, dz_is_compact, dW, lddw,
                         zero_fill_dropped, cuda_stream);
}

ard_status ard_compact_weight_cols(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, ard_dtype dtype,
                                   int K, int N, const void* W, int ldw, void* Wk, int ldwk, void* cuda_stream) {
  ard_status st = check_common(ctx, pat, 0, K, N);
  if (st != ARD_OK) return st;
  if (!in_pat || !W || !Wk) return ARD_ERR_INVALID_ARG;
  st = check_in_pattern(ctx, pat, in_pat, K);
  if (st != ARD_OK) return st;
  if (dtype != ARD_F32 && dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (ldw < K || ldwk < K) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  return launch_compact_weight_cols(ctx, pat->d_hdr, in_pat->d_hdr, W, ldw, Wk, ldwk, N, K, dtype == ARD_F32 ? 4 : 2,
                                    (cudaStream_t)cuda_stream);
}

ard_status ard_expand_weight_grad_cols(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, ard_dtype dtype,
                                       int K, int N, const void* dWk, int lddwk, void* dW, int lddw, int zero_fill,
                                       void* cuda_stream) {
  ard_status st = check_common(ctx, pat, 0, K, N);
  if (st != ARD_OK) return st;
  if (!in_pat || !dWk || !dW || dWk == dW) return ARD_ERR_INVALID_ARG;
  st = check_in_pattern(ctx, pat, in_pat, K);
  if (st != ARD_OK) return st;
  if (dtype != ARD_F32 && dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (lddwk < K || lddw < K) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  return launch_expand_weight_grad_cols(ctx, pat->d_hdr, in_pat->d_hdr, dWk, lddwk, dW, lddw, N, K,
                                        dtype == ARD_F32 ? 4 : 2, zero_fill, (cudaStream_t)cuda_stream);
}

ard_status ard_bias_grad(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, int B, int N, const void* dZ, int lddz,
                         int dz_is_compact, float* db, int zero_fill_dropped, void* cuda_stream) {
  if (!ctx || !pat || pat->ctx != ctx || pat->kind != ARD_ROW) return ARD_ERR_INVALID_ARG;
  if (B < 0 || N != pat->N_dim) return ARD_ERR_SHAPE;
  if (!dZ || !db) return ARD_ERR_INVALID_ARG;
  if (dtype != ARD_F32 && dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (lddz < (dz_is_compact ? 1 : N)) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  return launch_bias_grad(ctx, pat->d_hdr, dZ, lddz, dz_is_compact ? 1 : 0, dtype == ARD_BF16, B, N, db,
                          zero_fill_dropped, (cudaStream_t)cuda_stream);
}

ard_status ard_sample_pattern_counter(ard_ctx* ctx, ard_pattern* pat, int dist_id, uint64_t seed, uint64_t iteration_base,
                                      uint64_t* iteration_counter, int advance, uint32_t stream_id,
                                      void* cuda_stream) {
  if (!ctx || !pat || pat->ctx != ctx || !iteration_counter) return ARD_ERR_INVALID_ARG;
  if (dist_id < 0 || dist_id >= ARD_MAX_DISTRIBUTIONS) return ARD_ERR_INVALID_ARG;
  const ArdDistribution& d = ctx->dist[dist_id];
  if (d.ndp == 0 || d.ndp > pat->units) return ARD_ERR_DISTRIBUTION;
  DeviceGuard guard(ctx->device);
  pat->dp_bound = d.ndp;
  pat->generation++;
  return launch_sampler(ctx, pat, d.d_cdf, d.ndp, seed, iteration_base, stream_id, 0, 0, (cudaStream_t)cuda_stream,
                        reinterpret_cast<unsigned long long*>(iteration_counter), advance ? 1 : 0);
}

// ---------------------------------------------------------------------------------------------------

// One launch for the four gate blocks when the tensor-core path can take the operands; otherwise four
// calls of the single-gate products.
ard_status ard_lstm_gate_gemm(ard_ctx* ctx, const ard_pattern* pat, int B, int KH, int H, const void* XH, int ldxh,
                              const void* W, int ldw, float* Z, int ldz_gate, void* cuda_stream) {
  ard_status st = check_common(ctx, pat, B, KH, H);
  if (st != ARD_OK) return st;
  if (!XH || !W || !Z) return ARD_ERR_INVALID_ARG;
  if (pat->kind != ARD_ROW) return ARD_ERR_INVALID_ARG;
  if (ldxh < KH || ldw < KH || ldz_gate < H) return ARD_ERR_SHAPE;
  if (B == 0) return ARD_OK;
  DeviceGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const char* Wc = reinterpret_cast<const char*>(W);
  ard_status el = ctx->path == ARD_PATH_CUDA_CORE
                      ? ARD_ERR_UNSUPPORTED
                      : tc_eligible(ctx, pat, ARD_BF16, B, KH, H, XH, ldxh, W, ldw, Z, 4 * ldz_gate, 4);
  if (el == ARD_OK && (ldz_gate % 8 != 0 || ((size_t)H * ldw * 2) % 16 != 0)) el = ARD_ERR_ALIGNMENT;
  if (el != ARD_OK) {
    if (ctx->path == ARD_PATH_TENSOR_CORE) return el;
    for (int g = 0; g < 4; ++g) {
      st = ard_fwd(ctx, pat, ARD_BF16, B, KH, H, 1.0f, XH, ldxh, Wc + (size_t)g * H * ldw * 2, ldw, Z + (size_t)g * ldz_gate,
                   4 * ldz_gate, (ard_outmode)(ARD_OUT_COMPACT | ARD_FLAG_OUT_F32), cuda_stream);
      if (st != ARD_OK) return st;
    }
    return ARD_OK;
  }
  TcArgs t = {};
  GemmArgs g = {};
  fill_common(g, ctx, pat, B, KH, H, 1.0f);
  g.A0 = XH; g.lda0 = ldxh; g.A1 = W; g.lda1 = ldw; g.out = Z; g.ldo = 4 * ldz_gate;
  g.out_is_f32 = 1;
  t.g = g;
  t.ts = ldz_gate;
  t.bn = 0;
  st = get_maps(ctx, XH, B, KH, ldxh, 0, MAP_PLAIN, 0, 128, 64, &t.mapA);
  if (st != ARD_OK) return st;
  t.mapA_indexed = 0;
  for (int gate = 0; gate < 4; ++gate) {
    st = get_maps(ctx, Wc + (size_t)gate * H * ldw * 2, H, KH, ldw, H, MAP_STRIDED_ROWS, pat->dp_bound, 64, 64,
                  &t.mapB4[gate]);
    if (st != ARD_OK) return st;
    t.mapA4[gate] = t.mapA;
  }
  t.mapB = t.mapB4[0];
  t.mapB_indexed = 1;
  return launch_lstm_tc(ctx, 0, t, s);
}

// Tensor-core form of the adjoint gate product over `kout` consecutive columns of [x | h]:
//   out[:, k] (+)= sum_g sum_j dZ[:, g*ldz_gate + j] * Wcols[g*H + keep[j]][k],   k < kout,
// where Wcols points at the first of those columns of the weight.  The caller has checked eligibility.
static ard_status lstm_gate_gemm_bwd_tc(ard_ctx* ctx, const ard_pattern* pat, int B, int kout, int H, const void* dZ,
                                        int ldz_gate, const void* Wcols, int ldw, float* out, int ldo, int accumulate,
                                        cudaStream_t s) {
  const char* Wc = reinterpret_cast<const char*>(Wcols);
  const char* dZc = reinterpret_cast<const char*>(dZ);
  TcArgs t = {};
  GemmArgs g = {};
  fill_common(g, ctx, pat, B, kout, H, 1.0f);
  g.A0 = dZ; g.lda0 = 4 * ldz_gate; g.A1 = Wcols; g.lda1 = ldw; g.out = out; g.ldo = ldo;
  g.flag0 = 1;
  g.out_is_f32 = 1;
  g.accumulate = accumulate ? 1 : 0;
  t.g = g;
  t.ts = ldz_gate;
  t.bn = ctx->force_bn;
  for (int gate = 0; gate < 4; ++gate) {
    ard_status st = get_maps(ctx, dZc + (size_t)gate * ldz_gate * 2, B, H, 4 * ldz_gate, H, MAP_COMPACT_COLS,
                             pat->dp_bound, 128, 64, &t.mapA4[gate]);
    if (st != ARD_OK) return st;
    st = get_maps(ctx, Wc + (size_t)gate * H * ldw * 2, H, kout, ldw, H, MAP_STRIDED_ROWS, pat->dp_bound, 64, 64,
                  &t.mapB4[gate]);
    if (st != ARD_OK) return st;
  }
  t.mapA = t.mapA4[0];
  t.mapB = t.mapB4[0];
  t.mapA_indexed = t.mapB_indexed = 1;
  return launch_lstm_tc(ctx, 1, t, s);
}

ard_status ard_lstm_gate_gemm_bwd(ard_ctx* ctx, const ard_pattern* pat, int B, int KH, int H, const void* dZ,
                                  int ldz_gate, const void* W, int ldw, float* dXH, int lddxh, int accumulate,
                                  void* cuda_stream) {
  ard_status st = check_common(ctx, pat, B, KH, H);
  if (st != ARD_OK) return st;
  if (!dZ || !W || !dXH) return ARD_ERR_INVALID_ARG;
  if (pat->kind != ARD_ROW) return ARD_ERR_INVALID_ARG;
  if (ldz_gate < 1 || ldw < KH || lddxh < KH) return ARD_ERR_SHAPE;
  if (B == 0) return ARD_OK;
  DeviceGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const char* Wc = reinterpret_cast<const char*>(W);
  const char* dZc = reinterpret_cast<const char*>(dZ);
  ard_status el = ctx->path == ARD_PATH_CUDA_CORE
                      ? ARD_ERR_UNSUPPORTED
                      : tc_eligible(ctx, pat, ARD_BF16, B, KH, H, dZ, 4 * ldz_gate, W, ldw, dXH, lddxh, 4);
  if (el == ARD_OK && (ldz_gate % 8 != 0 || ((size_t)H * ldw * 2) % 16 != 0)) el = ARD_ERR_ALIGNMENT;
  if (el != ARD_OK) {
    if (ctx->path == ARD_PATH_TENSOR_CORE) return el;
    for (int g = 0; g < 4; ++g) {
      const int flags = 1 | ARD_FLAG_OUT_F32 | ((accumulate || g > 0) ? ARD_FLAG_ACCUMULATE : 0);
      st = ard_bwd_data(ctx, pat, ARD_BF16, B, KH, H, 1.0f, dZc + (size_t)g * ldz_gate * 2, 4 * ldz_gate, flags,
                        Wc + (size_t)g * H * ldw * 2, ldw, dXH, lddxh, cuda_stream);
      if (st != ARD_OK) return st;
    }
    return ARD_OK;
  }
  return lstm_gate_gemm_bwd_tc(ctx, pat, B, KH, H, dZ, ldz_gate, W, ldw, dXH, lddxh, accumulate, s);
}

ard_status ard_lstm_gates(ard_ctx* ctx, const ard_pattern* pat, ard_dtype h_dtype, int B, int H, float alpha,
                          const float* Z, int ldz_gate, const float* bias, const float* c_prev, int ldc, float* c,
                          void* h, int ldh, int h_scatter, float* gates_saved, void* cuda_stream) {
  if (!ctx || !pat || pat->ctx != ctx || !Z || !c_prev || !c || !h) return ARD_ERR_INVALID_ARG;
  if (pat->kind != ARD_ROW || pat->N_dim != H) return ARD_ERR_SHAPE;
  if (B < 0 || B > 65535 || H < 1) return ARD_ERR_INVALID_ARG;
  if (h_dtype != ARD_F32 && h_dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (ldz_gate < 1 || ldc < 1 || ldh < 1 || (h_scatter && ldh < H)) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  return launch_lstm_gates(ctx, pat, h_dtype, B, H, alpha, Z, ldz_gate, bias, c_prev, ldc, c, h, ldh, h_scatter,
                           gates_saved, (cudaStream_t)cuda_stream);
}

ard_status ard_lstm_gates_bwd(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dz_dtype, int B, int H, float alpha,
                              const float* gates_saved, const float* c_prev, const float* c, int ldc,
                              const float* dh, int lddh, int dh_scatter, float* dc_inout, void* dZ, int ldz_gate,
                              void* cuda_stream) {
  if (!ctx || !pat || pat->ctx != ctx || !gates_saved || !c_prev || !c || !dh || !dc_inout || !dZ)
    return ARD_ERR_INVALID_ARG;
  if (pat->kind != ARD_ROW || pat->N_dim != H) return ARD_ERR_SHAPE;
  if (B < 0 || B > 65535 || H < 1) return ARD_ERR_INVALID_ARG;
  if (dz_dtype != ARD_F32 && dz_dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (ldz_gate < 1 || ldc < 1 || lddh < 1 || (dh_scatter && lddh < H)) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  return launch_lstm_gates_bwd(ctx, pat, dz_dtype, B, H, alpha, gates_saved, c_prev, c, ldc, dh, lddh, dh_scatter,
                               dc_inout, dZ, ldz_gate, (cudaStream_t)cuda_stream);
}

// Whole-sequence drivers: the time loop runs here, in native code, and only enqueues kernels.
// gates_ready: the input half of every step's pre-activations is already in G (the caller multiplied it, e.g. over
// the kept outputs of the layer below); only the recurrence runs, which needs the one-kernel form.
static ard_status lstm_forward_impl(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H, float alpha,
                                    void* XH, const void* W, int ldw, const float* bias, float* C, float* G, float* Z,
                                    int gates_ready, void* cuda_stream) {
  if (!ctx || !pat || !XH || !W || !C || !G || (!Z && !gates_ready)) return ARD_ERR_INVALID_ARG;
  if (T < 0 || B < 0 || I < 0 || H < 1) return ARD_ERR_INVALID_ARG;
  const int KH = I + H;
  __nv_bfloat16* xh = reinterpret_cast<__nv_bfloat16*>(XH);
  // One cooperative kernel for the whole sequence when the layer fits it (the weight slice of 8 hidden
  // units per CTA in shared memory, all CTAs resident, at most 128 batch rows) and the operands meet the
  // TMA path's alignment rules; otherwise one gate product and one cell kernel per time step.
  if (ctx->lstm_persistent && ctx->path != ARD_PATH_CUDA_CORE && T >= 1 && B >= 1) {
    ard_status st = check_common(ctx, pat, B, KH, H);
    if (st != ARD_OK) return st;
    if (pat->kind != ARD_ROW) return ARD_ERR_INVALID_ARG;
    if (ldw < KH) return ARD_ERR_SHAPE;
    DeviceGuard guard(ctx->device);
    const char* Wc = reinterpret_cast<const char*>(W);
    if (tc_eligible(ctx, pat, ARD_BF16, B, KH, H, XH, KH, W, ldw, C, H, 4) == ARD_OK &&
        ((size_t)H * ldw * 2) % 16 == 0 && lstm_persistent_fits(ctx, B, H, H)) {
      cudaStream_t s = (cudaStream_t)cuda_stream;
      TcMap mapXH;
      TcMap mapW[4];
      // 1. The input half for all steps at once: G[t][:, g*H + j] = x_t . W[g*H + keep[j]][0:I]  (T*B rows).
      if (I > 0 && !gates_ready) {
        TcArgs t = {};
        GemmArgs g = {};
        fill_common(g, ctx, pat, T * B, I, H, 1.0f);
        g.A0 = XH; g.lda0 = KH; g.A1 = W; g.lda1 = ldw; g.out = G; g.ldo = 4 * H;
        g.out_is_f32 = 1;
        t.g = g;
        t.ts = H;
        t.bn = 0;
        st = get_maps(ctx, XH, T * B, I, KH, 0, MAP_PLAIN, 0, 128, 64, &t.mapA);
        if (st != ARD_OK) return st;
        t.mapA_indexed = 0;
        for (int gate = 0; gate < 4; ++gate) {
          st = get_maps(ctx, Wc + (size_t)gate * H * ldw * 2, H, I, ldw, H, MAP_STRIDED_ROWS, pat->dp_bound, 64, 64,
                        &t.mapB4[gate]);
          if (st != ARD_OK) return st;
          t.mapA4[gate] = t.mapA;
        }
        t.mapB = t.mapB4[0];
        t.mapB_indexed = 1;
        st = launch_lstm_tc(ctx, 0, t, s);
        if (st != ARD_OK) return st;
      }
      // 2. The recurrence: one kernel, recurrent half of the weight resident in shared memory.
      st = get_maps(ctx, XH, (T + 1) * B, KH, KH, 0, MAP_PLAIN, 0, 64, 64, &mapXH);
      if (st != ARD_OK) return st;
      for (int gate = 0; gate < 4; ++gate) {
        st = get_maps(ctx, Wc + (size_t)gate * H * ldw * 2, H, KH, ldw, H, MAP_STRIDED_ROWS, pat->dp_bound, 8, 64,
                      &mapW[gate]);
        if (st != ARD_OK) return st;
      }
      // 2b. Under a pattern the recurrence contracts over the kept units of h_{t-1} alone: its operand is a compact
      // copy of h in context scratch (two buffers, the kernel fills them).
      TcMap mapHc;
      const bool compact_h = ctx->lstm_compact_h && pat->dp_bound > 1 && ctx->d_lstm_hc != nullptr && H <= ARD_LSTM_HC_LD;
      if (compact_h) {
        st = get_maps(ctx, ctx->d_lstm_hc, 2 * B, ARD_LSTM_HC_LD, ARD_LSTM_HC_LD, 0, MAP_PLAIN, 0, 64, 64, &mapHc);
        if (st != ARD_OK) return st;
      }
      st = launch_lstm_forward_persistent(ctx, pat, T, B, I, H, I, H, I > 0 ? 1 : 0, alpha, mapXH, mapW,
                                          compact_h ? &mapHc : nullptr, W, ldw, XH, bias, C, G, s);
      if (st != ARD_ERR_UNSUPPORTED) return st;
      // not launchable as one kernel right now: the per-step path below recomputes everything
    }
  }
  if (gates_ready) return ARD_ERR_UNSUPPORTED;  // the per-step path multiplies [x, h] as one operand
  for (int t = 0; t < T; ++t) {
    __nv_bfloat16* xh_t = xh + (size_t)t * B * KH;
    __nv_bfloat16* h_out = xh + (size_t)(t + 1) * B * KH + I;  // h_t lands in the operand of step t+1
    ard_status st = ard_lstm_gate_gemm(ctx, pat, B, KH, H, xh_t, KH, W, ldw, Z, H, cuda_stream);
    if (st != ARD_OK) return st;
    st = ard_lstm_gates(ctx, pat, ARD_BF16, B, H, alpha, Z, H, bias, C + (size_t)t * B * H, H,
                        C + (size_t)(t + 1) * B * H, h_out, KH, 1, G + (size_t)t * B * 4 * H, cuda_stream);
    if (st != ARD_OK) return st;
  }
  return ARD_OK;
}

ard_status ard_lstm_forward(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H, float alpha, void* XH,
                            const void* W, int ldw, const float* bias, float* C, float* G, float* Z,
                            void* cuda_stream) {
  return lstm_forward_impl(ctx, pat, T, B, I, H, alpha, XH, W, ldw, bias, C, G, Z, 0, cuda_stream);
}

ard_status ard_lstm_forward_from_gates(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H, float alpha,
                                       void* XH, const void* W, int ldw, const float* bias, float* C, float* G,
                                       void* cuda_stream) {
  if (I < 1) return ARD_ERR_INVALID_ARG;
  return lstm_forward_impl(ctx, pat, T, B, I, H, alpha, XH, W, ldw, bias, C, G, nullptr, 1, cuda_stream);
}

// recurrent_only: the recurrence (gate gradients DZ) and the weight gradient of the recurrent half,
// dW[:, I : I+H]; the input half (dx and dW[:, 0 : I]) is left to the caller.  Needs the one-kernel form.
static ard_status lstm_backward_impl(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H, float alpha,
                                     const void* XH, const void* W, int ldw, const float* C, const float* G,
                                     const float* dH_last, float* D, float* dc, void* DZ, float* dW,
                                     int recurrent_only, void* cuda_stream) {
  if (!ctx || !pat || !XH || !W || !C || !G || !dH_last || !D || !dc || !DZ || !dW) return ARD_ERR_INVALID_ARG;
  if (T < 1 || B < 0 || I < 0 || H < 1) return ARD_ERR_INVALID_ARG;
  const int KH = I + H;
  __nv_bfloat16* dz = reinterpret_cast<__nv_bfloat16*>(DZ);
  // One cooperative kernel for the recurrence of the whole sequence when the layer fits it, followed by the
  // input half of d[x, h] as one product over all T*B rows; otherwise the two kernels per time step below.
  bool recurrence_done = false;
  if (ctx->lstm_persistent && ctx->path != ARD_PATH_CUDA_CORE && B >= 1 && I > 0) {
    ard_status st = check_common(ctx, pat, B, KH, H);
    if (st != ARD_OK) return st;
    if (pat->kind != ARD_ROW) return ARD_ERR_INVALID_ARG;
    if (ldw < KH) return ARD_ERR_SHAPE;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const char* Wc = reinterpret_cast<const char*>(W);
    const char* dZc = reinterpret_cast<const char*>(DZ);
    if (tc_eligible(ctx, pat, ARD_BF16, T * B, KH, H, DZ, 4 * H, W, ldw, D, KH, 4) == ARD_OK &&
        ((size_t)H * ldw * 2) % 16 == 0 && I % 8 == 0 && lstm_persistent_bwd_fits(ctx, B, H)) {
      TcMap mapDZ[4];
      TcMap mapW[4];
      for (int gate = 0; gate < 4; ++gate) {
        st = get_maps(ctx, dZc + (size_t)gate * H * 2, T * B, H, 4 * H, H, MAP_COMPACT_COLS, pat->dp_bound, 64, 64,
                      &mapDZ[gate]);
        if (st != ARD_OK) return st;
        st = get_maps(ctx, Wc + (size_t)gate * H * ldw * 2, H, KH, ldw, H, MAP_STRIDED_ROWS, pat->dp_bound, 64, 64,
                      &mapW[gate]);
        if (st != ARD_OK) return st;
      }
      st = launch_lstm_backward_persistent(ctx, pat, T, B, I, H, alpha, mapDZ, mapW, W, ldw, C, G, dH_last, D, dc, DZ, s);
      if (st == ARD_OK) {
        // dx_t for all t: the x halves of D are overwritten
        if (!recurrent_only) st = lstm_gate_gemm_bwd_tc(ctx, pat, T * B, I, H, DZ, H, W, ldw, D, KH, 0, s);
        if (st != ARD_OK) return st;
        recurrence_done = true;
      } else if (st != ARD_ERR_UNSUPPORTED) {
        return st;
      }
    }
  }
  if (recurrent_only && !recurrence_done) return ARD_ERR_UNSUPPORTED;
  for (int t = T - 1; t >= 0 && !recurrence_done; --t) {
    const float* dh = (t == T - 1) ? dH_last : D + (size_t)(t + 1) * B * KH + I;
    const int lddh = (t == T - 1) ? H : KH;
    ard_status st = ard_lstm_gates_bwd(ctx, pat, ARD_BF16, B, H, alpha, G + (size_t)t * B * 4 * H,
                                       C + (size_t)t * B * H, C + (size_t)(t + 1) * B * H, H, dh, lddh, 1, dc,
                                       dz + (size_t)t * B * 4 * H, H, cuda_stream);
    if (st != ARD_OK) return st;
    st = ard_lstm_gate_gemm_bwd(ctx, pat, B, KH, H, dz + (size_t)t * B * 4 * H, H, W, ldw, D + (size_t)t * B * KH, KH,
                                1, cuda_stream);
    if (st != ARD_OK) return st;
  }
  // Weight gradient over all T*B rows: the four gate blocks in one tensor-core launch when the operands
  // allow it (the M tiles of the four gates share one tile loop), else one product per gate.
  // (recurrent_only: the columns of the h half alone -- operand, output and fan-in extent start at column I)
  const int wcol0 = recurrent_only ? I : 0, wcols = recurrent_only ? H : KH;
  const void* XHw = reinterpret_cast<const __nv_bfloat16*>(XH) + wcol0;
  float* dWw = dW + wcol0;
  const bool w_tc = ctx->path != ARD_PATH_CUDA_CORE && H % 8 == 0 && wcols % 8 == 0 && wcol0 % 8 == 0 &&
                    tc_eligible(ctx, pat, ARD_BF16, T * B, KH, H, DZ, 4 * H, XH, KH, dW, KH, 4) == ARD_OK;
  if (recurrent_only && !w_tc) return ARD_ERR_UNSUPPORTED;
  if (w_tc) {
    TcArgs t = {};
    GemmArgs g = {};
    fill_common(g, ctx, pat, T * B, wcols, H, 1.0f);
    g.A0 = DZ; g.lda0 = 4 * H; g.A1 = XHw; g.lda1 = KH; g.out = dWw; g.ldo = KH;
    g.flag0 = 1;
    g.flag1 = 1;  // rows of dropped units are written as zero
    g.out_is_f32 = 1;
    ard_status st = ARD_OK;
    const char* dZc = reinterpret_cast<const char*>(DZ);
    for (int gate = 0; gate < 4 && st == ARD_OK; ++gate)
      st = get_maps(ctx, dZc + (size_t)gate * H * 2, T * B, H, 4 * H, H, MAP_COMPACT_COLS, pat->dp_bound, 64, 64,
                    &t.mapA4[gate]);
    if (st == ARD_OK) st = get_maps(ctx, XHw, T * B, wcols, KH, 0, MAP_PLAIN, 0, 64, 64, &t.mapB);
    if (st != ARD_OK) return st;
    t.mapA = t.mapA4[0];
    t.mapA_indexed = 1;
    t.mapB_indexed = 0;
    t.g = g;
    t.ts = 0;
    t.bn = ctx->force_bn;
    return launch_lstm_tc(ctx, 2, t, (cudaStream_t)cuda_stream);
  }
  for (int g = 0; g < 4; ++g) {  // one product per gate
    ard_status st = ard_bwd_weight(ctx, pat, ARD_BF16, ARD_F32, T * B, KH, H, 1.0f, XH, KH, dz + (size_t)g * H, 4 * H,
                                   1, dW + (size_t)g * H * KH, KH, 1, cuda_stream);
    if (st != ARD_OK) return st;
  }
  return ARD_OK;
}

ard_status ard_lstm_backward(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H, float alpha,
                             const void* XH, const void* W, int ldw, const float* C, const float* G,
                             const float* dH_last, float* D, float* dc, void* DZ, float* dW, void* cuda_stream) {
  return lstm_backward_impl(ctx, pat, T, B, I, H, alpha, XH, W, ldw, C, G, dH_last, D, dc, DZ, dW, 0, cuda_stream);
}

ard_status ard_lstm_backward_recurrent(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H, float alpha,
                                       const void* XH, const void* W, int ldw, const float* C, const float* G,
                                       const float* dH_last, float* D, float* dc, void* DZ, float* dW,
                                       void* cuda_stream) {
  return lstm_backward_impl(ctx, pat, T, B, I, H, alpha, XH, W, ldw, C, G, dH_last, D, dc, DZ, dW, 1, cuda_stream);
}

ard_status ard_compact_cols(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, int rows, int N, const void* src,
                            int ld_src, void* dst, int ld_dst, void* cuda_stream) {
  if (!ctx || !pat || pat->ctx != ctx || pat->kind != ARD_ROW || !src || !dst) return ARD_ERR_INVALID_ARG;
  if (dtype != ARD_F32 && dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (rows < 0 || N != pat->N_dim || ld_src < N || ld_dst < 1) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  return launch_gather_cols(ctx, pat->d_hdr, pat->d_idx, src, ld_src, dst, ld_dst, rows, dtype == ARD_F32 ? 4 : 2, N, 0,
                            (cudaStream_t)cuda_stream);
}

ard_status ard_expand_cols(ard_ctx* ctx, const ard_pattern* pat, ard_dtype src_dtype, int rows, int N, float alpha,
                           const void* src, int ld_src, float* dst, int ld_dst, void* cuda_stream) {
  if (!ctx || !pat || pat->ctx != ctx || pat->kind != ARD_ROW || !src || !dst) return ARD_ERR_INVALID_ARG;
  if (src_dtype != ARD_F32 && src_dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (rows < 0 || N != pat->N_dim || ld_src < 1 || ld_dst < N) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  return launch_expand_cols(ctx, pat->d_hdr, src, ld_src, src_dtype == ARD_BF16, dst, ld_dst, rows, N, alpha,
                            (cudaStream_t)cuda_stream);
}

// ---- products over the kept rows of a convolution layer's input matrix (Sec. 5.2.1) -----------------
static ard_status rows_check(ard_ctx* ctx, const ard_rows* rows, int M, int K, int N, const void* p0, int ld0,
                             const void* p1, int ld1, const void* po, int ldo, int out_es) {
  if (!ctx || !rows || rows->ctx != ctx || !p0 || !p1 || !po) return ARD_ERR_INVALID_ARG;
  if (M != rows->M || K < 1 || N < 1) return ARD_ERR_SHAPE;
  if (ctx->encode_fn == nullptr) return ARD_ERR_UNSUPPORTED;
  if (!aligned16(p0) || !aligned16(p1) || !aligned16(po)) return ARD_ERR_ALIGNMENT;
  if (ld0 % 8 || ld1 % 8 || ((size_t)ldo * out_es) % 16 || K % 8 || N % 8) return ARD_ERR_ALIGNMENT;
  return ARD_OK;
}

ard_status ard_rows_fwd(ard_ctx* ctx, const ard_rows* rows, int M, int K, int N, float alpha, const void* A, int lda,
                        const void* W, int ldw, void* Y, int ldy, void* cuda_stream) {
  ard_status st = rows_check(ctx, rows, M, K, N, A, lda, W, ldw, Y, ldy, 2);
  if (st != ARD_OK) return st;
  if (lda < K || ldw < K || ldy < N) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  TcArgs t = {};
  GemmArgs g = {};
  g.hdr = rows->d_hdr;
  g.B = M; g.K = K; g.N = N;
  g.alpha = alpha;
  g.out = Y; g.ldo = ldy;
  g.status = ctx->d_status;
  st = get_maps(ctx, A, M, K, lda, 0, MAP_PLAIN, 0, 1, 64, &t.mapA);   // gathered: one row of 64 k per piece
  if (st != ARD_OK) return st;
  st = get_maps(ctx, W, N, K, ldw, 0, MAP_PLAIN, 0, 64, 64, &t.mapB);  // boxes [64 neurons][64 k]
  if (st != ARD_OK) return st;
  t.g = g;
  t.bn = ctx->force_bn;
  st = launch_zero_dropped_rows(ctx, rows, Y, ldy * 2, N * 2, s);
  if (st != ARD_OK) return st;
  return launch_rows_tc(ctx, OP_FWD, t, rows->d_idx, nullptr, 0, nullptr, 0, s);
}

ard_status ard_rows_bwd_data(ard_ctx* ctx, const ard_rows* rows, int M, int K, int N, float alpha, const void* dY,
                             int lddy, const void* W, int ldw, void* dA, int ldda, void* cuda_stream) {
  ard_status st = rows_check(ctx, rows, M, K, N, dY, lddy, W, ldw, dA, ldda, 2);
  if (st != ARD_OK) return st;
  if (lddy < N || ldw < K || ldda < K) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  TcArgs t = {};
  GemmArgs g = {};
  g.hdr = rows->d_hdr;
  g.B = M; g.K = K; g.N = N;
  g.alpha = alpha;
  g.out = dA; g.ldo = ldda;
  g.status = ctx->d_status;
  st = get_maps(ctx, dY, M, N, lddy, 0, MAP_PLAIN, 0, 1, 64, &t.mapA);  // gathered: one row of 64 n per piece
  if (st != ARD_OK) return st;
  st = get_maps(ctx, W, N, K, ldw, 0, MAP_PLAIN, 0, 64, 64, &t.mapB);  // read MN-major: boxes [64 neurons][64 k]
  if (st != ARD_OK) return st;
  t.g = g;
  t.bn = ctx->force_bn;
  st = launch_zero_dropped_rows(ctx, rows, dA, ldda * 2, K * 2, s);
  if (st != ARD_OK) return st;
  return launch_rows_tc(ctx, OP_BWD_DATA, t, rows->d_idx, nullptr, 0, nullptr, 0, s);
}

ard_status ard_rows_bwd_weight(ard_ctx* ctx, const ard_rows* rows, ard_dtype dW_dtype, int M, int K, int N, float alpha,
                               const void* A, int lda, const void* dY, int lddy, void* dW, int lddw,
                               void* cuda_stream) {
  if (dW_dtype != ARD_F32 && dW_dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  ard_status st = rows_check(ctx, rows, M, K, N, A, lda, dY, lddy, dW, lddw, dW_dtype == ARD_F32 ? 4 : 2);
  if (st != ARD_OK) return st;
  if (lda < K || lddy < N || lddw < K) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  TcArgs t = {};
  GemmArgs g = {};
  g.hdr = rows->d_hdr;
  g.B = M; g.K = K; g.N = N;
  g.alpha = alpha;
  g.out = dW; g.ldo = lddw;
  g.out_is_f32 = dW_dtype == ARD_F32;
  g.status = ctx->d_status;
  // both operands are gathered along the contraction by the kernel's loading warps (plain pointers, no descriptor)
  st = get_maps(ctx, dY, M, N, lddy, 0, MAP_PLAIN, 0, 1, 64, &t.mapA);   // placeholders: the kernel's parameter block
  if (st != ARD_OK) return st;                                            // always carries two descriptors
  t.mapB = t.mapA;
  t.g = g;
  t.bn = ctx->force_bn;
  return launch_rows_tc(ctx, OP_BWD_WEIGHT, t, rows->d_idx, dY, lddy, A, lda, (cudaStream_t)cuda_stream);
}

// ---- the same products on compact operands (the dense small matrices of Sec. 5.2.1, step 2) ----------
ard_status ard_rows_gather(ard_ctx* ctx, const ard_rows* rows, int M, int width, const void* src, int ld_src, void* dst,
                           int ld_dst, void* cuda_stream) {
  if (!ctx || !rows || rows->ctx != ctx || !src || !dst) return ARD_ERR_INVALID_ARG;
  if (M != rows->M || width < 1 || ld_src < width || ld_dst < width) return ARD_ERR_SHAPE;
  if (!aligned16(src) || !aligned16(dst) || width % 8 || ld_src % 8 || ld_dst % 8) return ARD_ERR_ALIGNMENT;
  DeviceGuard guard(ctx->device);
  return launch_rows_gather(ctx, rows, src, ld_src * 2, dst, ld_dst * 2, width * 2, (cudaStream_t)cuda_stream);
}

static int rows_capacity(int M) { return (M + 63) / 64 * 64; }

ard_status ard_rows_fwd_compact(ard_ctx* ctx, const ard_rows* rows, int M, int K, int N, float alpha, const void* Ak,
                                int ldak, const void* W, int ldw, void* Y, int ldy, void* cuda_stream) {
  ard_status st = rows_check(ctx, rows, M, K, N, Ak, ldak, W, ldw, Y, ldy, 2);
  if (st != ARD_OK) return st;
  if (ldak < K || ldw < K || ldy < N) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  TcArgs t = {};
  GemmArgs g = {};
  g.hdr = rows->d_hdr;
  g.B = M; g.K = K; g.N = N;
  g.alpha = alpha;
  g.out = Y; g.ldo = ldy;
  g.flag0 = ARD_OUT_COMPACT;
  g.status = ctx->d_status;
  g.ext_mode = 1;
  g.ridx = rows->d_idx;
  st = get_maps(ctx, Ak, rows_capacity(M), K, ldak, 0, MAP_PLAIN, 0, 128, 64, &t.mapA);  // [128 rows][64 k]
  if (st != ARD_OK) return st;
  st = get_maps(ctx, W, N, K, ldw, 0, MAP_PLAIN, 0, 64, 64, &t.mapB);  // [64 neurons][64 k]
  if (st != ARD_OK) return st;
  t.g = g;
  t.bn = ctx->force_bn;
  st = launch_zero_dropped_rows(ctx, rows, Y, ldy * 2, N * 2, s);
  if (st != ARD_OK) return st;
  return launch_gemm_tc(ctx, ARD_ROW, OP_FWD, t, s);
}

ard_status ard_rows_bwd_data_compact(ard_ctx* ctx, const ard_rows* rows, int M, int K, int N, float alpha, const void* dYk,
                                     int lddyk, const void* W, int ldw, void* dA, int ldda, void* cuda_stream) {
  ard_status st = rows_check(ctx, rows, M, K, N, dYk, lddyk, W, ldw, dA, ldda, 2);
  if (st != ARD_OK) return st;
  if (lddyk < N || ldw < K || ldda < K) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  TcArgs t = {};
  GemmArgs g = {};
  g.hdr = rows->d_hdr;
  g.B = M; g.K = K; g.N = N;
  g.alpha = alpha;
  g.out = dA; g.ldo = ldda;
  g.flag0 = 1;
  g.status = ctx->d_status;
  g.ext_mode = 1;
  g.ridx = rows->d_idx;
  st = get_maps(ctx, dYk, rows_capacity(M), N, lddyk, 0, MAP_PLAIN, 0, 128, 64, &t.mapA);  // [128 rows][64 n]
  if (st != ARD_OK) return st;
  st = get_maps(ctx, W, N, K, ldw, 0, MAP_PLAIN, 0, 64, 64, &t.mapB);  // read MN-major: [64 neurons][64 k]
  if (st != ARD_OK) return st;
  t.g = g;
  t.bn = ctx->force_bn;
  st = launch_zero_dropped_rows(ctx, rows, dA, ldda * 2, K * 2, s);
  if (st != ARD_OK) return st;
  return launch_gemm_tc(ctx, ARD_ROW, OP_BWD_DATA, t, s);
}

ard_status ard_rows_bwd_weight_compact(ard_ctx* ctx, const ard_rows* rows, ard_dtype dW_dtype, int M, int K, int N,
                                       float alpha, const void* Ak, int ldak, const void* dYk, int lddyk, void* dW,
                                       int lddw, void* cuda_stream) {
  if (dW_dtype != ARD_F32 && dW_dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  ard_status st = rows_check(ctx, rows, M, K, N, Ak, ldak, dYk, lddyk, dW, lddw, dW_dtype == ARD_F32 ? 4 : 2);
  if (st != ARD_OK) return st;
  if (ldak < K || lddyk < N || lddw < K) return ARD_ERR_SHAPE;
  DeviceGuard guard(ctx->device);
  TcArgs t = {};
  GemmArgs g = {};
  g.hdr = rows->d_hdr;
  g.B = M; g.K = K; g.N = N;
  g.alpha = alpha;
  g.out = dW; g.ldo = lddw;
  g.flag0 = 1;
  g.out_is_f32 = dW_dtype == ARD_F32;
  g.status = ctx->d_status;
  g.ext_mode = 2;
  // both operands read along the rows of the list: boxes [64 list rows][64 columns]
  st = get_maps(ctx, dYk, rows_capacity(M), N, lddyk, 0, MAP_PLAIN, 0, 64, 64, &t.mapA);
  if (st != ARD_OK) return st;
  st = get_maps(ctx, Ak, rows_capacity(M), K, ldak, 0, MAP_PLAIN, 0, 64, 64, &t.mapB);
  if (st != ARD_OK) return st;
  t.g = g;
  t.bn = ctx->force_bn;
  return launch_gemm_tc(ctx, ARD_ROW, OP_BWD_WEIGHT, t, (cudaStream_t)cuda_stream);
}

// Gathers and the three products of one iteration in one call, the output-gradient half (gather of dY,
// backward-data) on the context's side stream beside the input half (gather of A, forward); the weight gradient
// waits for both gathered matrices.  Each product fills the GPU here, but its dependent launches leave tails and
// ramps that the other half covers.
ard_status ard_rows_products(ard_ctx* ctx, const ard_rows* rows, ard_dtype dW_dtype, int M, int K, int N, float alpha,
                             const void* A, int lda, const void* W, int ldw, const void* dY, int lddy, void* Ak,
                             int ldak, void* dYk, int lddyk, void* Y, int ldy, void* dA, int ldda, void* dW, int lddw,
                             void* cuda_stream) {
  if (!ctx || !rows || rows->ctx != ctx) return ARD_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const bool streams = ctx->mlp_two_streams && ard_side_streams(ctx, s);
  SharedTailOff tail_guard(ctx, streams);
  cudaStream_t side = streams ? ctx->side_stream : s;
  DeviceGuard guard(ctx->device);
  if (streams) {
    ARD_CUDA_OK(cudaEventRecord(ctx->ev[100], s));
    ARD_CUDA_OK(cudaStreamWaitEvent(side, ctx->ev[100], 0));
  }
  ard_status st = ard_rows_gather(ctx, rows, M, N, dY, lddy, dYk, lddyk, side);
  if (streams) ARD_CUDA_OK(cudaEventRecord(ctx->ev[101], side));
  ard_status st2 = st == ARD_OK ? ard_rows_bwd_data_compact(ctx, rows, M, K, N, alpha, dYk, lddyk, W, ldw, dA, ldda, side) : st;
  ard_status st3 = ard_rows_gather(ctx, rows, M, K, A, lda, Ak, ldak, s);
  if (streams) ARD_CUDA_OK(cudaStreamWaitEvent(s, ctx->ev[101], 0));
  ard_status st4 = (st == ARD_OK && st3 == ARD_OK)
                       ? ard_rows_bwd_weight_compact(ctx, rows, dW_dtype, M, K, N, alpha, Ak, ldak, dYk, lddyk, dW, lddw, s)
                       : (st != ARD_OK ? st : st3);
  ard_status st5 = st3 == ARD_OK ? ard_rows_fwd_compact(ctx, rows, M, K, N, alpha, Ak, ldak, W, ldw, Y, ldy, s) : st3;
  if (streams) {  // join whatever was enqueued, also after an error, so that a capture is not left forked
    ARD_CUDA_OK(cudaEventRecord(ctx->ev[102], side));
    ARD_CUDA_OK(cudaStreamWaitEvent(s, ctx->ev[102], 0));
  }
  for (ard_status r : {st, st2, st3, st4, st5})
    if (r != ARD_OK) return r;
  return ARD_OK;
}

ard_status ard_last_device_status(ard_ctx* ctx, void* cuda_stream) {
  if (!ctx) return ARD_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  int v = 0;
  ARD_CUDA_OK(cudaMemcpyAsync(&v, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, s));
  ARD_CUDA_OK(cudaStreamSynchronize(s));
  if (v != 0) {
    ARD_CUDA_OK(cudaMemsetAsync(ctx->d_status, 0, sizeof(int), s));
    ARD_CUDA_OK(cudaStreamSynchronize(s));
  }
  return (ard_status)v;
}

uint64_t ard_launch_count(const ard_ctx* ctx) { return ctx ? ctx->launches : 0; }

}  // extern "C"
