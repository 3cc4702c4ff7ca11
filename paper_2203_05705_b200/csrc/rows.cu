// Row-based sensitivity-aware dropout of a convolution layer's input matrix (Sec. 5.1, Sec. 5.2.1):
// sensitivity prediction per region, one Bernoulli draw per row, compaction of the kept rows into a
// device-resident list.  Nothing returns to the host; the products that follow read the list.
#include "ard_internal.h"
#include "philox.h"

namespace {

template <typename T> __device__ __forceinline__ float val_f(T v);
template <> __device__ __forceinline__ float val_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float val_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// Sec. 5.1, steps 2-4.  The sampled values are taken in runs of c neighbouring values of a row.  c = 1 is the
// text's statement (every value drawn on its own) and the default of the entry point; with c = gcd(Kc, 32) a run is
// what one memory transaction delivers (64 bytes of bf16), where isolated values cost a transaction each
// (3.8 M scattered reads and 208 MB of DRAM traffic per prediction on a 32768 x 2304 matrix, 41 us against 11).
// One warp per region of x rows by the whole width; lane l takes the runs l, l + 32, ...: run d is chosen by word
// (d mod 4) of the Philox block (d div 4) as run number floor(word * Cn / 2^32), runs numbered row-major.
template <typename T>
__global__ void __launch_bounds__(256) sensitivity_kernel(const T* A, int lda, int M, int Kc, int x, int regions,
                                                          int c, int n_runs, int need, float threshold, uint32_t P_sens,
                                                          uint32_t P_insens, unsigned long long seed,
                                                          unsigned long long iteration, uint32_t stream_id,
                                                          uint32_t* P_region) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int lane = threadIdx.x & 31;
  const int g = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (g >= regions) return;
  const unsigned int per_row = (unsigned int)(Kc / c);
  const unsigned long long Cn = (unsigned long long)x * per_row;
  // 16-byte pieces when every run starts on a 16-byte boundary
  constexpr int VEC = 16 / (int)sizeof(T);
  const bool wide = (c % VEC) == 0 && ((size_t)lda * sizeof(T)) % 16 == 0 && (reinterpret_cast<uintptr_t>(A) & 15) == 0;
  int count = 0;
  for (int d = lane; d < n_runs; d += 32) {
    uint32_t w[4] = {(uint32_t)iteration, (uint32_t)(iteration >> 32), (uint32_t)g, (stream_id << 16) | (uint32_t)(d >> 2)};
    philox4x32_10(w, (uint32_t)seed, (uint32_t)(seed >> 32));
    const uint32_t word = (d & 3) == 0 ? w[0] : ((d & 3) == 1 ? w[1] : ((d & 3) == 2 ? w[2] : w[3]));
    const unsigned int run = (unsigned int)(((unsigned long long)word * Cn) >> 32);  // < Cn < 2^32
    const unsigned int roff = run / per_row;
    const long long row = (long long)g * x + roff;
    if (row >= M) continue;  // nothing exceeds the threshold below the last row
    const T* p = A + (size_t)row * lda + (size_t)(run - roff * per_row) * c;
    if (wide) {
      for (int e = 0; e < c; e += VEC) {
        const uint4 v = *reinterpret_cast<const uint4*>(p + e);
        const T* t = reinterpret_cast<const T*>(&v);
#pragma unroll
        for (int u = 0; u < VEC; ++u) count += val_f<T>(t[u]) > threshold ? 1 : 0;
      }
    } else {
      for (int e = 0; e < c; ++e) count += val_f<T>(p[e]) > threshold ? 1 : 0;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) count += __shfl_xor_sync(0xffffffffu, count, o);
  if (lane == 0) P_region[g] = count >= need ? P_sens : P_insens;
}

__global__ void __launch_bounds__(256) fill_probability_kernel(uint32_t* P_region, int regions, uint32_t P) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  for (int g = blockIdx.x * 256 + threadIdx.x; g < regions; g += gridDim.x * 256) P_region[g] = P;
}

// Sec. 5.2.1: row r is dropped iff its Philox word is below the probability of its region.  Two launches:
// every CTA draws 2048 consecutive rows (8 per thread), scans the kept counts and parks its kept rows,
// compacted, in a staging array together with its count; then every CTA adds the counts of the CTAs before
// it and copies its run to its place in the list, which therefore comes out ascending.  hdr mimics a
// pattern header (dp = b = 1).
constexpr int ROWS_PER_CTA = 2048;

__global__ void __launch_bounds__(256) rows_draw_kernel(int32_t* stage, int32_t* counts, uint8_t* kept_flag,
                                                        const uint32_t* P_region, int M, int x, unsigned long long seed,
                                                        unsigned long long iteration, uint32_t stream_id) {
  __shared__ int s_warp[8];
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r0 = blockIdx.x * ROWS_PER_CTA + tid * 8;
  unsigned keepbits = 0;
  int mine = 0;
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const int r = r0 + q;
    if (r >= M) break;
    uint32_t c[4] = {(uint32_t)iteration, (uint32_t)(iteration >> 32), (uint32_t)r, (stream_id << 16) | 0xFFFFu};
    philox4x32_10(c, (uint32_t)seed, (uint32_t)(seed >> 32));
    const bool keep = !(c[0] < P_region[r / x]);
    kept_flag[r] = keep ? 1 : 0;
    if (keep) { keepbits |= 1u << q; ++mine; }
  }
  int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  int before = 0;
#pragma unroll
  for (int w = 0; w < 8; ++w)
    if (w < warp) before += s_warp[w];
  int out = blockIdx.x * ROWS_PER_CTA + before + incl - mine;
#pragma unroll
  for (int q = 0; q < 8; ++q)
    if (keepbits & (1u << q)) stage[out++] = r0 + q;
  if (tid == 255) counts[blockIdx.x] = before + incl;
}

__global__ void __launch_bounds__(256) rows_compact_kernel(int32_t* hdr, int32_t* idx, const int32_t* stage,
                                                           const int32_t* counts, int M) {
  __shared__ int s_part[8];
  __shared__ int s_base;
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int sum = 0;
  for (int b = tid; b < (int)blockIdx.x; b += 256) sum += counts[b];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) s_part[warp] = sum;
  __syncthreads();
  if (tid == 0) {
    int v = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) v += s_part[w];
    s_base = v;
  }
  __syncthreads();
  const int base = s_base, n = counts[blockIdx.x];
  for (int j = tid; j < n; j += 256) idx[base + j] = stage[blockIdx.x * ROWS_PER_CTA + j];
  if (blockIdx.x == gridDim.x - 1 && tid == 0) {
    hdr[HDR_KIND] = 2;
    hdr[HDR_DP] = 1;
    hdr[HDR_B] = 1;
    hdr[HDR_NKEEP] = base + n;
    hdr[HDR_UNITS] = M;
    hdr[HDR_TR] = 0;
    hdr[HDR_TC] = 0;
    hdr[HDR_TS] = 0;
    hdr[HDR_MAPIDX] = 0;
  }
}

// Dropped rows of an output matrix are zero (Sec. 5.2.1: only the kept rows are filled back).
__global__ void __launch_bounds__(256) zero_dropped_rows_kernel(const uint8_t* kept_flag, int M, void* out, int ld_bytes,
                                                                int row_bytes) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  for (int r = blockIdx.x; r < M; r += gridDim.x) {
    if (kept_flag[r]) continue;
    char* row = reinterpret_cast<char*>(out) + (size_t)r * ld_bytes;
    if ((row_bytes & 15) == 0 && (ld_bytes & 15) == 0 && (reinterpret_cast<uintptr_t>(out) & 15) == 0) {
      for (int o = threadIdx.x * 16; o < row_bytes; o += 256 * 16) *reinterpret_cast<uint4*>(row + o) = make_uint4(0, 0, 0, 0);
    } else {
      for (int o = threadIdx.x * 2; o < row_bytes; o += 256 * 2) *reinterpret_cast<uint16_t*>(row + o) = 0;
    }
  }
}

// The dense, small input matrix of Sec. 5.2.1 (step 2): row j of dst is row idx[j] of src, j < n_keep; the rows
// up to the next multiple of 64 are zero, so that a contraction over the list can run in whole 64-row blocks.
// One warp per row, 16-byte pieces, a few of them in flight per lane.
__global__ void __launch_bounds__(256) rows_gather_kernel(const int32_t* hdr, const int32_t* idx, const uint4* src,
                                                          size_t ld_src16, uint4* dst, size_t ld_dst16, int row16) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int n_keep = hdr[HDR_NKEEP];
  const int n_pad = (n_keep + 63) / 64 * 64;
  const int lane = threadIdx.x & 31;
  const int warps = (int)gridDim.x * 8;
  for (int j = (int)blockIdx.x * 8 + (threadIdx.x >> 5); j < n_pad; j += warps) {
    uint4* d = dst + (size_t)j * ld_dst16;
    if (j < n_keep) {
      const uint4* sp = src + (size_t)idx[j] * ld_src16;
      for (int c = lane; c < row16; c += 128) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (c + 32 * u < row16) v[u] = sp[c + 32 * u];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (c + 32 * u < row16) d[c + 32 * u] = v[u];
      }
    } else {
      for (int c = lane; c < row16; c += 32) d[c] = make_uint4(0u, 0u, 0u, 0u);
    }
  }
}

}  // namespace

ard_status launch_rows_gather(ard_ctx* ctx, const ard_rows* rows, const void* src, int ld_src_bytes, void* dst,
                              int ld_dst_bytes, int row_bytes, cudaStream_t s) {
  if (rows->M == 0 || row_bytes == 0) return ARD_OK;
  const int want = (rows->M + 7) / 8;
  const int grid = want < ctx->sm_count * 8 ? want : ctx->sm_count * 8;
  ARD_CUDA_OK(ard_launch(ctx, rows_gather_kernel, dim3(grid), dim3(256), 0, s, (const int32_t*)rows->d_hdr,
                         (const int32_t*)rows->d_idx, (const uint4*)src, (size_t)(ld_src_bytes / 16), (uint4*)dst,
                         (size_t)(ld_dst_bytes / 16), row_bytes / 16));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

ard_status launch_sensitivity(ard_ctx* ctx, ard_rows* rows, ard_dtype dtype, const void* A, int lda, int Kc, int c,
                              int n_runs, int need, float threshold, uint32_t P_sens, uint32_t P_insens, uint64_t seed,
                              uint64_t iteration, uint32_t stream_id, cudaStream_t s) {
  const int regions = rows->regions;
  dim3 grid((regions + 7) / 8);
  if (dtype == ARD_F32)
    ARD_CUDA_OK(ard_launch(ctx, sensitivity_kernel<float>, grid, dim3(256), 0, s, (const float*)A, lda, rows->M, Kc, rows->x,
                           regions, c, n_runs, need, threshold, P_sens, P_insens, (unsigned long long)seed,
                           (unsigned long long)iteration, stream_id, rows->d_P));
  else
    ARD_CUDA_OK(ard_launch(ctx, sensitivity_kernel<__nv_bfloat16>, grid, dim3(256), 0, s, (const __nv_bfloat16*)A, lda,
                           rows->M, Kc, rows->x, regions, c, n_runs, need, threshold, P_sens, P_insens,
                           (unsigned long long)seed, (unsigned long long)iteration, stream_id, rows->d_P));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

ard_status launch_fill_probability(ard_ctx* ctx, ard_rows* rows, uint32_t P, cudaStream_t s) {
  ARD_CUDA_OK(ard_launch(ctx, fill_probability_kernel, dim3((rows->regions + 255) / 256), dim3(256), 0, s, rows->d_P,
                         rows->regions, P));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

ard_status launch_rows_sample(ard_ctx* ctx, ard_rows* rows, uint64_t seed, uint64_t iteration, uint32_t stream_id,
                              cudaStream_t s) {
  const int nb = (rows->M + ROWS_PER_CTA - 1) / ROWS_PER_CTA;
  ARD_CUDA_OK(ard_launch(ctx, rows_draw_kernel, dim3(nb), dim3(256), 0, s, rows->d_stage, rows->d_counts, rows->d_flag,
                         (const uint32_t*)rows->d_P, rows->M, rows->x, (unsigned long long)seed,
                         (unsigned long long)iteration, stream_id));
  ARD_CUDA_OK(ard_launch(ctx, rows_compact_kernel, dim3(nb), dim3(256), 0, s, rows->d_hdr, rows->d_idx,
                         (const int32_t*)rows->d_stage, (const int32_t*)rows->d_counts, rows->M));
  ctx->launches += 2;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

ard_status launch_zero_dropped_rows(ard_ctx* ctx, const ard_rows* rows, void* out, int ld_bytes, int row_bytes,
                                    cudaStream_t s) {
  if (rows->M == 0 || row_bytes == 0) return ARD_OK;
  const int grid = rows->M < ctx->sm_count * 16 ? rows->M : ctx->sm_count * 16;
  ARD_CUDA_OK(ard_launch(ctx, zero_dropped_rows_kernel, dim3(grid), dim3(256), 0, s, (const uint8_t*)rows->d_flag, rows->M,
                         out, ld_bytes, row_bytes));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

// ---- C ABI -----------------------------------------------------------------------------------------
namespace {
struct DevGuard {
  int prev = -1;
  bool switched = false;
  explicit DevGuard(int dev) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != dev) switched = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DevGuard() {
    if (switched) cudaSetDevice(prev);
  }
};

uint32_t quantise_probability(double p) {
  const double v = floor(p * 4294967296.0);
  return v >= 4294967295.0 ? 4294967295u : (uint32_t)v;
}
}  // namespace

extern "C" {

ard_status ard_rows_create(ard_ctx* ctx, ard_rows** out, int M, int region_rows) {
  if (!ctx || !out || M < 1 || region_rows < 1) return ARD_ERR_INVALID_ARG;
  *out = nullptr;
  DevGuard guard(ctx->device);
  ard_rows* r = new (std::nothrow) ard_rows();
  if (!r) return ARD_ERR_NOMEM;
  r->ctx = ctx;
  r->M = M;
  r->x = region_rows;
  r->regions = (M + region_rows - 1) / region_rows;
  r->d_hdr = nullptr; r->d_idx = nullptr; r->d_flag = nullptr; r->d_P = nullptr;
  // one allocation: header | kept list (padded to 64 entries: the products read whole 64-row blocks of it) | P | flags
  const size_t n_idx = ((size_t)M + 63) / 64 * 64 + 64;
  const size_t n_cta = ((size_t)M + 2047) / 2048;
  const size_t bytes = sizeof(int32_t) * (HDR_WORDS + 2 * n_idx + n_cta) + sizeof(uint32_t) * r->regions + (size_t)M;
  char* base = nullptr;
  if (cudaMalloc(reinterpret_cast<void**>(&base), bytes) != cudaSuccess) {
    delete r;
    return ARD_ERR_NOMEM;
  }
  cudaMemset(base, 0, bytes);
  r->d_hdr = reinterpret_cast<int32_t*>(base);
  r->d_idx = r->d_hdr + HDR_WORDS;
  r->d_stage = r->d_idx + n_idx;
  r->d_counts = r->d_stage + n_idx;
  r->d_P = reinterpret_cast<uint32_t*>(r->d_counts + n_cta);
  r->d_flag = reinterpret_cast<uint8_t*>(r->d_P + r->regions);
  *out = r;
  return ARD_OK;
}

ard_status ard_rows_destroy(ard_rows* rows) {
  if (!rows) return ARD_ERR_INVALID_ARG;
  DevGuard guard(rows->ctx->device);
  cudaDeviceSynchronize();
  cudaFree(rows->d_hdr);
  delete rows;
  return ARD_OK;
}

ard_status ard_sensitivity_predict(ard_ctx* ctx, ard_rows* rows, ard_dtype dtype, const void* A, int lda, int Kc,
                                   double k_frac, int run_len, double t_frac, float threshold, double m_prob,
                                   double n_prob, uint64_t seed, uint64_t iteration, uint32_t stream_id,
                                   void* cuda_stream) {
  if (!ctx || !rows || rows->ctx != ctx || !A) return ARD_ERR_INVALID_ARG;
  if (dtype != ARD_F32 && dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (Kc < 1 || lda < Kc) return ARD_ERR_SHAPE;
  if (!(k_frac > 0.0 && k_frac <= 1.0) || !(t_frac >= 0.0 && t_frac <= 1.0)) return ARD_ERR_INVALID_ARG;
  if (!(m_prob >= 0.0 && m_prob <= 1.0) || !(n_prob >= 0.0 && n_prob <= 1.0) || stream_id > 0xFFFFu) return ARD_ERR_INVALID_ARG;
  if (run_len < 1 || Kc % run_len != 0) return ARD_ERR_INVALID_ARG;
  const int c = run_len;  // values per run
  const double Cn = (double)rows->x * (double)(Kc / c);
  if (Cn >= 4294967296.0) return ARD_ERR_UNSUPPORTED;  // run numbers are 32-bit
  const double rd = floor(k_frac * Cn + 0.5);
  const long long n_runs = rd < 1.0 ? 1 : (long long)rd;
  if ((n_runs + 3) / 4 > 65535) return ARD_ERR_UNSUPPORTED;  // the block index shares a counter word with the stream id
  const long long samples = n_runs * c;
  if (samples >= (1ll << 31)) return ARD_ERR_UNSUPPORTED;
  const int need = (int)ard_exact_need(t_frac, samples);
  DevGuard guard(ctx->device);
  return launch_sensitivity(ctx, rows, dtype, A, lda, Kc, c, (int)n_runs, need, threshold, quantise_probability(m_prob),
                            quantise_probability(n_prob), seed, iteration, stream_id, (cudaStream_t)cuda_stream);
}

ard_status ard_rows_set_probability(ard_ctx* ctx, ard_rows* rows, double p, void* cuda_stream) {
  if (!ctx || !rows || rows->ctx != ctx || !(p >= 0.0 && p <= 1.0)) return ARD_ERR_INVALID_ARG;
  DevGuard guard(ctx->device);
  return launch_fill_probability(ctx, rows, quantise_probability(p), (cudaStream_t)cuda_stream);
}

ard_status ard_rows_sample(ard_ctx* ctx, ard_rows* rows, uint64_t seed, uint64_t iteration, uint32_t stream_id,
                           void* cuda_stream) {
  if (!ctx || !rows || rows->ctx != ctx || stream_id > 0xFFFFu) return ARD_ERR_INVALID_ARG;
  DevGuard guard(ctx->device);
  return launch_rows_sample(ctx, rows, seed, iteration, stream_id, (cudaStream_t)cuda_stream);
}

ard_status ard_rows_to_host(const ard_rows* rows, int32_t* n_keep, int32_t* idx, size_t idx_capacity,
                            uint32_t* region_probability, void* cuda_stream) {
  if (!rows) return ARD_ERR_INVALID_ARG;
  DevGuard guard(rows->ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  int32_t hdr[HDR_WORDS];
  ARD_CUDA_OK(cudaMemcpyAsync(hdr, rows->d_hdr, sizeof(hdr), cudaMemcpyDeviceToHost, s));
  ARD_CUDA_OK(cudaStreamSynchronize(s));
  if (n_keep) *n_keep = hdr[HDR_NKEEP];
  if (idx && idx_capacity > 0) {
    const size_t n = (size_t)hdr[HDR_NKEEP] < idx_capacity ? (size_t)hdr[HDR_NKEEP] : idx_capacity;
    ARD_CUDA_OK(cudaMemcpyAsync(idx, rows->d_idx, n * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  }
  if (region_probability)
    ARD_CUDA_OK(cudaMemcpyAsync(region_probability, rows->d_P, (size_t)rows->regions * sizeof(uint32_t),
                                cudaMemcpyDeviceToHost, s));
  ARD_CUDA_OK(cudaStreamSynchronize(s));
  return ARD_OK;
}

}  // extern "C"
