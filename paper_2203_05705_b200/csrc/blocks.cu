// Block-based sensitivity-aware dropout of a convolution layer's input matrix (Sec. 5.1, Sec. 5.2.2):
// per-block sensitivity counts, the bound on sensitive blocks per group, one Bernoulli draw per block, and
// the kept blocks written as the index lists of a tile pattern whose "weight" is the input matrix.  The
// three products then are the tile-pattern products with the operands' roles exchanged (see ard.h).
// Nothing returns to the host.
#include "ard_internal.h"
#include "philox.h"

#include <math.h>

#include <new>

struct ard_blocks {
  ard_ctx* ctx;
  int M, Kc, ts, G, Q;   // G = M/ts groups of Q = Kc/ts blocks
  ard_pattern* pat;      // tile pattern over [Kc x M]: tile (r, c) = (block j along Kc, group g)
  int32_t* d_count;      // [G*Q] sampled values above the threshold
  uint8_t* d_sens;       // [G*Q] 1 = sensitive
  uint8_t* d_keep;       // [G*Q] 1 = kept
};

namespace {

template <typename T> __device__ __forceinline__ float val_f(T v);
template <> __device__ __forceinline__ float val_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float val_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// Sec. 5.1, step 2 with a block as the region.  The sampled values are taken in runs of c neighbouring values of
// a row.  c = 1 is the text's statement (every value drawn on its own) and the default of the entry point; with
// c = gcd(ts, 32) a run is what one memory transaction delivers (64 bytes of bf16), where isolated values cost a
// transaction each and make this kernel read more than the kept blocks themselves.
// One warp per block (g, j); lane l takes the runs l, l + 32, ...: run d is chosen by word (d mod 4) of the
// Philox block (d div 4) as run number floor(word * Cn / 2^32), runs numbered row-major inside the block.
template <typename T>
__global__ void __launch_bounds__(256) block_count_kernel(const T* A, int lda, int ts, int Q, int nblocks, int c,
                                                          int n_runs, float threshold, unsigned long long seed,
                                                          unsigned long long iteration, uint32_t stream_id,
                                                          int32_t* counts) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int lane = threadIdx.x & 31;
  const int blk = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (blk >= nblocks) return;
  const int g = blk / Q, j = blk - g * Q;
  const T* base = A + (size_t)g * ts * lda + (size_t)j * ts;
  const unsigned int per_row = (unsigned int)(ts / c);
  const unsigned long long Cn = (unsigned long long)ts * per_row;
  // 16-byte pieces when every run starts on a 16-byte boundary
  constexpr int VEC = 16 / (int)sizeof(T);
  const bool wide = (c % VEC) == 0 && ((size_t)lda * sizeof(T)) % 16 == 0 && (reinterpret_cast<uintptr_t>(A) & 15) == 0 &&
                    ((size_t)ts * sizeof(T)) % 16 == 0;
  int count = 0;
  for (int d = lane; d < n_runs; d += 32) {
    uint32_t w[4] = {(uint32_t)iteration, (uint32_t)(iteration >> 32), (uint32_t)blk, (stream_id << 16) | (uint32_t)(d >> 2)};
    philox4x32_10(w, (uint32_t)seed, (uint32_t)(seed >> 32));
    const uint32_t word = (d & 3) == 0 ? w[0] : ((d & 3) == 1 ? w[1] : ((d & 3) == 2 ? w[2] : w[3]));
    const unsigned int run = (unsigned int)(((unsigned long long)word * Cn) >> 32);  // < Cn
    const unsigned int roff = run / per_row;
    const T* p = base + (size_t)roff * lda + (size_t)(run - roff * per_row) * c;
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
  if (lane == 0) counts[blk] = count;
}

// Sec. 5.2.2: in its group a block is sensitive iff its count reaches `need` and fewer than `cap` blocks
// of the group come before it in the order (count descending, index ascending).  One thread per block.
__global__ void __launch_bounds__(256) block_label_kernel(const int32_t* counts, int Q, int nblocks, int need, int cap,
                                                          uint8_t* sens) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int blk = blockIdx.x * 256 + threadIdx.x;
  if (blk >= nblocks) return;
  const int g = blk / Q, j = blk - g * Q;
  const int mine = counts[blk];
  int before = 0;
  for (int o = 0; o < Q; ++o) {
    const int c = counts[g * Q + o];
    before += (c > mine || (c == mine && o < j)) ? 1 : 0;   // such a block also reaches `need` if this one does
  }
  sens[blk] = (mine >= need && before < cap) ? 1 : 0;
}

__global__ void __launch_bounds__(256) block_fill_label_kernel(uint8_t* sens, int nblocks, uint8_t v) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int blk = blockIdx.x * 256 + threadIdx.x;
  if (blk < nblocks) sens[blk] = v;
}

// Block blk is dropped iff its Philox word is below the probability of its label.
__global__ void __launch_bounds__(256) block_draw_kernel(const uint8_t* sens, int nblocks, uint32_t P_sens,
                                                         uint32_t P_insens, unsigned long long seed,
                                                         unsigned long long iteration, uint32_t stream_id,
                                                         uint8_t* keep) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int blk = blockIdx.x * 256 + threadIdx.x;
  if (blk >= nblocks) return;
  uint32_t c[4] = {(uint32_t)iteration, (uint32_t)(iteration >> 32), (uint32_t)blk, (stream_id << 16) | 0xFFFFu};
  philox4x32_10(c, (uint32_t)seed, (uint32_t)(seed >> 32));
  keep[blk] = (c[0] < (sens[blk] ? P_sens : P_insens)) ? 0 : 1;
}

// Exclusive prefix sum of ptr[0..n) in place, ptr[n] = total; every thread of the CTA calls it.
// Each thread sums a contiguous run, the runs' sums are scanned through shared memory.
constexpr int LIST_THREADS = 1024;
__device__ void block_exclusive_scan(int32_t* ptr, int n, int* s_warp /* [33] */) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per = (n + LIST_THREADS - 1) / LIST_THREADS;
  const int lo = min(tid * per, n), hi = min(lo + per, n);
  int sum = 0;
  for (int i = lo; i < hi; ++i) sum += ptr[i];
  int incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = s_warp[lane], wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += v;
    }
    s_warp[lane] = wi - w;  // exclusive over warps
    if (lane == 31) s_warp[32] = wi;
  }
  __syncthreads();
  int run = s_warp[warp] + incl - sum;
  for (int i = lo; i < hi; ++i) {
    const int v = ptr[i];
    ptr[i] = run;
    run += v;
  }
  if (tid == 0) ptr[n] = s_warp[32];
  __syncthreads();
}

// The kept blocks as the lists of a tile pattern with Tr = Q tile-rows (blocks along Kc) and Tc = G
// tile-columns (groups): idx = r*G + c ascending; grouped by tile-column (col_ptr, col_idx = r ascending)
// and by tile-row (row_ptr, row_idx = c ascending).  One CTA: the lists are a few thousand entries.
// draw != 0: the CTA first draws the kept flags itself (small block counts: saves a launch).
// in_smem != 0: the flags and the two pointer arrays live in shared memory while the lists are built (every
// phase otherwise waits for a round trip to global memory); the pointer arrays are copied out at the end.
__global__ void __launch_bounds__(LIST_THREADS) block_lists_kernel(uint8_t* keep, const uint8_t* sens, int draw, int in_smem,
                                                                   uint32_t P_sens, uint32_t P_insens,
                                                                   unsigned long long seed, unsigned long long iteration,
                                                                   uint32_t stream_id, int G, int Q, int ts, int kind,
                                                                   int32_t* hdr, int32_t* idx, int32_t* col_ptr,
                                                                   int32_t* col_idx, int32_t* row_ptr, int32_t* row_idx) {
  __shared__ int s_warp[33];
  extern __shared__ int32_t s_dyn[];
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = LIST_THREADS / 32;
  const int nblocks = G * Q;
  int32_t* cp = in_smem ? s_dyn : col_ptr;
  int32_t* rp = in_smem ? s_dyn + (G + 1) : row_ptr;
  uint8_t* s_keep = reinterpret_cast<uint8_t*>(s_dyn + (G + 1) + (Q + 1));
  const uint8_t* kp = in_smem ? s_keep : keep;
  if (draw) {
    for (int blk = tid; blk < nblocks; blk += LIST_THREADS) {
      uint32_t c[4] = {(uint32_t)iteration, (uint32_t)(iteration >> 32), (uint32_t)blk, (stream_id << 16) | 0xFFFFu};
      philox4x32_10(c, (uint32_t)seed, (uint32_t)(seed >> 32));
      const uint8_t k = (c[0] < (sens[blk] ? P_sens : P_insens)) ? 0 : 1;
      keep[blk] = k;
      if (in_smem) s_keep[blk] = k;
    }
    __syncthreads();
  } else if (in_smem) {
    for (int blk = tid; blk < nblocks; blk += LIST_THREADS) s_keep[blk] = keep[blk];
    __syncthreads();
  }
  // counts per group (a warp per group, lanes across its blocks) and per tile-row (lanes across the groups)
  for (int g = warp; g < G; g += nwarps) {
    int cnt = 0;
    for (int j0 = 0; j0 < Q; j0 += 32) cnt += __popc(__ballot_sync(0xffffffffu, j0 + lane < Q && kp[g * Q + j0 + lane]));
    if (lane == 0) cp[g] = cnt;
  }
  for (int j = warp; j < Q; j += nwarps) {
    int cnt = 0;
    for (int g0 = 0; g0 < G; g0 += 32) cnt += __popc(__ballot_sync(0xffffffffu, g0 + lane < G && kp[(g0 + lane) * Q + j]));
    if (lane == 0) rp[j] = cnt;
  }
  __syncthreads();
  block_exclusive_scan(cp, G, s_warp);
  block_exclusive_scan(rp, Q, s_warp);
  for (int g = warp; g < G; g += nwarps) {
    int o = cp[g];
    for (int j0 = 0; j0 < Q; j0 += 32) {
      const bool k = j0 + lane < Q && kp[g * Q + j0 + lane];
      const unsigned m = __ballot_sync(0xffffffffu, k);
      if (k) col_idx[o + __popc(m & ((1u << lane) - 1u))] = j0 + lane;
      o += __popc(m);
    }
  }
  for (int j = warp; j < Q; j += nwarps) {
    int o = rp[j];
    for (int g0 = 0; g0 < G; g0 += 32) {
      const bool k = g0 + lane < G && kp[(g0 + lane) * Q + j];
      const unsigned m = __ballot_sync(0xffffffffu, k);
      if (k) {
        const int at = o + __popc(m & ((1u << lane) - 1u));
        row_idx[at] = g0 + lane;
        idx[at] = j * G + g0 + lane;
      }
      o += __popc(m);
    }
  }
  if (in_smem) {
    for (int g = tid; g <= G; g += LIST_THREADS) col_ptr[g] = cp[g];
    for (int j = tid; j <= Q; j += LIST_THREADS) row_ptr[j] = rp[j];
  }
  if (tid == 0) {
    hdr[HDR_KIND] = kind;
    hdr[HDR_DP] = 1;   // no period: the list kernels never use it
    hdr[HDR_B] = 1;
    hdr[HDR_NKEEP] = rp[Q];
    hdr[HDR_UNITS] = G * Q;
    hdr[HDR_TR] = Q;
    hdr[HDR_TC] = G;
    hdr[HDR_TS] = ts;
    hdr[HDR_MAPIDX] = 0;
  }
}

// Dropped blocks of the input gradient are zero.  dA [M][Kc]; a CTA per dropped block.
__global__ void __launch_bounds__(256) zero_dropped_blocks_kernel(const uint8_t* keep, int nblocks, int Q, int ts, void* dA,
                                                                  int ld_bytes, int elem_bytes) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int row_bytes = ts * elem_bytes;  // ts is a multiple of 64: whole 16-byte pieces when the base is aligned
  const bool wide = (ld_bytes & 15) == 0 && (reinterpret_cast<uintptr_t>(dA) & 15) == 0;
  for (int blk = blockIdx.x; blk < nblocks; blk += gridDim.x) {
    if (keep[blk]) continue;
    const int g = blk / Q, j = blk - g * Q;
    char* base = reinterpret_cast<char*>(dA) + (size_t)g * ts * ld_bytes + (size_t)j * row_bytes;
    if (wide) {
      const int per_row = row_bytes >> 4;
      for (int e = threadIdx.x; e < ts * per_row; e += 256) {
        const int r = e / per_row, q = e - r * per_row;
        *reinterpret_cast<uint4*>(base + (size_t)r * ld_bytes + (size_t)q * 16) = make_uint4(0, 0, 0, 0);
      }
    } else {
      const int per_row = row_bytes >> 1;
      for (int e = threadIdx.x; e < ts * per_row; e += 256) {
        const int r = e / per_row, q = e - r * per_row;
        *reinterpret_cast<uint16_t*>(base + (size_t)r * ld_bytes + (size_t)q * 2) = 0;
      }
    }
  }
}

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

// A pattern whose lists have no period: keeps the tile products on their list form.
constexpr int IRREGULAR_DP_BOUND = 1 << 20;

// The tensor-core path or an error: the CUDA-core weight-gradient kernel decides "kept" from (dp, b).
struct PathGuard {
  ard_ctx* ctx;
  ard_path prev;
  explicit PathGuard(ard_ctx* c) : ctx(c), prev(c->path) { c->path = ARD_PATH_TENSOR_CORE; }
  ~PathGuard() { ctx->path = prev; }
};

}  // namespace

extern "C" {

ard_status ard_blocks_create(ard_ctx* ctx, ard_blocks** out, int M, int Kc, int ts) {
  if (!ctx || !out) return ARD_ERR_INVALID_ARG;
  *out = nullptr;
  if (M < 1 || Kc < 1 || ts < 1 || M % ts || Kc % ts) return ARD_ERR_SHAPE;
  if ((long long)(M / ts) * (Kc / ts) > (1ll << 24)) return ARD_ERR_UNSUPPORTED;
  DevGuard guard(ctx->device);
  ard_blocks* b = new (std::nothrow) ard_blocks();
  if (!b) return ARD_ERR_NOMEM;
  b->ctx = ctx;
  b->M = M; b->Kc = Kc; b->ts = ts; b->G = M / ts; b->Q = Kc / ts;
  b->pat = nullptr; b->d_count = nullptr;
  ard_status st = ard_pattern_create(ctx, &b->pat, ARD_TILE, Kc, M, ts);
  if (st != ARD_OK) { delete b; return st; }
  const size_t n = (size_t)b->G * b->Q;
  char* base = nullptr;
  if (cudaMalloc(reinterpret_cast<void**>(&base), n * (sizeof(int32_t) + 2)) != cudaSuccess) {
    ard_pattern_destroy(b->pat);
    delete b;
    return ARD_ERR_NOMEM;
  }
  cudaMemset(base, 0, n * (sizeof(int32_t) + 2));
  b->d_count = reinterpret_cast<int32_t*>(base);
  b->d_sens = reinterpret_cast<uint8_t*>(b->d_count + n);
  b->d_keep = b->d_sens + n;
  cudaMemset(b->d_keep, 1, n);  // matches the fresh pattern: everything kept
  *out = b;
  return ARD_OK;
}

ard_status ard_blocks_destroy(ard_blocks* b) {
  if (!b) return ARD_ERR_INVALID_ARG;
  DevGuard guard(b->ctx->device);
  cudaDeviceSynchronize();
  cudaFree(b->d_count);
  ard_pattern_destroy(b->pat);
  delete b;
  return ARD_OK;
}

ard_status ard_blocks_predict(ard_ctx* ctx, ard_blocks* b, ard_dtype dtype, const void* A, int lda, double k_frac,
                              int run_len, double t_frac, float threshold, int cap, uint64_t seed, uint64_t iteration,
                              uint32_t stream_id, void* cuda_stream) {
  if (!ctx || !b || b->ctx != ctx || !A) return ARD_ERR_INVALID_ARG;
  if (dtype != ARD_F32 && dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (lda < b->Kc) return ARD_ERR_SHAPE;
  if (!(k_frac > 0.0) || k_frac > 1.0 || !(t_frac >= 0.0) || t_frac > 1.0 || cap < 0 || stream_id >= 65536u)
    return ARD_ERR_INVALID_ARG;
  if (run_len < 1 || b->ts % run_len != 0) return ARD_ERR_INVALID_ARG;
  const int c = run_len;  // values per run
  const long long Cn = (long long)b->ts * (b->ts / c);
  const double rd = floor(k_frac * (double)Cn + 0.5);
  const long long n_runs_ll = rd < 1.0 ? 1 : (long long)rd;
  if ((n_runs_ll + 3) / 4 > 65535) return ARD_ERR_UNSUPPORTED;
  const int n_runs = (int)n_runs_ll;
  const long long samples = n_runs_ll * c;
  if (samples >= (1ll << 31)) return ARD_ERR_UNSUPPORTED;
  const int need = (int)ard_exact_need(t_frac, samples);
  DevGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int nblocks = b->G * b->Q;
  if (dtype == ARD_F32)
    ARD_CUDA_OK(ard_launch(ctx, block_count_kernel<float>, dim3((nblocks + 7) / 8), dim3(256), 0, s, (const float*)A, lda,
                           b->ts, b->Q, nblocks, c, n_runs, threshold, (unsigned long long)seed,
                           (unsigned long long)iteration, stream_id, b->d_count));
  else
    ARD_CUDA_OK(ard_launch(ctx, block_count_kernel<__nv_bfloat16>, dim3((nblocks + 7) / 8), dim3(256), 0, s,
                           (const __nv_bfloat16*)A, lda, b->ts, b->Q, nblocks, c, n_runs, threshold,
                           (unsigned long long)seed, (unsigned long long)iteration, stream_id, b->d_count));
  ARD_CUDA_OK(ard_launch(ctx, block_label_kernel, dim3((nblocks + 255) / 256), dim3(256), 0, s,
                         (const int32_t*)b->d_count, b->Q, nblocks, need, cap, b->d_sens));
  ctx->launches += 2;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

ard_status ard_blocks_set_label(ard_ctx* ctx, ard_blocks* b, int sensitive, void* cuda_stream) {
  if (!ctx || !b || b->ctx != ctx) return ARD_ERR_INVALID_ARG;
  DevGuard guard(ctx->device);
  const int nblocks = b->G * b->Q;
  ARD_CUDA_OK(ard_launch(ctx, block_fill_label_kernel, dim3((nblocks + 255) / 256), dim3(256), 0, (cudaStream_t)cuda_stream,
                         b->d_sens, nblocks, (uint8_t)(sensitive ? 1 : 0)));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

ard_status ard_blocks_sample(ard_ctx* ctx, ard_blocks* b, double m_prob, double n_prob, uint64_t seed,
                             uint64_t iteration, uint32_t stream_id, void* cuda_stream) {
  if (!ctx || !b || b->ctx != ctx) return ARD_ERR_INVALID_ARG;
  if (!(m_prob >= 0.0) || m_prob > 1.0 || !(n_prob >= 0.0) || n_prob > 1.0 || stream_id >= 65536u)
    return ARD_ERR_INVALID_ARG;
  DevGuard guard(ctx->device);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int nblocks = b->G * b->Q;
  ard_pattern* p = b->pat;
  const uint32_t Pm = quantise_probability(m_prob), Pn = quantise_probability(n_prob);
  // few blocks: the list kernel's CTA draws them itself; the flags and pointer arrays in shared memory if they fit
  const int fused = nblocks <= 65536 ? 1 : 0;
  const size_t smem = ((size_t)(b->G + 1) + (size_t)(b->Q + 1)) * sizeof(int32_t) + (size_t)nblocks;
  const int in_smem = smem <= 40960 ? 1 : 0;
  if (!fused) {
    ARD_CUDA_OK(ard_launch(ctx, block_draw_kernel, dim3((nblocks + 255) / 256), dim3(256), 0, s, (const uint8_t*)b->d_sens,
                           nblocks, Pm, Pn, (unsigned long long)seed, (unsigned long long)iteration, stream_id, b->d_keep));
    ctx->launches++;
  }
  ARD_CUDA_OK(ard_launch(ctx, block_lists_kernel, dim3(1), dim3(LIST_THREADS), in_smem ? smem : 0, s, b->d_keep,
                         (const uint8_t*)b->d_sens, fused, in_smem, Pm, Pn, (unsigned long long)seed,
                         (unsigned long long)iteration, stream_id, b->G, b->Q, b->ts, (int)ARD_TILE, p->d_hdr, p->d_idx,
                         p->d_col_ptr, p->d_col_idx, p->d_row_ptr, p->d_row_idx));
  ctx->launches++;
  p->dp_bound = IRREGULAR_DP_BOUND;
  p->generation++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

// Roles: the tile products see the filters as their batch operand X' [N][Kc] and the input matrix as their
// weight W' [M][Kc] (neuron-major), so the result is the output matrix transposed, Yt [N][M].
ard_status ard_blocks_fwd(ard_ctx* ctx, const ard_blocks* b, int N, float alpha, const void* A, int lda, const void* W,
                          int ldw, void* Yt, int ldyt, void* cuda_stream) {
  if (!ctx || !b || b->ctx != ctx) return ARD_ERR_INVALID_ARG;
  PathGuard path(ctx);
  return ard_fwd(ctx, b->pat, ARD_BF16, N, b->Kc, b->M, alpha, W, ldw, A, lda, Yt, ldyt, ARD_OUT_SCATTER_ZEROFILL,
                 cuda_stream);
}

ard_status ard_blocks_bwd_weight(ard_ctx* ctx, const ard_blocks* b, int N, float alpha, const void* A, int lda,
                                 const void* dYt, int lddyt, void* dW, int lddw, void* cuda_stream) {
  if (!ctx || !b || b->ctx != ctx) return ARD_ERR_INVALID_ARG;
  PathGuard path(ctx);
  return ard_bwd_data(ctx, b->pat, ARD_BF16, N, b->Kc, b->M, alpha, dYt, lddyt, 0, A, lda, dW, lddw, cuda_stream);
}

ard_status ard_blocks_bwd_input(ard_ctx* ctx, const ard_blocks* b, ard_dtype dA_dtype, int N, float alpha, const void* dYt,
                                int lddyt, const void* W, int ldw, void* dA, int ldda, int zero_fill_dropped,
                                void* cuda_stream) {
  if (!ctx || !b || b->ctx != ctx || !dA) return ARD_ERR_INVALID_ARG;
  if (dA_dtype != ARD_F32 && dA_dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (ldda < b->Kc) return ARD_ERR_SHAPE;
  if (N < 1) return ARD_ERR_SHAPE;  // the empty-batch branch of the tile product is not a list kernel
  DevGuard guard(ctx->device);
  if (zero_fill_dropped) {
    const int es = dA_dtype == ARD_F32 ? 4 : 2;
    const int nblocks = b->G * b->Q;
    const int grid = nblocks < ctx->sm_count * 32 ? nblocks : ctx->sm_count * 32;
    ARD_CUDA_OK(ard_launch(ctx, zero_dropped_blocks_kernel, dim3(grid), dim3(256), 0, (cudaStream_t)cuda_stream,
                           (const uint8_t*)b->d_keep, nblocks, b->Q, b->ts, dA, ldda * es, es));
    ctx->launches++;
    ARD_CUDA_OK(cudaGetLastError());
  }
  PathGuard path(ctx);
  return ard_bwd_weight(ctx, b->pat, ARD_BF16, dA_dtype, N, b->Kc, b->M, alpha, W, ldw, dYt, lddyt, 0, dA, ldda, 0,
                        cuda_stream);
}

ard_status ard_blocks_products(ard_ctx* ctx, const ard_blocks* b, ard_dtype dA_dtype, int N, float alpha, const void* A,
                               int lda, const void* W, int ldw, const void* dYt, int lddyt, void* Yt, int ldyt, void* dW,
                               int lddw, void* dA, int ldda, int zero_fill_dropped, void* cuda_stream) {
  if (!ctx || !b || b->ctx != ctx || !dA) return ARD_ERR_INVALID_ARG;
  if (dA_dtype != ARD_F32 && dA_dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (ldda < b->Kc || N < 1) return ARD_ERR_SHAPE;
  DevGuard guard(ctx->device);
  if (zero_fill_dropped) {
    // On the stream that will run the input gradient (the context's third stream when ard_layer_products forks),
    // so that clearing the dropped blocks runs beside the forward product instead of ahead of everything.
    cudaStream_t s = (cudaStream_t)cuda_stream, zs = s;
    if (ctx->mlp_two_streams && ard_side_streams(ctx, s)) {
      ARD_CUDA_OK(cudaEventRecord(ctx->ev[103], s));
      ARD_CUDA_OK(cudaStreamWaitEvent(ctx->aux_stream, ctx->ev[103], 0));
      zs = ctx->aux_stream;
    }
    const int es = dA_dtype == ARD_F32 ? 4 : 2;
    const int nblocks = b->G * b->Q;
    const int grid = nblocks < ctx->sm_count * 32 ? nblocks : ctx->sm_count * 32;
    ARD_CUDA_OK(ard_launch(ctx, zero_dropped_blocks_kernel, dim3(grid), dim3(256), 0, zs, (const uint8_t*)b->d_keep, nblocks,
                           b->Q, b->ts, dA, ldda * es, es));
    ctx->launches++;
    ARD_CUDA_OK(cudaGetLastError());
  }
  PathGuard path(ctx);
  return ard_layer_products(ctx, b->pat, ARD_BF16, dA_dtype, N, b->Kc, b->M, alpha, W, ldw, A, lda, dYt, lddyt, Yt, ldyt,
                            ARD_OUT_SCATTER_ZEROFILL, dW, lddw, dA, ldda, 0, cuda_stream);
}

ard_status ard_blocks_to_host(const ard_blocks* b, int32_t* counts, uint8_t* sensitive, uint8_t* keep,
                              void* cuda_stream) {
  if (!b) return ARD_ERR_INVALID_ARG;
  DevGuard guard(b->ctx->device);
  ARD_CUDA_OK(cudaStreamSynchronize((cudaStream_t)cuda_stream));
  const size_t n = (size_t)b->G * b->Q;
  if (counts) ARD_CUDA_OK(cudaMemcpy(counts, b->d_count, n * sizeof(int32_t), cudaMemcpyDeviceToHost));
  if (sensitive) ARD_CUDA_OK(cudaMemcpy(sensitive, b->d_sens, n, cudaMemcpyDeviceToHost));
  if (keep) ARD_CUDA_OK(cudaMemcpy(keep, b->d_keep, n, cudaMemcpyDeviceToHost));
  return ARD_OK;
}

const ard_pattern* ard_blocks_pattern(const ard_blocks* b) { return b ? b->pat : nullptr; }

}  // extern "C"
