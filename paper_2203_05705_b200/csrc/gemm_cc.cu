// CUDA-core family of the compacted GEMMs: fp32 (or bf16) operands, fp32 FFMA accumulation.
//
// This is the path of the fp32 layers (a single tcgen05 tf32 pass keeps 10 mantissa bits and
// cannot reach 1e-5) and the fall-back for bf16 shapes whose alignment the TMA path cannot take.
// One generic 32x32x32 shared-memory tiled kernel; what differs per product is only how the
// logical operand element (m, k), (n, k) maps to memory and which contraction indices exist:
// dropped neurons / tiles are skipped through the index lists, never multiplied by zero.
#include "ard_internal.h"

namespace {

constexpr int T_M = 32, T_N = 32, T_K = 32, CC_THREADS = 256;

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

__device__ __forceinline__ void store_out(void* out, size_t off, float v, int out_is_f32, int accumulate = 0) {
  if (out_is_f32) {
    float* p = reinterpret_cast<float*>(out) + off;
    *p = accumulate ? *p + v : v;
  } else {
    __nv_bfloat16* p = reinterpret_cast<__nv_bfloat16*>(out) + off;
    *p = __float2bfloat16_rn(accumulate ? __bfloat162float(*p) + v : v);
  }
}

// KIND: 0 row, 1 tile.  OP: GemmOp.
template <typename T, int KIND, int OP>
__global__ void __launch_bounds__(CC_THREADS) gemm_cc_kernel(GemmArgs g, int ts) {
  __shared__ float As[T_K][T_M + 1];
  __shared__ float Bs[T_K][T_N + 1];

  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int dp = g.hdr[HDR_DP], b = g.hdr[HDR_B], n_keep = g.hdr[HDR_NKEEP];
  const int Tc = g.hdr[HDR_TC];
  // No __restrict__ / read-only loads on anything an earlier kernel of the stream wrote: this kernel may
  // become resident before that kernel has finished (see pdl_wait_prior_grids), and the non-coherent
  // load path may then serve a line another resident kernel brought in before the data was rewritten.
  const T* P0 = reinterpret_cast<const T*>(g.A0);
  const T* P1 = reinterpret_cast<const T*>(g.A1);

  int M, N, nk;
  const int m0 = blockIdx.y * T_M, n0 = blockIdx.x * T_N;
  const int32_t* klist = nullptr;  // tile patterns: contraction runs over ts-wide blocks klist[0..]
  if (KIND == 0) {
    // fan-in extent: all K inputs, or the kept outputs of the layer that produced the input
    const int kin = g.hdr_in != nullptr ? g.hdr_in[HDR_NKEEP] : g.K;
    if (OP == OP_FWD) { M = g.B; N = n_keep; nk = kin; }
    else if (OP == OP_BWD_DATA) { M = g.B; N = kin; nk = n_keep; }
    else { M = n_keep; N = kin; nk = g.B; }
  } else {
    if (OP == OP_FWD) {
      M = g.B; N = g.N;
      if (n0 >= N) return;
      const int c = n0 / ts;
      klist = g.col_idx + g.col_ptr[c];
      nk = (g.col_ptr[c + 1] - g.col_ptr[c]) * ts;
    } else if (OP == OP_BWD_DATA) {
      M = g.B; N = g.K;
      if (n0 >= N) return;
      const int r = n0 / ts;
      klist = g.row_idx + g.row_ptr[r];
      nk = (g.row_ptr[r + 1] - g.row_ptr[r]) * ts;
    } else {
      M = g.N; N = g.K; nk = g.B;
    }
  }
  if (m0 >= M || n0 >= N) return;

  if (KIND == 1 && OP == OP_BWD_WEIGHT) {
    const int lin = (n0 / ts) * Tc + (m0 / ts);  // tile (r, c) = (k-block, neuron-block), 0-based t-1
    const bool kept = lin >= b - 1 && (lin - (b - 1)) % dp == 0;
    if (!kept) {
      if (g.flag1) {
        for (int e = threadIdx.x; e < T_M * T_N; e += CC_THREADS) {
          const int m = m0 + e / T_N, n = n0 + e % T_N;
          if (m < M && n < N) store_out(g.out, (size_t)m * g.ldo + n, 0.f, g.out_is_f32);
        }
      }
      return;
    }
  }

  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float acc[2][2] = {{0.f, 0.f}, {0.f, 0.f}};

  for (int k0 = 0; k0 < nk; k0 += T_K) {
    for (int e = threadIdx.x; e < T_K * T_M; e += CC_THREADS) {
      // operand A: element (m, kk)
      int kk, m;
      if ((KIND == 0 && OP == OP_BWD_WEIGHT) || (KIND == 1 && OP == OP_BWD_WEIGHT)) { m = e % T_M; kk = e / T_M; }
      else { kk = e % T_K; m = e / T_K; }
      float v = 0.f;
      const int gm = m0 + m, gk = k0 + kk;
      if (gm < M && gk < nk) {
        size_t off;
        if (KIND == 0) {
          if (OP == OP_FWD) off = (size_t)gm * g.lda0 + gk;
          else if (OP == OP_BWD_DATA) off = (size_t)gm * g.lda0 + (g.flag0 ? gk : g.idx[gk]);
          else off = (size_t)gk * g.lda0 + (g.flag0 ? gm : g.idx[gm]);
        } else {
          if (OP == OP_BWD_WEIGHT) off = (size_t)gk * g.lda0 + gm;
          else off = (size_t)gm * g.lda0 + (size_t)klist[gk / ts] * ts + gk % ts;
        }
        v = to_f<T>(P0[off]);
      }
      As[kk][m] = v;
    }
    for (int e = threadIdx.x; e < T_K * T_N; e += CC_THREADS) {
      // operand B: element (n, kk)
      int kk, n;
      if (OP == OP_FWD) { kk = e % T_K; n = e / T_K; }
      else { n = e % T_N; kk = e / T_N; }
      float v = 0.f;
      const int gn = n0 + n, gk = k0 + kk;
      if (gn < N && gk < nk) {
        size_t off;
        if (KIND == 0) {
          // with a feeding pattern the weight is packed in both dimensions (row j = j-th kept neuron)
          if (OP == OP_FWD) off = (size_t)(g.hdr_in != nullptr ? gn : g.idx[gn]) * g.lda1 + gk;
          else if (OP == OP_BWD_DATA) off = (size_t)(g.hdr_in != nullptr ? gk : g.idx[gk]) * g.lda1 + gn;
          else off = (size_t)gk * g.lda1 + gn;
        } else {
          const size_t kidx = (OP == OP_BWD_WEIGHT) ? (size_t)gk : (size_t)klist[gk / ts] * ts + gk % ts;
          if (OP == OP_FWD) off = (size_t)gn * g.lda1 + kidx;
          else if (OP == OP_BWD_DATA) off = kidx * g.lda1 + gn;
          else off = kidx * g.lda1 + gn;
        }
        v = to_f<T>(P1[off]);
      }
      Bs[kk][n] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < T_K; ++kk) {
      const float a0 = As[kk][ty * 2], a1 = As[kk][ty * 2 + 1];
      const float b0 = Bs[kk][tx * 2], b1 = Bs[kk][tx * 2 + 1];
      acc[0][0] = fmaf(a0, b0, acc[0][0]);
      acc[0][1] = fmaf(a0, b1, acc[0][1]);
      acc[1][0] = fmaf(a1, b0, acc[1][0]);
      acc[1][1] = fmaf(a1, b1, acc[1][1]);
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int m = m0 + ty * 2 + i, n = n0 + tx * 2 + j;
      if (m >= M || n >= N) continue;
      size_t off;
      if (KIND == 0 && OP == OP_FWD) off = (size_t)m * g.ldo + (g.flag0 == ARD_OUT_SCATTER_ZEROFILL ? g.idx[n] : n);
      else if (KIND == 0 && OP == OP_BWD_WEIGHT) off = (size_t)(g.hdr_in != nullptr ? m : g.idx[m]) * g.ldo + n;
      else off = (size_t)m * g.ldo + n;
      float v = acc[i][j];
      if (KIND == 0 && OP == OP_FWD) {
        // layer step: bias, then the activation, then the rescale (Sec. 3.2, last paragraph)
        if (g.bias != nullptr) v += g.bias[g.idx[n]];
        if (g.relu) v = fmaxf(v, 0.f);
      }
      v *= g.alpha;
      if (KIND == 0 && OP == OP_BWD_DATA && g.act != nullptr) {
        // adjoint of the producing layer's ReLU: nothing flows where its output was not positive
        if (!(to_f<T>(reinterpret_cast<const T*>(g.act)[(size_t)m * g.ldact + n]) > 0.f)) v = 0.f;
      }
      store_out(g.out, off, v, g.out_is_f32, g.accumulate);
    }
}

// ---- layers with at most 16 neurons (an output layer) -----------------------------------------------
// The tiled kernel above would give such a layer a handful of CTAs, each walking the whole fan-in alone.
// Forward: one CTA per batch row; every thread walks a strided share of the fan-in with one accumulator
// per kept neuron, then the CTA adds the shares (fixed order).  Backward-weight: 32 fan-in columns per CTA,
// the batch rows dealt to its 8 warps, one accumulator per kept neuron, warp sums added in warp order.
constexpr int SKINNY_N = 16;

template <typename T>
__global__ void __launch_bounds__(256) skinny_fwd_kernel(GemmArgs g) {
  __shared__ float part[8][SKINNY_N];
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int n_keep = g.hdr[HDR_NKEEP];
  const int kin = g.hdr_in != nullptr ? g.hdr_in[HDR_NKEEP] : g.K;
  const int m = blockIdx.x;
  const T* X = reinterpret_cast<const T*>(g.A0) + (size_t)m * g.lda0;
  const T* W = reinterpret_cast<const T*>(g.A1);
  float acc[SKINNY_N];
#pragma unroll
  for (int n = 0; n < SKINNY_N; ++n) acc[n] = 0.f;
  int rows[SKINNY_N];
#pragma unroll
  for (int n = 0; n < SKINNY_N; ++n) rows[n] = n < n_keep ? (g.hdr_in != nullptr ? n : g.idx[n]) : 0;
  for (int k = threadIdx.x; k < kin; k += 256) {
    const float x = to_f<T>(X[k]);
#pragma unroll
    for (int n = 0; n < SKINNY_N; ++n)
      if (n < n_keep) acc[n] = fmaf(x, to_f<T>(W[(size_t)rows[n] * g.lda1 + k]), acc[n]);
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int n = 0; n < SKINNY_N; ++n) {
    float v = acc[n];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) part[warp][n] = v;
  }
  __syncthreads();
  if (threadIdx.x < n_keep) {
    const int n = threadIdx.x;
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) v += part[w][n];
    if (g.bias != nullptr) v += g.bias[g.idx[n]];
    if (g.relu) v = fmaxf(v, 0.f);
    v *= g.alpha;
    const size_t off = (size_t)m * g.ldo + (g.flag0 == ARD_OUT_SCATTER_ZEROFILL ? g.idx[n] : n);
    store_out(g.out, off, v, g.out_is_f32, g.accumulate);
  }
  if (g.flag0 == ARD_OUT_SCATTER_ZEROFILL && threadIdx.x >= 32 && threadIdx.x < 32 + g.N) {
    // full-width output: the dropped neurons' entries of this row are zero (no separate clearing pass)
    const int o = threadIdx.x - 32, dp = g.hdr[HDR_DP], bb = g.hdr[HDR_B] - 1;
    if (!(o >= bb && (o - bb) % dp == 0)) store_out(g.out, (size_t)m * g.ldo + o, 0.f, g.out_is_f32);
  }
}

template <typename T>
__global__ void __launch_bounds__(256) skinny_bwd_weight_kernel(GemmArgs g) {
  // 32 fan-in columns per CTA; its 8 warps take every eighth batch row and their sums are added in warp order
  __shared__ float part[8][SKINNY_N][33];
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int n_keep = g.hdr[HDR_NKEEP];
  const int kin = g.hdr_in != nullptr ? g.hdr_in[HDR_NKEEP] : g.K;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int k = blockIdx.x * 32 + lane;
  if (blockIdx.x * 32 >= kin) return;
  const T* dY = reinterpret_cast<const T*>(g.A0);
  const T* X = reinterpret_cast<const T*>(g.A1);
  int cols[SKINNY_N];
#pragma unroll
  for (int n = 0; n < SKINNY_N; ++n) cols[n] = n < n_keep ? (g.flag0 ? n : g.idx[n]) : 0;
  float acc[SKINNY_N];
#pragma unroll
  for (int n = 0; n < SKINNY_N; ++n) acc[n] = 0.f;
  if (k < kin) {
#pragma unroll 4
    for (int r = warp; r < g.B; r += 8) {
      const float x = to_f<T>(X[(size_t)r * g.lda1 + k]);
      const T* dy = dY + (size_t)r * g.lda0;
#pragma unroll
      for (int n = 0; n < SKINNY_N; ++n)
        if (n < n_keep) acc[n] = fmaf(to_f<T>(dy[cols[n]]), x, acc[n]);
    }
  }
#pragma unroll
  for (int n = 0; n < SKINNY_N; ++n) part[warp][n][lane] = acc[n];
  __syncthreads();
  // 32 columns x up to 16 neurons = up to 512 outputs for 256 threads
  for (int o = threadIdx.x; o < 32 * n_keep; o += 256) {
    const int n = o >> 5, c = o & 31;
    const int kk = blockIdx.x * 32 + c;
    if (kk >= kin) continue;
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) v += part[w][n][c];
    store_out(g.out, (size_t)(g.hdr_in != nullptr ? n : g.idx[n]) * g.ldo + kk, g.alpha * v, g.out_is_f32, g.accumulate);
  }
  if (g.flag1) {
    // rows of dropped neurons, this CTA's 32 columns
    const int dp = g.hdr[HDR_DP], bb = g.hdr[HDR_B] - 1;
    for (int o = threadIdx.x; o < 32 * g.N; o += 256) {
      const int row = o >> 5, kk = blockIdx.x * 32 + (o & 31);
      if (kk < kin && !(row >= bb && (row - bb) % dp == 0)) store_out(g.out, (size_t)row * g.ldo + kk, 0.f, g.out_is_f32);
    }
  }
}

template <typename T, int KIND, int OP>
void launch_one(const ard_ctx* ctx, const GemmArgs& a, int ts, int Mmax, int Nmax, cudaStream_t s) {
  dim3 grid((Nmax + T_N - 1) / T_N, (Mmax + T_M - 1) / T_M);
  (void)ard_launch(ctx, gemm_cc_kernel<T, KIND, OP>, grid, dim3(CC_THREADS), 0, s, a, ts);  // errors: cudaGetLastError
}

template <typename T>
void dispatch(const ard_ctx* ctx, ard_kind kind, GemmOp op, const GemmArgs& a, int ts, cudaStream_t s) {
  // The grid covers the largest problem any pattern can produce (dp = 1); CTAs beyond the
  // sampled extent read the header and exit.
  if (kind == ARD_ROW) {
    if (op == OP_FWD) launch_one<T, 0, OP_FWD>(ctx, a, ts, a.B, a.N, s);
    else if (op == OP_BWD_DATA) launch_one<T, 0, OP_BWD_DATA>(ctx, a, ts, a.B, a.K, s);
    else launch_one<T, 0, OP_BWD_WEIGHT>(ctx, a, ts, a.N, a.K, s);
  } else {
    if (op == OP_FWD) launch_one<T, 1, OP_FWD>(ctx, a, ts, a.B, a.N, s);
    else if (op == OP_BWD_DATA) launch_one<T, 1, OP_BWD_DATA>(ctx, a, ts, a.B, a.K, s);
    else launch_one<T, 1, OP_BWD_WEIGHT>(ctx, a, ts, a.N, a.K, s);
  }
}

}  // namespace

ard_status launch_gemm_cc(ard_ctx* ctx, ard_kind kind, GemmOp op, ard_dtype dtype, const GemmArgs& a, int ts,
                          cudaStream_t s) {
  if ((a.B == 0 && op != OP_BWD_WEIGHT) || a.K == 0 || a.N == 0) return ARD_OK;
  const size_t es_out = a.out_is_f32 ? 4 : 2;
  // Row patterns: dropped outputs are cleared by a strided memset before the kept ones are written.
  const bool small_layer = kind == ARD_ROW && a.N <= SKINNY_N && (op == OP_FWD ? a.B > 0 : op == OP_BWD_WEIGHT);
  if (small_layer) {
    // the kernels for a handful of neurons write their own zeros
  } else if (kind == ARD_ROW && op == OP_FWD && a.flag0 == ARD_OUT_SCATTER_ZEROFILL) {
    ARD_CUDA_OK(cudaMemset2DAsync(a.out, (size_t)a.ldo * es_out, 0, (size_t)a.N * es_out, a.B, s));
  }
  if (!small_layer && kind == ARD_ROW && op == OP_BWD_WEIGHT && a.flag1) {
    ARD_CUDA_OK(cudaMemset2DAsync(a.out, (size_t)a.ldo * es_out, 0, (size_t)a.K * es_out, a.N, s));
  }
  if (kind == ARD_ROW && a.N <= SKINNY_N && op == OP_FWD && a.B > 0) {
    if (dtype == ARD_F32) (void)ard_launch(ctx, skinny_fwd_kernel<float>, dim3(a.B), dim3(256), 0, s, a);
    else (void)ard_launch(ctx, skinny_fwd_kernel<__nv_bfloat16>, dim3(a.B), dim3(256), 0, s, a);
  } else if (kind == ARD_ROW && a.N <= SKINNY_N && op == OP_BWD_WEIGHT) {
    if (dtype == ARD_F32) (void)ard_launch(ctx, skinny_bwd_weight_kernel<float>, dim3((a.K + 31) / 32), dim3(256), 0, s, a);
    else (void)ard_launch(ctx, skinny_bwd_weight_kernel<__nv_bfloat16>, dim3((a.K + 31) / 32), dim3(256), 0, s, a);
  } else if (dtype == ARD_F32) {
    dispatch<float>(ctx, kind, op, a, ts, s);
  } else {
    dispatch<__nv_bfloat16>(ctx, kind, op, a, ts, s);
  }
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}
