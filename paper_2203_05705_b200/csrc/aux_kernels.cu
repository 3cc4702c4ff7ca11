// Small memory-bound kernels around the GEMMs: column compaction of a full-width gradient and the
// fused LSTM cell update (forward and adjoint) on the kept hidden units.
#include "ard_internal.h"
#include "sm100_ptx.h"

namespace {

// dst[r][j] = src[r][keep[j]], j < n_keep.  The kept columns of a row pattern (Sec. 3.1) stride the
// contiguous dimension, which a TMA box cannot do, so the tensor-core backward GEMMs read this copy.
template <typename T>
__global__ void __launch_bounds__(256) gather_cols_kernel(const int32_t* hdr, const T* src,
                                                          int ld_src, T* dst, int ld_dst, int rows) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int n_keep = hdr[HDR_NKEEP], dp = hdr[HDR_DP], b = hdr[HDR_B];
  const int j = blockIdx.x * 256 + threadIdx.x;
  if (j >= n_keep) return;
  const int col = b - 1 + j * dp;
  for (int r = blockIdx.y; r < rows; r += gridDim.y) dst[(size_t)r * ld_dst + j] = src[(size_t)r * ld_src + col];
}

// The adjoint of the gather, with a rescale: dst[r][b-1 + j*dp] = alpha * src[r][j] for j < n_keep, every other
// column of dst zero (fp32 out).  Used to hand a gradient that arrives over kept units only to a consumer that
// wants it full width (the upstream gradient of an LSTM layer whose outputs were dropped).
template <typename T>
__global__ void __launch_bounds__(256) expand_cols_kernel(const int32_t* hdr, const T* src, int ld_src, float* dst,
                                                          int ld_dst, int rows, int N, float alpha) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int dp = hdr[HDR_DP], bb = hdr[HDR_B] - 1;
  const int c = blockIdx.x * 256 + threadIdx.x;
  if (c >= N) return;
  const int rel = c - bb;
  const bool kept = rel >= 0 && rel % dp == 0;
  const int j = kept ? rel / dp : 0;
  for (int r = blockIdx.y; r < rows; r += gridDim.y) {
    float v = 0.f;
    if (kept) {
      if (sizeof(T) == 2) v = alpha * __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(src)[(size_t)r * ld_src + j]);
      else v = alpha * reinterpret_cast<const float*>(src)[(size_t)r * ld_src + j];
    }
    dst[(size_t)r * ld_dst + c] = v;
  }
}

// Faster form for 2-byte elements with 16-byte aligned rows.  Each warp owns two private slices of
// shared memory: one bulk copy (the copy engine, not the load unit, whose queue holds about 20 KB of
// 16-byte requests per SM) brings the source span of a pass into one slice while the warp compacts the
// other slice in place and writes it out with 16-byte stores.  No block-wide barrier, so the warps of a
// block overlap each other's latency.  The wait on a copy is bounded; a timeout sets *status and ends
// the warp.
// With skip_dense != 0 a dense pattern (dp = 1) is left alone: the GEMM then reads the original matrix.
constexpr int GATHER_WARPS = 4;
constexpr int GATHER_SPAN = 2048;  // staged source elements per slice (4 KiB)

struct GatherItem {
  int r, j0, nout, a0, off, count, n16;
};

__global__ void __launch_bounds__(GATHER_WARPS * 32)
gather_cols_staged_kernel(const int32_t* hdr, const uint16_t* src, int ld_src,
                          uint16_t* dst, int ld_dst, int rows, int n_cols, int skip_dense, int* status) {
  __shared__ __align__(128) uint16_t smem[GATHER_WARPS][2][GATHER_SPAN + 64];
  __shared__ __align__(8) uint64_t bars[GATHER_WARPS][2];
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  if (lane == 0) {
    mbar_init(smem_u32(&bars[wib][0]), 1);
    mbar_init(smem_u32(&bars[wib][1]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int n_keep = hdr[HDR_NKEEP], dp = hdr[HDR_DP], bb = hdr[HDR_B] - 1;
  if (skip_dense && dp == 1) return;
  const long long warp_id = (long long)blockIdx.x * GATHER_WARPS + wib;
  const long long n_warps = (long long)gridDim.x * GATHER_WARPS;
  // outputs per warp pass (multiple of 8): whatever the period, a pass fills its staging slice
  const int outs = ((GATHER_SPAN - 8) / dp) & ~7;
  if (outs < 8) {
    // period too long for the staging slice: element-wise copy
    for (long long e = warp_id * 32 + lane; e < (long long)rows * n_keep; e += n_warps * 32) {
      const int r = (int)(e / n_keep), j = (int)(e % n_keep);
      dst[(size_t)r * ld_dst + j] = src[(size_t)r * ld_src + bb + (long long)j * dp];
    }
    return;
  }
  const int chunks = (n_keep + outs - 1) / outs;
  const long long total = (long long)rows * chunks;
  auto describe = [&](long long item) {
    GatherItem g;
    g.r = (int)(item / chunks);
    const int ch = (int)(item - (long long)g.r * chunks);
    g.j0 = ch * outs;
    g.nout = min(outs, n_keep - g.j0);
    const int s0 = bb + g.j0 * dp;  // first source column
    g.a0 = s0 & ~7;                 // 16-byte aligned start
    g.off = s0 - g.a0;
    g.count = bb + (g.j0 + g.nout - 1) * dp - g.a0 + 1;  // <= n_cols - a0
    // whole 16-byte pieces inside the row go through the copy engine, a ragged end (< 8 elements) by lanes
    g.n16 = min((g.count + 7) & ~7, (n_cols - g.a0) & ~7);
    return g;
  };
  // starts the copy of an item into a slice; every lane's earlier accesses to the slice were fenced
  auto fetch = [&](const GatherItem& g, int slot) {
    uint16_t* buf = smem[wib][slot];
    const uint16_t* srow = src + (size_t)g.r * ld_src;
    if (lane == 0 && g.n16 > 0) {
      const uint32_t bar = smem_u32(&bars[wib][slot]);
      mbar_arrive_expect_tx(bar, (uint32_t)g.n16 * 2u);
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(smem_u32(buf)), "l"(srow + g.a0), "r"((uint32_t)g.n16 * 2u), "r"(bar)
                   : "memory");
    }
    for (int i = g.n16 + lane; i < g.count; i += 32) buf[i] = srow[g.a0 + i];
  };
  uint32_t phase[2] = {0u, 0u};
  long long item = warp_id;
  if (item >= total) return;
  GatherItem cur = describe(item);
  fetch(cur, 0);
  for (int k = 0;; ++k) {
    const int slot = k & 1;
    const long long next_item = item + n_warps;
    GatherItem nxt = cur;
    if (next_item < total) {
      nxt = describe(next_item);
      fetch(nxt, slot ^ 1);
    }
    if (cur.n16 > 0) {
      const uint32_t bar = smem_u32(&bars[wib][slot]);
      bool ok = mbar_try_wait(bar, phase[slot]);
      for (int poll = 0; poll < 4000 && !ok; ++poll) ok = mbar_try_wait_hint(bar, phase[slot], 1000000u);
      if (!ok) {
        if (lane == 0) atomicMax(status, (int)ARD_ERR_TIMEOUT);
        if (next_item < total && nxt.n16 > 0) {  // the copy into the other slice: give it the same time, then leave
          const uint32_t bar2 = smem_u32(&bars[wib][slot ^ 1]);
          bool done = false;
          for (int poll = 0; poll < 4000 && !done; ++poll) done = mbar_try_wait_hint(bar2, phase[slot ^ 1], 1000000u);
        }
        return;
      }
      phase[slot] ^= 1u;
    }
    __syncwarp();
    uint16_t* buf = smem[wib][slot];
    const int off = cur.off, nout = cur.nout;
    uint16_t* drow = dst + (size_t)cur.r * ld_dst + cur.j0;
    // Compact the slice in place, consecutive lanes taking consecutive outputs (a lane that took eight
    // outputs in a row read shared memory at a stride of 16 * dp bytes: up to 32 lanes on one bank).  Output
    // j lands at element j <= off + j * dp, and the sources of a batch are all in registers before any of
    // its outputs is written, so nothing is overwritten before it is read.
    for (int j = 0; j < nout; j += 256) {
      uint16_t v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int jj = j + 32 * i + lane;
        v[i] = jj < nout ? buf[off + jj * dp] : (uint16_t)0;
      }
      __syncwarp();
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int jj = j + 32 * i + lane;
        if (jj < nout) buf[jj] = v[i];
      }
      __syncwarp();
    }
    for (int t = lane; t * 8 < nout; t += 32) {
      if (t * 8 + 8 <= nout) {
        *reinterpret_cast<uint4*>(drow + t * 8) = *reinterpret_cast<const uint4*>(buf + t * 8);
      } else {
        for (int i = t * 8; i < nout; ++i) drow[i] = buf[i];
      }
    }
    fence_proxy_async_smem();  // this lane's accesses to the slice, before a later pass's copy overwrites it
    __syncwarp();
    if (next_item >= total) break;
    item = next_item;
    cur = nxt;
  }
}

__device__ __forceinline__ float sigmoidf_(float x) { return 1.f / (1.f + __expf(-x)); }

template <typename HT>
__global__ void __launch_bounds__(256)
lstm_gates_kernel(const int32_t* hdr, int B, int H, float alpha, const float* Z,
                  int ldz, const float* bias, const float* c_prev, int ldc,
                  float* c, HT* h, int ldh, int h_scatter,
                  float* gates_saved) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int n_keep = hdr[HDR_NKEEP], dp = hdr[HDR_DP], b = hdr[HDR_B];
  const int i = blockIdx.y;
  const int x = blockIdx.x * 256 + threadIdx.x;  // unit (scatter) or kept index (compact)
  int j, u;
  if (h_scatter) {
    u = x;
    if (u >= H) return;
    const bool kept = u >= b - 1 && (u - (b - 1)) % dp == 0;
    if (!kept) {
      h[(size_t)i * ldh + u] = HT(0.f);
      return;
    }
    j = (u - (b - 1)) / dp;
  } else {
    j = x;
    if (j >= n_keep) return;
    u = b - 1 + j * dp;
  }
  const float* z = Z + (size_t)i * 4 * ldz;
  float zi = z[0 * ldz + j], zf = z[1 * ldz + j], zg = z[2 * ldz + j], zo = z[3 * ldz + j];
  if (bias) {
    zi += bias[0 * H + u];
    zf += bias[1 * H + u];
    zg += bias[2 * H + u];
    zo += bias[3 * H + u];
  }
  const float gi = sigmoidf_(zi), gf = sigmoidf_(zf), gg = tanhf(zg), go = sigmoidf_(zo);
  const float cn = gf * c_prev[(size_t)i * ldc + j] + gi * gg;
  c[(size_t)i * ldc + j] = cn;
  const float hv = alpha * go * tanhf(cn);
  h[(size_t)i * ldh + (h_scatter ? u : j)] = HT(hv);
  if (gates_saved) {
    float* gs = gates_saved + (size_t)i * 4 * ldc;
    gs[0 * ldc + j] = gi;
    gs[1 * ldc + j] = gf;
    gs[2 * ldc + j] = gg;
    gs[3 * ldc + j] = go;
  }
}

template <typename ZT>
__global__ void __launch_bounds__(256)
lstm_gates_bwd_kernel(const int32_t* hdr, int B, int H, float alpha,
                      const float* gates_saved, const float* c_prev,
                      const float* c, int ldc, const float* dh, int lddh, int dh_scatter,
                      float* dc_inout, ZT* dZ, int ldz) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int n_keep = hdr[HDR_NKEEP], dp = hdr[HDR_DP], b = hdr[HDR_B];
  const int i = blockIdx.y;
  const int j = blockIdx.x * 256 + threadIdx.x;
  if (j >= n_keep) return;
  const int u = b - 1 + j * dp;
  const float* gs = gates_saved + (size_t)i * 4 * ldc;
  const float gi = gs[0 * ldc + j], gf = gs[1 * ldc + j], gg = gs[2 * ldc + j], go = gs[3 * ldc + j];
  const float cp = c_prev[(size_t)i * ldc + j];
  const float tc = tanhf(c[(size_t)i * ldc + j]);
  const float dhv = dh[(size_t)i * lddh + (dh_scatter ? u : j)];
  const float d_o = dhv * alpha * tc;
  const float dc = dc_inout[(size_t)i * ldc + j] + dhv * alpha * go * (1.f - tc * tc);
  const float d_i = dc * gg, d_g = dc * gi, d_f = dc * cp;
  dc_inout[(size_t)i * ldc + j] = dc * gf;
  ZT* dz = dZ + (size_t)i * 4 * ldz;
  dz[0 * ldz + j] = ZT(d_i * gi * (1.f - gi));
  dz[1 * ldz + j] = ZT(d_f * gf * (1.f - gf));
  dz[2 * ldz + j] = ZT(d_g * (1.f - gg * gg));
  dz[3 * ldz + j] = ZT(d_o * go * (1.f - go));
}

// ---- layer-step helpers (Sec. 3.1: the weight is compacted along the fan-in too when the layer that
// feeds it ran under a row pattern) -----------------------------------------------------------------
//
// Wk[j][i] = W[keep[j]][keep_in[i]], compact in both dimensions (row j = j-th kept neuron of `hdr`, i < n_in).
// Columns n_in up to the next multiple of 64 (or ldwk) and rows n_keep up to the next multiple of 64 (or N)
// are written as zero, so that the last 64-deep contraction block of the forward and of the backward-data
// product multiplies zeros.  Rows are packed (and not left at their neuron's position) because the products
// read them in boxes of 64 rows: with a period of 8 and a 16 KiB pitch the rows of a box would be 128 KiB
// apart, which halves the speed of the box loads.  Eight outputs per thread (one 16- or 32-byte store).
template <typename T>
__global__ void __launch_bounds__(256) compact_weight_cols_kernel(const int32_t* hdr,
                                                                  const int32_t* hdr_in,
                                                                  const T* W, int ldw, T* Wk,
                                                                  int ldwk, int N, int vec_ok) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int n_keep = hdr[HDR_NKEEP], dp = hdr[HDR_DP], bb = hdr[HDR_B] - 1;
  const int n_in = hdr_in[HDR_NKEEP], dpi = hdr_in[HDR_DP], bi = hdr_in[HDR_B] - 1;
  const int padded = min(ldwk, (n_in + 63) / 64 * 64);
  const int rows_padded = min(N, (n_keep + 63) / 64 * 64);
  const int groups = (padded + 7) / 8;
  for (int i = blockIdx.y; i < rows_padded; i += gridDim.y) {
    const bool real = i < n_keep;
    const size_t row = (size_t)bb + (size_t)i * dp;
    const T* src = W + (real ? row : 0) * ldw + bi;
    T* dst = Wk + (size_t)i * ldwk;
    for (int g = blockIdx.x * 256 + threadIdx.x; g < groups; g += gridDim.x * 256) {
      const int j0 = g * 8;
      __align__(16) T v[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) v[q] = (real && j0 + q < n_in) ? src[(size_t)(j0 + q) * dpi] : T(0.f);
      if (vec_ok && j0 + 8 <= padded) {
        if (sizeof(T) == 2) {
          *reinterpret_cast<uint4*>(dst + j0) = *reinterpret_cast<const uint4*>(v);
        } else {
          reinterpret_cast<uint4*>(dst + j0)[0] = reinterpret_cast<const uint4*>(v)[0];
          reinterpret_cast<uint4*>(dst + j0)[1] = reinterpret_cast<const uint4*>(v)[1];
        }
      } else {
#pragma unroll
        for (int q = 0; q < 8; ++q)
          if (j0 + q < padded) dst[j0 + q] = v[q];
      }
    }
  }
}

// The inverse for the gradient: dW[keep[j]][keep_in[i]] = dWk[j][i]; with zero_fill
// every other entry of dW [N][K] (dropped neurons, dropped inputs) is written as zero, without it they
// are left alone.  One output row per blockIdx.y step, consecutive threads write consecutive columns.
template <typename T>
__global__ void __launch_bounds__(256) expand_weight_grad_cols_kernel(const int32_t* hdr,
                                                                      const int32_t* hdr_in,
                                                                      const T* dWk, int lddwk,
                                                                      T* dW, int lddw, int N, int K,
                                                                      int zero_fill) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int dp = hdr[HDR_DP], bb = hdr[HDR_B] - 1;
  const int dpi = hdr_in[HDR_DP], bi = hdr_in[HDR_B] - 1;
  for (int n = blockIdx.y; n < N; n += gridDim.y) {
    const bool kept_row = n >= bb && (n - bb) % dp == 0;
    if (!kept_row && !zero_fill) continue;
    const T* src = dWk + (size_t)(kept_row ? (n - bb) / dp : 0) * lddwk;  // packed row of this neuron
    T* dst = dW + (size_t)n * lddw;
    for (int k = blockIdx.x * 256 + threadIdx.x; k < K; k += gridDim.x * 256) {
      const bool kept = kept_row && k >= bi && (k - bi) % dpi == 0;
      if (kept) dst[k] = src[(k - bi) / dpi];
      else if (zero_fill) dst[k] = T(0.f);
    }
  }
}

// Bias gradient of a layer step: db[n] = sum over the batch of dZ[:, n] for the kept neurons (Sec. 3.1:
// a dropped neuron takes no part in the iteration); dropped entries are zeroed on request.
// A block owns 32 consecutive neurons; its 8 row groups add their rows in a fixed order.
template <typename T>
__global__ void __launch_bounds__(256) bias_grad_kernel(const int32_t* hdr, const T* dZ,
                                                        int lddz, int dz_is_compact, int B, int N,
                                                        float* db, int zero_fill) {
  __shared__ float part[8][33];
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int dp = hdr[HDR_DP], bb = hdr[HDR_B] - 1;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int n = blockIdx.x * 32 + tx;
  const bool kept = n < N && n >= bb && (n - bb) % dp == 0;
  float acc = 0.f;
  if (kept) {
    const int col = dz_is_compact ? (n - bb) / dp : n;
    for (int r = ty; r < B; r += 8) acc += (float)dZ[(size_t)r * lddz + col];
  }
  part[ty][tx] = acc;
  __syncthreads();
  if (ty == 0 && n < N) {
    float sum = 0.f;
#pragma unroll
    for (int q = 0; q < 8; ++q) sum += part[q][tx];
    if (kept) db[n] = sum;
    else if (zero_fill) db[n] = 0.f;
  }
}

// Wide form of the expansion for 16-byte aligned rows: a thread assembles 8 consecutive output columns
// (one 16-byte store for bf16, two for fp32) from the at most 8 compact entries that fall into them.
template <typename T>
__global__ void __launch_bounds__(256) expand_weight_grad_cols_wide_kernel(const int32_t* hdr, const int32_t* hdr_in,
                                                                           const T* dWk, int lddwk, T* dW, int lddw,
                                                                           int N, int K, int zero_fill) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int dp = hdr[HDR_DP], bb = hdr[HDR_B] - 1;
  const int dpi = hdr_in[HDR_DP], bi = hdr_in[HDR_B] - 1;
  const int groups = K / 8;  // the caller guarantees K % 8 == 0
  for (int n = blockIdx.y; n < N; n += gridDim.y) {
    const bool kept_row = n >= bb && (n - bb) % dp == 0;
    if (!kept_row && !zero_fill) continue;
    const T* src = dWk + (size_t)(kept_row ? (n - bb) / dp : 0) * lddwk;  // packed row of this neuron
    T* dst = dW + (size_t)n * lddw;
    for (int g = blockIdx.x * 256 + threadIdx.x; g < groups; g += gridDim.x * 256) {
      const int k0 = g * 8;
      __align__(16) T v[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) v[q] = T(0.f);
      bool any = false;
      if (kept_row) {
        // first kept input at or after k0, then every dpi-th
        int k = k0 <= bi ? bi : bi + ((k0 - bi + dpi - 1) / dpi) * dpi;
        int j = (k - bi) / dpi;
        for (; k < k0 + 8; k += dpi, ++j) {
          const T x = src[j];
#pragma unroll
          for (int q = 0; q < 8; ++q)
            if (q == k - k0) v[q] = x;
          any = true;
        }
      }
      if (!any && !zero_fill) continue;
      if (!zero_fill) {
        // only the kept entries may be touched
#pragma unroll
        for (int q = 0; q < 8; ++q)
          if (k0 + q >= bi && (k0 + q - bi) % dpi == 0) dst[k0 + q] = v[q];
      } else if (sizeof(T) == 2) {
        *reinterpret_cast<uint4*>(dst + k0) = *reinterpret_cast<const uint4*>(v);
      } else {
        reinterpret_cast<uint4*>(dst + k0)[0] = reinterpret_cast<const uint4*>(v)[0];
        reinterpret_cast<uint4*>(dst + k0)[1] = reinterpret_cast<const uint4*>(v)[1];
      }
    }
  }
}

// Wide form of the bias gradient for compact 16-byte aligned bf16 dZ and many rows: the batch is cut into
// gridDim.y slices; a block adds its slice of 256 compact columns (a lane owns 8 columns of a row, a warp
// every eighth row of the slice), parks the 256 sums in scratch and the block that arrives last for its
// columns adds the slices in slice order, so the result does not depend on the arrival order.
constexpr int BIAS_WIDE_COLS = 256;

__global__ void __launch_bounds__(256) bias_grad_wide_kernel(const int32_t* hdr, const __nv_bfloat16* dZ, int lddz,
                                                             int compact, int B, int N, float* db, int zero_fill,
                                                             float* partial, int* counters) {
  __shared__ float red[8][BIAS_WIDE_COLS + 8];
  __shared__ int s_last;
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int dp = hdr[HDR_DP], bb = hdr[HDR_B] - 1;
  const int n_keep = compact ? hdr[HDR_NKEEP] : N;  // columns of dZ that are added (full width: all of them)
  const int c0 = blockIdx.x * BIAS_WIDE_COLS;
  if (c0 >= n_keep) return;
  const int S = gridDim.y, y = blockIdx.y;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (compact && zero_fill && y == 0) {
    // dropped neurons between this block's first kept neuron and the next block's (the last block: to N)
    const int lo = c0 == 0 ? 0 : bb + c0 * dp;
    const int hi = (c0 + BIAS_WIDE_COLS >= n_keep) ? N : bb + (c0 + BIAS_WIDE_COLS) * dp;
    for (int o = lo + threadIdx.x; o < hi; o += 256)
      if (!(o >= bb && (o - bb) % dp == 0)) db[o] = 0.f;
  }
  const int rows_per = (B + S - 1) / S;
  const int r0 = y * rows_per, r1 = min(B, r0 + rows_per);
  const int c = c0 + lane * 8;
  float acc[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) acc[q] = 0.f;
  if (c < n_keep) {
    for (int r = r0 + warp; r < r1; r += 8) {
      const uint4 x = *reinterpret_cast<const uint4*>(dZ + (size_t)r * lddz + c);
      const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        acc[2 * q] += __uint_as_float(w[q] << 16);
        acc[2 * q + 1] += __uint_as_float(w[q] & 0xFFFF0000u);
      }
    }
  }
#pragma unroll
  for (int q = 0; q < 8; ++q) red[warp][lane * 8 + q] = acc[q];
  __syncthreads();
  const int col = threadIdx.x;  // one compact column per thread from here on
  float sum = 0.f;
#pragma unroll
  for (int w8 = 0; w8 < 8; ++w8) sum += red[w8][col];
  const int n_cols_total = gridDim.x * BIAS_WIDE_COLS;
  __stcg(partial + (size_t)y * n_cols_total + c0 + col, sum);
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = (atomicAdd(counters + blockIdx.x, 1) == S - 1) ? 1 : 0;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (threadIdx.x == 0) counters[blockIdx.x] = 0;  // armed again for the next launch
  if (c0 + col < n_keep) {
    float total = 0.f;
    for (int yy = 0; yy < S; ++yy) total += __ldcg(partial + (size_t)yy * n_cols_total + c0 + col);
    if (compact) {
      db[bb + (c0 + col) * dp] = total;
    } else {
      // full width: the sums of dropped columns (whose entries are never values) are discarded
      const int o = c0 + col;
      if (o >= bb && (o - bb) % dp == 0) db[o] = total;
      else if (zero_fill) db[o] = 0.f;
    }
  }
}

// Tile patterns, backward-weight: the dropped tiles of dW are zero (Sec. 3.2).  One CTA per dropped tile
// (kept tiles are written by the product and skipped here), so a dense pattern costs nothing and a
// pattern of period dp writes (dp-1)/dp of dW instead of all of it.
__global__ void __launch_bounds__(256) zero_dropped_tiles_kernel(const int32_t* hdr, void* dW, int lddw, int ts, int Tr,
                                                                 int Tc, int elem_bytes) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int dp = hdr[HDR_DP], bb = hdr[HDR_B] - 1;
  if (dp == 1) return;
  const int row_bytes = ts * elem_bytes;
  const bool wide = (row_bytes & 15) == 0 && (((size_t)lddw * elem_bytes) & 15) == 0 && (reinterpret_cast<uintptr_t>(dW) & 15) == 0;
  for (int lin = blockIdx.x; lin < Tr * Tc; lin += gridDim.x) {
    if (lin >= bb && (lin - bb) % dp == 0) continue;  // kept
    const int r = lin / Tc, c = lin - r * Tc;         // tile-row along the fan-in, tile-column along the neurons
    char* base = reinterpret_cast<char*>(dW) + ((size_t)c * ts * lddw + (size_t)r * ts) * elem_bytes;
    if (wide) {
      const int per_row = row_bytes >> 4;
      for (int e = threadIdx.x; e < ts * per_row; e += 256) {
        const int n = e / per_row, q = e - n * per_row;
        *reinterpret_cast<uint4*>(base + (size_t)n * lddw * elem_bytes + (size_t)q * 16) = make_uint4(0, 0, 0, 0);
      }
    } else {
      const int per_row = row_bytes >> 1;
      for (int e = threadIdx.x; e < ts * per_row; e += 256) {
        const int n = e / per_row, q = e - n * per_row;
        *reinterpret_cast<uint16_t*>(base + (size_t)n * lddw * elem_bytes + (size_t)q * 2) = 0;
      }
    }
  }
}

}  // namespace

ard_status launch_gather_cols(ard_ctx* ctx, const int32_t* hdr, const int32_t* idx, const void* src, int ld_src,
                              void* dst, int ld_dst, int rows, int elem_bytes, int max_cols, int skip_dense,
                              cudaStream_t s) {
  (void)idx;
  if (rows == 0 || max_cols == 0) return ARD_OK;
  const bool vec_ok = elem_bytes == 2 && ld_src % 8 == 0 && ld_dst % 8 == 0 &&
                      (reinterpret_cast<uintptr_t>(src) & 15) == 0 && (reinterpret_cast<uintptr_t>(dst) & 15) == 0;
  if (vec_ok) {
    ARD_CUDA_OK(ard_launch(ctx, gather_cols_staged_kernel, dim3(ctx->sm_count * 6), dim3(GATHER_WARPS * 32), 0, s, hdr,
                           (const uint16_t*)src, ld_src, (uint16_t*)dst, ld_dst, rows, max_cols, skip_dense, ctx->d_status));
  } else {
    dim3 grid((max_cols + 255) / 256, rows < 1024 ? rows : 1024);
    if (elem_bytes == 2)
      ARD_CUDA_OK(ard_launch(ctx, gather_cols_kernel<uint16_t>, grid, dim3(256), 0, s, hdr, (const uint16_t*)src, ld_src,
                             (uint16_t*)dst, ld_dst, rows));
    else
      ARD_CUDA_OK(ard_launch(ctx, gather_cols_kernel<uint32_t>, grid, dim3(256), 0, s, hdr, (const uint32_t*)src, ld_src,
                             (uint32_t*)dst, ld_dst, rows));
  }
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

ard_status launch_expand_cols(ard_ctx* ctx, const int32_t* hdr, const void* src, int ld_src, int src_is_bf16, float* dst,
                              int ld_dst, int rows, int N, float alpha, cudaStream_t s) {
  if (rows == 0 || N == 0) return ARD_OK;
  dim3 grid((N + 255) / 256, rows < 2048 ? rows : 2048);
  if (src_is_bf16)
    ARD_CUDA_OK(ard_launch(ctx, expand_cols_kernel<uint16_t>, grid, dim3(256), 0, s, hdr, (const uint16_t*)src, ld_src, dst,
                           ld_dst, rows, N, alpha));
  else
    ARD_CUDA_OK(ard_launch(ctx, expand_cols_kernel<float>, grid, dim3(256), 0, s, hdr, (const float*)src, ld_src, dst, ld_dst,
                           rows, N, alpha));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

ard_status launch_lstm_gates(ard_ctx* ctx, const ard_pattern* pat, ard_dtype h_dtype, int B, int H, float alpha,
                             const float* Z, int ldz_gate, const float* bias, const float* c_prev, int ldc, float* c,
                             void* h, int ldh, int h_scatter, float* gates_saved, cudaStream_t s) {
  if (B == 0 || H == 0) return ARD_OK;
  dim3 grid((H + 255) / 256, B);
  if (h_dtype == ARD_F32)
    ARD_CUDA_OK(ard_launch(ctx, lstm_gates_kernel<float>, grid, dim3(256), 0, s, (const int32_t*)pat->d_hdr, B, H, alpha, Z,
                           ldz_gate, bias, c_prev, ldc, c, (float*)h, ldh, h_scatter, gates_saved));
  else
    ARD_CUDA_OK(ard_launch(ctx, lstm_gates_kernel<__nv_bfloat16>, grid, dim3(256), 0, s, (const int32_t*)pat->d_hdr, B, H,
                           alpha, Z, ldz_gate, bias, c_prev, ldc, c, (__nv_bfloat16*)h, ldh, h_scatter, gates_saved));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

ard_status launch_lstm_gates_bwd(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dz_dtype, int B, int H, float alpha,
                                 const float* gates_saved, const float* c_prev, const float* c, int ldc,
                                 const float* dh, int lddh, int dh_scatter, float* dc_inout, void* dZ, int ldz_gate,
                                 cudaStream_t s) {
  if (B == 0 || H == 0) return ARD_OK;
  dim3 grid((H + 255) / 256, B);
  if (dz_dtype == ARD_F32)
    ARD_CUDA_OK(ard_launch(ctx, lstm_gates_bwd_kernel<float>, grid, dim3(256), 0, s, (const int32_t*)pat->d_hdr, B, H, alpha,
                           gates_saved, c_prev, c, ldc, dh, lddh, dh_scatter, dc_inout, (float*)dZ, ldz_gate));
  else
    ARD_CUDA_OK(ard_launch(ctx, lstm_gates_bwd_kernel<__nv_bfloat16>, grid, dim3(256), 0, s, (const int32_t*)pat->d_hdr, B,
                           H, alpha, gates_saved, c_prev, c, ldc, dh, lddh, dh_scatter, dc_inout, (__nv_bfloat16*)dZ,
                           ldz_gate));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

ard_status launch_compact_weight_cols(ard_ctx* ctx, const int32_t* hdr, const int32_t* hdr_in, const void* W, int ldw,
                                      void* Wk, int ldwk, int N, int K, int elem_bytes, cudaStream_t s) {
  if (N == 0 || K == 0) return ARD_OK;
  const int vec_ok = (reinterpret_cast<uintptr_t>(Wk) & 15) == 0 && ((size_t)ldwk * elem_bytes) % 16 == 0 && ldwk % 8 == 0;
  dim3 grid((K / 8 + 255) / 256 > 0 ? (K / 8 + 255) / 256 : 1, N < 65535 ? N : 65535);
  if (elem_bytes == 2)
    ARD_CUDA_OK(ard_launch(ctx, compact_weight_cols_kernel<__nv_bfloat16>, grid, dim3(256), 0, s, hdr, hdr_in,
                           (const __nv_bfloat16*)W, ldw, (__nv_bfloat16*)Wk, ldwk, N, vec_ok));
  else
    ARD_CUDA_OK(ard_launch(ctx, compact_weight_cols_kernel<float>, grid, dim3(256), 0, s, hdr, hdr_in, (const float*)W,
                           ldw, (float*)Wk, ldwk, N, vec_ok));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

ard_status launch_expand_weight_grad_cols(ard_ctx* ctx, const int32_t* hdr, const int32_t* hdr_in, const void* dWk,
                                          int lddwk, void* dW, int lddw, int N, int K, int elem_bytes, int zero_fill,
                                          cudaStream_t s) {
  if (N == 0 || K == 0) return ARD_OK;
  const bool wide = K % 8 == 0 && lddw % 8 == 0 && (reinterpret_cast<uintptr_t>(dW) & 15) == 0;
  if (wide) {
    dim3 gridw((K / 8 + 255) / 256, N < 65535 ? N : 65535);
    if (elem_bytes == 2)
      ARD_CUDA_OK(ard_launch(ctx, expand_weight_grad_cols_wide_kernel<__nv_bfloat16>, gridw, dim3(256), 0, s, hdr, hdr_in,
                             (const __nv_bfloat16*)dWk, lddwk, (__nv_bfloat16*)dW, lddw, N, K, zero_fill));
    else
      ARD_CUDA_OK(ard_launch(ctx, expand_weight_grad_cols_wide_kernel<float>, gridw, dim3(256), 0, s, hdr, hdr_in,
                             (const float*)dWk, lddwk, (float*)dW, lddw, N, K, zero_fill));
    ctx->launches++;
    ARD_CUDA_OK(cudaGetLastError());
    return ARD_OK;
  }
  dim3 grid((K + 1023) / 1024, N < 65535 ? N : 65535);
  if (elem_bytes == 2)
    ARD_CUDA_OK(ard_launch(ctx, expand_weight_grad_cols_kernel<__nv_bfloat16>, grid, dim3(256), 0, s, hdr, hdr_in,
                           (const __nv_bfloat16*)dWk, lddwk, (__nv_bfloat16*)dW, lddw, N, K, zero_fill));
  else
    ARD_CUDA_OK(ard_launch(ctx, expand_weight_grad_cols_kernel<float>, grid, dim3(256), 0, s, hdr, hdr_in,
                           (const float*)dWk, lddwk, (float*)dW, lddw, N, K, zero_fill));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

ard_status launch_bias_grad(ard_ctx* ctx, const int32_t* hdr, const void* dZ, int lddz, int dz_is_compact,
                            int is_bf16, int B, int N, float* db, int zero_fill, cudaStream_t s) {
  if (N == 0) return ARD_OK;
  // 512 rows or more of aligned bf16: the batch is cut into slices that are added in a fixed order (with
  // fewer rows the plain form below is faster: 2 us against 5 us at 128 rows)
  const int xblocks = (N + BIAS_WIDE_COLS - 1) / BIAS_WIDE_COLS;
  int slices = B / 64;
  if (slices > 32) slices = 32;
  if (is_bf16 && N % 8 == 0 && slices >= 8 && lddz % 8 == 0 && (reinterpret_cast<uintptr_t>(dZ) & 15) == 0 &&
      ctx->d_sk_ws != nullptr && (size_t)slices * xblocks * BIAS_WIDE_COLS * sizeof(float) <= sk_ws_bytes(ctx->sm_count) &&
      (size_t)xblocks * sizeof(int) <= sk_cnt_bytes(ctx->sm_count)) {
    ARD_CUDA_OK(ard_launch(ctx, bias_grad_wide_kernel, dim3(xblocks, slices), dim3(256), 0, s, hdr,
                           (const __nv_bfloat16*)dZ, lddz, dz_is_compact, B, N, db, zero_fill,
                           reinterpret_cast<float*>(ctx->d_sk_ws),
                           ctx->d_sk_cnt));
    ctx->launches++;
    ARD_CUDA_OK(cudaGetLastError());
    return ARD_OK;
  }
  dim3 grid((N + 31) / 32);
  if (is_bf16)
    ARD_CUDA_OK(ard_launch(ctx, bias_grad_kernel<__nv_bfloat16>, grid, dim3(256), 0, s, hdr, (const __nv_bfloat16*)dZ,
                           lddz, dz_is_compact, B, N, db, zero_fill));
  else
    ARD_CUDA_OK(ard_launch(ctx, bias_grad_kernel<float>, grid, dim3(256), 0, s, hdr, (const float*)dZ, lddz,
                           dz_is_compact, B, N, db, zero_fill));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

ard_status launch_zero_dropped_tiles(ard_ctx* ctx, const ard_pattern* pat, void* dW, int lddw, int elem_bytes,
                                     cudaStream_t s) {
  const int tiles = pat->Tr * pat->Tc;
  if (tiles == 0) return ARD_OK;
  const int grid = tiles < ctx->sm_count * 32 ? tiles : ctx->sm_count * 32;
  ARD_CUDA_OK(ard_launch(ctx, zero_dropped_tiles_kernel, dim3(grid), dim3(256), 0, s, (const int32_t*)pat->d_hdr, dW, lddw,
                         pat->ts, pat->Tr, pat->Tc, elem_bytes));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}
