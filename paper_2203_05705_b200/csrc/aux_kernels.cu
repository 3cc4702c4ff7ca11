// Small memory-bound kernels around the GEMMs: column compaction of a full-width gradient and the
// fused LSTM cell update (forward and adjoint) on the kept hidden units.
#include "ard_internal.h"

namespace {

// dst[r][j] = src[r][keep[j]], j < n_keep.  The kept columns of a row pattern (Sec. 3.1) stride the
// contiguous dimension, which a TMA box cannot do, so the tensor-core backward GEMMs read this copy.
template <typename T>
__global__ void __launch_bounds__(256) gather_cols_kernel(const int32_t* __restrict__ hdr, const T* __restrict__ src,
                                                          int ld_src, T* __restrict__ dst, int ld_dst, int rows) {
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int n_keep = hdr[HDR_NKEEP], dp = hdr[HDR_DP], b = hdr[HDR_B];
  const int j = blockIdx.x * 256 + threadIdx.x;
  if (j >= n_keep) return;
  const int col = b - 1 + j * dp;
  for (int r = blockIdx.y; r < rows; r += gridDim.y) dst[(size_t)r * ld_dst + j] = src[(size_t)r * ld_src + col];
}

// Faster form for 2-byte elements with 16-byte aligned rows.  Each warp owns a private slice of
// shared memory: it pulls the source span of up to 256 outputs with coalesced 16-byte loads (all of
// a lane's loads are issued before any is consumed), then every lane assembles 8 kept values into one
// 16-byte store.  No block-wide barrier, so the warps of a block overlap each other's latency.
// With skip_dense != 0 a dense pattern (dp = 1) is left alone: the GEMM then reads the original matrix.
constexpr int GATHER_WARPS = 4;
constexpr int GATHER_SPAN = 4096;  // staged source elements per warp (8 KiB)

__global__ void __launch_bounds__(GATHER_WARPS * 32)
gather_cols_staged_kernel(const int32_t* __restrict__ hdr, const uint16_t* __restrict__ src, int ld_src,
                          uint16_t* __restrict__ dst, int ld_dst, int rows, int n_cols, int skip_dense) {
  __shared__ __align__(16) uint16_t smem[GATHER_WARPS][GATHER_SPAN + 8];
  pdl_launch_dependents();
  pdl_wait_prior_grids();
  const int n_keep = hdr[HDR_NKEEP], dp = hdr[HDR_DP], bb = hdr[HDR_B] - 1;
  if (skip_dense && dp == 1) return;
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const long long warp_id = (long long)blockIdx.x * GATHER_WARPS + wib;
  const long long n_warps = (long long)gridDim.x * GATHER_WARPS;
  int outs = ((GATHER_SPAN - 8) / dp) & ~7;  // outputs per warp pass (multiple of 8)
  if (outs > 256) outs = 256;
  if (outs < 8) {
    // period too long for the staging slice: element-wise copy
    for (long long e = warp_id * 32 + lane; e < (long long)rows * n_keep; e += n_warps * 32) {
      const int r = (int)(e / n_keep), j = (int)(e % n_keep);
      dst[(size_t)r * ld_dst + j] = src[(size_t)r * ld_src + bb + (long long)j * dp];
    }
    return;
  }
  uint16_t* buf = smem[wib];
  const int chunks = (n_keep + outs - 1) / outs;
  for (long long item = warp_id; item < (long long)rows * chunks; item += n_warps) {
    const int r = (int)(item / chunks), ch = (int)(item - (long long)r * chunks);
    const int j0 = ch * outs;
    const int nout = min(outs, n_keep - j0);
    const int s0 = bb + j0 * dp;  // first source column
    const int a0 = s0 & ~7;       // 16-byte aligned start
    const int count = bb + (j0 + nout - 1) * dp - a0 + 1;
    const uint16_t* srow = src + (size_t)r * ld_src;
    for (int v = lane; v * 8 < count; v += 32) {
      const int col = a0 + 8 * v;
      if (col + 8 <= ld_src) {
        // asynchronous 16-byte copy: every piece of the span is in flight at once
        const uint32_t saddr = (uint32_t)__cvta_generic_to_shared(buf + 8 * v);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(saddr), "l"(srow + col) : "memory");
      } else {
        for (int i = 0; i < 8; ++i) buf[8 * v + i] = (col + i < n_cols) ? srow[col + i] : (uint16_t)0;
      }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncwarp();
    const int off = s0 - a0;
    uint16_t* drow = dst + (size_t)r * ld_dst + j0;
    const int t = lane;
    if (t * 8 + 8 <= nout) {
      uint32_t w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t lo = buf[off + (t * 8 + 2 * i) * dp], hi = buf[off + (t * 8 + 2 * i + 1) * dp];
        w[i] = lo | (hi << 16);
      }
      *reinterpret_cast<uint4*>(drow + t * 8) = make_uint4(w[0], w[1], w[2], w[3]);
    } else {
      for (int i = t * 8; i < nout && i < t * 8 + 8; ++i) drow[i] = buf[off + i * dp];
    }
    __syncwarp();
  }
}

__device__ __forceinline__ float sigmoidf_(float x) { return 1.f / (1.f + __expf(-x)); }

template <typename HT>
__global__ void __launch_bounds__(256)
lstm_gates_kernel(const int32_t* __restrict__ hdr, int B, int H, float alpha, const float* __restrict__ Z,
                  int ldz, const float* __restrict__ bias, const float* __restrict__ c_prev, int ldc,
                  float* __restrict__ c, HT* __restrict__ h, int ldh, int h_scatter,
                  float* __restrict__ gates_saved) {
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
lstm_gates_bwd_kernel(const int32_t* __restrict__ hdr, int B, int H, float alpha,
                      const float* __restrict__ gates_saved, const float* __restrict__ c_prev,
                      const float* __restrict__ c, int ldc, const float* __restrict__ dh, int lddh, int dh_scatter,
                      float* __restrict__ dc_inout, ZT* __restrict__ dZ, int ldz) {
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
                           (const uint16_t*)src, ld_src, (uint16_t*)dst, ld_dst, rows, max_cols, skip_dense));
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
