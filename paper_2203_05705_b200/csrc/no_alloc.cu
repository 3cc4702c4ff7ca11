// ard_bwd_data_static_scratch: backward-data for a row pattern that allocates nothing.
//
// Who needs this: code that may not allocate device memory at the moment it calls the layer -- an
// inference / training server that froze its memory plan after start-up, a plug-in running inside a
// host application that owns the allocator, or a caller sitting on a stream whose owner forbids
// cudaMalloc / cudaFree because both synchronise the whole device.  ard_bwd_data needs a context
// workspace that ard_create allocated for it; this entry point needs none and never allocates.
//
// How: the compacted copy of dY (kept columns only) that the GEMM reads lives in a fixed array that
// is part of the library image, so every GPU that loads libard.so carries ARD_STATIC_SCRATCH_BYTES
// of it until the process exits.  A small gather kernel fills it, then the CUDA-core GEMM kernel
// consumes it.  All calls on one device share that one array: it still holds the previous call's
// data when the next call starts (every element the GEMM reads is rewritten first, so nothing has
// to be cleared), and two calls that overlap on the GPU -- different streams, or different host
// threads -- would overwrite each other's copy.  Serialise them.
#include "ard_internal.h"

namespace {

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress; device
// code could name it directly, host code must never pass it to a kernel as if it were an address.
static __device__ __align__(256) unsigned char g_static_scratch[ARD_STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
void* g_scratch_addr[MAX_DEVICES] = {};  // device address of g_static_scratch, per device

// dst[r][j] = src[r][b-1 + j*dp] for j < n_keep: the kept columns of a row pattern (Sec. 3.1, Eq. 1),
// written densely.  `dst` is the static scratch array.
template <typename T>
__global__ void __launch_bounds__(256)
gather_into_static_scratch_kernel(const int32_t* hdr, const T* src, int ld_src,
                                  T* dst, int ld_dst, int rows) {
  const int n_keep = hdr[HDR_NKEEP], dp = hdr[HDR_DP], bb = hdr[HDR_B] - 1;
  for (long long e = (long long)blockIdx.x * 256 + threadIdx.x; e < (long long)rows * n_keep;
       e += (long long)gridDim.x * 256) {
    const int r = (int)(e / n_keep), j = (int)(e % n_keep);
    dst[(size_t)r * ld_dst + j] = src[(size_t)r * ld_src + bb + (size_t)j * dp];
  }
}

}  // namespace

extern "C" ard_status ard_bwd_data_static_scratch(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, int B, int K,
                                                  int N, float alpha, const void* dY, int lddy, const void* W,
                                                  int ldw, void* dX, int lddx, void* cuda_stream) {
  if (!ctx || !pat || pat->ctx != ctx || !dY || !W || !dX) return ARD_ERR_INVALID_ARG;
  if (dtype != ARD_F32 && dtype != ARD_BF16) return ARD_ERR_INVALID_ARG;
  if (pat->kind != ARD_ROW) return ARD_ERR_UNSUPPORTED;
  if (B < 0 || K != pat->K_dim || N != pat->N_dim) return ARD_ERR_SHAPE;
  if (lddy < N || ldw < K || lddx < K) return ARD_ERR_SHAPE;
  if (B > 65535 * 32) return ARD_ERR_UNSUPPORTED;
  if (ctx->device < 0 || ctx->device >= MAX_DEVICES) return ARD_ERR_UNSUPPORTED;
  const size_t es = dtype == ARD_F32 ? 4 : 2;
  // Worst case is the dense pattern: all N columns are kept.
  if ((size_t)B * (size_t)N * es > (size_t)ARD_STATIC_SCRATCH_BYTES) return ARD_ERR_NOMEM;
  if (B == 0) return ARD_OK;

  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess || cudaSetDevice(ctx->device) != cudaSuccess) return ARD_ERR_CUDA;
  ard_status st = ARD_OK;
  // Set-up, once per device and with that device current: ask the runtime where this device's copy
  // of the array lives.
  if (g_scratch_addr[ctx->device] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) st = ARD_ERR_CUDA;
    else g_scratch_addr[ctx->device] = p;
  }
  if (st == ARD_OK) {
    void* scratch = g_scratch_addr[ctx->device];
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const int ldc = N;
    const long long total = (long long)B * N;
    int blocks = (int)((total + 255) / 256 < (long long)ctx->sm_count * 16 ? (total + 255) / 256
                                                                            : (long long)ctx->sm_count * 16);
    if (blocks < 1) blocks = 1;
    if (dtype == ARD_F32)
      gather_into_static_scratch_kernel<float><<<blocks, 256, 0, s>>>(pat->d_hdr, (const float*)dY, lddy,
                                                                     (float*)scratch, ldc, B);
    else
      gather_into_static_scratch_kernel<uint16_t><<<blocks, 256, 0, s>>>(pat->d_hdr, (const uint16_t*)dY, lddy,
                                                                        (uint16_t*)scratch, ldc, B);
    ctx->launches++;
    if (cudaGetLastError() != cudaSuccess) st = ARD_ERR_CUDA;
    if (st == ARD_OK) {
      GemmArgs g = {};
      g.hdr = pat->d_hdr;
      g.idx = pat->d_idx;
      g.col_ptr = g.col_idx = g.row_ptr = g.row_idx = nullptr;
      g.B = B; g.K = K; g.N = N;
      g.alpha = alpha;
      g.A0 = scratch; g.lda0 = ldc;   // compact dY
      g.A1 = W; g.lda1 = ldw;
      g.out = dX; g.ldo = lddx;
      g.flag0 = 1;                    // columns are already compact
      g.flag1 = 0;
      g.out_is_f32 = dtype == ARD_F32;
      g.accumulate = 0;
      g.status = ctx->d_status;
      st = launch_gemm_cc(ctx, ARD_ROW, OP_BWD_DATA, dtype, g, 0, s);
    }
  }
  cudaSetDevice(prev);
  return st;
}
