// Device-side pattern sampler (Sec. 3.4) and kept-unit list emitter (Sec. 3.1 Eq. 1, Sec. 3.2).
//
// One CTA per call.  Thread 0 runs Philox4x32-10 on the (seed, iteration, stream) counter, picks
// the period dp from the integer cumulative table of K and the bias b uniformly from {1..dp};
// all threads then write the header and the lists the GEMM kernels read.  Nothing returns to the
// host, so the GEMMs that follow on the same stream need no synchronisation.
#include "ard_internal.h"
#include "philox.h"

namespace {

constexpr int SAMPLER_THREADS = 1024;  // tile patterns; row patterns launch 256 (fewer lists to fill)
constexpr int SCAN_CAP = 2048;  // tile-columns whose running count fits in shared memory

__global__ void __launch_bounds__(SAMPLER_THREADS)
ard_sample_kernel(int32_t* __restrict__ hdr, int32_t* __restrict__ idx, int32_t* __restrict__ col_ptr,
                  int32_t* __restrict__ col_idx, int32_t* __restrict__ row_ptr, int32_t* __restrict__ row_idx,
                  const unsigned long long* __restrict__ cdf, int ndp, unsigned long long seed,
                  unsigned long long iteration, uint32_t stream_id, int forced_dp, int forced_b, int kind,
                  int units, int Tr, int Tc, int ts, unsigned long long* __restrict__ counter, int advance) {
  __shared__ int s_dp, s_b;
  const int nthreads = (int)blockDim.x;
  __shared__ unsigned long long s_cdf[64];
  pdl_launch_dependents();
  pdl_wait_prior_grids();  // earlier kernels may still be reading the lists this kernel rewrites
  // The cumulative table is searched by one thread; short tables are fetched by all threads at once first,
  // so that the search does not pay one global-memory round trip per probe.
  const bool cdf_smem = forced_dp <= 0 && ndp <= 64;
  if (cdf_smem && (int)threadIdx.x < ndp) s_cdf[threadIdx.x] = cdf[threadIdx.x];
  __syncthreads();
  if (threadIdx.x == 0) {
    int dp, b;
    if (forced_dp > 0) {
      dp = forced_dp;
      b = forced_b;
    } else {
      // A device-resident counter lets a captured graph draw a fresh pattern at every replay.
      if (counter != nullptr) {
        const unsigned long long n = *counter;
        iteration += n;
        if (advance) *counter = n + 1ull;
      }
      uint32_t c[4] = {(uint32_t)iteration, (uint32_t)(iteration >> 32), stream_id, 0u};
      philox4x32_10(c, (uint32_t)seed, (uint32_t)(seed >> 32));
      // dp = smallest i with r0 < c_i; the table is non-decreasing and ends at 2^32.
      int lo = 0, hi = ndp - 1;  // answer index in [0, ndp-1]
      const unsigned long long r0 = c[0];
      while (lo < hi) {
        int mid = (lo + hi) >> 1;
        const unsigned long long cm = cdf_smem ? s_cdf[mid] : cdf[mid];
        if (r0 < cm) hi = mid; else lo = mid + 1;
      }
      dp = lo + 1;
      b = 1 + (int)(((unsigned long long)c[1] * (unsigned long long)dp) >> 32);
    }
    s_dp = dp;
    s_b = b;
  }
  __syncthreads();
  const int dp = s_dp, b = s_b;
  const int n_keep = (units - b) / dp + 1;
  if (threadIdx.x == 0) {
    hdr[HDR_KIND] = kind;
    hdr[HDR_DP] = dp;
    hdr[HDR_B] = b;
    hdr[HDR_NKEEP] = n_keep;
    hdr[HDR_UNITS] = units;
    hdr[HDR_TR] = Tr;
    hdr[HDR_TC] = Tc;
    hdr[HDR_TS] = ts;
    hdr[HDR_MAPIDX] = dp * (dp - 1) / 2 + (b - 1);
  }
  // Eq. 1 on the 1-based unit index i = b + j*dp  ->  0-based b-1 + j*dp, ascending.
  for (int j = threadIdx.x; j < n_keep; j += nthreads) idx[j] = b - 1 + j * dp;
  if (kind != ARD_TILE) return;

  // Tiles are numbered row-major, so the ascending list is already grouped by tile-row.
  for (int j = threadIdx.x; j < n_keep; j += nthreads) row_idx[j] = (b - 1 + j * dp) % Tc;
  for (int r = threadIdx.x; r <= Tr; r += nthreads) {
    // kept tiles with 0-based linear index < r*Tc
    const long long lim = (long long)r * Tc;  // count of j with b-1 + j*dp < lim
    int cnt = 0;
    if (lim > b - 1) cnt = (int)((lim - 1 - (b - 1)) / dp) + 1;
    row_ptr[r] = cnt;
  }
  // Group by tile-column: count, prefix-sum, fill.  A warp takes a column at a time with its lanes across
  // the tile-rows, so a column costs Tr/32 ballots instead of a serial walk; the running sum over the
  // columns lives in shared memory when the grid is narrow enough (a dependent chain through global
  // memory would cost a round trip per column).
  __shared__ int s_cnt[SCAN_CAP];
  const bool in_smem = Tc <= SCAN_CAP;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = nthreads / 32;
  auto kept = [&](int r, int c) {
    const int lin = r * Tc + c - (b - 1);
    return r < Tr && lin >= 0 && lin % dp == 0;
  };
  for (int c = warp; c < Tc; c += nwarps) {
    int cnt = 0;
    for (int r0 = 0; r0 < Tr; r0 += 32) cnt += __popc(__ballot_sync(0xffffffffu, kept(r0 + lane, c)));
    if (lane == 0) { if (in_smem) s_cnt[c] = cnt; else col_ptr[c + 1] = cnt; }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    if (in_smem) {
      for (int c = 0; c < Tc; ++c) { const int n = s_cnt[c]; s_cnt[c] = run; run += n; }
    } else {
      col_ptr[0] = 0;
      for (int c = 0; c < Tc; ++c) { run += col_ptr[c + 1]; col_ptr[c + 1] = run; }
    }
  }
  __syncthreads();
  if (in_smem) {
    for (int c = threadIdx.x; c < Tc; c += nthreads) col_ptr[c] = s_cnt[c];
    if (threadIdx.x == 0) col_ptr[Tc] = n_keep;
  }
  for (int c = warp; c < Tc; c += nwarps) {
    int o = in_smem ? s_cnt[c] : col_ptr[c];
    for (int r0 = 0; r0 < Tr; r0 += 32) {
      const bool k = kept(r0 + lane, c);
      const unsigned m = __ballot_sync(0xffffffffu, k);
      if (k) col_idx[o + __popc(m & ((1u << lane) - 1u))] = r0 + lane;  // ascending rows
      o += __popc(m);
    }
  }
}

}  // namespace

ard_status launch_sampler(ard_ctx* ctx, ard_pattern* pat, const unsigned long long* d_cdf, int ndp, uint64_t seed,
                          uint64_t iteration, uint32_t stream_id, int forced_dp, int forced_b, cudaStream_t s,
                          unsigned long long* d_counter, int advance) {
  ARD_CUDA_OK(ard_launch(ctx, ard_sample_kernel, dim3(1), dim3(pat->kind == ARD_TILE ? SAMPLER_THREADS : 256), 0, s, pat->d_hdr, pat->d_idx,
                         pat->d_col_ptr, pat->d_col_idx, pat->d_row_ptr, pat->d_row_idx, d_cdf, ndp,
                         (unsigned long long)seed, (unsigned long long)iteration, stream_id, forced_dp, forced_b,
                         (int)pat->kind, pat->units, pat->Tr, pat->Tc, pat->ts, d_counter, advance));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}
