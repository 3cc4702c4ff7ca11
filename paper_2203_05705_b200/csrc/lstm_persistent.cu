// Whole-sequence LSTM forward in one cooperative kernel (Sec. 7: the LSTM layer under a row pattern on
// its hidden units; one pattern serves every time step).
//
// The per-step path launches a gate product and a cell kernel per time step, and each launch costs
// more than the 64-row product itself.  Here the recurrence runs inside one kernel:
//   - the input half of the gate pre-activations does not depend on the recurrence: the caller computes
//     x_t . W_x for all steps with one large product beforehand and leaves it where the gate activations
//     of step t will be stored; the kernel adds it in its epilogue and handles the recurrent half only
//     (it can also take the whole [x_t, h_{t-1}] row, at the price of a larger resident slice);
//   - every CTA owns 8 kept hidden units, i.e. 32 gate columns (i|f|g|o x 8), and loads its slice of
//     the weight, [32 rows][H] bf16, into shared memory once (TMA, rows b-1 + j*dp of each gate block
//     through the same strided descriptors the forward product uses);
//   - per step it loads its contraction columns of [x_t, h_{t-1}] (64-row TMA boxes of 64 columns) into a
//     buffer that holds all of them at once; the lanes of the producer warp issue one box each, so all
//     loads of a step are in flight together (one thread issuing box after box, with a barrier hand-off
//     per box, was measured at ~410 SM cycles per box, which paced the whole step); the boxes arrive on
//     four barriers, so the MMAs of the first quarter start while the rest is in flight; it multiplies
//     the row with the
//     resident slice (tcgen05.mma, M = 128, N = 32, accumulator in tensor memory, double-buffered over
//     steps);
//   - four warps move the accumulator rows to shared memory, then all 14 compute warps apply the cell
//     update to the (batch row, unit) pairs, keep c in registers, and write h_t (bf16) into the operand
//     of step t+1 and, after signalling, c_t and the gate activations for BPTT;
//   - columns of x, if the kernel is given any, are loaded ahead; the h columns wait for the grid-wide
//     barrier that says h_{t-1} is complete;
//   - under a pattern (period > 1) the dropped units of h_{t-1} are exact zeros, so the contraction runs over
//     the kept units only: the cell update also writes h_t into a compact copy (column j = j-th kept unit, two
//     buffers in context scratch), which is the operand of step t+1, and the slice holds the kept fan-in
//     columns of the weight only.  Those stride the weight's contiguous dimension, which a TMA box cannot
//     follow, so the CTA gathers its slice with plain loads, once per sequence, straight into the swizzled
//     layout the MMA reads.  A step's loads and MMAs shrink with the kept count (forward of 35 steps, batch 64,
//     H = 1024: 218 -> 189 us at a period of 2, 204 -> 146 us at 8).
// The grid barrier is an arrival counter in global memory: after its stores and a fence each CTA adds 1,
// and the producer thread of each CTA polls for t * (number of CTAs with units) before it loads the
// h half of step t.  The launch is cooperative, so all CTAs are resident; every wait is bounded (2 s)
// and a CTA that gives up sets the status word, which the others poll, so the kernel always returns.
#include "ard_internal.h"
#include "sm100_ptx.h"

namespace {

constexpr int LP_UNITS = 8;                  // kept hidden units per CTA
constexpr int LP_N = 4 * LP_UNITS;           // gate columns per CTA
constexpr int LP_BK = 64;                    // contraction block: 64 bf16 = one 128-byte swizzle row
constexpr int LP_MAX_BLOCKS = 32;            // contraction blocks per step: one lane of the producer warp each
constexpr int LP_GROUPS = 4;                 // the blocks of a step arrive on this many barriers
constexpr int LP_ROW_BOX = 64 * LP_BK * 2;   // one TMA box of the activations: 64 batch rows x 64 columns
constexpr int LP_W_BLOCK = LP_N * LP_BK * 2; // one contraction block of the resident weight slice
constexpr int LP_THREADS = 512;              // warps 0-10 cell update (0-3 also read TMEM: lane quadrant = warp),
constexpr int LP_MATH = 352;                 //   warp 11 TMA producer, warps 12-15 MMA issuers (one per group)
constexpr int LP_ZS_LD = LP_N + 1;           // staged pre-activations: [128 rows][33] floats
constexpr int LP_ZS_BYTES = 128 * LP_ZS_LD * 4;
constexpr int LP_PAIRS_MAX = (128 * LP_UNITS + LP_MATH - 1) / LP_MATH;  // (row, unit) pairs per thread

struct LstmFwdParams {
  TcMap mapXH;    // [(T+1)*B][I+H], boxes of 64 rows x 64 columns (used as encoded)
  TcMap mapW[4];  // per gate: [H rows][I+H], boxes of 8 rows x 64 columns; specialised to the kept rows by the kernel
  TcMap mapHc;    // [2*B][ldhc]: the compact copies of h_{t-1} and h_t, boxes of 64 rows x 64 columns
  CUtensorMap* tm_slots;  // this launch's descriptor scratch: ARD_TM_LSTM_SLOTS slots per block
  const int32_t* hdr;
  int T, B, I, H;
  int kx0, klen;      // contraction columns [kx0, kx0 + klen) of [x | h] this kernel multiplies
  const __nv_bfloat16* W;  // the weight itself, [4H][ldw]: its kept recurrent columns are gathered by the kernel
  int ldw;
  __nv_bfloat16* Hc;  // two buffers [B][ldhc]: column j = the j-th kept unit (nullptr: no compact recurrence)
  int ldhc;
  int add_zx;         // the products of the other columns are waiting in G[t] (same layout as the gates)
  float alpha;
  __nv_bfloat16* XH;
  const float* bias;  // [4][H] or nullptr
  float* C;           // [T+1][B][H] compact
  float* G;           // [T][B][4H]: gate blocks of width H, compact inside a block
  unsigned int* bar;  // arrival counter, zero at launch
  int* status;
};

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Waits until the arrival counter reaches `target`.  Gives up after the time limit or when another CTA
// has already recorded a failure.
__device__ bool grid_wait(const unsigned int* bar, unsigned int target, volatile int* abort_flag, int* status) {
  if (ld_acquire_u32(bar) >= target) return true;
  const unsigned long long t0 = global_ns();
  for (int spin = 1;; ++spin) {
    if (ld_acquire_u32(bar) >= target) return true;
    if (*abort_flag) return false;
    if ((spin & 63) == 0) {
      if (*reinterpret_cast<volatile int*>(status) != 0) { *abort_flag = 1; return false; }
      if (global_ns() - t0 > WAIT_LIMIT_NS) {
        *abort_flag = 1;
        atomicMax(status, (int)ARD_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

__host__ __device__ inline bool lstm_fwd_zs_shared(int kx0, int I, int nkb, int a_block) {
  return kx0 >= I && nkb * a_block >= LP_ZS_BYTES;
}

__device__ __forceinline__ float sigmoid_fast(float x) { return 1.f / (1.f + __expf(-x)); }
__device__ __forceinline__ float tanh_fast(float x) { return 1.f - 2.f / (1.f + __expf(2.f * x)); }

__global__ void __launch_bounds__(LP_THREADS, 1) ard_lstm_forward_kernel(const __grid_constant__ LstmFwdParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw_addr);

  const int KH = p.I + p.H;
  int nkb = (p.klen + LP_BK - 1) / LP_BK;
  // The activation row buffer comes first and the weight slice right after it: a block holds one or two
  // 64-row boxes, the MMA always reads 128 rows, and for a batch of at most 64 rows the upper half of
  // what it reads is the next block (or the start of the weight slice); those accumulator rows are
  // never used.
  const int row_boxes = (p.B + 63) / 64;
  const uint32_t a_block = (uint32_t)row_boxes * LP_ROW_BOX;
  const uint32_t sA = base;
  const uint32_t sW = base + (uint32_t)nkb * a_block;         // nkb blocks of 4 KiB
  // The staged pre-activations share the start of the row buffer when every block of a step waits for the grid-wide
  // barrier (no x columns): they are written after the step's MMAs have completed and read before this CTA releases
  // h_t, and the next loads are issued only after every CTA has released.  Without them the kernel stays below
  // 196 KB of shared memory at H = 1024; one carve-out step higher (228 KB, next to no L1 left) this kernel was
  // measured 1.5 % slower and the BPTT kernel 4 %.
  const bool zs_shared = lstm_fwd_zs_shared(p.kx0, p.I, nkb, (int)a_block);
  float* zs = reinterpret_cast<float*>(zs_shared ? smem : smem + (sW - base) + (size_t)nkb * LP_W_BLOCK);
  const uint32_t bar_base = sW + (uint32_t)nkb * LP_W_BLOCK + (zs_shared ? 0 : LP_ZS_BYTES);  // gfull[4], tfull[2], tempty[2], wfull
  auto gfull_bar = [&](int g) { return bar_base + 8u * g; };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (LP_GROUPS + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (LP_GROUPS + 2 + a); };
  const uint32_t wfull_bar = bar_base + 8u * (LP_GROUPS + 4);
  const uint32_t hready_bar = bar_base + 8u * (LP_GROUPS + 5);  // h_{t-1} is complete (relayed from the grid barrier)
  uint8_t* misc = smem + (bar_base - base) + 8 * (LP_GROUPS + 6);
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);
  int gsz = (nkb + LP_GROUPS - 1) / LP_GROUPS;                // blocks per arrival group

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int g = 0; g < LP_GROUPS; ++g) mbar_init(gfull_bar(g), 1);
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), LP_GROUPS);  // one commit per MMA issuer
      mbar_init(tempty_bar(a), 4);         // one arrival per TMEM-reading warp
    }
    mbar_init(wfull_bar, 1);
    mbar_init(hready_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 15) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_ptr_smem)), 2 * LP_GROUPS * LP_N);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_smem;
  pdl_wait_prior_grids();

  const int dp = p.hdr[HDR_DP], bb = p.hdr[HDR_B] - 1, n_keep = p.hdr[HDR_NKEEP];
  const int n_active = (n_keep + LP_UNITS - 1) / LP_UNITS;  // CTAs that own units (the others only tear down)
  const int j0 = (int)blockIdx.x * LP_UNITS;                // first kept unit (compact index) of this CTA
  const bool active = (int)blockIdx.x < n_active;
  const int xblocks = p.I > p.kx0 ? (p.I - p.kx0) / LP_BK : 0;  // contraction blocks that hold only x columns
  // Under a pattern the dropped units of h_{t-1} are exact zeros (Sec. 3.1), so the recurrent contraction runs over
  // the kept units alone: the operand of a step is the compact copy of h_{t-1} (column j = j-th kept unit) that the
  // cell update writes beside the full-width one, and the weight slice holds the kept fan-in columns only.  Those
  // stride the weight's contiguous dimension, which no TMA box can follow, so the CTA gathers its slice itself,
  // once per sequence, straight into the swizzled layout the MMA reads.
  const bool compact = dp > 1 && p.Hc != nullptr && p.kx0 == p.I;
  const int hs = compact ? 1 : 0;  // the compact h_0 is made by the kernel: one more grid-wide hand-over, before step 0
  if (compact) {
    nkb = (n_keep + LP_BK - 1) / LP_BK;
    gsz = (nkb + LP_GROUPS - 1) / LP_GROUPS;
    if (active) {
      const int nchunks = nkb * 8;  // 16-byte pieces of a slice row
      for (int task = threadIdx.x; task < LP_N * nchunks; task += LP_THREADS) {
        const int r = task / nchunks, ch = task - r * nchunks;
        const int g = r >> 3, k = r & 7, j = j0 + k;
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        if (j < n_keep) {
          const __nv_bfloat16* src = p.W + ((size_t)g * p.H + bb + (size_t)j * dp) * p.ldw + p.I + bb + (size_t)ch * 8 * dp;
          uint32_t e[8];
#pragma unroll
          for (int q = 0; q < 8; ++q)
            e[q] = (ch * 8 + q < n_keep) ? (uint32_t)__ldg(reinterpret_cast<const unsigned short*>(src) + (size_t)q * dp) : 0u;
#pragma unroll
          for (int q = 0; q < 4; ++q) w[q] = e[2 * q] | (e[2 * q + 1] << 16);
        }
        // 128-byte swizzle: the 16-byte piece c of row k of an 8-row group sits at piece c ^ k
        uint8_t* dst = smem + (sW - base) + (size_t)(ch >> 3) * LP_W_BLOCK + g * (LP_UNITS * LP_BK * 2) + k * 128 + (((ch & 7) ^ k) << 4);
        *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
      }
      fence_proxy_async_smem();  // generic-proxy stores -> the tensor core's reads
    }
    __syncthreads();
  }

  if (active) {
    if (warp == 11) {
      // ===================== weight loader and barrier relay =====================
      // Loads the weight slice (lane = contraction block), then relays the grid barrier of every step to
      // the warps of this CTA through a shared-memory barrier.
      // The gates' weight descriptors become those of the kept rows (the weight area, still empty, is the work area).
      if (compact) {
        // the slice is in place already (gathered by the whole CTA above)
        if (lane == 0) mbar_arrive(wfull_bar);
      } else {
        CUtensorMap* slots = p.tm_slots + (size_t)blockIdx.x * ARD_TM_LSTM_SLOTS;
        const CUtensorMap* mapW[4];
#pragma unroll
        for (int g = 0; g < 4; ++g)
          mapW[g] = tensormap_specialise(&p.mapW[g], dp, bb + 1, n_keep, smem + (sW - base) + 128 * g, slots + g, lane);
        fence_proxy_async_smem();
        const int kb = lane;
        if (kb < nkb && dp > 1) {
#pragma unroll
          for (int g = 0; g < 4; ++g) tensormap_acquire(mapW[g]);
        }
        if (lane == 0) mbar_arrive_expect_tx(wfull_bar, (uint32_t)nkb * LP_W_BLOCK);
        __syncwarp();
        if (kb < nkb) {
#pragma unroll
          for (int g = 0; g < 4; ++g)
            tma_load_2d(sW + kb * LP_W_BLOCK + g * (LP_UNITS * LP_BK * 2), mapW[g], wfull_bar, p.kx0 + kb * LP_BK, j0);
        }
      }
      if (lane == 0) {
        for (int t = 1 - hs; t < p.T; ++t) {
          // h_{t-1} is complete when every CTA with units has arrived t times (once more with a compact h_0)
          if (!grid_wait(p.bar, (unsigned)(t + hs) * (unsigned)n_active, abort_flag, p.status)) break;
          mbar_arrive(hready_bar);
        }
      }
    } else if (warp >= 12) {
      // ===================== loaders and MMA issuers: warp 12 + g owns the contraction blocks of group g =====================
      // Lanes 0 .. gsz-1 issue one TMA box each (a single thread issuing box after box was measured at
      // ~410 cycles per box, and the lanes of ONE warp still issue one after the other, ~70 cycles each,
      // so the four groups are issued by four warps side by side).  Lane 0 then issues the MMAs of the
      // group: a tcgen05.mma this narrow (N = 32) costs ~110 cycles to issue whatever its shape, so one
      // thread issuing all 4 * nkb of a step would pace the step; the four warps issue their quarters side
      // by side into four accumulators, which the epilogue adds.
      const int g = warp - 12;
      const int kb0 = g * gsz, kb1 = min(nkb, kb0 + gsz);
      const int kb = kb0 + lane;
      const bool mine = kb < kb1;
      const CUtensorMap* mapXH = compact ? &p.mapHc.tm : &p.mapXH.tm;  // kernel parameters, used as encoded
      const uint32_t idesc = make_idesc(LP_N, false, false, 128);
      bool ok = (lane != 0) || mbar_wait(wfull_bar, 0u, abort_flag, p.status);
      for (int t = 0; t < p.T; ++t) {
        const int acc = t & 1;
        // this group's part of the row buffer is free once the MMAs of the previous step have completed
        if (ok && t > 0 && !mbar_wait(tfull_bar((t - 1) & 1), (uint32_t)((t - 1) >> 1) & 1u, abort_flag, p.status)) ok = false;
        if (!__all_sync(0xffffffffu, ok)) break;
        if (lane == 0 && kb0 < kb1) mbar_arrive_expect_tx(gfull_bar(g), (uint32_t)(kb1 - kb0) * a_block);
        __syncwarp();
        auto issue = [&]() {
          // full width: columns of [x_t | h_{t-1}], rows of step t; compact: the buffer that holds h_{t-1}
          const int x = compact ? kb * LP_BK : p.kx0 + kb * LP_BK, y = compact ? (t & 1) * p.B : t * p.B;
          for (int rb = 0; rb < row_boxes; ++rb)
            tma_load_2d(sA + kb * a_block + rb * LP_ROW_BOX, mapXH, gfull_bar(g), x, y + rb * 64);
        };
        if (mine && kb < xblocks) issue();  // columns of x do not depend on the recurrence
        if (t + hs > 0 && kb1 > xblocks) {
          // the other columns are h_{t-1}
          if (!mbar_wait(hready_bar, (uint32_t)(t - 1 + hs) & 1u, abort_flag, p.status)) ok = false;
          if (!__all_sync(0xffffffffu, ok)) break;
          asm volatile("fence.proxy.async.global;" ::: "memory");  // generic-proxy stores of other CTAs -> TMA reads
        }
        if (mine && kb >= xblocks) issue();
        if (lane == 0) {
          if (!mbar_wait(tempty_bar(acc), ((uint32_t)(t >> 1) & 1u) ^ 1u, abort_flag, p.status)) ok = false;
          if (ok && kb0 < kb1) {
            if (!mbar_wait(gfull_bar(g), (uint32_t)t & 1u, abort_flag, p.status)) ok = false;
            if (ok) {
              tc_fence_after();
              const uint32_t d_tmem = tmem_base + (uint32_t)((acc * LP_GROUPS + g) * LP_N);
              // descriptors by addition: the start-address field counts 16-byte units
              uint64_t ad = make_desc(sA + kb0 * a_block, 16, 1024), bd = make_desc(sW + kb0 * LP_W_BLOCK, 16, 1024);
              for (int k2 = kb0; k2 < kb1; ++k2, ad += a_block >> 4, bd += LP_W_BLOCK >> 4) {
#pragma unroll
                for (int s = 0; s < LP_BK / 16; ++s)
                  tc_mma_bf16(d_tmem, ad + 2 * s, bd + 2 * s, idesc, (k2 != kb0 || s != 0) ? 1u : 0u);
              }
            }
          }
          if (ok) tc_commit(tfull_bar(acc));  // this quarter is complete; with all four, the row buffer may be overwritten
        }
        __syncwarp();
      }
    } else {
      // ===================== cell update (warps 0-10) =====================
      const int tid = threadIdx.x;  // 0 .. LP_MATH-1
      const size_t ldxh = (size_t)KH;
      const int npairs = p.B * LP_UNITS;            // (batch row, unit) pairs of this CTA; pair q = row * 8 + k
      const int nvalid = min(LP_UNITS, n_keep - j0);  // units this CTA really owns (>= 1)
      float creg[LP_PAIRS_MAX];
#pragma unroll
      for (int i = 0; i < LP_PAIRS_MAX; ++i) {
        const int q = tid + i * LP_MATH;
        const int row = q >> 3, k = q & 7;
        creg[i] = (q < npairs && k < nvalid) ? p.C[(size_t)row * p.H + j0 + k] : 0.f;
      }
      if (compact) {
        // the compact copy of h_0 (buffer 0): this CTA's units of every row; the last CTA with units also clears
        // the columns up to the next multiple of 64 in both buffers (they meet the zeros of the weight slice)
        for (int q = tid; q < npairs; q += LP_MATH) {
          const int row = q >> 3, k = q & 7;
          if (k < nvalid) p.Hc[(size_t)row * p.ldhc + j0 + k] = p.XH[(size_t)row * ldxh + p.I + bb + (size_t)(j0 + k) * dp];
        }
        if ((int)blockIdx.x == n_active - 1) {
          const int npad = nkb * LP_BK - n_keep;
          for (int q = tid; q < 2 * p.B * npad; q += LP_MATH) {
            const int row = q / npad, c = q - row * npad;
            p.Hc[(size_t)row * p.ldhc + n_keep + c] = __float2bfloat16_rn(0.f);
          }
        }
        asm volatile("bar.sync 1, 352;" ::: "memory");
        if (tid == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.bar) : "memory");
      }
      bool ok = true;
      for (int t = 0; t < p.T && ok; ++t) {
        const int acc = t & 1;
        // what does not depend on the recurrence is fetched before the wait: x_t . W_x and the bias
        float zadd[LP_PAIRS_MAX][4];
#pragma unroll
        for (int i = 0; i < LP_PAIRS_MAX; ++i) {
          const int q = tid + i * LP_MATH;
          const int row = q >> 3, k = q & 7;
          zadd[i][0] = zadd[i][1] = zadd[i][2] = zadd[i][3] = 0.f;
          if (q < npairs && k < nvalid) {
            if (p.add_zx) {  // left in the slot of this step's gate activations
              const float* zx = p.G + ((size_t)t * p.B + row) * 4 * p.H + j0 + k;
#pragma unroll
              for (int g = 0; g < 4; ++g) zadd[i][g] = __ldcg(zx + (size_t)g * p.H);
            }
            if (p.bias) {
              const int u = bb + (j0 + k) * dp;
#pragma unroll
              for (int g = 0; g < 4; ++g) zadd[i][g] += p.bias[g * p.H + u];
            }
          }
        }
        if (warp < 4) {
          // accumulator rows -> shared memory
          if (!mbar_wait(tfull_bar(acc), (uint32_t)(t >> 1) & 1u, abort_flag, p.status)) ok = false;
          if (ok) {
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(acc * LP_GROUPS * LP_N);
            const int ngroups = (nkb + gsz - 1) / gsz;  // accumulators that received MMAs
            uint32_t z[32], y[32];
            tmem_ld32(t_row, z);
            tmem_ld_wait();
            for (int c = 1; c < ngroups; ++c) {
              tmem_ld32(t_row + (uint32_t)(c * LP_N), y);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; ++i) z[i] = __float_as_uint(__uint_as_float(z[i]) + __uint_as_float(y[i]));
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));  // the accumulator is in registers now
            const int r = warp * 32 + lane;
            if (r < p.B) {
#pragma unroll
              for (int i = 0; i < 32; ++i) zs[r * LP_ZS_LD + i] = __uint_as_float(z[i]);
            }
          }
        }
        // every compute thread learns about a failed wait through the flag in shared memory
        asm volatile("bar.sync 2, 352;" ::: "memory");
        if (*abort_flag) { ok = false; break; }
        // Cell update (Sec. 7).  h first, because the other CTAs wait for it; c_t and the gate
        // activations, which only BPTT reads, after the CTA has signalled.
        float gi[LP_PAIRS_MAX], gf[LP_PAIRS_MAX], gg[LP_PAIRS_MAX], go[LP_PAIRS_MAX];
#pragma unroll
        for (int i = 0; i < LP_PAIRS_MAX; ++i) {
          const int q = tid + i * LP_MATH;
          const int row = q >> 3, k = q & 7;
          if (q < npairs && k < nvalid) {
            const int u = bb + (j0 + k) * dp;
            const float* zr = zs + row * LP_ZS_LD;
            const float zi = zr[k] + zadd[i][0], zf = zr[LP_UNITS + k] + zadd[i][1];
            const float zg = zr[2 * LP_UNITS + k] + zadd[i][2], zo = zr[3 * LP_UNITS + k] + zadd[i][3];
            gi[i] = sigmoid_fast(zi);
            gf[i] = sigmoid_fast(zf);
            gg[i] = tanh_fast(zg);
            go[i] = sigmoid_fast(zo);
            creg[i] = gf[i] * creg[i] + gi[i] * gg[i];
            const __nv_bfloat16 h = __float2bfloat16_rn(p.alpha * go[i] * tanh_fast(creg[i]));
            p.XH[((size_t)(t + 1) * p.B + row) * ldxh + p.I + u] = h;
            if (compact) p.Hc[((size_t)((t + 1) & 1) * p.B + row) * p.ldhc + j0 + k] = h;
          }
        }
        // publish h_t: all stores of the CTA, then one release-add for the CTA (the staged sums may lie in the row
        // buffer, which the TMA unit overwrites next: generic-proxy accesses first)
        fence_proxy_async_smem();
        asm volatile("bar.sync 1, 352;" ::: "memory");
        if (tid == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.bar) : "memory");
#pragma unroll
        for (int i = 0; i < LP_PAIRS_MAX; ++i) {
          const int q = tid + i * LP_MATH;
          const int row = q >> 3, k = q & 7;
          if (q < npairs && k < nvalid) {
            p.C[((size_t)(t + 1) * p.B + row) * p.H + j0 + k] = creg[i];
            float* g_out = p.G + ((size_t)t * p.B + row) * 4 * p.H + j0 + k;
            g_out[0] = gi[i];
            g_out[p.H] = gf[i];
            g_out[2 * p.H] = gg[i];
            g_out[3 * p.H] = go[i];
          }
        }
      }
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncwarp();  // lanes that left their role's loop one by one arrive at the block-wide barrier together
  __syncthreads();
  if (warp == 15) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 2 * LP_GROUPS * LP_N);
  }
}


// ======================================================================================================
// Whole-sequence BPTT recurrence (Sec. 7), the counterpart of the kernel above.
//
// Per step t = T-1 .. 0 the recurrence needs  dh_t = upstream_t + dz_{t+1} . W_h  (contraction over the
// 4 * n_keep kept gate rows, output over the hidden units), then the cell adjoint gives dz_t.  Every SM
// would need all of dz_{t+1} if the output units were simply dealt out, so the product is cut both ways:
// CTA (s, r) owns the 64 hidden-unit COLUMNS 64 s .. 64 s + 63 of the recurrent weight (all of them, kept
// or not: the columns of a kept-unit set are strided and cannot be boxed) and the r-th eighth of the
// contraction blocks; its slice of the weight (at most 8 boxes of 64 gate rows x 64 columns, MN-major B
// operand straight from the neuron-major weight) stays in shared memory for the whole sequence.  A step is
//   A. wait until dz_{t+1} is complete (grid barrier), TMA-load this CTA's blocks of it, multiply
//      (tcgen05.mma M = 128, N = 64, four issuing warps with an accumulator each), park the 64-column
//      partial sums in global memory, arrive;
//   B. wait until all partial sums are there (grid barrier); the threads that own a kept unit among this
//      CTA's 8 columns 64 s + 8 r .. + 7 add the 8 partial sums in a fixed order, add the upstream gradient,
//      store the total (the caller's D holds it afterwards), apply the cell adjoint with dc in a register,
//      store dz_t (bf16, the operand of the next step and of the weight-gradient products), arrive.
// After t = 0 one more product gives the gradient of h_0.  The input half of d[x, h] and the weight
// gradient are large products over all T*B rows that the caller runs afterwards.
// Grid barriers are phases of one arrival counter: every CTA arrives exactly once per phase and only
// after it has passed the previous phase, so the count p * (number of CTAs) identifies phase p.
constexpr int LB_COLS = 64;    // weight columns (hidden units, kept or not) per CTA
constexpr int LB_KPARTS = 8;   // CTAs sharing the contraction of one column slice
constexpr int LB_OWN = LB_COLS / LB_KPARTS;  // columns whose cell adjoint this CTA computes
constexpr int LB_MAX_BLOCKS = 8;             // contraction blocks of one CTA (64 gate rows each)
constexpr int LB_W_BLOCK = 64 * LB_COLS * 2; // one resident weight box
constexpr int LB_THREADS = 512;              // warps 0-10 adjoint (0-3 also read TMEM), 11 relay, 12-15 load + MMA
constexpr int LB_MATH = 352;
constexpr int LB_PAIRS_MAX = (128 * LB_OWN + LB_MATH - 1) / LB_MATH;
// Few kept units (all contraction blocks of a step fit the row buffer): the cut along the contraction is dropped.
// A CTA owns LC_UNITS KEPT units, holds their fan-out weights over all 4 * n_keep kept gate rows (gathered by the
// kernel, K-major) and contracts the whole of dz_{t+1} itself: one grid-wide barrier per step instead of two, no
// partial sums through global memory.
constexpr int LC_UNITS = 8;                    // kept units per CTA
constexpr int LC_N = 16;                       // MMA width (the instruction's minimum at 128 rows): units 8-15 are zeros
constexpr int LC_W_BLOCK = LC_N * LP_BK * 2;   // one contraction block of the resident weight slice
constexpr int LC_ZS_LD = LC_UNITS + 1;         // staged recurrent sums: [128 rows][9] floats
constexpr int LC_ZS_BYTES = 128 * LC_ZS_LD * 4;
constexpr int LB_BAR_BYTES = 1024;             // barriers and flags at the start of shared memory
constexpr int LB_SMEM_BYTES = 227 * 1024;      // the kernel always asks for all of it (one CTA per SM anyway)
static_assert(LC_UNITS == LB_OWN, "both forms give a thread the same number of (row, unit) pairs");

struct LstmBwdParams {
  TcMap mapDZ[4];  // per gate: [T*B rows][H columns], boxes 64 x 64; the kernel limits them to the n_keep compact columns
  TcMap mapW[4];   // per gate: [H rows][I+H columns], boxes 64 x 64; the kernel turns them into the kept rows
  CUtensorMap* tm_slots;  // this launch's descriptor scratch: ARD_TM_LSTM_SLOTS slots per block
  const int32_t* hdr;
  int T, B, I, H;
  float alpha;
  const float* C;        // [T+1][B][H] compact
  const float* G;        // [T][B][4H]
  const float* dH_last;  // [B][H] full width
  float* D;              // [T][B][I+H]
  float* dc;             // [B][H] compact, in/out
  __nv_bfloat16* DZ;     // [T][B][4H]: gate blocks of width H, compact inside a block
  float* partial;        // [CTA][128][64]
  unsigned int* bar;
  int* status;
  const __nv_bfloat16* W;  // the weight itself, [4H][ldw] (the compact form gathers its slice from it)
  int ldw;
  int compact_ok;          // the compact form may be used when the drawn pattern allows it
  int smem_bytes;          // dynamic shared memory of this launch
};

__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
}

// The compact form of the BPTT recurrence (see LC_UNITS).  Barriers gfull[4], tfull and hready of the caller's set.
__device__ __forceinline__ void lstm_backward_compact(const LstmBwdParams& p, uint8_t* smem, uint32_t base, uint32_t bar_base,
                                                      uint32_t tmem_base, volatile int* abort_flag, int dp, int bb,
                                                      int n_keep) {
  auto gfull_bar = [&](int g) { return bar_base + 8u * g; };
  const uint32_t tfull_bar = bar_base + 8u * LP_GROUPS;
  const uint32_t hready_bar = bar_base + 8u * (LP_GROUPS + 2);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KH = p.I + p.H, T = p.T;
  const int row_boxes = (p.B + 63) / 64;
  const uint32_t a_block = (uint32_t)row_boxes * LP_ROW_BOX;
  const int nb = (n_keep + 63) / 64;                  // contraction blocks per gate
  const int nblk = 4 * nb;                            // ... per step; block = gate * nb + jb
  const int gsz = (nblk + LP_GROUPS - 1) / LP_GROUPS; // blocks per loader / MMA warp
  const int n_active = (n_keep + LC_UNITS - 1) / LC_UNITS;
  const bool active = (int)blockIdx.x < n_active;
  const int j0 = (int)blockIdx.x * LC_UNITS;          // first kept unit (compact index) of this CTA
  const uint32_t sA = base + LB_BAR_BYTES;            // the blocks of dz_{t+1}
  const uint32_t sW = sA + (uint32_t)nblk * a_block;  // the weight slice
  float* zs = reinterpret_cast<float*>(smem + (sW - base) + (size_t)nblk * LC_W_BLOCK);

  if (active) {
    // Weight slice, K-major: row r = unit j0 + r, column (gate, i) = W[gate * H + keep[i]][I + keep[j0 + r]], in the
    // 128-byte swizzle (16-byte piece c of row r of an 8-row group sits at piece c ^ r); rows 8-15 and what lies
    // beyond the kept counts are zeros.
    for (int task = threadIdx.x; task < nblk * LC_N * 8; task += LB_THREADS) {
      const int kb = task >> 7, r = (task >> 3) & 15, c = task & 7;
      const int g = kb / nb, jb = kb - g * nb;
      uint32_t w[4] = {0u, 0u, 0u, 0u};
      if (r < LC_UNITS && j0 + r < n_keep) {
        const int i0 = jb * 64 + c * 8;
        const unsigned short* src = reinterpret_cast<const unsigned short*>(p.W) +
                                    ((size_t)g * p.H + bb + (size_t)i0 * dp) * p.ldw + p.I + bb + (size_t)(j0 + r) * dp;
        uint32_t e[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) e[q] = (i0 + q < n_keep) ? (uint32_t)__ldg(src + (size_t)q * dp * p.ldw) : 0u;
#pragma unroll
        for (int q = 0; q < 4; ++q) w[q] = e[2 * q] | (e[2 * q + 1] << 16);
      }
      uint8_t* dst = smem + (sW - base) + (size_t)kb * LC_W_BLOCK + (r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4);
      *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    fence_proxy_async_smem();  // generic-proxy stores -> the tensor core's reads
  }
  __syncthreads();
  if (!active) return;

  CUtensorMap* slots = p.tm_slots + (size_t)blockIdx.x * ARD_TM_LSTM_SLOTS;
  if (warp == 11) {
    // ===================== descriptors of the compact gradient columns, barrier relay =====================
#pragma unroll
    for (int g = 0; g < 4; ++g)
      tensormap_specialise(&p.mapDZ[g], dp, bb + 1, n_keep, reinterpret_cast<uint8_t*>(zs) + 128 * g, slots + 4 + g, lane);
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
      for (int ph = 1; ph <= T; ++ph) {
        // dz of time index T - ph is complete when every CTA with units has arrived ph times
        if (!grid_wait(p.bar, (unsigned)ph * (unsigned)n_active, abort_flag, p.status)) break;
        mbar_arrive(hready_bar);
      }
    }
  } else if (warp >= 12) {
    // ===================== loaders and MMA issuers (group g4 = warp - 12) =====================
    const int g4 = warp - 12;
    const int kb0 = g4 * gsz, kb1 = min(nblk, kb0 + gsz);
    const int kb = kb0 + lane;
    const bool mine = kb < kb1;
    int gate = 0, jb = 0;
    if (mine) {
      gate = kb / nb;
      jb = kb - gate * nb;
    }
    const CUtensorMap* mdz = slots + 4 + gate;
    const uint32_t idesc = make_idesc(LC_N, false, false, 128);
    bool ok = true;
    for (int k = 1; k <= T; ++k) {
      if (ok && !mbar_wait(hready_bar, (uint32_t)(k - 1) & 1u, abort_flag, p.status)) ok = false;
      if (!__all_sync(0xffffffffu, ok)) break;
      if (k == 1 && mine) tensormap_acquire(mdz);  // written by warp 11 ahead of its first arrival on hready_bar
      if (kb0 < kb1) {
        asm volatile("fence.proxy.async.global;" ::: "memory");  // generic-proxy stores of other CTAs -> TMA reads
        if (lane == 0) mbar_arrive_expect_tx(gfull_bar(g4), (uint32_t)(kb1 - kb0) * a_block);
        __syncwarp();
        if (mine)
          for (int rb = 0; rb < row_boxes; ++rb)
            tma_load_2d(sA + kb * a_block + rb * LP_ROW_BOX, mdz, gfull_bar(g4), jb * 64, (T - k) * p.B + rb * 64);
        if (lane == 0) {
          if (!mbar_wait(gfull_bar(g4), (uint32_t)(k - 1) & 1u, abort_flag, p.status)) ok = false;
          if (ok) {
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(g4 * LB_COLS);
            uint64_t ad = make_desc(sA + kb0 * a_block, 16, 1024), bd = make_desc(sW + kb0 * LC_W_BLOCK, 16, 1024);
            for (int k2 = kb0; k2 < kb1; ++k2, ad += a_block >> 4, bd += LC_W_BLOCK >> 4) {
#pragma unroll
              for (int s = 0; s < LP_BK / 16; ++s)
                tc_mma_bf16(d_tmem, ad + 2 * s, bd + 2 * s, idesc, (k2 != kb0 || s != 0) ? 1u : 0u);
            }
          }
        }
      }
      if (lane == 0 && ok) {
        if (kb0 < kb1) tc_commit(tfull_bar);
        else mbar_arrive(tfull_bar);
      }
      __syncwarp();
    }
  } else {
    // ===================== recurrent sums and cell adjoint (warps 0-10) =====================
    const int tid = threadIdx.x;
    const int npairs = p.B * LC_UNITS;  // (batch row, owned unit) pairs; pair q = row * 8 + kk
    const size_t ldd = (size_t)KH;
    float dcreg[LB_PAIRS_MAX];
    int jj[LB_PAIRS_MAX];  // kept index of the pair's unit, -1 beyond the kept count or the batch
#pragma unroll
    for (int i = 0; i < LB_PAIRS_MAX; ++i) {
      const int q = tid + i * LB_MATH;
      const int row = q >> 3, j = j0 + (q & 7);
      jj[i] = (q < npairs && j < n_keep) ? j : -1;
      dcreg[i] = jj[i] >= 0 ? p.dc[(size_t)row * p.H + j] : 0.f;
    }
    bool ok = true;
    for (int k = 0; k <= T && ok; ++k) {
      const int t = T - 1 - k;  // time index whose dh is formed in this round (-1: the gradient of h_0)
      float pg[LB_PAIRS_MAX][6], ups[LB_PAIRS_MAX];
#pragma unroll
      for (int i = 0; i < LB_PAIRS_MAX; ++i) {
        ups[i] = 0.f;
        if (jj[i] >= 0 && t >= 0) {
          const int row = (tid + i * LB_MATH) >> 3, j = jj[i], u = bb + j * dp;
          const float* gs = p.G + ((size_t)t * p.B + row) * 4 * p.H + j;
          pg[i][0] = __ldcg(gs);
          pg[i][1] = __ldcg(gs + p.H);
          pg[i][2] = __ldcg(gs + 2 * p.H);
          pg[i][3] = __ldcg(gs + 3 * p.H);
          pg[i][4] = __ldcg(p.C + ((size_t)t * p.B + row) * p.H + j);
          pg[i][5] = __ldcg(p.C + ((size_t)(t + 1) * p.B + row) * p.H + j);
          ups[i] = (t == T - 1) ? p.dH_last[(size_t)row * p.H + u]
                                : __ldcg(p.D + ((size_t)(t + 1) * p.B + row) * ldd + p.I + u);
        }
      }
      if (k >= 1) {
        if (warp < 4) {
          if (!mbar_wait(tfull_bar, (uint32_t)(k - 1) & 1u, abort_flag, p.status)) ok = false;
          if (ok) {
            tc_fence_after();
            const int row = warp * 32 + lane;
            const uint32_t t_row = tmem_base + ((uint32_t)(warp * 32) << 16);
            const int ngroups = (nblk + gsz - 1) / gsz;
            uint32_t z[8], y[8];
            tmem_ld8(t_row, z);
            tmem_ld_wait();
            for (int c = 1; c < ngroups; ++c) {
              tmem_ld8(t_row + (uint32_t)(c * LB_COLS), y);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 8; ++i) z[i] = __float_as_uint(__uint_as_float(z[i]) + __uint_as_float(y[i]));
            }
            tc_fence_before();
#pragma unroll
            for (int i = 0; i < 8; ++i) zs[row * LC_ZS_LD + i] = __uint_as_float(z[i]);
          }
        }
        asm volatile("bar.sync 2, 352;" ::: "memory");
        if (*abort_flag) { ok = false; break; }
      }
#pragma unroll
      for (int i = 0; i < LB_PAIRS_MAX; ++i) {
        if (jj[i] < 0) continue;
        const int q = tid + i * LB_MATH;
        const int row = q >> 3, j = jj[i], u = bb + j * dp;
        const float rec = k >= 1 ? zs[row * LC_ZS_LD + (q & 7)] : 0.f;
        if (t < 0) {  // gradient of h_0: added to what the caller left in the h half of D[0]
          p.D[(size_t)row * ldd + p.I + u] += rec;
          continue;
        }
        float dh;
        if (t == T - 1) {
          dh = ups[i];
        } else {
          dh = ups[i] + rec;  // upstream gradient of h_t plus the recurrent part
          p.D[((size_t)(t + 1) * p.B + row) * ldd + p.I + u] = dh;
        }
        const float gi = pg[i][0], gf = pg[i][1], gg = pg[i][2], go = pg[i][3];
        const float cp = pg[i][4];
        const float tc = tanh_fast(pg[i][5]);
        const float d_o = dh * p.alpha * tc;
        const float dcv = dcreg[i] + dh * p.alpha * go * (1.f - tc * tc);
        dcreg[i] = dcv * gf;
        __nv_bfloat16* dz = p.DZ + ((size_t)t * p.B + row) * 4 * p.H + j;
        dz[0] = __float2bfloat16_rn(dcv * gg * gi * (1.f - gi));
        dz[p.H] = __float2bfloat16_rn(dcv * cp * gf * (1.f - gf));
        dz[2 * p.H] = __float2bfloat16_rn(dcv * gi * (1.f - gg * gg));
        dz[3 * p.H] = __float2bfloat16_rn(d_o * go * (1.f - go));
      }
      if (t >= 0) {
        asm volatile("bar.sync 1, 352;" ::: "memory");
        if (tid == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.bar) : "memory");
      }
    }
    if (ok) {
#pragma unroll
      for (int i = 0; i < LB_PAIRS_MAX; ++i)
        if (jj[i] >= 0) p.dc[(size_t)((tid + i * LB_MATH) >> 3) * p.H + jj[i]] = dcreg[i];
    }
  }
}

__global__ void __launch_bounds__(LB_THREADS, 1) ard_lstm_backward_kernel(const __grid_constant__ LstmBwdParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw_addr);

  const int KH = p.I + p.H;
  const int row_boxes = (p.B + 63) / 64;
  const uint32_t a_block = (uint32_t)row_boxes * LP_ROW_BOX;
  const uint32_t bar_base = base;                               // gfull[4], tfull, wfull, hready, pready; flags
  const uint32_t sA = base + LB_BAR_BYTES;                      // LB_MAX_BLOCKS blocks of dz
  const uint32_t sW = sA + LB_MAX_BLOCKS * a_block;             // LB_MAX_BLOCKS weight boxes (the MMA's 128-row read of
                                                                 // the last dz block ends inside this region)
  auto gfull_bar = [&](int g) { return bar_base + 8u * g; };
  const uint32_t tfull_bar = bar_base + 8u * LP_GROUPS;
  const uint32_t wfull_bar = bar_base + 8u * (LP_GROUPS + 1);
  const uint32_t hready_bar = bar_base + 8u * (LP_GROUPS + 2);   // dz of the previous step is complete
  const uint32_t pready_bar = bar_base + 8u * (LP_GROUPS + 3);   // all partial sums of this step are parked
  uint8_t* misc = smem + (bar_base - base) + 8 * (LP_GROUPS + 4);
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(misc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int g = 0; g < LP_GROUPS; ++g) mbar_init(gfull_bar(g), 1);
    mbar_init(tfull_bar, LP_GROUPS);
    mbar_init(wfull_bar, 1);
    mbar_init(hready_bar, 1);
    mbar_init(pready_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 15) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_ptr_smem)), LP_GROUPS * LB_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_smem;
  pdl_wait_prior_grids();

  const int dp = p.hdr[HDR_DP], bb = p.hdr[HDR_B] - 1, n_keep = p.hdr[HDR_NKEEP];
  // Descriptors of this pattern: slots 0-3 the gates' kept weight rows, 4-7 the gates' compact gradient columns.
  // Warp 11 writes them (below) before its first arrival on hready_bar; the loading lanes acquire them after
  // their first wait on that barrier.
  CUtensorMap* slots = p.tm_slots + (size_t)blockIdx.x * ARD_TM_LSTM_SLOTS;
  auto map_of = [&](const TcMap* m, int slot) -> const CUtensorMap* { return dp == 1 ? &m->tm : slots + slot; };
  const int n_cta = (int)gridDim.x;
  const int s_idx = (int)blockIdx.x / LB_KPARTS, r_idx = (int)blockIdx.x % LB_KPARTS;
  const int c0 = s_idx * LB_COLS;                       // first weight column (hidden unit) of the slice
  const int nb = (n_keep + 63) / 64;                    // contraction blocks per gate
  const int per = (4 * nb + LB_KPARTS - 1) / LB_KPARTS; // blocks per CTA (<= LB_MAX_BLOCKS, checked by the host)
  const int blk0 = r_idx * per;
  const int nblk = max(0, min(per, 4 * nb - blk0));     // this CTA's blocks blk0 .. blk0 + nblk - 1; block = gate * nb + jb
  const int parts = (4 * nb + per - 1) / per;           // CTAs of a slice that have blocks
  const int gsz = (nblk + LP_GROUPS - 1) / LP_GROUPS;   // blocks per loader / MMA warp
  const int T = p.T;

  // few kept units: every block of a step fits the row buffer beside the slice of one CTA's units
  const bool compact = p.compact_ok && dp > 1 &&
                       LB_BAR_BYTES + 4 * nb * ((int)a_block + LC_W_BLOCK) + LC_ZS_BYTES <= p.smem_bytes - 1024;
  if (compact) {
    lstm_backward_compact(p, smem, base, bar_base, tmem_base, abort_flag, dp, bb, n_keep);
  } else if (warp == 11) {
    // ===================== weight loader and barrier relay =====================
    // the weight area, still empty, is the work area of the eight descriptors
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      tensormap_specialise(&p.mapW[g], dp, bb + 1, n_keep, smem + (sW - base) + 128 * g, slots + g, lane);
      tensormap_specialise(&p.mapDZ[g], dp, bb + 1, n_keep, smem + (sW - base) + 128 * (4 + g), slots + 4 + g, lane);
    }
    fence_proxy_async_smem();
    const int kb = lane;
    if (kb < nblk) {
      const int blk = blk0 + kb, g = blk / nb, jb = blk - g * nb;
      const CUtensorMap* mw = map_of(&p.mapW[g], g);
      if (dp > 1) tensormap_acquire(mw);
      if (lane == 0) mbar_arrive_expect_tx(wfull_bar, (uint32_t)nblk * LB_W_BLOCK);
      __syncwarp(__activemask());
      tma_load_2d(sW + kb * LB_W_BLOCK, mw, wfull_bar, p.I + c0, jb * 64);
    }
    __syncwarp();
    if (lane == 0) {
      for (int ph = 1; ph <= 2 * T; ++ph) {
        if (!grid_wait(p.bar, (unsigned)ph * (unsigned)n_cta, abort_flag, p.status)) break;
        mbar_arrive((ph & 1) ? hready_bar : pready_bar);
      }
    }
  } else if (warp >= 12) {
    // ===================== loaders and MMA issuers (group g = warp - 12) =====================
    const int g4 = warp - 12;
    const int kb0 = g4 * gsz, kb1 = min(nblk, kb0 + gsz);
    const int kb = kb0 + lane;
    const bool mine = kb < kb1;
    int gate = 0, jb = 0;
    if (mine) {
      const int blk = blk0 + kb;
      gate = blk / nb;
      jb = blk - gate * nb;
    }
    const CUtensorMap* mdz = map_of(&p.mapDZ[gate], 4 + gate);
    const uint32_t idesc = make_idesc(LB_COLS, false, true, 128);
    bool ok = (lane != 0) || nblk == 0 || mbar_wait(wfull_bar, 0u, abort_flag, p.status);
    for (int k = 1; k <= T; ++k) {
      // dz of time index T - k is complete
      if (ok && !mbar_wait(hready_bar, (uint32_t)(k - 1) & 1u, abort_flag, p.status)) ok = false;
      if (!__all_sync(0xffffffffu, ok)) break;
      if (k == 1 && mine && dp > 1) tensormap_acquire(mdz);  // written by warp 11 ahead of its first arrival on hready_bar
      if (kb0 < kb1) {
        asm volatile("fence.proxy.async.global;" ::: "memory");  // generic-proxy stores of other CTAs -> TMA reads
        if (lane == 0) mbar_arrive_expect_tx(gfull_bar(g4), (uint32_t)(kb1 - kb0) * a_block);
        __syncwarp();
        if (mine)
          for (int rb = 0; rb < row_boxes; ++rb)
            tma_load_2d(sA + kb * a_block + rb * LP_ROW_BOX, mdz, gfull_bar(g4), jb * 64,
                        (T - k) * p.B + rb * 64);
        if (lane == 0) {
          if (!mbar_wait(gfull_bar(g4), (uint32_t)(k - 1) & 1u, abort_flag, p.status)) ok = false;
          if (ok) {
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(g4 * LB_COLS);
            for (int k2 = kb0; k2 < kb1; ++k2) {
              const uint32_t a0 = sA + k2 * a_block, b0 = sW + k2 * LB_W_BLOCK;
#pragma unroll
              for (int s = 0; s < LP_BK / 16; ++s)  // A K-major: 32 bytes per step; B MN-major: 16 k-rows = 2048 bytes
                tc_mma_bf16(d_tmem, make_desc(a0 + s * 32, 16, 1024), make_desc(b0 + s * 2048, 64 * LP_BK * 2, 1024), idesc,
                            (k2 != kb0 || s != 0) ? 1u : 0u);
            }
          }
        }
      }
      if (lane == 0 && ok && nblk > 0) {
        if (kb0 < kb1) tc_commit(tfull_bar);
        else mbar_arrive(tfull_bar);
      }
      __syncwarp();
    }
  } else {
    // ===================== partial sums and cell adjoint (warps 0-10) =====================
    const int tid = threadIdx.x;  // 0 .. LB_MATH-1
    const int npairs = p.B * LB_OWN;  // (batch row, owned column) pairs; pair q = row * 8 + cc
    const size_t ldd = (size_t)KH;
    float dcreg[LB_PAIRS_MAX];
    int jj[LB_PAIRS_MAX];  // kept index of the pair's unit, -1 if the column is a dropped unit or out of range
#pragma unroll
    for (int i = 0; i < LB_PAIRS_MAX; ++i) {
      const int q = tid + i * LB_MATH;
      const int row = q >> 3, u = c0 + r_idx * LB_OWN + (q & 7);
      const int rel = u - bb;
      jj[i] = (q < npairs && u < p.H && rel >= 0 && rel % dp == 0) ? rel / dp : -1;
      dcreg[i] = jj[i] >= 0 ? p.dc[(size_t)row * p.H + jj[i]] : 0.f;
    }
    float* my_partial = p.partial + (size_t)blockIdx.x * 128 * LB_COLS;
    const float* slice_partial = p.partial + (size_t)(s_idx * LB_KPARTS) * 128 * LB_COLS;
    bool ok = true;
    for (int k = 0; k <= T && ok; ++k) {
      const int t = T - 1 - k;  // time index whose dh is formed in this round (-1: the gradient of h_0)
      // what does not depend on the recurrence is fetched before the waits: gate activations, cell states
      float pg[LB_PAIRS_MAX][6];
#pragma unroll
      for (int i = 0; i < LB_PAIRS_MAX; ++i) {
        if (jj[i] >= 0 && t >= 0) {
          const int row = (tid + i * LB_MATH) >> 3, j = jj[i];
          const float* gs = p.G + ((size_t)t * p.B + row) * 4 * p.H + j;
          pg[i][0] = __ldcg(gs);
          pg[i][1] = __ldcg(gs + p.H);
          pg[i][2] = __ldcg(gs + 2 * p.H);
          pg[i][3] = __ldcg(gs + 3 * p.H);
          pg[i][4] = __ldcg(p.C + ((size_t)t * p.B + row) * p.H + j);
          pg[i][5] = __ldcg(p.C + ((size_t)(t + 1) * p.B + row) * p.H + j);
        }
      }
      if (k >= 1) {
        // ---- phase A: park this CTA's partial sums ----
        // Every CTA passes the previous phase before it arrives for this one, also a CTA that has no
        // contraction blocks: the arrival count identifies a phase only if nobody is two arrivals ahead.
        if (!mbar_wait(hready_bar, (uint32_t)(k - 1) & 1u, abort_flag, p.status)) ok = false;
        if (ok && warp < 4 && nblk > 0) {
          if (!mbar_wait(tfull_bar, (uint32_t)(k - 1) & 1u, abort_flag, p.status)) ok = false;
          if (ok) {
            tc_fence_after();
            const int row = warp * 32 + lane;
            const uint32_t t_row = tmem_base + ((uint32_t)(warp * 32) << 16);
            const int ngroups = (nblk + gsz - 1) / gsz;
#pragma unroll 1
            for (int half = 0; half < 2; ++half) {
              uint32_t z[32], y[32];
              tmem_ld32(t_row + (uint32_t)(half * 32), z);
              tmem_ld_wait();
              for (int c = 1; c < ngroups; ++c) {
                tmem_ld32(t_row + (uint32_t)(c * LB_COLS + half * 32), y);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) z[i] = __float_as_uint(__uint_as_float(z[i]) + __uint_as_float(y[i]));
              }
              if (row < p.B) {
                float4* dst = reinterpret_cast<float4*>(my_partial + (size_t)row * LB_COLS + half * 32);
#pragma unroll
                for (int i = 0; i < 8; ++i)
                  __stcg(dst + i, make_float4(__uint_as_float(z[4 * i]), __uint_as_float(z[4 * i + 1]),
                                              __uint_as_float(z[4 * i + 2]), __uint_as_float(z[4 * i + 3])));
              }
            }
            tc_fence_before();
          }
        }
        asm volatile("bar.sync 1, 352;" ::: "memory");
        if (*abort_flag) { ok = false; break; }
        if (tid == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.bar) : "memory");
        // ---- all partial sums of the slice are parked ----
        if (!mbar_wait(pready_bar, (uint32_t)(k - 1) & 1u, abort_flag, p.status)) ok = false;
        asm volatile("bar.sync 2, 352;" ::: "memory");
        if (*abort_flag) { ok = false; break; }
      }
      // ---- phase B: total gradient of h_t, cell adjoint, dz_t ----
      // All loads of all owned (row, unit) pairs are issued before the first is consumed: the partial sums
      // come from L2 and a chain of dependent round trips would cost more than the whole product.
      float recs[LB_PAIRS_MAX], ups[LB_PAIRS_MAX];
#pragma unroll
      for (int i = 0; i < LB_PAIRS_MAX; ++i) {
        recs[i] = 0.f;
        ups[i] = 0.f;
        if (jj[i] < 0) continue;
        const int q = tid + i * LB_MATH;
        const int row = q >> 3, cc = r_idx * LB_OWN + (q & 7), u = c0 + cc;
        float part[LB_KPARTS];
#pragma unroll
        for (int rp = 0; rp < LB_KPARTS; ++rp)
          part[rp] = (k >= 1 && rp < parts) ? __ldcg(slice_partial + ((size_t)rp * 128 + row) * LB_COLS + cc) : 0.f;
        if (t >= 0)
          ups[i] = (t == T - 1) ? p.dH_last[(size_t)row * p.H + u]
                                : __ldcg(p.D + ((size_t)(t + 1) * p.B + row) * ldd + p.I + u);
        float rec = 0.f;
#pragma unroll
        for (int rp = 0; rp < LB_KPARTS; ++rp) rec += part[rp];  // fixed order: same bits every launch
        recs[i] = rec;
      }
#pragma unroll
      for (int i = 0; i < LB_PAIRS_MAX; ++i) {
        if (jj[i] < 0) continue;
        const int q = tid + i * LB_MATH;
        const int row = q >> 3, cc = r_idx * LB_OWN + (q & 7), u = c0 + cc, j = jj[i];
        const float rec = recs[i];
        if (t < 0) {  // gradient of h_0: added to what the caller left in the h half of D[0]
          p.D[(size_t)row * ldd + p.I + u] += rec;
          continue;
        }
        float dh;
        if (t == T - 1) {
          dh = ups[i];
        } else {
          dh = ups[i] + rec;  // upstream gradient of h_t plus the recurrent part
          p.D[((size_t)(t + 1) * p.B + row) * ldd + p.I + u] = dh;
        }
        const float gi = pg[i][0], gf = pg[i][1], gg = pg[i][2], go = pg[i][3];
        const float cp = pg[i][4];
        const float tc = tanh_fast(pg[i][5]);
        const float d_o = dh * p.alpha * tc;
        const float dcv = dcreg[i] + dh * p.alpha * go * (1.f - tc * tc);
        dcreg[i] = dcv * gf;
        __nv_bfloat16* dz = p.DZ + ((size_t)t * p.B + row) * 4 * p.H + j;
        dz[0] = __float2bfloat16_rn(dcv * gg * gi * (1.f - gi));
        dz[p.H] = __float2bfloat16_rn(dcv * cp * gf * (1.f - gf));
        dz[2 * p.H] = __float2bfloat16_rn(dcv * gi * (1.f - gg * gg));
        dz[3 * p.H] = __float2bfloat16_rn(d_o * go * (1.f - go));
      }
      if (t >= 0) {
        asm volatile("bar.sync 1, 352;" ::: "memory");
        if (tid == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.bar) : "memory");
      }
    }
    if (ok) {
#pragma unroll
      for (int i = 0; i < LB_PAIRS_MAX; ++i)
        if (jj[i] >= 0) p.dc[(size_t)((tid + i * LB_MATH) >> 3) * p.H + jj[i]] = dcreg[i];
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncwarp();  // lanes that left their role's loop one by one arrive at the block-wide barrier together
  __syncthreads();
  if (warp == 15) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, LP_GROUPS * LB_COLS);
  }
}

}  // namespace

// Dynamic shared memory for klen contraction columns and batch B: the row buffer, the weight slice, the
// staged pre-activations, barriers, and slack for the 1024-byte alignment.
static size_t lstm_fwd_smem_bytes(int klen, int B, int kx0 = 0, int I = 1) {
  const size_t nkb = (size_t)(klen + LP_BK - 1) / LP_BK;
  const size_t a_block = (size_t)((B + 63) / 64) * LP_ROW_BOX;
  const size_t zs = lstm_fwd_zs_shared(kx0, I, (int)nkb, (int)a_block) ? 0 : LP_ZS_BYTES;
  return nkb * a_block + nkb * LP_W_BLOCK + zs + 8 * (LP_GROUPS + 6) + 16 + 1024;
}

// Can the whole-sequence kernel run this layer on this device?  (Shared memory for the weight slice, one
// CTA per 8 hidden units all resident at once, one 128-row tile of batch.)
bool lstm_persistent_fits(ard_ctx* ctx, int B, int klen, int H) {
  if (B < 1 || B > 128 || H < 1 || klen < 1) return false;
  if ((klen + LP_BK - 1) / LP_BK > LP_MAX_BLOCKS) return false;
  const size_t smem = lstm_fwd_smem_bytes(klen, B);
  if (smem > 227 * 1024) return false;  // the row of activations and the weight slice must both be resident
  static int probed[64] = {};
  const int dev = ctx->device & 63;
  if (probed[dev] == 0) {
    int n = 0;
    if (cudaFuncSetAttribute(ard_lstm_forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
            cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, ard_lstm_forward_kernel, LP_THREADS, smem) != cudaSuccess ||
        n < 1)
      probed[dev] = -1;
    else
      probed[dev] = 1;
  }
  if (probed[dev] < 1) return false;
  return (H + LP_UNITS - 1) / LP_UNITS <= ctx->sm_count;  // one CTA per SM, all resident at once
}

ard_status launch_lstm_forward_persistent(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H,
                                          int kx0, int klen, int add_zx, float alpha, const TcMap& mapXH, const TcMap mapW[4],
                                          const TcMap* mapHc, const void* W, int ldw, void* XH, const float* bias, float* C, float* G, cudaStream_t s) {
  if ((H + LP_UNITS - 1) / LP_UNITS > ARD_TM_LSTM_BLOCKS) return ARD_ERR_UNSUPPORTED;
  LstmFwdParams p;
  p.mapXH = mapXH;
  for (int g = 0; g < 4; ++g) p.mapW[g] = mapW[g];
  p.tm_slots = ctx->d_tm_slots + (size_t)ARD_TM_SM_MAX * ARD_TM_SLOTS;
  p.hdr = pat->d_hdr;
  p.T = T; p.B = B; p.I = I; p.H = H;
  p.kx0 = kx0; p.klen = klen; p.add_zx = add_zx;
  p.mapHc = mapHc ? *mapHc : mapXH;
  p.W = reinterpret_cast<const __nv_bfloat16*>(W);
  p.ldw = ldw;
  p.Hc = mapHc ? reinterpret_cast<__nv_bfloat16*>(ctx->d_lstm_hc) : nullptr;
  p.ldhc = ARD_LSTM_HC_LD;
  p.alpha = alpha;
  p.XH = reinterpret_cast<__nv_bfloat16*>(XH);
  p.bias = bias;
  p.C = C;
  p.G = G;
  p.bar = ctx->d_grid_bar;
  p.status = ctx->d_status;
  ARD_CUDA_OK(cudaMemsetAsync(ctx->d_grid_bar, 0, sizeof(unsigned int), s));
  // h_1 .. h_T: zeros at the dropped units (the kernel stores the kept ones)
  ARD_CUDA_OK(cudaMemset2DAsync(p.XH + (size_t)B * (I + H) + I, (size_t)(I + H) * 2, 0, (size_t)H * 2, (size_t)T * B, s));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((H + LP_UNITS - 1) / LP_UNITS);  // sized for dp = 1; CTAs without units leave at once
  cfg.blockDim = dim3(LP_THREADS);
  cfg.dynamicSmemBytes = lstm_fwd_smem_bytes(klen, B, kx0, I);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs resident: they wait for one another
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t err = cudaLaunchKernelEx(&cfg, ard_lstm_forward_kernel, p);
  if (err == cudaErrorCooperativeLaunchTooLarge || err == cudaErrorLaunchOutOfResources) {
    // the device cannot hold all CTAs at once right now (SMs taken by another context, a smaller
    // partition): nothing was enqueued, the caller falls back to the per-step path
    (void)cudaGetLastError();
    return ARD_ERR_UNSUPPORTED;
  }
  if (err != cudaSuccess) return ARD_ERR_CUDA;
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

// ---- whole-sequence BPTT recurrence ----
// Shared memory of the BPTT kernel.  The form is chosen on the device from the drawn pattern, so the launch asks for
// what either may need: 8 row blocks and 8 weight boxes behind the barriers for the form with partial sums, 16 row
// blocks and slice blocks for the compact form (more kept units than that take the other form).  Asking for all
// 227 KB instead cost the form with partial sums 4 % (390 -> 407 us per backward pass at H = 1024, batch 64).
static size_t lstm_bwd_smem_bytes(int B, int compact_ok) {
  static_assert((size_t)LB_MAX_BLOCKS * 2 * LP_ROW_BOX + (size_t)LB_MAX_BLOCKS * LB_W_BLOCK + LB_BAR_BYTES + 1024 <= LB_SMEM_BYTES,
                "the form with partial sums does not fit");
  const size_t a_block = (size_t)((B + 63) / 64) * LP_ROW_BOX;
  const size_t sums = LB_MAX_BLOCKS * a_block + (size_t)LB_MAX_BLOCKS * LB_W_BLOCK + LB_BAR_BYTES + 1024;
  if (!compact_ok) return sums;
  // room for the compact form up to 4 blocks per gate (256 kept units), or whatever the other form needs
  const size_t compact = 16 * (a_block + LC_W_BLOCK) + LC_ZS_BYTES + LB_BAR_BYTES + 1024;
  const size_t want = compact > sums ? compact : sums;
  return want < (size_t)LB_SMEM_BYTES ? want : (size_t)LB_SMEM_BYTES;
}

size_t lstm_bwd_partial_bytes(int sm_count) { return (size_t)sm_count * 128 * LB_COLS * sizeof(float); }

bool lstm_persistent_bwd_fits(ard_ctx* ctx, int B, int H) {
  if (B < 1 || B > 128 || H < 1 || H > 1024) return false;  // at most 8 contraction blocks per CTA
  if (ctx->d_lstm_partial == nullptr) return false;
  if ((H + LB_COLS - 1) / LB_COLS * LB_KPARTS > ctx->sm_count) return false;  // one CTA per SM, all resident at once
  static int probed[64] = {};
  const int dev = ctx->device & 63;
  if (probed[dev] == 0) {
    int n = 0;
    if (cudaFuncSetAttribute(ard_lstm_backward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) !=
            cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, ard_lstm_backward_kernel, LB_THREADS, lstm_bwd_smem_bytes(128, 1)) !=
            cudaSuccess ||
        n < 1)
      probed[dev] = -1;
    else
      probed[dev] = 1;
  }
  return probed[dev] == 1;
}

ard_status launch_lstm_backward_persistent(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H, float alpha,
                                           const TcMap mapDZ[4], const TcMap mapW[4], const void* W, int ldw,
                                           const float* C, const float* G, const float* dH_last, float* D, float* dc,
                                           void* DZ, cudaStream_t s) {
  if ((H + LB_COLS - 1) / LB_COLS * LB_KPARTS > ARD_TM_LSTM_BLOCKS) return ARD_ERR_UNSUPPORTED;
  LstmBwdParams p;
  for (int g = 0; g < 4; ++g) { p.mapDZ[g] = mapDZ[g]; p.mapW[g] = mapW[g]; }
  p.tm_slots = ctx->d_tm_slots + (size_t)ARD_TM_SM_MAX * ARD_TM_SLOTS;
  p.hdr = pat->d_hdr;
  p.T = T; p.B = B; p.I = I; p.H = H;
  p.alpha = alpha;
  p.C = C; p.G = G; p.dH_last = dH_last; p.D = D; p.dc = dc;
  p.DZ = reinterpret_cast<__nv_bfloat16*>(DZ);
  p.partial = ctx->d_lstm_partial;
  p.bar = ctx->d_grid_bar;
  p.status = ctx->d_status;
  p.W = reinterpret_cast<const __nv_bfloat16*>(W);
  p.ldw = ldw;
  p.compact_ok = ctx->lstm_compact_h;
  p.smem_bytes = (int)lstm_bwd_smem_bytes(B, p.compact_ok);
  ARD_CUDA_OK(cudaMemsetAsync(ctx->d_grid_bar, 0, sizeof(unsigned int), s));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((H + LB_COLS - 1) / LB_COLS * LB_KPARTS);
  cfg.blockDim = dim3(LB_THREADS);
  cfg.dynamicSmemBytes = lstm_bwd_smem_bytes(B, p.compact_ok);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs resident: they wait for one another
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t err = cudaLaunchKernelEx(&cfg, ard_lstm_backward_kernel, p);
  if (err == cudaErrorCooperativeLaunchTooLarge || err == cudaErrorLaunchOutOfResources) {
    (void)cudaGetLastError();
    return ARD_ERR_UNSUPPORTED;  // nothing was enqueued: the caller takes the per-step path
  }
  if (err != cudaSuccess) return ARD_ERR_CUDA;
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}
