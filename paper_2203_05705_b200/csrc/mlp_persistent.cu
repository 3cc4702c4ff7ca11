// One training iteration of a small stack of fully connected layers under row patterns in ONE cooperative
// kernel (Sec. 3.1: a layer fed by a dropped layer multiplies compact matrices on both sides; Sec. 3.2, last
// paragraph: product -> activation -> dropout per layer; Sec. 3.4: a new pattern per iteration).
//
// With a batch of at most 128 rows every product of the iteration is a single row tile: a few microseconds of
// work that, launched on its own, costs as much again in set-up and in the gap to the launch that depends on
// it.  Here the iteration is a sequence of stages inside one kernel, separated by grid-wide barriers:
//   stage s < H (H hidden layers): the forward product of hidden layer s.  Its epilogue adds the bias, applies
//     the activation and the rescale and stores the kept neurons' outputs compact, bf16.  The output layer has at
//     most 16 neurons, so the epilogue of the last hidden layer also forms that layer's input gradient (ten
//     multiply-adds per element, no product to wait for).  Beside it, on CUDA cores: in stage 0 the kept lists of
//     the patterns and the packed copies W[keep][keep_in] of the later layers' weights; in every forward stage the
//     zero rows of that layer's weight gradient;
//   stage H + t (t < H), layer l = H-1-t: the input-gradient product of layer l (its epilogue applies the ReLU
//     adjoint and the rescale of layer l-1 and stores compact bf16) and the weight-gradient product of layer l (its
//     epilogue writes the kept rows of the full-width gradient, zeros between the kept fan-in columns); beside
//     them, on CUDA cores, the bias gradient, and at t = 0 the output layer's own product and gradients.
// Roles of a CTA: warp 0 requests the operands (TMA boxes, one ring stage per lane), warps 1-2 issue the products
// (tcgen05.mma, M = 128 = the batch rows, or 128 kept neurons for a weight gradient; alternate 64-deep blocks of a
// tile go into accumulators of their own in tensor memory, because one thread needs ~0.2 us to issue a block's
// four instructions, as long as the block takes to arrive), warps 3-6 are the epilogue (they add the two
// accumulators in a fixed order), warps 7-10 do the CUDA-core work of the stage at the same time.  The forward
// weight arrives in boxes of 16, 32 or 64 rows, so that a tile is as narrow as it takes to spread a product over
// all SMs: what bounds a tile is its 128-row operand streaming through one SM.
// The patterns are drawn by every CTA for itself (a few hundred instructions).  Every wait is bounded; a CTA that
// gives up records the status, which the others poll at the grid barrier.
#include "ard_internal.h"
#include "philox.h"
#include "sm100_ptx.h"

namespace {


constexpr int MP_MAX_LAYERS = 4;                    // hidden layers + the output layer
constexpr int MP_NI = 2;                            // issuing warps = accumulators per tile
constexpr int MP_EPI_WARPS = 4;
constexpr int MP_CC_WARPS = 4;                      // warps that do the CUDA-core work of a stage
constexpr int MP_EPI_W0 = 1 + MP_NI;                // warp 0 producer, 1..NI issuers, then epilogue, then CUDA-core warps
constexpr int MP_CC_W0 = MP_EPI_W0 + MP_EPI_WARPS;
constexpr int MP_WARPS = MP_CC_W0 + MP_CC_WARPS;
constexpr int MP_THREADS = MP_WARPS * 32;
constexpr int MP_CC_THREADS = MP_CC_WARPS * 32;
constexpr int MP_BK = 64;
constexpr int MP_A_BYTES = 128 * MP_BK * 2;         // 128 rows (or 2 x 64 MN-major columns) of one block
constexpr int MP_B_BYTES = 64 * MP_BK * 2;
constexpr int MP_STAGE_BYTES = MP_A_BYTES + MP_B_BYTES;
constexpr int MP_STAGES = 7;
constexpr int MP_ACC_COLS = 64;                     // tensor-memory columns per accumulator
constexpr int MP_TMEM_COLS = MP_NI * MP_ACC_COLS <= 128 ? 128 : 256;
#ifndef MP_SPIN
#define MP_SPIN 4096
#endif
constexpr int MP_SMALL_N = 16;                      // widest output layer
constexpr int MP_STG_LD = 65;
constexpr int MP_STG_WORDS = 32 * MP_STG_LD;        // per epilogue warp: 4 x 16 x 16 output weights + 64 biases, or
                                                    //   32 rows x 36 words of ReLU bits, or 32 x 65 staged sums
constexpr int MP_STG_OFF = MP_STAGES * MP_STAGE_BYTES;
constexpr int MP_SDO_OFF = MP_STG_OFF + MP_EPI_WARPS * MP_STG_WORDS * 4;   // [128][MP_SMALL_N] floats
constexpr int MP_BAR_OFF = MP_SDO_OFF + 128 * MP_SMALL_N * 4;
constexpr int MP_NBARS = 2 * MP_STAGES + MP_NI + 1;
constexpr int MP_CDF_OFF = (MP_BAR_OFF + 8 * MP_NBARS + 15) / 16 * 16;
constexpr int MP_MISC_OFF = MP_CDF_OFF + 64 * 8;
constexpr int MP_SMEM = MP_MISC_OFF + 128 + 2 * (MP_MAX_LAYERS - 1) * 2 * 112 + 64 + 1024;   // + slack for the 1024-byte alignment of the ring
static_assert(MP_SMEM <= 227 * 1024, "shared memory of the iteration kernel");

enum { JT_F = 0, JT_BD = 1, JT_BW = 2 };

struct MpLayer {
  int K, N, ldw;
  int relu, dW_is_f32, sample;
  float alpha;
  uint32_t stream_id;
  const __nv_bfloat16* W;
  const float* bias;
  __nv_bfloat16* Wk;
  __nv_bfloat16* A;
  __nv_bfloat16* dZ;
  void* dW;
  float* db;
  int32_t* hdr;
  int32_t* idx;
  int Tr, Tc, ts;  // what the header of a row pattern holds in the tile fields
};

struct MpParams {
  // Whole-matrix descriptors.  "k": boxes of 128 rows x 64 columns (the 128-row operand, contraction along the
  // row); "m": boxes of 64 x 64 (an operand whose contraction runs down the rows).
  TcMap mapXk, mapXm;                 // [B][K_0]
  TcMap mapAk[MP_MAX_LAYERS - 1];     // activations of hidden layer l, [B][N_l]
  TcMap mapAm[MP_MAX_LAYERS - 1];
  TcMap mapdZk[MP_MAX_LAYERS - 1];    // their gradients
  TcMap mapdZm[MP_MAX_LAYERS - 1];
  TcMap mapWf[MP_MAX_LAYERS - 1][3];  // forward weight in boxes of 16 / 32 / 64 rows x 64 columns: layer 0 the weight
                                      //   itself (kept rows: fitted by the kernel), else the packed copy
  TcMap mapWb[MP_MAX_LAYERS - 1];     // the same matrices in boxes of 64 x 64 (input gradient)
  MpLayer layer[MP_MAX_LAYERS];
  int L, B;
  int ldx, lddout, lddx;
  const __nv_bfloat16* X;
  const __nv_bfloat16* dOut;
  __nv_bfloat16* dX;
  CUtensorMap* tm_slots;
  const unsigned long long* cdf;
  int ndp;
  int any_sampled;
  unsigned long long seed, iteration_base;
  unsigned long long* counter;
  unsigned int* bar;
  int* status;
};

struct LayerRt { int dp, bb, n, npad; };  // period, offset - 1, kept neurons, the latter rounded up to 64

constexpr int MP_MAX_MINE = 40;  // most tiles of one product a CTA can be dealt (checked on the host)
struct GemmJob {
  int type, l;
  int items, nkb, nt, ntn;
  int mine;                  // tiles of this CTA
  short tile[MP_MAX_MINE];   // their numbers
};
static_assert(sizeof(GemmJob) <= 112, "room per product in shared memory");

__device__ __forceinline__ unsigned int mp_ld_acquire(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__device__ bool mp_grid_wait(const unsigned int* bar, unsigned int target, volatile int* abort_flag, int* status) {
  if (mp_ld_acquire(bar) >= target) return true;
  const unsigned long long t0 = global_ns();
  for (int spin = 1;; ++spin) {
    if (mp_ld_acquire(bar) >= target) return true;
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

// mbar_wait out of line: the fast path (the phase is already complete) stays inline, the polling loop with its
// clock reads and status updates exists once.
__device__ __noinline__ bool mp_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  return mbar_wait(bar, parity, abort_flag, status);
}
__device__ __forceinline__ bool mp_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  // The hand-offs of this kernel are microseconds apart and each of them is on the critical path of its stage, so
  // the waiting thread polls (a few ten microseconds at most) before it lets the hardware park it.
#pragma unroll 1
  for (int spin = 0; spin < MP_SPIN; ++spin)
    if (mbar_try_wait(bar, parity)) return true;
  return mp_wait_slow(bar, parity, abort_flag, status);
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}

__device__ __forceinline__ uint32_t mp_pack(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ bool bf16_bits_positive(uint32_t bits) {  // > 0: sign clear, not zero, not NaN
  return !(bits & 0x8000u) && (bits & 0x7FFFu) != 0u && (bits & 0x7FFFu) <= 0x7F80u;
}
// 16 consecutive bf16 of one row, 32-byte aligned
__device__ __forceinline__ void store16_bf16(__nv_bfloat16* dst, const float (&v)[16]) {
  uint4* d = reinterpret_cast<uint4*>(dst);
  d[0] = make_uint4(mp_pack(v[0], v[1]), mp_pack(v[2], v[3]), mp_pack(v[4], v[5]), mp_pack(v[6], v[7]));
  d[1] = make_uint4(mp_pack(v[8], v[9]), mp_pack(v[10], v[11]), mp_pack(v[12], v[13]), mp_pack(v[14], v[15]));
}

// The helpers below read the kernel's parameters and are inlined for that reason: behind a call the parameter
// block is reached through a generic pointer, i.e. by loads that go to the L2 instead of the constant bank, a
// memory round trip per field on the critical path of every stage.

// The products of stage st and the tiles of this CTA, written by one thread into shared memory (all stages are set
// up at the start of the kernel).  Tiles are dealt round-robin.  A stage with two products deals the second one (the
// weight gradient: many short tiles) past the CTAs that hold a tile of the first (the input gradient: few tiles
// with a long contraction) for as many rounds as that tile is worth, when enough other CTAs are left.
__device__ __forceinline__ int mp_make_jobs(const MpParams& p, const LayerRt* rt, int H, int G, int cta, int st,
                                            GemmJob* job) {
  int njobs = 0;
  if (st < H) {
    const int l = st;
    GemmJob& j = job[njobs++];
    j.type = JT_F; j.l = l;
    j.nt = (rt[l].n + 15) / 16 <= G ? 16 : ((rt[l].n + 31) / 32 <= G ? 32 : 64);
    j.items = (rt[l].n + j.nt - 1) / j.nt;
    j.nkb = l == 0 ? (p.layer[0].K + MP_BK - 1) / MP_BK : rt[l - 1].npad / MP_BK;
    j.ntn = 1;
  } else {
    const int l = H - 1 - (st - H);
    const int nin = l == 0 ? p.layer[0].K : rt[l - 1].n;
    if (l > 0 || p.dX != nullptr) {
      GemmJob& j = job[njobs++];
      j.type = JT_BD; j.l = l;
      j.nt = 64;
      j.items = (nin + 63) / 64;
      j.nkb = rt[l].npad / MP_BK;
      j.ntn = 1;
    }
    GemmJob& j = job[njobs++];
    j.type = JT_BW; j.l = l;
    j.nt = 64;
    j.ntn = (nin + 63) / 64;
    j.items = ((rt[l].n + 127) / 128) * j.ntn;
    j.nkb = (p.B + MP_BK - 1) / MP_BK;
  }
  // first product: tile cta, cta + G, ...
  {
    GemmJob& j = job[0];
    j.mine = 0;
    for (int i = cta; i < j.items && j.mine < MP_MAX_MINE; i += G) j.tile[j.mine++] = (short)i;
  }
  if (njobs > 1) {
    GemmJob& j = job[1];
    const int nbd = min(job[0].items, G);
    int skip = min(4, job[0].nkb / 8);           // rounds in which the holders of a long tile are passed over
    if ((G - nbd) * 2 < G) skip = 0;
    j.mine = 0;
    int next = 0;                                 // first tile of the current round
    for (int r = 0; next < j.items && j.mine < MP_MAX_MINE; ++r) {
      if (r < skip) {
        if (cta >= nbd && next + (cta - nbd) < j.items) j.tile[j.mine++] = (short)(next + (cta - nbd));
        next += G - nbd;
      } else {
        // the rounds after that start behind the long tiles' holders, so that those come last
        const int slot = cta >= nbd ? cta - nbd : cta + (G - nbd);
        if (next + slot < j.items) j.tile[j.mine++] = (short)(next + slot);
        next += G;
      }
    }
  }
  return njobs;
}

// CUDA-core work of stage 0, done by thread gtid of gthreads: the CUDA-core warps of every CTA (ct = 0 .. MP_CC_THREADS-1
// inside the CTA) and, in the CTAs that have no tile of the first product, the other warps too (ct = -1).  Every
// loop here is bound by memory latency: a thread issues a batch of independent loads before it uses the first.
__device__ __forceinline__ void mp_forward_jobs(const MpParams& p, const LayerRt* rt, int H, int cta, int G, int ct,
                                                int gtid, int gthreads) {
  {
    // (a) headers and kept lists of the patterns, as the sampler kernel leaves them: the last CTAs, one per layer
    const int l = G - 1 - cta;
    if (ct >= 0 && l < H && p.layer[l].sample) {
      const MpLayer& y = p.layer[l];
      if (ct == 0) {
        y.hdr[HDR_KIND] = ARD_ROW;
        y.hdr[HDR_DP] = rt[l].dp;
        y.hdr[HDR_B] = rt[l].bb + 1;
        y.hdr[HDR_NKEEP] = rt[l].n;
        y.hdr[HDR_UNITS] = y.N;
        y.hdr[HDR_TR] = y.Tr;
        y.hdr[HDR_TC] = y.Tc;
        y.hdr[HDR_TS] = y.ts;
        y.hdr[HDR_MAPIDX] = rt[l].dp * (rt[l].dp - 1) / 2 + rt[l].bb;
      }
#pragma unroll 1
      for (int jx = ct; jx < rt[l].n; jx += MP_CC_THREADS) y.idx[jx] = rt[l].bb + jx * rt[l].dp;
    }
    // (b) packed weights of the layers behind a dropped layer: Wk[i][j] = W[bb + i dp][bi + j dpi], zeros up to the
    //     next multiples of 64 both ways.  A thread reads 16 bytes of a kept row (8 fan-in columns) and stores those
    //     that are kept, so the kept rows are read once, in whole lines; four pieces are in flight per thread.
#pragma unroll 1
    for (int l2 = 1; l2 <= H; ++l2) {
      const MpLayer& y = p.layer[l2];
      const int dpi = rt[l2 - 1].dp, bi = rt[l2 - 1].bb, nin = rt[l2 - 1].n;
      const int cols_padded = min(y.ldw, rt[l2 - 1].npad);
      const int rows_padded = l2 == H ? y.N : min(y.N, rt[l2].npad);
      const int nkeep = rt[l2].n;
      const uint32_t magic = (uint32_t)(0x100000000ull / (unsigned)dpi) + 1u;  // exact x / dpi for x < 2^16
      const int vecs = y.K / 8;                 // 16-byte pieces of a weight row
      const int units = nkeep * vecs;
#pragma unroll 1
      for (int u0 = gtid; u0 < units; u0 += 4 * gthreads) {
        uint4 v[4];
        int ik[4], c0[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int u = u0 + k * gthreads;
          ik[k] = -1;
          c0[k] = 0;
          v[k] = make_uint4(0u, 0u, 0u, 0u);
          if (u < units) {
            ik[k] = u / vecs;
            c0[k] = (u - ik[k] * vecs) * 8;
            v[k] = *reinterpret_cast<const uint4*>(y.W + ((size_t)rt[l2].bb + (size_t)ik[k] * rt[l2].dp) * y.ldw + c0[k]);
          }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (ik[k] < 0) continue;
          __nv_bfloat16* dst = y.Wk + (size_t)ik[k] * y.ldw;
          if (dpi == 1) {
            *reinterpret_cast<uint4*>(dst + c0[k]) = v[k];
          } else {
            // the kept ones among these 8 columns (Eq. 1), one short store each
            int rel = c0[k] - bi, e0 = 0;
            if (rel < 0) { e0 = -rel; rel = 0; }
            else {
              const int jq0 = (int)__umulhi((uint32_t)(rel + dpi - 1), magic);
              e0 = jq0 * dpi - rel;
              rel = jq0 * dpi;
            }
            int jq = (int)__umulhi((uint32_t)rel, magic);  // packed column of the first kept one
#pragma unroll 1
            for (int e = e0; e < 8 && jq < nin; e += dpi, ++jq) {
              const uint32_t w = e < 2 ? v[k].x : (e < 4 ? v[k].y : (e < 6 ? v[k].z : v[k].w));
              dst[jq] = __ushort_as_bfloat16((unsigned short)((w >> ((e & 1) * 16)) & 0xFFFFu));
            }
          }
        }
      }
      // zeros behind the kept columns of the kept rows, and the rows up to the next multiple of 64
      const int padc = cols_padded - nin;
#pragma unroll 1
      for (int u = gtid; u < nkeep * padc; u += gthreads) {
        const int i = u / padc;
        y.Wk[(size_t)i * y.ldw + nin + (u - i * padc)] = __float2bfloat16_rn(0.f);
      }
      const int padr = rows_padded - nkeep, g8 = cols_padded / 8;
#pragma unroll 1
      for (int u = gtid; u < padr * g8; u += gthreads) {
        const int i = u / g8;
        *reinterpret_cast<uint4*>(y.Wk + (size_t)(nkeep + i) * y.ldw + (u - i * g8) * 8) = make_uint4(0u, 0u, 0u, 0u);
      }
    }
  }
}

// What the weight-gradient products do not write is zero (Sec. 3.1): the rows of the dropped neurons, and in a
// layer fed by a dropped layer also everything between the kept fan-in columns, so there the whole matrix is
// cleared and the product stores its values into it.  A stream of stores that nothing in the forward stages waits
// for: it is cut into as many parts as there are forward stages and part st is written in stage st, one CUDA-core
// warp of the grid per row, beside the tiles.  (The barriers between the stages order it before the products.)
__device__ __forceinline__ void mp_zero_fill(const MpParams& p, const LayerRt* rt, int H, int st, int cta, int G, int ct) {
  const int lane = ct & 31, cw = ct >> 5;
  const int gwarps = G * MP_CC_WARPS, gwarp = cta + G * cw;
  int total = 0;
  for (int l = 0; l < H; ++l) total += (l > 0 && rt[l - 1].dp > 1) ? p.layer[l].N : p.layer[l].N - rt[l].n;
  const int lo = total * st / H, hi = total * (st + 1) / H;  // a few thousand rows: 32 bits suffice
#pragma unroll 1
  for (int g = lo + gwarp; g < hi; g += gwarps) {
    int l = 0, dr = g;
    for (;;) {
      const int cnt = (l > 0 && rt[l - 1].dp > 1) ? p.layer[l].N : p.layer[l].N - rt[l].n;
      if (dr < cnt) break;
      dr -= cnt;
      ++l;
    }
    const MpLayer& y = p.layer[l];
    const int dp = rt[l].dp, bb = rt[l].bb;
    int r = dr;
    bool dropped = true;
    if (l > 0 && rt[l - 1].dp > 1) {
      dropped = !(r >= bb && (r - bb) % dp == 0);
    } else if (dr >= bb) {
      // the dr-th dropped neuron: the bb neurons before the first kept one, then dp - 1 behind every kept one
      const int x = dr - bb, ii = x / (dp - 1);
      r = bb + ii * dp + 1 + (x - ii * (dp - 1));
    }
    const int per_row = y.dW_is_f32 ? y.K / 4 : y.K / 8;  // 16-byte pieces (K is a multiple of 8)
    uint4* d = reinterpret_cast<uint4*>(reinterpret_cast<char*>(y.dW) + (size_t)r * y.ldw * (y.dW_is_f32 ? 4 : 2));
#pragma unroll 4
    for (int e = lane; e < per_row; e += 32) d[e] = make_uint4(0u, 0u, 0u, 0u);
    if (lane == 0 && dropped && y.db != nullptr) y.db[r] = 0.f;
  }
}

// CUDA-core work of a backward stage: the bias gradient of layer l; at the first backward stage also the output
// layer's product, weight gradient and bias gradient.  All of it is cut into warp-sized items in ONE numbering, so
// that the CUDA-core warps of the grid take an item or two each and the different jobs run side by side (one job
// after the other, each would pay its own memory round trips).  The CTAs are numbered from the end: the first ones
// have the long tiles.  sdO: the loss gradient as floats, [MP_SMALL_N][128] (output-major), in shared memory since the kernel's start.
//   column item: two kept neurons of layer l, 16 lanes each (8 batch rows per lane, one batch of loads): their bias
//     gradient and, at the first backward stage (l = H-1), their columns of the output layer's weight gradient;
//   output item: two batch rows x two output neurons, lanes across the kept inputs in 16-byte pieces (the zeros
//     behind the kept columns of both operands are multiplied along);
//   bias item of the output layer: one output neuron, four batch rows per lane.
__device__ __forceinline__ void mp_backward_jobs(const MpParams& p, const LayerRt* rt, int H, int st, const float* sdO,
                                                 int cta, int G, int ct) {
  const int lane = ct & 31, cw = ct >> 5;
  const int l = H - 1 - (st - H);
  const MpLayer& y = p.layer[l];
  const MpLayer& yo = p.layer[H];
  const MpLayer& yh = p.layer[H - 1];
  const bool first = st == H;
  const int rcta = G - 1 - cta;
  const int gwarps = G * MP_CC_WARPS, gwarp = rcta + G * cw;  // consecutive items go to different CTAs
  const int dpi = rt[H - 1].dp, bi = rt[H - 1].bb;
  const int n_col = (first || y.db != nullptr) ? (rt[l].n + 1) / 2 : 0;
  const int opairs = (yo.N + 1) / 2;
  const int n_out = first ? ((p.B + 1) / 2) * opairs : 0;
  const int n_dbo = (first && yo.db != nullptr) ? yo.N : 0;
  const int pieces = min(yo.ldw, rt[H - 1].npad) / 8;
#pragma unroll 1
  for (int it = gwarp; it < n_col + n_out + n_dbo; it += gwarps) {
    if (it < n_col) {
      const int jc = it * 2 + (lane & 1), sl = lane >> 1;
      const bool col_ok = jc < rt[l].n;
      float g[8], a[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int r = sl * 8 + k;
        g[k] = (col_ok && r < p.B) ? __bfloat162float(__ldcg(y.dZ + (size_t)r * y.N + jc)) : 0.f;
        a[k] = (first && col_ok && r < p.B) ? __bfloat162float(__ldcg(yh.A + (size_t)r * yh.N + jc)) : 0.f;
      }
      if (y.db != nullptr) {
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) s += g[k];
#pragma unroll
        for (int off = 2; off < 32; off <<= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (sl == 0 && col_ok) y.db[rt[l].bb + (size_t)jc * rt[l].dp] = s;
      }
      if (first) {
        // two outputs per round, their reductions side by side
        const size_t c = (size_t)bi + (size_t)jc * dpi;
#pragma unroll 1
        for (int o = 0; o < yo.N; o += 2) {
          const bool two = o + 1 < yo.N;
          float s0 = 0.f, s1 = 0.f;
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            s0 += sdO[o * 128 + sl * 8 + k] * a[k];
            s1 += sdO[(two ? o + 1 : o) * 128 + sl * 8 + k] * a[k];
          }
#pragma unroll
          for (int off = 2; off < 32; off <<= 1) {
            s0 += __shfl_xor_sync(0xffffffffu, s0, off);
            s1 += __shfl_xor_sync(0xffffffffu, s1, off);
          }
          if (sl == 0 && col_ok) {
            if (yo.dW_is_f32) {
              reinterpret_cast<float*>(yo.dW)[(size_t)o * yo.ldw + c] = s0;
              if (two) reinterpret_cast<float*>(yo.dW)[(size_t)(o + 1) * yo.ldw + c] = s1;
            } else {
              reinterpret_cast<__nv_bfloat16*>(yo.dW)[(size_t)o * yo.ldw + c] = __float2bfloat16_rn(s0);
              if (two) reinterpret_cast<__nv_bfloat16*>(yo.dW)[(size_t)(o + 1) * yo.ldw + c] = __float2bfloat16_rn(s1);
            }
          }
        }
      }
    } else if (it < n_col + n_out) {
      const int e = it - n_col;
      const int rp = e / opairs, op = e - rp * opairs;
      const int r0 = 2 * rp, o0 = 2 * op;
      const bool r1ok = r0 + 1 < p.B, o1ok = o0 + 1 < yo.N;
      const uint4* pa0 = reinterpret_cast<const uint4*>(yh.A + (size_t)r0 * yh.N);
      const uint4* pa1 = reinterpret_cast<const uint4*>(yh.A + (size_t)(r1ok ? r0 + 1 : r0) * yh.N);
      const uint4* pw0 = reinterpret_cast<const uint4*>(yo.Wk + (size_t)o0 * yo.ldw);
      const uint4* pw1 = reinterpret_cast<const uint4*>(yo.Wk + (size_t)(o1ok ? o0 + 1 : o0) * yo.ldw);
      float s00 = 0.f, s01 = 0.f, s10 = 0.f, s11 = 0.f;
#pragma unroll 1
      for (int c0 = lane; c0 < pieces; c0 += 64) {
        uint4 a0[2], a1[2], w0[2], w1[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const int c = c0 + 32 * k;
          const bool in = c < pieces;
          const uint4 z = make_uint4(0u, 0u, 0u, 0u);
          a0[k] = in ? __ldcg(pa0 + c) : z;
          a1[k] = in ? __ldcg(pa1 + c) : z;
          w0[k] = in ? __ldcg(pw0 + c) : z;
          w1[k] = in ? __ldcg(pw1 + c) : z;
        }
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          const uint32_t x0[4] = {a0[k].x, a0[k].y, a0[k].z, a0[k].w}, x1[4] = {a1[k].x, a1[k].y, a1[k].z, a1[k].w};
          const uint32_t u0[4] = {w0[k].x, w0[k].y, w0[k].z, w0[k].w}, u1[4] = {w1[k].x, w1[k].y, w1[k].z, w1[k].w};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float x0l = __uint_as_float(x0[q] << 16), x0h = __uint_as_float(x0[q] & 0xFFFF0000u);
            const float x1l = __uint_as_float(x1[q] << 16), x1h = __uint_as_float(x1[q] & 0xFFFF0000u);
            const float u0l = __uint_as_float(u0[q] << 16), u0h = __uint_as_float(u0[q] & 0xFFFF0000u);
            const float u1l = __uint_as_float(u1[q] << 16), u1h = __uint_as_float(u1[q] & 0xFFFF0000u);
            s00 += x0l * u0l; s00 += x0h * u0h;
            s01 += x0l * u1l; s01 += x0h * u1h;
            s10 += x1l * u0l; s10 += x1h * u0h;
            s11 += x1l * u1l; s11 += x1h * u1h;
          }
        }
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        s00 += __shfl_xor_sync(0xffffffffu, s00, off);
        s01 += __shfl_xor_sync(0xffffffffu, s01, off);
        s10 += __shfl_xor_sync(0xffffffffu, s10, off);
        s11 += __shfl_xor_sync(0xffffffffu, s11, off);
      }
      if (lane < 4) {
        const int r = r0 + (lane >> 1), o = o0 + (lane & 1);
        const float sv = lane == 0 ? s00 : (lane == 1 ? s01 : (lane == 2 ? s10 : s11));
        if (r < p.B && o < yo.N) {
          float z = sv + (yo.bias != nullptr ? yo.bias[o] : 0.f);
          if (yo.relu) z = fmaxf(z, 0.f);
          yo.A[(size_t)r * yo.N + o] = __float2bfloat16_rn(yo.alpha * z);
        }
      }
    } else {
      const int o = it - n_col - n_out;
      float s = 0.f;
#pragma unroll
      for (int k = 0; k < 4; ++k) s += sdO[o * 128 + lane * 4 + k];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
      if (lane == 0) yo.db[o] = s;
    }
  }
  // the output layer's weight gradient is zero at the dropped fan-in columns
  if (first && dpi > 1) {
    const int gthreads = G * MP_CC_THREADS, gtid = rcta * MP_CC_THREADS + ct;
#pragma unroll 1
    for (int u = gtid; u < yo.N * yo.K; u += gthreads) {
      const int o = u / yo.K, c = u - o * yo.K;
      const int rel = c - bi;
      if (rel >= 0 && rel % dpi == 0) continue;
      if (yo.dW_is_f32) reinterpret_cast<float*>(yo.dW)[(size_t)o * yo.ldw + c] = 0.f;
      else reinterpret_cast<__nv_bfloat16*>(yo.dW)[(size_t)o * yo.ldw + c] = __float2bfloat16_rn(0.f);
    }
  }
}

__global__ void __launch_bounds__(MP_THREADS, 1) ard_mlp_persistent_kernel(const __grid_constant__ MpParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw_addr);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = (int)gridDim.x, cta = (int)blockIdx.x;
  const int H = p.L - 1;  // hidden layers; layer H is the output layer

  const uint32_t bar_base = base + MP_BAR_OFF;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (MP_STAGES + s); };
  auto tfull_bar = [&](int w) { return bar_base + 8u * (2 * MP_STAGES + w); };
  const uint32_t tempty_bar = bar_base + 8u * (2 * MP_STAGES + MP_NI);
  unsigned long long* s_cdf = reinterpret_cast<unsigned long long*>(smem + MP_CDF_OFF);
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(smem + MP_MISC_OFF);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + MP_MISC_OFF + 4);
  volatile int* stop_flag = reinterpret_cast<volatile int*>(smem + MP_MISC_OFF + 8);
  volatile int* s_njobs = reinterpret_cast<volatile int*>(smem + MP_MISC_OFF + 96);  // [stage]
  LayerRt* s_rt = reinterpret_cast<LayerRt*>(smem + MP_MISC_OFF + 16);  // [MP_MAX_LAYERS]
  unsigned long long* s_count = reinterpret_cast<unsigned long long*>(smem + MP_MISC_OFF + 16 + 16 * MP_MAX_LAYERS);
  GemmJob* jobs = reinterpret_cast<GemmJob*>(smem + MP_MISC_OFF + 128);  // [stage][2]

  // A block-wide barrier counts a warp once, whichever of its lanes execute it: every warp first waits for its own
  // lanes (the lanes of the producer warp and lane 0 of the issuing warps come out of their loops one by one).
  auto block_sync = [&]() {
    __syncwarp();
    __syncthreads();
  };

  // ---- set-up: barriers, tensor memory, the patterns of this iteration ----
  if (tid == 0) {
    for (int s = 0; s < MP_STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int w = 0; w < MP_NI; ++w) mbar_init(tfull_bar(w), 1);
    mbar_init(tempty_bar, MP_EPI_WARPS);
    *abort_flag = 0;
    *stop_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_ptr_smem)), MP_TMEM_COLS);
    tmem_relinquish();
  }
  if (p.any_sampled && tid < p.ndp) s_cdf[tid] = p.cdf[tid];
  if (warp >= MP_CC_W0) {
    // the loss gradient as floats, output-major [MP_SMALL_N][128]: an input of the iteration, read by the epilogue
    // of the last hidden layer and by the output layer's gradients
    float* sdO = reinterpret_cast<float*>(smem + MP_SDO_OFF);
    const MpLayer& yo = p.layer[H];
    const int ct = tid - MP_CC_W0 * 32;
    float dv[128 * MP_SMALL_N / MP_CC_THREADS];
#pragma unroll
    for (int k = 0; k < 128 * MP_SMALL_N / MP_CC_THREADS; ++k) {
      const int e = ct + k * MP_CC_THREADS;
      const int o = e >> 7, r = e & 127;
      dv[k] = (r < p.B && o < yo.N) ? __bfloat162float(p.dOut[(size_t)r * p.lddout + o]) : 0.f;
    }
#pragma unroll
    for (int k = 0; k < 128 * MP_SMALL_N / MP_CC_THREADS; ++k) sdO[ct + k * MP_CC_THREADS] = dv[k];
  }
  if (tid == 64) *s_count = (p.any_sampled && p.counter != nullptr) ? *p.counter : 0ull;
  tc_fence_before();
  block_sync();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_smem;
  if (tid <= H) {
    // Every CTA draws for itself (Sec. 3.4): Philox on (iteration, layer stream), the period from the integer
    // cumulative table of K, the offset uniform in 1..dp.  A layer that is not sampled keeps what its header holds.
    const MpLayer& y = p.layer[tid];
    int dp, b;
    if (y.sample) {
      const unsigned long long iteration = p.iteration_base + *s_count;
      uint32_t c[4] = {(uint32_t)iteration, (uint32_t)(iteration >> 32), y.stream_id, 0u};
      philox4x32_10(c, (uint32_t)p.seed, (uint32_t)(p.seed >> 32));
      int lo = 0, hi = p.ndp - 1;
      const unsigned long long r0 = c[0];
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (r0 < s_cdf[mid]) hi = mid; else lo = mid + 1;
      }
      dp = lo + 1;
      b = 1 + (int)(((unsigned long long)c[1] * (unsigned long long)dp) >> 32);
    } else {
      dp = y.hdr[HDR_DP];
      b = y.hdr[HDR_B];
    }
    LayerRt r;
    r.dp = dp;
    r.bb = b - 1;
    r.n = (y.N - b) / dp + 1;
    r.npad = (r.n + 63) / 64 * 64;
    s_rt[tid] = r;
  }
  block_sync();
  // the patterns and the stage's products are read from shared memory: indexed by layer they would otherwise sit
  // in local memory, for whose lines the 200 KB of shared memory leave almost no L1
  const LayerRt* rt = s_rt;
  if (tid < 2 * H) s_njobs[tid] = mp_make_jobs(p, rt, H, G, cta, tid, jobs + 2 * tid);
  block_sync();

  // per-role running counters: contraction blocks and tiles this CTA has been through
  int gblk = 0, git = 0;
  unsigned int barrier_no = 0;
  const int n_stages = 2 * H;
  const int nt0 = jobs[0].nt;  // tile width of layer 0

  // The first layer's weight is read in place: its kept rows are b-1, b-1+dp, ... (Eq. 1), which a descriptor
  // with the pitch dp x ldw follows.  The producer warp fits the two box shapes it will use to the pattern.
  const int v0 = nt0 == 16 ? 0 : (nt0 == 32 ? 1 : 2);
  const CUtensorMap* mapW0f = &p.mapWf[0][v0].tm;
  const CUtensorMap* mapW0b = &p.mapWb[0].tm;
  if (warp == 0) {
    // every descriptor of the iteration is asked for now: the first copy through a descriptor the TMA unit has
    // not seen waits for the descriptor itself, a memory round trip at the head of every stage
    {
      const TcMap* first = &p.mapXk;
      constexpr int NMAPS = 2 + 4 * (MP_MAX_LAYERS - 1) + 3 * (MP_MAX_LAYERS - 1) + (MP_MAX_LAYERS - 1);
      if (lane < NMAPS) asm volatile("prefetch.tensormap [%0];" ::"l"(&first[lane].tm) : "memory");
    }
    CUtensorMap* slots = p.tm_slots + (size_t)cta * ARD_TM_LSTM_SLOTS;
    mapW0f = tensormap_specialise(&p.mapWf[0][v0], rt[0].dp, rt[0].bb + 1, rt[0].n, smem, slots, lane);
    mapW0b = tensormap_specialise(&p.mapWb[0], rt[0].dp, rt[0].bb + 1, rt[0].n, smem + 128, slots + 1, lane);
    fence_proxy_async_smem();
    if (mapW0f != &p.mapWf[0][v0].tm) tensormap_acquire(mapW0f);
    if (mapW0b != &p.mapWb[0].tm) tensormap_acquire(mapW0b);
    if (lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(mapW0f) : "memory");
    if (lane == 1) asm volatile("prefetch.tensormap [%0];" ::"l"(mapW0b) : "memory");
  }

  // The output weights of a tile's neurons of the last hidden layer (columns bb + j dp of the output layer's
  // weight), [chunk][output][16], into an epilogue warp's own staging block: no other warp is waited for.  All
  // loads of a round are issued before the first one is used: rolled up, each would wait for the one before it.
  auto stage_out_weights = [&](float* stg, int t, int nt, int lane_) {
    const MpLayer& yo = p.layer[H];
    const int l = H - 1;
    const int total = (nt / 16) * 256;
#pragma unroll 1
    for (int e0 = 0; e0 < total; e0 += 512) {
      float wv[16];
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        const int e = e0 + lane_ + 32 * k;
        const int o = (e >> 4) & 15;
        const int col = t * nt + (e >> 8) * 16 + (e & 15);
        wv[k] = 0.f;
        if (e < total && o < yo.N && col < rt[l].n)
          wv[k] = __bfloat162float(yo.W[(size_t)o * yo.ldw + rt[l].bb + (size_t)col * rt[l].dp]);
      }
#pragma unroll
      for (int k = 0; k < 16; ++k)
        if (e0 + lane_ + 32 * k < total) stg[e0 + lane_ + 32 * k] = wv[k];
    }
  };
  // With more than one hidden layer the last one's product is stages away: its first tile's output weights are
  // fetched now, off that stage's critical path (the stages before it leave this part of the staging block alone).
  if (H > 1 && warp >= MP_EPI_W0 && warp < MP_CC_W0 && jobs[2 * (H - 1)].mine > 0)
    stage_out_weights(reinterpret_cast<float*>(smem + MP_STG_OFF) + (warp - MP_EPI_W0) * MP_STG_WORDS,
                      jobs[2 * (H - 1)].tile[0], jobs[2 * (H - 1)].nt, lane);

  for (int st = 0; st < n_stages; ++st) {
    // ---- the products of this stage (set up by thread 0 before the barrier that opened the stage) ----
    const int njobs = s_njobs[st];
    const GemmJob* job = jobs + 2 * st;
    // no tile in the first stage: the warps of the tile pipeline help to pack the weights
    const bool helper = st == 0 && warp < MP_CC_W0 && job[0].mine == 0;
    if (helper) {
      // (their work is below, with the CUDA-core warps')
    } else if (warp == 0) {
      // ===================== producer =====================
      // Lane s owns ring stage s: it waits for the stage, announces the bytes and issues the two or three boxes
      // of every block that falls on its stage, so up to MP_STAGES blocks are requested at once (one thread
      // issuing box after box, with a barrier hand-off each, paces at ~400 cycles per box).
      int stage_blocks = 0;  // contraction blocks of this CTA in this stage
      for (int q = 0; q < njobs; ++q) stage_blocks += job[q].mine * job[q].nkb;
      if (lane < MP_STAGES) {
        int d = (lane - gblk % MP_STAGES + MP_STAGES) % MP_STAGES;  // this lane's first block among the stage's blocks
        int seq0 = 0;
        bool ok = true;
#pragma unroll 1
        for (int q = 0; q < njobs && ok; ++q) {
          const GemmJob& j = job[q];
          const int l = j.l;
          const CUtensorMap* ma;
          const CUtensorMap* mb;
          if (j.type == JT_F) {
            ma = l == 0 ? &p.mapXk.tm : &p.mapAk[l - 1].tm;
            mb = l == 0 ? mapW0f : &p.mapWf[l][j.nt == 16 ? 0 : (j.nt == 32 ? 1 : 2)].tm;
          } else if (j.type == JT_BD) {
            ma = &p.mapdZk[l].tm;
            mb = l == 0 ? mapW0b : &p.mapWb[l].tm;
          } else {
            ma = &p.mapdZm[l].tm;
            mb = l == 0 ? &p.mapXm.tm : &p.mapAm[l - 1].tm;
          }
          const uint32_t bytes = (uint32_t)(MP_A_BYTES + (j.type == JT_F ? j.nt * 128 : MP_B_BYTES));
#pragma unroll 1
          for (int ti = 0; ti < j.mine && ok; ++ti, seq0 += j.nkb) {
            const int t = j.tile[ti];
#pragma unroll 1
            for (; d < seq0 + j.nkb; d += MP_STAGES) {
              const int kb = d - seq0;
              const uint32_t phase = (uint32_t)((gblk + d) / MP_STAGES) & 1u;
              if (!mp_wait(empty_bar(lane), phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
              const uint32_t sA = base + lane * MP_STAGE_BYTES;
              const uint32_t sB = sA + MP_A_BYTES;
              mbar_arrive_expect_tx(full_bar(lane), bytes);
              const int kx = kb * MP_BK;
              if (j.type == JT_F) {
                tma_load_2d(sA, ma, full_bar(lane), kx, 0);
                tma_load_2d(sB, mb, full_bar(lane), kx, t * j.nt);
              } else if (j.type == JT_BD) {
                tma_load_2d(sA, ma, full_bar(lane), kx, 0);
                tma_load_2d(sB, mb, full_bar(lane), t * 64, kx);
              } else {
                const int mt = t / j.ntn, ni = t - mt * j.ntn;
                tma_load_2d(sA, ma, full_bar(lane), mt * 128, kx);
                tma_load_2d(sA + 8192u, ma, full_bar(lane), mt * 128 + 64, kx);
                tma_load_2d(sB, mb, full_bar(lane), ni * 64, kx);
              }
            }
          }
        }
      }
      gblk += stage_blocks;
    } else if (warp <= MP_NI) {
      // ===================== MMA issuers: warp 1 + w takes blocks w, w + NI, ... of a tile =====================
      const int w = warp - 1;
      if (lane == 0) {
        bool ok = true;
#pragma unroll 1
        for (int q = 0; q < njobs && ok; ++q) {
          const GemmJob& j = job[q];
          const bool a_mn = j.type == JT_BW, b_mn = j.type != JT_F;
          const uint64_t desc_a_hi = a_mn ? make_desc(0, 64 * MP_BK * 2, 1024) : make_desc(0, 16, 1024);
          const uint64_t desc_b_hi = b_mn ? make_desc(0, 64 * MP_BK * 2, 1024) : make_desc(0, 16, 1024);
          const uint32_t idesc = make_idesc(j.nt, a_mn, b_mn, 128);
          const uint32_t d_tmem = tmem_base + (uint32_t)(w * MP_ACC_COLS);
#pragma unroll 1
          for (int ti = 0; ti < j.mine && ok; ++ti, ++git, gblk += j.nkb) {
            // the epilogue warps have taken the previous tile's sums out of the accumulators
            if (!mp_wait(tempty_bar, ((uint32_t)git & 1u) ^ 1u, abort_flag, p.status)) { ok = false; break; }
            tc_fence_after();
#pragma unroll 1
            for (int kb = w; kb < j.nkb; kb += MP_NI) {
              const int g = gblk + kb;
              const int stage = g % MP_STAGES;
              const uint32_t phase = (uint32_t)(g / MP_STAGES) & 1u;
              if (!mp_wait(full_bar(stage), phase, abort_flag, p.status)) { ok = false; break; }
              tc_fence_after();
              const uint32_t sA = base + stage * MP_STAGE_BYTES;
              const uint64_t ad0 = desc_a_hi | (uint64_t)((sA & 0x3FFFFu) >> 4);
              const uint64_t bd0 = desc_b_hi | (uint64_t)(((sA + MP_A_BYTES) & 0x3FFFFu) >> 4);
#pragma unroll
              for (int s = 0; s < MP_BK / 16; ++s) {
                const uint64_t ad = ad0 + (uint64_t)(s * (a_mn ? 128 : 2));
                const uint64_t bd = bd0 + (uint64_t)(s * (b_mn ? 128 : 2));
                tc_mma_bf16(d_tmem, ad, bd, idesc, (kb != w || s != 0) ? 1u : 0u);
              }
              tc_commit(empty_bar(stage));
            }
            if (!ok) break;
            if (w < j.nkb) tc_commit(tfull_bar(w));
            else mbar_arrive(tfull_bar(w));  // no block of this tile was this warp's
          }
        }
      }
    } else if (warp < MP_CC_W0) {
      // ===================== epilogue warps =====================
      const int quad = warp & 3;     // the tensor-memory lanes a warp may read: 32 x (warp id mod 4)
      float* stg = reinterpret_cast<float*>(smem + MP_STG_OFF) + (warp - MP_EPI_W0) * MP_STG_WORDS;
      const int row = quad * 32 + lane;  // accumulator row of this thread
      const bool row_ok = row < p.B;
      bool ok = true;
#pragma unroll 1
      for (int q = 0; q < njobs && ok; ++q) {
        const GemmJob& j = job[q];
        const int l = j.l;
        const MpLayer& y = p.layer[l];
        const int nacc = min(MP_NI, j.nkb);
        const bool fused_dz = j.type == JT_F && l == H - 1;  // the output layer's input gradient rides along
        const MpLayer& yo = p.layer[H];
        const int nch = j.nt / 16;  // 16-column chunks of the tile
        // weight gradient: where the kept fan-in columns go (Eq. 1)
        const int dpi = (j.type == JT_BW && l > 0) ? rt[l - 1].dp : 1, bi = (j.type == JT_BW && l > 0) ? rt[l - 1].bb : 0;
        const int nin = l == 0 ? y.K : rt[l - 1].n;
#pragma unroll 1
        for (int ti = 0; ti < j.mine && ok; ++ti, ++git) {
          const int t = j.tile[ti];
          // ---- what does not depend on the accumulators is fetched while the products run ----
          __syncwarp();
          if (j.type == JT_F) {
            // biases of the tile's neurons behind the (at most) 1024 staged output weights
#pragma unroll
            for (int k = 0; k < 2; ++k) {
              const int jj = lane + 32 * k, jc = t * j.nt + jj;
              stg[1024 + jj] = (y.bias != nullptr && jj < j.nt && jc < rt[l].n) ? __ldg(y.bias + rt[l].bb + (size_t)jc * rt[l].dp) : 0.f;
            }
            if (fused_dz) {
              // the first tile's output weights were staged before the first stage (see below)
              if (ti > 0 || H == 1) stage_out_weights(stg, t, j.nt, lane);
            }
          } else if (j.type == JT_BD && l > 0) {
            // the bf16 outputs of the layer below, this thread's 64 columns (ReLU adjoint): 8 x 16 bytes at
            // words 36 r .. of the staging block
            const MpLayer& yp = p.layer[l - 1];
            uint4 a[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
              a[k] = make_uint4(0u, 0u, 0u, 0u);
              if (yp.relu && row_ok) a[k] = __ldcg(reinterpret_cast<const uint4*>(yp.A + (size_t)row * yp.N + t * 64) + k);
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) reinterpret_cast<uint4*>(stg + lane * 36)[k] = a[k];
          }
          __syncwarp();
          bool all = true;
#pragma unroll
          for (int w = 0; w < MP_NI; ++w) all = all && mp_wait(tfull_bar(w), (uint32_t)git & 1u, abort_flag, p.status);
          if (!all) { ok = false; break; }
          tc_fence_after();
          if (j.type == JT_BW) {
            // Weight gradient: accumulator row = kept neuron mt*128 + row, columns = kept fan-in ni*64 ...  The whole
            // 32 x 64 block of the warp leaves tensor memory first; then the warp stores one neuron's 64 values after
            // the other at the kept fan-in columns (Eq. 1) of the full-width gradient.  Everything between and around
            // them was cleared in the forward stages (mp_zero_fill): one SM stores ~25 GB/s, so a tile that wrote its
            // whole span with the zeros in it (256 KB at a period of 8) took 12 us, while the clearing is spread over
            // all SMs and the stages in which the tensor cores set the pace.
#pragma unroll 1
            for (int ch = 0; ch < nch; ++ch) {
              float acc[16];
#pragma unroll
              for (int e = 0; e < 16; ++e) acc[e] = 0.f;
              {
                static_assert(MP_NI == 2, "two accumulators are read side by side");
                uint32_t r0[16], r1[16];
                const uint32_t ta = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(ch * 16);
                tmem_ld16(ta, r0);
                if (nacc > 1) tmem_ld16(ta + MP_ACC_COLS, r1);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 16; ++e) acc[e] = __uint_as_float(r0[e]) + (nacc > 1 ? __uint_as_float(r1[e]) : 0.f);
              }
#pragma unroll
              for (int e = 0; e < 16; ++e) stg[lane * MP_STG_LD + ch * 16 + e] = acc[e];
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar);
            const int mt = t / j.ntn, ni = t - mt * j.ntn;
            const int i0 = mt * 128 + quad * 32;
            const int nrows = min(32, rt[l].n - i0);
            const int jn = min(64, nin - ni * 64);  // kept fan-in columns of this tile
            if (dpi == 1) {
              // contiguous fan-in (the first layer, or a dense layer below): 16 bytes per lane, so an instruction
              // writes two whole 256-byte row pieces (fp32) or four of 128 bytes (bf16).  A store instruction costs a
              // warp ~150 cycles here whatever its width, so the width is what sets the epilogue's pace.
              __syncwarp();
              if (y.dW_is_f32) {
                const int sub = lane >> 4, pc = (lane & 15) * 4;
#pragma unroll 1
                for (int rr = sub; rr < nrows; rr += 2) {
                  if (pc < jn) {
                    const float* sp = stg + rr * MP_STG_LD + pc;
                    float* d = reinterpret_cast<float*>(y.dW) + ((size_t)rt[l].bb + (size_t)(i0 + rr) * rt[l].dp) * y.ldw + ni * 64 + pc;
                    *reinterpret_cast<float4*>(d) = make_float4(sp[0], sp[1], sp[2], sp[3]);
                  }
                }
              } else {
                const int sub = lane >> 3, pc = (lane & 7) * 8;
#pragma unroll 1
                for (int rr = sub; rr < nrows; rr += 4) {
                  if (pc < jn) {
                    const float* sp = stg + rr * MP_STG_LD + pc;
                    __nv_bfloat16* d = reinterpret_cast<__nv_bfloat16*>(y.dW) + ((size_t)rt[l].bb + (size_t)(i0 + rr) * rt[l].dp) * y.ldw + ni * 64 + pc;
                    *reinterpret_cast<uint4*>(d) = make_uint4(mp_pack(sp[0], sp[1]), mp_pack(sp[2], sp[3]), mp_pack(sp[4], sp[5]), mp_pack(sp[6], sp[7]));
                  }
                }
              }
            } else {
#pragma unroll 1
              for (int rr = 0; rr < nrows; ++rr) {
                const size_t off = ((size_t)rt[l].bb + (size_t)(i0 + rr) * rt[l].dp) * y.ldw + bi;
                const float* sp = stg + rr * MP_STG_LD;
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                  const int jj = lane + 32 * k;
                  if (jj < jn) {
                    const size_t c = off + (size_t)(ni * 64 + jj) * dpi;
                    if (y.dW_is_f32) reinterpret_cast<float*>(y.dW)[c] = sp[jj];
                    else reinterpret_cast<__nv_bfloat16*>(y.dW)[c] = __float2bfloat16_rn(sp[jj]);
                  }
                }
              }
            }
            continue;
          }
#pragma unroll 1
          for (int ch = 0; ch < nch; ++ch) {
            // this chunk of the tile: the accumulators added in issuing-warp order
            float acc[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) acc[e] = 0.f;
            {
              uint32_t r0[16], r1[16];
              const uint32_t ta = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(ch * 16);
              tmem_ld16(ta, r0);
              if (nacc > 1) tmem_ld16(ta + MP_ACC_COLS, r1);
              tmem_ld_wait();
#pragma unroll
              for (int e = 0; e < 16; ++e) acc[e] = __uint_as_float(r0[e]) + (nacc > 1 ? __uint_as_float(r1[e]) : 0.f);
            }
            if (ch == nch - 1) {  // the accumulators may be overwritten from here on
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(tempty_bar);
            }
            if (j.type == JT_F) {
              const int j0 = t * j.nt + ch * 16;
              float dz[16];
#pragma unroll
              for (int e = 0; e < 16; ++e) {
                float z = 0.f;
                if (j0 + e < rt[l].n) {
                  z = acc[e] + stg[1024 + ch * 16 + e];
                  if (y.relu) z = fmaxf(z, 0.f);
                  z *= y.alpha;
                }
                acc[e] = z;
              }
              if (fused_dz) {
#pragma unroll
                for (int e = 0; e < 16; ++e) dz[e] = 0.f;
                const float* sdOe = reinterpret_cast<const float*>(smem + MP_SDO_OFF) + row;
#pragma unroll 1
                for (int o = 0; o < yo.N; ++o) {
                  const float g = sdOe[o * 128];
                  const float4* wq = reinterpret_cast<const float4*>(stg + (ch * MP_SMALL_N + o) * 16);
#pragma unroll
                  for (int q4 = 0; q4 < 4; ++q4) {
                    const float4 w4 = wq[q4];
                    dz[4 * q4] += g * w4.x;
                    dz[4 * q4 + 1] += g * w4.y;
                    dz[4 * q4 + 2] += g * w4.z;
                    dz[4 * q4 + 3] += g * w4.w;
                  }
                }
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                  const uint32_t bits = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(acc[e]));
                  const bool pass = !y.relu || bf16_bits_positive(bits);
                  dz[e] = (j0 + e < rt[l].n && pass) ? y.alpha * dz[e] : 0.f;
                }
              }
              if (row_ok) {
                store16_bf16(y.A + (size_t)row * y.N + j0, acc);
                if (fused_dz) store16_bf16(y.dZ + (size_t)row * y.N + j0, dz);
              }
            } else if (j.type == JT_BD) {
              const int j0 = t * 64 + ch * 16;
              if (l > 0) {
                const MpLayer& yp = p.layer[l - 1];
                const int np = rt[l - 1].n;
                const uint4 k0 = reinterpret_cast<const uint4*>(stg + lane * 36)[2 * ch];
                const uint4 k1 = reinterpret_cast<const uint4*>(stg + lane * 36)[2 * ch + 1];
                const uint32_t wb[8] = {k0.x, k0.y, k0.z, k0.w, k1.x, k1.y, k1.z, k1.w};
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                  const uint32_t bits = (wb[e >> 1] >> ((e & 1) * 16)) & 0xFFFFu;
                  const bool pass = !yp.relu || bf16_bits_positive(bits);
                  acc[e] = (j0 + e < np && pass) ? yp.alpha * acc[e] : 0.f;
                }
                if (row_ok) store16_bf16(yp.dZ + (size_t)row * yp.N + j0, acc);
              } else if (row_ok) {
                const int K0 = p.layer[0].K;
                __nv_bfloat16* d = p.dX + (size_t)row * p.lddx + j0;
                if (j0 + 16 <= K0) {
                  store16_bf16(d, acc);
                } else {
#pragma unroll
                  for (int e = 0; e < 16; ++e)
                    if (j0 + e < K0) d[e] = __float2bfloat16_rn(acc[e]);
                }
              }
            }
          }
          // the last forward tile also clears the columns up to the next multiple of 64: they are multiplied (by
          // the zeros of the packed weight) when this matrix is an operand
          if (j.type == JT_F && t == j.items - 1 && row_ok) {
            const uint4 z4 = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll 1
            for (int c0 = (t + 1) * j.nt; c0 < rt[l].npad; c0 += 16) {
              uint4* d = reinterpret_cast<uint4*>(y.A + (size_t)row * y.N + c0);
              d[0] = z4; d[1] = z4;
              if (fused_dz) {
                uint4* d2 = reinterpret_cast<uint4*>(y.dZ + (size_t)row * y.N + c0);
                d2[0] = z4; d2[1] = z4;
              }
            }
          }
        }
      }
    } else {
      // ===================== CUDA-core warps: the rest of the stage, beside the tiles =====================
      const int ct = tid - MP_CC_W0 * 32;
      if (st >= H) {
        const float* sdO = reinterpret_cast<const float*>(smem + MP_SDO_OFF);
        mp_backward_jobs(p, rt, H, st, sdO, cta, G, ct);
      }
      if (st < H) mp_zero_fill(p, rt, H, st, cta, G, ct);
    }

    if (st == 0 && (warp >= MP_CC_W0 || helper)) {
      // kept lists and packed weights: the CUDA-core warps of every CTA and the idle warps of the CTAs without a tile
      const int T = min(G, job[0].items);  // CTAs 0 .. T-1 have a tile
      const int gthreads = G * MP_CC_THREADS + (G - T) * (MP_CC_W0 * 32);
      const int gtid = helper ? G * MP_CC_THREADS + (cta - T) * (MP_CC_W0 * 32) + tid : cta * MP_CC_THREADS + (tid - MP_CC_W0 * 32);
      mp_forward_jobs(p, rt, H, cta, G, helper ? -1 : tid - MP_CC_W0 * 32, gtid, gthreads);
    }

    // ---- grid-wide barrier (none behind the last stage) ----
    if (st + 1 < n_stages) {
      block_sync();
      if (tid == 0) {
        __threadfence();
        atomicAdd(p.bar, 1u);
        ++barrier_no;
        mp_grid_wait(p.bar, barrier_no * (unsigned int)G, abort_flag, p.status);
        *stop_flag = *abort_flag;
        // the draw of this iteration has been read by every CTA: the next launch draws the next one
        if (st == 0 && cta == 0 && p.any_sampled && p.counter != nullptr && !*abort_flag) *p.counter = *s_count + 1ull;
      }
      block_sync();
      // what other CTAs stored with ordinary stores is read by TMA from here on
      asm volatile("fence.proxy.async.global;" ::: "memory");
      if (*stop_flag) break;
    }
  }

  // ---- teardown ----
  tc_fence_before();
  block_sync();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, MP_TMEM_COLS);
  }
}

bool aligned16(const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) == 0; }

}  // namespace

// Runs the iteration in the kernel above if the stack fits it; ARD_ERR_UNSUPPORTED (nothing enqueued) tells the
// caller to take the call-by-call path.
ard_status launch_mlp_persistent(ard_ctx* ctx, const ard_mlp_layer* layers, int n_layers, int B, const void* X, int ldx,
                                 const void* dOut, int lddout, void* dX, int lddx, int dist_id, uint64_t seed,
                                 uint64_t iteration_base, uint64_t* iteration_counter, cudaStream_t s) {
  if (n_layers < 2 || n_layers > MP_MAX_LAYERS || B < 1 || B > 128) return ARD_ERR_UNSUPPORTED;
  if (ctx->sm_count > ARD_TM_LSTM_BLOCKS) return ARD_ERR_UNSUPPORTED;
  if (!aligned16(X) || ldx % 8 != 0 || (dX != nullptr && (!aligned16(dX) || lddx % 8 != 0))) return ARD_ERR_UNSUPPORTED;
  const int H = n_layers - 1;
  bool any_sampled = false;
  for (int l = 0; l < n_layers; ++l) {
    const ard_mlp_layer& y = layers[l];
    if (y.pat->kind != ARD_ROW || y.pat->units != y.N) return ARD_ERR_UNSUPPORTED;
    if (y.K % 8 != 0 || y.ldw % 8 != 0 || y.ldw < y.K || !aligned16(y.W) || !aligned16(y.dW)) return ARD_ERR_UNSUPPORTED;
    if (l > 0 && (!y.Wk || !aligned16(y.Wk))) return ARD_ERR_UNSUPPORTED;
    if (l < H) {
      // no CTA may be dealt more tiles of a product than its list holds (half of the SMs is the fewest the weight
      // gradient is spread over)
      const int bw_tiles = ((y.N + 127) / 128) * ((y.K + 63) / 64), half = ctx->sm_count / 2 > 0 ? ctx->sm_count / 2 : 1;
      if ((bw_tiles + half - 1) / half + 5 > MP_MAX_MINE || y.N > 32767 || y.K > 32767) return ARD_ERR_UNSUPPORTED;
      if (!y.compact_out || y.N % 64 != 0 || !y.dZ || !aligned16(y.A) || !aligned16(y.dZ)) return ARD_ERR_UNSUPPORTED;
      if (y.sample) any_sampled = true;
    } else {
      // the output layer: narrow, dense, not sampled
      if (y.N > MP_SMALL_N || y.compact_out || y.sample || y.pat->dp_bound != 1) return ARD_ERR_UNSUPPORTED;
    }
  }
  const ArdDistribution* d = nullptr;
  if (any_sampled) {
    if (dist_id < 0 || dist_id >= ARD_MAX_DISTRIBUTIONS || !iteration_counter) return ARD_ERR_UNSUPPORTED;
    d = &ctx->dist[dist_id];
    if (d->ndp == 0 || d->ndp > 64) return ARD_ERR_UNSUPPORTED;
    for (int l = 0; l < H; ++l)
      if (layers[l].sample && d->ndp > layers[l].pat->units) return ARD_ERR_UNSUPPORTED;
  }
  static int probed[64] = {};
  const int dev = ctx->device & 63;
  if (probed[dev] == 0) {
    int n = 0;
    if (cudaFuncSetAttribute(ard_mlp_persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MP_SMEM) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, ard_mlp_persistent_kernel, MP_THREADS, MP_SMEM) != cudaSuccess ||
        n < 1)
      probed[dev] = -1;
    else
      probed[dev] = 1;
  }
  if (probed[dev] < 1) { (void)cudaGetLastError(); return ARD_ERR_UNSUPPORTED; }

  MpParams p = {};
  p.L = n_layers; p.B = B;
  p.ldx = ldx; p.lddout = lddout; p.lddx = lddx;
  p.X = reinterpret_cast<const __nv_bfloat16*>(X);
  p.dOut = reinterpret_cast<const __nv_bfloat16*>(dOut);
  p.dX = reinterpret_cast<__nv_bfloat16*>(dX);
  p.tm_slots = ctx->d_tm_slots + (size_t)ARD_TM_SM_MAX * ARD_TM_SLOTS;
  p.cdf = d ? d->d_cdf : nullptr;
  p.ndp = d ? d->ndp : 0;
  p.any_sampled = any_sampled ? 1 : 0;
  p.seed = seed; p.iteration_base = iteration_base;
  p.counter = reinterpret_cast<unsigned long long*>(iteration_counter);
  p.bar = ctx->d_grid_bar;
  p.status = ctx->d_status;
  ard_status st = ard_encode_tcmap(ctx, X, B, layers[0].K, ldx, 0, MAP_PLAIN, 128, 64, &p.mapXk);
  if (st == ARD_OK) st = ard_encode_tcmap(ctx, X, B, layers[0].K, ldx, 0, MAP_PLAIN, 64, 64, &p.mapXm);
  if (st != ARD_OK) return st;
  for (int l = 0; l < n_layers; ++l) {
    const ard_mlp_layer& y = layers[l];
    MpLayer& q = p.layer[l];
    q.K = y.K; q.N = y.N; q.ldw = y.ldw;
    q.relu = y.relu; q.dW_is_f32 = y.dW_is_f32; q.sample = y.sample;
    q.alpha = y.alpha;
    q.stream_id = (uint32_t)(l + 1);
    q.W = reinterpret_cast<const __nv_bfloat16*>(y.W);
    q.bias = y.bias;
    q.Wk = reinterpret_cast<__nv_bfloat16*>(y.Wk);
    q.A = reinterpret_cast<__nv_bfloat16*>(y.A);
    q.dZ = reinterpret_cast<__nv_bfloat16*>(y.dZ);
    q.dW = y.dW;
    q.db = y.db;
    q.hdr = y.pat->d_hdr;
    q.idx = y.pat->d_idx;
    q.Tr = y.pat->Tr; q.Tc = y.pat->Tc; q.ts = y.pat->ts;
    if (l < H) {
      st = ard_encode_tcmap(ctx, y.A, B, y.N, y.N, 0, MAP_PLAIN, 128, 64, &p.mapAk[l]);
      if (st == ARD_OK) st = ard_encode_tcmap(ctx, y.A, B, y.N, y.N, 0, MAP_PLAIN, 64, 64, &p.mapAm[l]);
      if (st == ARD_OK) st = ard_encode_tcmap(ctx, y.dZ, B, y.N, y.N, 0, MAP_PLAIN, 128, 64, &p.mapdZk[l]);
      if (st == ARD_OK) st = ard_encode_tcmap(ctx, y.dZ, B, y.N, y.N, 0, MAP_PLAIN, 64, 64, &p.mapdZm[l]);
      const void* wsrc = l == 0 ? y.W : y.Wk;  // layer 0 reads the weight in place (kept rows), the others the packed copy
      const int variant = l == 0 ? MAP_STRIDED_ROWS : MAP_PLAIN;
      const int units = l == 0 ? y.N : 0;
      for (int v = 0; v < 3 && st == ARD_OK; ++v)
        st = ard_encode_tcmap(ctx, wsrc, y.N, y.K, y.ldw, units, variant, 16 << v, 64, &p.mapWf[l][v]);
      if (st == ARD_OK) st = ard_encode_tcmap(ctx, wsrc, y.N, y.K, y.ldw, units, variant, 64, 64, &p.mapWb[l]);
      if (st != ARD_OK) return st;
    }
  }
  if (cudaMemsetAsync(ctx->d_grid_bar, 0, sizeof(unsigned int), s) != cudaSuccess) return ARD_ERR_CUDA;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ctx->sm_count);
  cfg.blockDim = dim3(MP_THREADS);
  cfg.dynamicSmemBytes = MP_SMEM;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs resident: they wait for one another
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t err = cudaLaunchKernelEx(&cfg, ard_mlp_persistent_kernel, p);
  if (err == cudaErrorCooperativeLaunchTooLarge || err == cudaErrorLaunchOutOfResources) {
    (void)cudaGetLastError();
    return ARD_ERR_UNSUPPORTED;
  }
  if (err != cudaSuccess) return ARD_ERR_CUDA;
  ctx->launches++;
  for (int l = 0; l < H; ++l) {
    if (!layers[l].sample) continue;
    layers[l].pat->dp_bound = d->ndp;
    layers[l].pat->generation++;
  }
  return ARD_OK;
}
