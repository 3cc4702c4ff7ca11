// tcgen05 family of the compacted GEMMs (bf16 operands, fp32 accumulation in tensor memory).
//
// One persistent, warp-specialised kernel template covers the six products (row / tile pattern x
// forward / backward-data / backward-weight).  Per CTA: warp 0 is the TMA producer, warp 1 issues
// tcgen05.mma and owns the TMEM allocation, warps 2..9 are the epilogue (two warps per TMEM lane
// quadrant, each taking half of the tile's columns).  Only the kept rows /
// tiles of the weight and the matching slices of the activations are ever staged into shared
// memory (Sec. 3.1, 3.2): a row pattern's kept neurons b-1, b-1+dp, ... are one TMA box of a
// descriptor whose row pitch is dp*ldw; a tile pattern's kept tiles come from the per-column /
// per-row lists the sampler emitted.  The pattern is read from device memory, so the launch does
// not depend on it: the grid is sized for the densest pattern and each CTA derives its own tile
// schedule from the header.
//
// Row patterns pick the N extent of the output tile (64, 128 or 256) on the device from the sampled
// n_keep, so that a sparse pattern still spreads over all SMs; the instruction descriptor, the
// number of TMA boxes per stage and the tile schedule follow that choice.
//
// The accumulator is double-buffered in TMEM (2 x BN columns), so the epilogue of one output tile
// overlaps the MMAs of the next.  Every wait on an mbarrier is bounded by a wall-clock limit;
// when it expires the CTA records ARD_ERR_TIMEOUT, all roles leave their loops, the TMEM
// allocation is released and the kernel returns normally.
#include "ard_internal.h"
#include <type_traits>

#include "sm100_ptx.h"

namespace {

constexpr int BM = 128;
constexpr int BK = 64;  // 64 bf16 = 128 bytes = one swizzle row
constexpr int TC_THREADS = 320;  // warp 0 producer, warp 1 MMA, warps 2..9 epilogue
constexpr int TC_THREADS_CLASS = TC_THREADS + 32;  // class form of the tile pattern: warp 10 is a second producer
constexpr int ROWS_GATHER_WARPS = 4;  // row-list products: warp 0 and warps 10..12 gather (one warp cannot issue enough copies)
constexpr int TC_THREADS_ROWS = TC_THREADS + 32 * (ROWS_GATHER_WARPS - 1);
constexpr int EPI_WARPS = 8;

enum TcMode {
  M_ROW_FWD = 0,
  M_ROW_BWD_DATA = 1,
  M_ROW_BWD_WEIGHT = 2,
  M_TILE_FWD = 3,
  M_TILE_BWD_DATA = 4,
  M_TILE_BWD_WEIGHT = 5,
  // Tile patterns, "class" form: tile-columns with equal (c mod dp) share one kept-row set and tile-rows
  // with equal (r mod s) share one kept-column set, so a tile pattern is a handful of dense products
  // over gathered 64-wide blocks; these modes build 256-wide output tiles from such blocks.
  M_TILEC_FWD = 6,
  M_TILEC_BWD_DATA = 7,
  M_TILEC_BWD_WEIGHT = 8,
  // LSTM gate products over the four gate blocks i|f|g|o of one weight in a single launch: the kept
  // units of gate g are the rows g*H + keep[j] of W, reached through one descriptor per gate.
  M_LSTM_FWD = 9,       // Z[:, g*ldz + j] = [x,h] . W[g*H + keep[j], :]
  M_LSTM_BWD_DATA = 10, // d[x,h] = sum_g dZ[:, g*ldz + j] . W[g*H + keep[j], :]
  M_LSTM_BWD_WEIGHT = 11, // dW[g*H + keep[j], :] = sum_rows dZ[:, g*ldz + j] . [x,h]   (M tiles: gate-major)
  // Products over an index list of kept ROWS of the input matrix (Sec. 5.2.1).  The kept rows follow no
  // stride, so the producer warps fetch them four at a time with TMA gather instructions (tile::gather4), which
  // fill a stage exactly as a box would; the weight arrives in ordinary boxes.
  M_ROWS_FWD = 12,        // Y[idx[j], :]  = A[idx[j], :] . W^T          (A gathered, K-major)
  M_ROWS_BWD_DATA = 13,   // dA[idx[j], :] = dY[idx[j], :] . W           (dY gathered, K-major)
  M_ROWS_BWD_WEIGHT = 14  // dW[n, :] = sum_j dY[idx[j], n] A[idx[j], :] (both gathered, MN-major)
};

__host__ __device__ constexpr bool a_is_mn(int mode) {
  return mode == M_ROW_BWD_WEIGHT || mode == M_TILE_BWD_WEIGHT || mode == M_TILEC_BWD_WEIGHT ||
         mode == M_LSTM_BWD_WEIGHT || mode == M_ROWS_BWD_WEIGHT;
}
__host__ __device__ constexpr bool b_is_mn(int mode) {
  return mode != M_ROW_FWD && mode != M_TILE_FWD && mode != M_TILEC_FWD && mode != M_LSTM_FWD && mode != M_ROWS_FWD;
}
__host__ __device__ constexpr bool is_rows_mode(int mode) { return mode >= M_ROWS_FWD && mode <= M_ROWS_BWD_WEIGHT; }
__host__ __device__ constexpr bool is_class_mode(int mode) { return mode >= M_TILEC_FWD && mode <= M_TILEC_BWD_WEIGHT; }
__host__ __device__ constexpr bool has_second_producer(int mode) {
  return is_class_mode(mode) || mode == M_TILE_FWD || mode == M_TILE_BWD_DATA || mode == M_TILE_BWD_WEIGHT;
}
__host__ __device__ constexpr int tc_threads(int mode) {
  return is_rows_mode(mode) ? TC_THREADS_ROWS : (has_second_producer(mode) ? TC_THREADS_CLASS : TC_THREADS);
}
__host__ __device__ constexpr int stages_for(int bn) { return bn == 256 ? 4 : (bn == 128 ? 6 : 8); }
__host__ __device__ constexpr int tmem_cols_for(int bn) { return 2 * bn < 32 ? 32 : 2 * bn; }

struct TcParams {
  CUtensorMap* tm_slots;  // descriptor scratch of the context (ARD_TM_SLOTS slots per SM)
  int mapA_indexed, mapB_indexed;
  const int32_t* hdr;
  const int32_t* idx;
  const int32_t* col_ptr;
  const int32_t* col_idx;
  const int32_t* row_ptr;
  const int32_t* row_idx;
  int B, K, N;  // batch, fan-in, neurons
  int ts;
  float alpha;
  void* out;
  int ldo;
  int out_is_f32;
  int scatter;    // row fwd: full-width output with zero fill
  int zero_fill;  // row bwd-weight: write zeros to dropped rows
  int force_bn;   // row modes: 0 = choose the N tile on the device, else a multiple of 32 in 64 .. 256
  int accumulate; // plain stores add to the existing output
  int band_m;     // M-tiles per raster band (0: one band)
  // Shared tiles (row modes): when the tile count is not a multiple of the worker count, the tiles
  // that do not fill a wave are cut along the contraction and shared by all workers.  sk_ws holds the
  // fp32 partial accumulators (two slots per worker), sk_cnt one arrival counter per (shared tile,
  // epilogue warp).
  float4* sk_ws;      // nullptr: every tile is computed by one worker
  int* sk_cnt;
  int sk_min_blocks;  // fewest contraction blocks worth a separate share
  int sk_min_gain;    // fewest contraction blocks sharing must take off the last wave to be used
  int* status;
  // Fused layer step (kernels instantiated with FUSED): see GemmArgs.
  const int32_t* hdr_in;
  const float* bias;
  int relu;
  const void* act;
  int ldact;
  // Row-list products: the kept-row list.  Forward and backward-data gather through descriptors; the weight
  // gradient, whose two operands both follow the list, gathers with asynchronous copies from these matrices.
  const int32_t* ridx;
  const __nv_bfloat16* gA;  // backward-weight: dY
  int ldgA;
  const __nv_bfloat16* gB;  // backward-weight: A
  int ldgB;
  // Row-list products on compact operands (FUSED row kernels): hdr is the row list's header, the layer itself is
  // dense.  1: the row extent of A and of the output is hdr[HDR_NKEEP] and output row m goes to row ridx[m]
  // (forward, backward-data); 2: the contraction runs over hdr[HDR_NKEEP] rows (backward-weight).
  int ext_mode;
  int sk_any;  // shared tiles also when the tiles do not fill one wave (long contractions, few tiles)
};

// The descriptors travel by value behind the scalar parameters: A and B, and for the LSTM gate products one per
// gate for either operand (maps[2 + g] for A, maps[6 + g] for B).
template <int NM>
struct TcParamsT : TcParams {
  TcMap maps[NM];
};
__host__ __device__ constexpr bool is_lstm_mode(int mode) { return mode >= M_LSTM_FWD && mode <= M_LSTM_BWD_WEIGHT; }
__host__ __device__ constexpr int nmaps(int mode) { return is_lstm_mode(mode) ? 10 : 2; }

// CTAS = 2: a cluster of two CTAs shares one 256 x BN output tile; each CTA stages its own 128 rows
// of A and half of the B rows, so a stage is smaller and the pipeline deeper.
template <int BN, int CTAS = 1>
struct SmemLayout {
  static constexpr int STAGES = stages_for(BN / CTAS);
  static constexpr int A_BYTES = BM * BK * 2;
  static constexpr int B_BYTES = (BN / CTAS) * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STG_OFF = STAGES * STAGE_BYTES;       // epilogue staging: 8 warps x 32 x 33 floats
  static constexpr int STG_BYTES = EPI_WARPS * 32 * 33 * 4;
  static constexpr int BAR_OFF = STG_OFF + STG_BYTES;        // full[S], empty[S], tfull[2], tempty[2]
  static constexpr int MISC_OFF = BAR_OFF + (2 * STAGES + 4) * 8;
  static constexpr int TOTAL = MISC_OFF + 32 + 1024;         // + slack for manual 1024-byte alignment
};

// Class modes: bytes of the staging area that hold the kept-tile list and the class table.
constexpr int CLASS_LIST_BYTES = 16384;
static_assert(CLASS_LIST_BYTES + EPI_WARPS * 32 * 17 * 4 <= EPI_WARPS * 32 * 33 * 4, "class staging does not fit");

// Element i of a 4-entry array without dynamic indexing (keeps the array in registers).
__device__ __forceinline__ int sel4(const int (&a)[4], int i) {
  return i == 0 ? a[0] : (i == 1 ? a[1] : (i == 2 ? a[2] : a[3]));
}
__device__ __forceinline__ const CUtensorMap* sel_map(const CUtensorMap* const (&a)[4], int i) {
  return i == 0 ? a[0] : (i == 1 ? a[1] : (i == 2 ? a[2] : a[3]));
}

// One piece of work of a CTA (pair): contraction blocks [kb0, kb1) of output tile t.
struct Unit {
  int t;
  int kb0, kb1;    // kb1 < 0: the whole tile
  int sk_tile;     // index of t among the shared tiles, -1 if this worker computes t alone
  int slot;        // which of the worker's two partial slots this piece uses
  int jfirst;      // first worker contributing to t
  int nsplit;      // number of contributing workers
};

constexpr int SK_SLOT_F4 = 1024;  // float4 per (epilogue warp, partial): 32 rows x 128 columns of fp32

// Tile schedule shared by the three roles.
struct TileInfo {
  int m0, n0;      // origin in GEMM space
  int nkb;         // number of 64-wide contraction blocks
  const int32_t* klist;  // tile patterns: kept block list for this output tile
  int kper;        // 64-blocks per pattern tile
  int out_row0;    // tile bwd-weight: first output row (neuron); LSTM bwd-weight: first row of the tile's gate block
  int gate;        // LSTM bwd-weight: gate of this tile
  int rows_valid;  // tile bwd-weight: rows of this tile that belong to the kept tile
  int bn;          // N extent of this tile (whole pair)
  int nbox;        // 64-wide B boxes this CTA stages
  int bx[4];       // their coordinates along the B operand's N axis (out of range: a box of zeros)
  int ax[2];       // MN-major A: coordinates of this CTA's two 64-row boxes
  int ocol[4];     // output column of each 64-column group of the tile (-1: nothing to write)
  int orow[2];     // class bwd-weight: output row of each 64-row group of this CTA (-1: nothing to write)
};

template <int BN, int MODE, int CTAS = 1, bool SHARE = false>
struct Sched {
  int dp, b, n_keep, Tc;
  int Mt, Nt, total;
  int M_gemm, N_gemm, Kc;  // GEMM extents (valid rows, valid cols, contraction length)
  int subm, subn;          // tile bwd-weight: sub-blocks per pattern tile
  int bn;                  // N extent of the output tile actually used (<= BN)
  int rank;                // CTA rank inside the pair (0 for single-CTA tiles)
  int workers;             // CTAs (or CTA pairs) sharing the tile loop
  // class modes
  int Tr, nclass, cstep;   // tile-rows; number of classes; distance between members of a class
  int h_items, light_q;    // class form: items of classes that keep something come first; see unit()
  const int32_t* list;     // kept-tile list the class modes walk (a shared-memory copy when it fits)
  const int4* ctab;        // per class {first item, list offset, list length, members} (shared memory)
  int qn, qm;              // pattern tiles per output tile along N and along M
  int lts;                 // log2 of the pattern tile size (64, 128 or 256 in the class modes)
  bool dense;              // class modes with dp = 1: nothing is dropped, plain dense tiling
  // shared tiles of the row modes
  int KT;                  // contraction blocks per tile
  int sk_tiles;            // tiles 0 .. sk_tiles-1 are shared along the contraction (0: none)
  int sk_S;                // workers sharing them
  int sk_blocks;           // their contraction blocks

  // compiled in only for the row products launched with the sharing enabled
  static constexpr bool SK_MODE = SHARE && (MODE == M_ROW_FWD || MODE == M_ROW_BWD_DATA || MODE == M_ROW_BWD_WEIGHT);

  // Workers that would share the `rem` tiles left over by `full` complete waves (0: not worth it).
  // The shared tiles are computed first, so that parking and adding their partial sums overlaps the
  // contraction of the tiles that follow; without a complete wave there is nothing to hide behind.
  __device__ static int sharing_workers(int full, int rem, int kt, int nworkers, int min_blocks, int min_gain,
                                        int any = 0) {
    if (rem == 0 || (full == 0 && !any)) return 0;
    const int S = min(nworkers, rem * kt / min_blocks);
    if (S <= rem) return 0;
    return kt - (rem * kt + S - 1) / S >= min_gain ? S : 0;
  }

  // kin: fan-in extent of the row products (K, or the kept outputs of the layer that feeds this one)
  // ext_mode: see TcParams (0 unless the kernel was instantiated with FUSED)
  __device__ void init(const TcParams& p, int rank_, int kin, int ext_mode = 0) {
    rank = rank_;
    workers = (int)gridDim.x / CTAS;
    dp = p.hdr[HDR_DP];
    b = p.hdr[HDR_B];
    n_keep = p.hdr[HDR_NKEEP];
    const int ext = n_keep;  // length of the row list when hdr is a row list's header
    if (ext_mode) { dp = 1; b = 1; n_keep = p.N; }
    Tc = p.hdr[HDR_TC];
    subm = subn = 1;
    KT = sk_tiles = sk_S = sk_blocks = 0;
    if (MODE == M_ROW_FWD) { M_gemm = ext_mode ? ext : p.B; N_gemm = n_keep; Kc = kin; }
    else if (MODE == M_ROW_BWD_DATA) { M_gemm = ext_mode ? ext : p.B; N_gemm = kin; Kc = n_keep; }
    else if (MODE == M_LSTM_FWD) { M_gemm = p.B; N_gemm = ((n_keep + 63) / 64) * 256; Kc = p.K; }
    else if (MODE == M_LSTM_BWD_DATA) { M_gemm = p.B; N_gemm = p.K; Kc = 4 * (((n_keep + 63) / 64) * 64); }
    else if (MODE == M_ROW_BWD_WEIGHT || MODE == M_LSTM_BWD_WEIGHT) { M_gemm = n_keep; N_gemm = kin; Kc = ext_mode ? ext : p.B; }
    else if (MODE == M_ROWS_FWD) { M_gemm = n_keep; N_gemm = p.N; Kc = p.K; }
    else if (MODE == M_ROWS_BWD_DATA) { M_gemm = n_keep; N_gemm = p.K; Kc = p.N; }
    else if (MODE == M_ROWS_BWD_WEIGHT) { M_gemm = p.N; N_gemm = p.K; Kc = n_keep; }
    else if (MODE == M_TILE_FWD || MODE == M_TILEC_FWD) { M_gemm = p.B; N_gemm = p.N; Kc = 0; }
    else if (MODE == M_TILE_BWD_DATA || MODE == M_TILEC_BWD_DATA) { M_gemm = p.B; N_gemm = p.K; Kc = 0; }
    else { M_gemm = p.N; N_gemm = p.K; Kc = p.B; }
    bn = BN;
    Tr = p.hdr[HDR_TR];
    nclass = cstep = qn = qm = 1;
    h_items = 0x7fffffff;
    light_q = 1;
    list = (MODE == M_TILEC_BWD_DATA) ? p.row_idx : p.col_idx;
    ctab = nullptr;
    lts = 31 - __clz(p.ts > 0 ? p.ts : 1);
    dense = is_class_mode(MODE) && dp == 1;
    if (dense) {
      // every tile is kept: the contraction runs over the whole operand
      Kc = (MODE == M_TILEC_FWD) ? p.K : (MODE == M_TILEC_BWD_DATA ? p.N : p.B);
      Mt = (M_gemm + BM * CTAS - 1) / (BM * CTAS);
      Nt = (N_gemm + bn - 1) / bn;
      total = Mt * Nt;
      return;
    }
    if (is_class_mode(MODE)) {
      qn = BN / p.ts;
      qm = (BM * CTAS) / p.ts;
      Mt = (M_gemm + BM * CTAS - 1) / (BM * CTAS);
      if (MODE == M_TILEC_BWD_DATA) {
        // tile-rows r and r' keep the same tile-columns when (r - r') * (Tc mod dp) = 0 (mod dp)
        int g = Tc % dp, a = dp;
        while (g) { const int tmp = a % g; a = g; g = tmp; }  // a = gcd(Tc mod dp, dp)
        cstep = dp / a;
        nclass = min(cstep, Tr);
      } else {
        cstep = dp;
        nclass = min(dp, Tc);
      }
      total = 0;  // filled in by build_class_table()
      return;
    }
    if (MODE == M_TILE_BWD_WEIGHT) {
      subm = (p.ts + BM - 1) / BM;
      subn = p.ts / BN;
      Mt = n_keep * subm;
      Nt = subn;
    } else {
      Mt = (M_gemm + BM * CTAS - 1) / (BM * CTAS);
      if (MODE == M_LSTM_BWD_WEIGHT) Mt *= 4;  // the M tiles of the four gate blocks, gate after gate
      if (MODE == M_ROW_FWD || MODE == M_ROW_BWD_DATA || MODE == M_ROW_BWD_WEIGHT || MODE == M_LSTM_BWD_DATA ||
          MODE == M_LSTM_BWD_WEIGHT || is_rows_mode(MODE)) {
        if (p.force_bn) {
          bn = p.force_bn;
        } else {
          // Fewest (waves x time per tile).  Narrow tiles re-read the A operand more often and use narrower
          // instructions; the time of a tile relative to a 256-wide one, measured per wave on dense
          // problems: pairs 0.92 / 0.83 / 0.78 / 0.76 at 224 / 192 / 160 / 128 columns, single CTAs 0.7 at
          // 128 and 0.55 at 64.  Ties go to the wider tile.
          // The forward products of CTA pairs try every multiple of 32 columns (the instruction takes any
          // multiple of 16; B still arrives in 64-row boxes, the last one partly unused).  Where B is read along its
          // contiguous dimension (both backward products) only 256 / 128 / 64 keep every box on a 128-byte
          // line; other widths were measured up to 20 % slower per tile there and are not tried.
          // Shared tiles cost each worker its share of their contraction plus some of the reduction.
          constexpr bool FLEX = CTAS == 2 && MODE == M_ROW_FWD;  // single CTAs: small, latency-bound problems
          const int kt = (Kc + BK - 1) / BK;
          int best_cost = 0x7fffffff;
          for (int cand = BN; cand >= 64 * CTAS; cand = FLEX ? cand - 32 : cand >> 1) {
            const int tiles = Mt * ((N_gemm + cand - 1) / cand);
            const int wpair = cand == 256 ? 100 : (cand == 224 ? 92 : (cand == 192 ? 83 : (cand == 160 ? 78 : 76)));
            const int wone = cand == 256 ? 100 : (cand == 128 ? 70 : 55);
            const int w16 = 16 * (FLEX ? wpair : wone);
            const int full = tiles / workers, rem = tiles % workers;
            const int S = (SK_MODE && p.sk_ws != nullptr && kt > 0)
                              ? sharing_workers(full, rem, kt, workers, p.sk_min_blocks, p.sk_min_gain, p.sk_any) : 0;
            int cost = full * w16;
            if (S > 0) cost += (((rem * kt + S - 1) / max(S, 1)) + p.sk_min_gain / 2) * w16 / max(kt, 1);
            else if (rem > 0) cost += w16;
            if (cost < best_cost) { best_cost = cost; bn = cand; }
          }
        }
      }
      Nt = (N_gemm + bn - 1) / bn;
    }
    total = Mt * Nt;
    KT = (Kc + BK - 1) / BK;
    sk_tiles = sk_S = sk_blocks = 0;
    if (SK_MODE && p.sk_ws != nullptr && KT > 0) {
      const int rem = total % workers;
      const int S = sharing_workers(total / workers, rem, KT, workers, p.sk_min_blocks, p.sk_min_gain, p.sk_any);
      if (S > 0) { sk_tiles = rem; sk_S = S; sk_blocks = rem * KT; }
    }
  }

  // Worker whose share holds contraction block x of the shared tiles (shares start at
  // floor(j * sk_blocks / sk_S)).
  __device__ int share_worker_of(int x) const { return (int)((((long long)x + 1) * sk_S - 1) / sk_blocks); }
  __device__ int share_start(int j) const { return (int)((long long)j * sk_blocks / sk_S); }

  // i-th piece of work of worker w: first the one or two pieces of its share of the shared tiles
  // 0 .. sk_tiles-1, then its own tiles sk_tiles + w, sk_tiles + w + workers, ...  Returns false when
  // there is none.
  __device__ bool unit(int w, int i, Unit& u) const {
    u.sk_tile = -1;
    u.slot = 0;
    u.jfirst = w;
    u.nsplit = 1;
    int n_shared = 0;
    if (SK_MODE && w < sk_S) {
      const int r0 = share_start(w), r1 = share_start(w + 1);
      const int tile0 = r0 / KT;
      n_shared = (r1 > (tile0 + 1) * KT) ? 2 : 1;
      if (i < n_shared) {
        const int tile = tile0 + i;
        const int lo = max(r0, tile * KT), hi = min(r1, (tile + 1) * KT);
        u.t = tile;
        u.kb0 = lo - tile * KT;
        u.kb1 = hi - tile * KT;
        u.jfirst = share_worker_of(tile * KT);
        u.nsplit = share_worker_of((tile + 1) * KT - 1) - u.jfirst + 1;
        if (u.nsplit > 1) { u.sk_tile = tile; u.slot = i; }
        return true;
      }
    }
    u.kb0 = 0;
    u.kb1 = -1;
    if (is_class_mode(MODE) && h_items < total) {
      // Some classes keep nothing: their items only write zeros, take no part in the producer's and the MMA
      // thread's loops and cost a fraction of the others.  The others are dealt round-robin; the zero items go,
      // light_q apiece, to the workers that got one item less in that round, and only what is left of them is
      // dealt to everybody.  (In plain round-robin order a forward product whose period divides the tile-column
      // count ran its few long items on workers that afterwards still took their full share of the zero items.)
      // Every worker takes its zero items FIRST: its epilogue warps write them while the first long item's
      // products run, instead of after the last one.
      const int a = h_items / workers, rem = h_items - a * workers;
      const int a_w = a + (w < rem ? 1 : 0);
      const int n_light = total - h_items;
      const int n_less = workers - rem;                        // workers rem .. workers-1 got one item less
      const int first_part = rem == 0 ? 0 : min(n_light, n_less * light_q);
      int n1 = 0;                                               // zero items this worker takes in the first part
      if (rem != 0 && w >= rem && first_part > w - rem) n1 = min(light_q, (first_part - (w - rem) + n_less - 1) / n_less);
      const int rest = n_light - first_part;
      const int n2 = rest > w ? (rest - w + workers - 1) / workers : 0;
      if (i < n1 + n2) {
        const int j = i < n1 ? (w - rem) + i * n_less : first_part + w + (i - n1) * workers;
        u.t = h_items + j;
        return true;
      }
      const int ih = i - (n1 + n2);
      u.t = w + ih * workers;
      return ih < a_w;
    }
    const int first = SK_MODE ? sk_tiles : 0;
    u.t = first + w + (i - n_shared) * workers;
    return u.t < total;
  }

  // ---- class modes ----
  __device__ int class_members(int c) const {  // pattern tiles in class c along the gathered axis
    const int extent = (MODE == M_TILEC_BWD_DATA) ? Tr : Tc;
    return (extent - 1 - c) / cstep + 1;
  }
  __device__ int class_items(int cnt, int len) const {  // output tiles of a class with cnt members
    if (MODE == M_TILEC_BWD_WEIGHT) return ((cnt + qm - 1) / qm) * ((len + qn - 1) / qn);
    return Mt * ((cnt + qn - 1) / qn);
  }
  // One warp fills the per-class table in shared memory (at most 64 classes: two per lane, so the list pointers of
  // all classes come back in one round trip; a single thread walking them took ~2.5 us of every launch); callers
  // synchronise.
  // Classes that keep something come first, the empty ones (whose items only write zeros) after them, each group
  // by class number; an entry is {first item, list offset, list length, members | class << 16}.  out[0] = number of
  // items, out[1] = items of the non-empty classes, out[2] = how many zero items cost about as much as one of the
  // others.
  __device__ static int warp_excl_scan(int v, int lane, int& total) {
    int x = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, d);
      if (lane >= d) x += y;
    }
    total = __shfl_sync(0xffffffffu, x, 31);
    return x - v;
  }
  __device__ void build_class_table(const TcParams& p, int4* tab, int* out, int lane) const {
    const int32_t* ptr = (MODE == M_TILEC_BWD_DATA) ? p.row_ptr : p.col_ptr;
    int off[2], len[2], cnt[2], items[2];
    bool valid[2], full[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int c = lane + 32 * h;
      valid[h] = c < nclass;
      off[h] = valid[h] ? ptr[c] : 0;
      len[h] = valid[h] ? ptr[c + 1] - off[h] : 0;
      cnt[h] = valid[h] ? class_members(c) : 0;
      items[h] = valid[h] ? class_items(cnt[h], len[h]) : 0;
      full[h] = valid[h] && len[h] != 0;
    }
    const unsigned lt = (1u << lane) - 1u;
    const unsigned mf0 = __ballot_sync(0xffffffffu, full[0]), mf1 = __ballot_sync(0xffffffffu, full[1]);
    const unsigned me0 = __ballot_sync(0xffffffffu, valid[0] && !full[0]), me1 = __ballot_sync(0xffffffffu, valid[1] && !full[1]);
    const int n_full = __popc(mf0) + __popc(mf1);
    int tA, tB, tC, tD;
    const int sA = warp_excl_scan(full[0] ? items[0] : 0, lane, tA);
    const int sB = warp_excl_scan(full[1] ? items[1] : 0, lane, tB);
    const int sC = warp_excl_scan(valid[0] && !full[0] ? items[0] : 0, lane, tC);
    const int sD = warp_excl_scan(valid[1] && !full[1] ? items[1] : 0, lane, tD);
    if (valid[0]) {
      const int slot = full[0] ? __popc(mf0 & lt) : n_full + __popc(me0 & lt);
      const int run = full[0] ? sA : tA + tB + sC;
      tab[slot] = make_int4(run, off[0], len[0], cnt[0] | (lane << 16));
    }
    if (valid[1]) {
      const int slot = full[1] ? __popc(mf0) + __popc(mf1 & lt) : n_full + __popc(me0) + __popc(me1 & lt);
      const int run = full[1] ? tA + sB : tA + tB + tC + sD;
      tab[slot] = make_int4(run, off[1], len[1], cnt[1] | ((lane + 32) << 16));
    }
    // contraction blocks of the non-empty classes' items
    long long blocks = (full[0] ? (long long)items[0] * len[0] : 0) + (full[1] ? (long long)items[1] * len[1] : 0);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) blocks += __shfl_xor_sync(0xffffffffu, blocks, d);
    blocks *= (p.ts >> 6);
    if (lane == 0) {
      const int heavy = tA + tB;
      out[0] = heavy + tC + tD;
      out[1] = heavy;
      // an item that only writes zeros takes about as long as 14 contraction blocks
      const int avg = heavy > 0 ? (int)(blocks / heavy) : 0;
      out[2] = min(64, max(1, (avg + 14) / 14));
    }
  }
  __device__ TileInfo class_tile(const TcParams& p, int t) const {
    TileInfo ti;
    ti.klist = nullptr;
    ti.kper = p.ts >> 6;
    ti.out_row0 = 0;
    ti.rows_valid = BM;
    ti.n0 = 0;
    const int tmask = p.ts - 1;   // the pattern tile size is a power of two here
    int sl = nclass - 1;
    while (sl > 0 && ctab[sl].x > t) --sl;  // table entry whose item range holds t
    const int4 ce = ctab[sl];
    t -= ce.x;
    const int cnt = ce.w & 0xffff, c = ce.w >> 16;
    const int lsub = lts - 6;     // log2 of the 64-wide boxes per pattern tile
    int nm;                       // pattern tiles along N in this output tile
    if (MODE == M_TILEC_BWD_WEIGHT) {
      const int32_t* rlist = list + ce.y;
      const int rn = ce.z;
      const int mtiles = (cnt + qm - 1) / qm;
      const int mi = t % mtiles, ni = t / mtiles;
      ti.m0 = 0;
      ti.nkb = (Kc + BK - 1) / BK;
#pragma unroll
      for (int k = 0; k < 2; ++k) {  // this CTA's two 64-row boxes of gathered neurons
        const int row = rank * BM + 64 * k;
        const int mem = mi * qm + (row >> lts);
        const int coord = (mem < cnt) ? (((c + mem * cstep) << lts) + (row & tmask)) : -1;
        ti.orow[k] = coord;
        ti.ax[k] = coord >= 0 ? coord : p.N;  // beyond the matrix: TMA fills zeros
      }
      const int j0 = ni * qn;
      nm = min(qn, rn - j0);
      ti.bn = ((nm << lts) + 64 * CTAS - 1) / (64 * CTAS) * (64 * CTAS);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int mem = j >> lsub;
        ti.ocol[j] = (mem < nm) ? ((rlist[j0 + mem] << lts) + ((j & ((1 << lsub) - 1)) << 6)) : -1;
      }
    } else {
      const int ntiles = (cnt + qn - 1) / qn;
      (void)ntiles;
      const int mt = t % Mt, v = t / Mt;
      ti.m0 = mt * BM * CTAS + rank * BM;
      ti.ax[0] = ti.m0; ti.ax[1] = ti.m0 + 64;
      ti.orow[0] = ti.orow[1] = 0;
      const int i0 = v * qn;
      nm = min(qn, cnt - i0);
      ti.bn = ((nm << lts) + 64 * CTAS - 1) / (64 * CTAS) * (64 * CTAS);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int mem = j >> lsub;
        ti.ocol[j] = (mem < nm) ? (((c + (i0 + mem) * cstep) << lts) + ((j & ((1 << lsub) - 1)) << 6)) : -1;
      }
      ti.klist = list + ce.y;
      ti.nkb = ce.z * ti.kper;
    }
    // this CTA's share of the B boxes
    const int oob = (MODE == M_TILEC_FWD) ? p.N : p.K;
    ti.nbox = ti.bn / 64 / CTAS;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int oc = sel4(ti.ocol, rank * ti.nbox + i);
      ti.bx[i] = (i < ti.nbox && oc >= 0) ? oc : oob;
    }
    return ti;
  }

  // PLAIN: the caller knows that the tiling is the plain dense one (class modes with dp = 1).  The roles of
  // the kernel are compiled once for each case: with both paths behind one run-time test the tile's
  // coordinates are opaque to the compiler in every per-block loop, which cost the dense draws of a tile
  // pattern 10 - 30 % against the same product under a row pattern.
  template <bool PLAIN>
  __device__ TileInfo tile(const TcParams& p, int t) const {
    if (is_class_mode(MODE) && !PLAIN) return class_tile(p, t);
    TileInfo ti = plain_tile(p, t);
    // affine block coordinates
    ti.bn = bn;
    ti.nbox = (bn / CTAS + 63) / 64;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      ti.bx[i] = ti.n0 + rank * (bn / CTAS) + 64 * i;
      ti.ocol[i] = ti.n0 + 64 * i;
    }
    ti.ax[0] = ti.m0; ti.ax[1] = ti.m0 + 64;
    ti.orow[0] = ti.m0; ti.orow[1] = ti.m0 + 64;
    if (MODE == M_LSTM_FWD) {
      // N tile = the same 64 kept units of all four gates; p.ts carries the gate block width of Z
      const int j0 = ti.n0 / 4;
      ti.n0 = j0;
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        ti.bx[g] = j0;
        ti.ocol[g] = g * p.ts + j0;
      }
    }
    return ti;
  }

  __device__ TileInfo plain_tile(const TcParams& p, int t) const {
    TileInfo ti;
    ti.klist = nullptr;
    ti.kper = 1;
    ti.out_row0 = 0;
    ti.rows_valid = BM;
    if (MODE == M_TILE_BWD_WEIGHT) {
      const int j = t / (subm * subn), rem = t % (subm * subn);
      const int sm = rem / subn, sn = rem % subn;
      const int lin = p.idx[j];
      const int r = lin / Tc, c = lin % Tc;
      ti.m0 = c * p.ts + sm * BM;
      ti.n0 = r * p.ts + sn * BN;
      ti.nkb = (Kc + BK - 1) / BK;
      ti.rows_valid = min(BM, p.ts - sm * BM);
      return ti;
    }
    // Raster order: bands of band_m M-tiles; inside a band the M index runs fastest, so the CTAs that
    // run together share a few B tiles and one band of A, and consecutive waves reuse that band from L2.
    int mt, nt;
    {
      const int bm = (p.band_m > 0 && p.band_m < Mt) ? p.band_m : Mt;
      const int per_band = bm * Nt;
      const int band = t / per_band, r = t - band * per_band;
      const int rows_in_band = min(bm, Mt - band * bm);
      nt = r / rows_in_band;
      mt = band * bm + (r - nt * rows_in_band);
    }
    ti.m0 = mt * BM * CTAS + rank * BM;  // this CTA's 128 rows of the tile
    ti.n0 = nt * bn;
    ti.gate = 0;
    if (MODE == M_LSTM_BWD_WEIGHT) {
      const int mt_gate = Mt >> 2;
      ti.gate = mt / mt_gate;
      ti.m0 = (mt - ti.gate * mt_gate) * BM * CTAS + rank * BM;  // row inside the gate's compact block
      ti.out_row0 = ti.gate * p.N;
    }
    if (MODE == M_TILE_FWD) {
      const int c = ti.n0 / p.ts;
      ti.klist = p.col_idx + p.col_ptr[c];
      ti.kper = p.ts / BK;
      ti.nkb = (p.col_ptr[c + 1] - p.col_ptr[c]) * ti.kper;
    } else if (MODE == M_TILE_BWD_DATA) {
      const int r = ti.n0 / p.ts;
      ti.klist = p.row_idx + p.row_ptr[r];
      ti.kper = p.ts / BK;
      ti.nkb = (p.row_ptr[r + 1] - p.row_ptr[r]) * ti.kper;
    } else {
      ti.nkb = (Kc + BK - 1) / BK;
    }
    return ti;
  }
};

// ---- epilogue helpers -------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Stores 32 consecutive values of one output row; `nvalid` of them exist.  The row start is 16-byte
// aligned whenever nvalid == 32 paths are taken (guaranteed by the host-side alignment checks).
__device__ __forceinline__ void store_row32(void* out, size_t row_off, int col, float (&v)[32], int nvalid,
                                            int out_is_f32, int accumulate = 0) {
  if (accumulate) {
    // read-modify-write of this thread's own 32 outputs
    if (out_is_f32) {
      const float* p = reinterpret_cast<const float*>(out) + row_off + col;
#pragma unroll
      for (int q = 0; q < 32; ++q)
        if (q < nvalid) v[q] += p[q];
    } else {
      const __nv_bfloat16* p = reinterpret_cast<const __nv_bfloat16*>(out) + row_off + col;
#pragma unroll
      for (int q = 0; q < 32; ++q)
        if (q < nvalid) v[q] += __bfloat162float(p[q]);
    }
  }
  if (out_is_f32) {
    float* p = reinterpret_cast<float*>(out) + row_off + col;
    if (nvalid >= 32) {
#pragma unroll
      for (int q = 0; q < 8; ++q)
        reinterpret_cast<float4*>(p)[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
    } else {
#pragma unroll
      for (int q = 0; q < 32; ++q)
        if (q < nvalid) p[q] = v[q];
    }
  } else {
    __nv_bfloat16* p = reinterpret_cast<__nv_bfloat16*>(out) + row_off + col;
    if (nvalid >= 32) {
#pragma unroll
      for (int q = 0; q < 4; ++q)
        reinterpret_cast<uint4*>(p)[q] =
            make_uint4(pack_bf16(v[8 * q], v[8 * q + 1]), pack_bf16(v[8 * q + 2], v[8 * q + 3]),
                       pack_bf16(v[8 * q + 4], v[8 * q + 5]), pack_bf16(v[8 * q + 6], v[8 * q + 7]));
    } else {
#pragma unroll
      for (int q = 0; q < 32; ++q)
        if (q < nvalid) p[q] = __float2bfloat16_rn(v[q]);
    }
  }
}

__device__ __forceinline__ void zero_row32(void* out, size_t row_off, int col, int nvalid, int out_is_f32) {
  float z[32];
#pragma unroll
  for (int q = 0; q < 32; ++q) z[q] = 0.f;
  store_row32(out, row_off, col, z, nvalid, out_is_f32);
}

// ---- the kernel -----------------------------------------------------------------------------------
template <int BN, int MODE, int CTAS, bool SHARE, bool FUSED>
__global__ void __launch_bounds__(tc_threads(MODE), 1)
ard_gemm_tc_kernel(const __grid_constant__ TcParamsT<nmaps(MODE)> p) {
  using L = SmemLayout<BN, CTAS>;
  const uint32_t rank = (CTAS == 2) ? cluster_ctarank() : 0u;  // rank 0 leads the pair and issues its MMAs
  constexpr int STAGES = L::STAGES;
  constexpr bool A_MN = a_is_mn(MODE), B_MN = b_is_mn(MODE);
  constexpr uint32_t TMEM_COLS = tmem_cols_for(BN);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw_addr);

  const uint32_t bar_base = base + L::BAR_OFF;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + 2 + a); };
  volatile uint32_t* tmem_ptr_smem = reinterpret_cast<volatile uint32_t*>(smem + L::MISC_OFF);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::MISC_OFF + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_launch_dependents();  // the next kernel of the stream may set up while this one runs

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      // weight gradient over a row list: one arrival per gathering lane besides the producer's
      mbar_init(full_bar(s), MODE == M_ROWS_BWD_WEIGHT ? 1 + 32 * ROWS_GATHER_WARPS : 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), EPI_WARPS * CTAS);  // the pair's epilogue warps all report to the leader
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    if (CTAS == 2) {
      tmem_alloc2(smem_u32(const_cast<uint32_t*>(tmem_ptr_smem)), TMEM_COLS);
      tmem_relinquish2();
    } else {
      tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_ptr_smem)), TMEM_COLS);
      tmem_relinquish();
    }
  }
  tc_fence_before();
  if (CTAS == 2) cluster_sync_all();  // both CTAs' barriers exist before anyone signals across the pair
  else __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_smem;
  // Everything above touched only this CTA's shared and tensor memory; from here on the kernel reads
  // what earlier kernels of the stream wrote (the pattern, the operands) and overwrites what they read.
  pdl_wait_prior_grids();

  Sched<BN, MODE, CTAS, SHARE> sch;
  sch.init(p, (int)rank, (FUSED && p.hdr_in != nullptr) ? p.hdr_in[HDR_NKEEP] : p.K, FUSED ? p.ext_mode : 0);
  if (is_class_mode(MODE) && !sch.dense) {
    // The producer reads one list entry per contraction block: keep the list in shared memory (the
    // staging area of the forward scatter epilogue is free in these modes) instead of paying a
    // global-memory round trip on its critical path.
    // The list and the per-class table (first item, list offset, length, members; one KiB) share the first
    // CLASS_LIST_BYTES of that area; the rest is the epilogue warps' staging (32 rows x 17 words each).
    const int n_list = p.hdr[HDR_NKEEP];
    int4* tab = reinterpret_cast<int4*>(smem + L::STG_OFF + CLASS_LIST_BYTES - 1024);
    int* total_smem = reinterpret_cast<int*>(smem + L::MISC_OFF + 8);  // [3]: items, items of non-empty classes, light_q
    int32_t* slist = reinterpret_cast<int32_t*>(smem + L::STG_OFF);
    const bool fits = n_list * 4 <= CLASS_LIST_BYTES - 1024;
    if (warp == 0) sch.build_class_table(p, tab, total_smem, lane);
    if (fits)
      for (int i = threadIdx.x; i < n_list; i += (int)blockDim.x) slist[i] = sch.list[i];
    __syncthreads();
    sch.ctab = tab;
    sch.total = total_smem[0];
    sch.h_items = total_smem[1];
    sch.light_q = total_smem[2];
    if (fits) sch.list = slist;
  }
  const int w0 = (int)blockIdx.x / CTAS;  // first tile of this CTA (pair)

  // The four roles, compiled for the class tiling and for the plain one (see Sched::tile).
  auto roles = [&](auto plain_tag) {
  constexpr bool PLAIN = decltype(plain_tag)::value;
  if (is_rows_mode(MODE) && (warp == 0 || warp >= 10)) {
    // ===================== gathering producers (4 warps) =====================
    // An index list has no stride a TMA box could follow, but the TMA unit takes four arbitrary rows per
    // instruction (tile::gather4 on a descriptor whose box is one row of 64 columns = 128 bytes high): the four
    // 128-byte pieces land one after the other, and since the 128-byte swizzle is a function of the shared-memory
    // address, a run of such instructions fills a stage exactly as one tall box would.  Forward and backward-data
    // take 32 of them per stage (128 rows of the list); one thread paces at several hundred cycles per
    // instruction, so they are dealt over lanes of four warps.  Rows past the end of the list get an index outside
    // the matrix: TMA fills zeros.  (The weight gradient gathers differently, see below.)
    const int gw = warp == 0 ? 0 : warp - 9;  // 0..3
    const CUtensorMap* mapG = &p.maps[0].tm;  // forward: A; backward-data: dY
    const CUtensorMap* mapB = &p.maps[1].tm;  // the weight (boxes)
    const int oob = p.B;                      // the first row the gathered matrices do not have
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    Unit un;
    for (int i = 0; ok && sch.unit(w0, i, un); ++i) {
      const TileInfo ti = sch.template tile<PLAIN>(p, un.t);
      // forward / backward-data: lanes 0..7 of warp gw own the rows 4*(8*gw + lane) .. + 3 of the tile for all blocks
      int r4[4] = {oob, oob, oob, oob};
      if (MODE != M_ROWS_BWD_WEIGHT && lane < 8) {
        const int m = ti.m0 + 4 * (8 * gw + lane);
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (m + q < sch.M_gemm) r4[q] = p.ridx[m + q];
      }
      // Weight gradient: both operands follow the list along the contraction, 16 x (2 + boxes of B) gather
      // instructions per block, and at the ~115 cycles a warp needs per instruction that is slower (378 us on the
      // 32768 x 2304 x 512 layer) than 16-byte asynchronous copies straight into the swizzled layout (261 us): eight
      // lanes fetch the eight chunks of one row, chunk c of row r goes to chunk c ^ (r & 7).  Lanes 0..15 of warp gw
      // own the contraction rows gw*16 .. gw*16 + 15 of a block; the next block's list entries are fetched while
      // this one is issued.
      const int sub = lane >> 3, ch = lane & 7;
      unsigned long long* rowtab = reinterpret_cast<unsigned long long*>(smem + L::STG_OFF) + gw * 64;
      int jcur = -1;
      if (MODE == M_ROWS_BWD_WEIGHT && lane < 16 && gw * 16 + lane < sch.Kc) jcur = p.ridx[gw * 16 + lane];
      for (int kb = 0; kb < ti.nkb; ++kb) {
        int jnext = -1;
        unsigned long long* tabA = rowtab + (kb & 1) * 32;  // [16] addresses in dY, then [16] in A
        if (MODE == M_ROWS_BWD_WEIGHT) {
          if (lane < 16) {
            tabA[lane] = jcur >= 0 ? (unsigned long long)(p.gA + (size_t)jcur * p.ldgA) : 0ull;
            tabA[16 + lane] = jcur >= 0 ? (unsigned long long)(p.gB + (size_t)jcur * p.ldgB) : 0ull;
            const int j = (kb + 1) * BK + gw * 16 + lane;
            if (kb + 1 < ti.nkb && j < sch.Kc) jnext = p.ridx[j];
          }
          __syncwarp();  // the table entries are read by other lanes below
        }
        int good = 1;
        if (lane == 0) good = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status) ? 1 : 0;
        good = __shfl_sync(0xffffffffu, good, 0);
        if (!good) { ok = false; break; }
        const uint32_t sA = base + stage * L::STAGE_BYTES;
        const uint32_t sB = sA + L::A_BYTES;
        const int kx = kb * BK;
        if (warp == 0 && lane == 0) {
          if (MODE == M_ROWS_BWD_WEIGHT) {
            mbar_arrive(full_bar(stage));
          } else {
            mbar_arrive_expect_tx(full_bar(stage), (uint32_t)(L::A_BYTES + ti.nbox * 64 * BK * 2));
#pragma unroll
            for (int bxi = 0; bxi < 4; ++bxi) {
              if (bxi < ti.nbox) {
                if (MODE == M_ROWS_FWD) tma_load_2d(sB + bxi * (64 * BK * 2), mapB, full_bar(stage), kx, ti.bx[bxi]);
                else tma_load_2d(sB + bxi * (64 * BK * 2), mapB, full_bar(stage), ti.bx[bxi], kx);
              }
            }
          }
        }
        if (MODE != M_ROWS_BWD_WEIGHT) {
          // [128 rows][64 k]: rows 4g .. 4g+3 at byte 512 g of the stage
          if (lane < 8)
            tma_gather4_2d(sA + (uint32_t)(8 * gw + lane) * 512u, mapG, full_bar(stage), kx, r4[0], r4[1], r4[2], r4[3]);
        } else {
          // boxes of [64 contraction rows][64 columns]: A operand = dY columns m0.., B operand = A columns n0..
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int jl = 4 * q + sub, jr = gw * 16 + jl;
            const unsigned long long pa = tabA[jl], pb = tabA[16 + jl];
            const uint32_t off = (uint32_t)jr * 128u + (uint32_t)((ch ^ (jr & 7)) << 4);
#pragma unroll
            for (int bxi = 0; bxi < BM / 64; ++bxi) {
              const int col = ti.ax[bxi] + 8 * ch;
              const bool in = pa != 0ull && col < sch.M_gemm;
              cp_async_16(sA + (uint32_t)bxi * (64 * BK * 2) + off,
                          in ? (const void*)(pa + (unsigned long long)col * 2ull) : (const void*)p.gA, in ? 16u : 0u);
            }
#pragma unroll
            for (int bxi = 0; bxi < 4; ++bxi) {
              if (bxi < ti.nbox) {
                const int col = ti.bx[bxi] + 8 * ch;
                const bool in = pb != 0ull && col < sch.N_gemm;
                cp_async_16(sB + (uint32_t)bxi * (64 * BK * 2) + off,
                            in ? (const void*)(pb + (unsigned long long)col * 2ull) : (const void*)p.gA, in ? 16u : 0u);
              }
            }
          }
          cp_async_mbar_arrive_noinc(full_bar(stage));
        }
        jcur = jnext;
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
    }
  } else if (warp == 0 || (has_second_producer(MODE) && warp == 10)) {
    // ===================== TMA producers =====================
    // In the class form of the tile pattern (and in the tile-list kernels) two threads issue the copies, lane 0 of warp 0 the even contraction
    // blocks (counted over all tiles of the CTA) and lane 0 of warp 10 the odd ones: there a thread spends ~160
    // cycles in each copy instruction, three or four per block, and one thread alone paced the product (0.44 us per
    // block where the MMAs need 0.34; -10 to -25 % per product with two).  Everywhere else one thread keeps up, and a
    // second one gains nothing (the row form's weight gradient was 4 % slower with the eleventh warp merely present):
    // only the class-form kernels and the tile-list kernels have warp 10, and it stays idle in the class form's
    // dense draws.
    constexpr bool TWO = has_second_producer(MODE) && !(is_class_mode(MODE) && PLAIN);
    // Warp 0 first turns the descriptors it was given into those of the sampled pattern (the first
    // operand stage is free until the first load and serves as the 128-byte work area of each); warp 10 works out
    // the same addresses and waits for it.
    const int me = warp == 0 ? 0 : 1;
    const int32_t* hin = (FUSED && p.hdr_in != nullptr) ? p.hdr_in : p.hdr;
    const uint32_t smid = sm_id();
    CUtensorMap* slots = p.tm_slots + (size_t)(smid < (uint32_t)ARD_TM_SM_MAX ? smid : 0u) * ARD_TM_SLOTS;
    auto special = [&](int mi, int indexed, int slot) -> const CUtensorMap* {
      const int32_t* h = indexed == 2 ? hin : p.hdr;
      if (indexed == 0) return &p.maps[mi].tm;
      if (me == 1) return tensormap_specialised_address(&p.maps[mi], h[HDR_DP], slots + slot);
      return tensormap_specialise(&p.maps[mi], h[HDR_DP], h[HDR_B], h[HDR_NKEEP], smem + 128 * slot, slots + slot, lane);
    };
    const CUtensorMap* mapA = special(0, p.mapA_indexed, 0);
    const CUtensorMap* mapB = special(1, p.mapB_indexed, 1);
    const CUtensorMap* mapA4[4] = {mapA, mapA, mapA, mapA};
    const CUtensorMap* mapB4[4] = {mapB, mapB, mapB, mapB};
    if (is_lstm_mode(MODE)) {
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        if (MODE == M_LSTM_BWD_DATA || MODE == M_LSTM_BWD_WEIGHT) mapA4[g] = special(2 + g, 1, 2 + g);
        if (MODE == M_LSTM_FWD || MODE == M_LSTM_BWD_DATA) mapB4[g] = special(6 + g, 1, 6 + g);
      }
    }
    if (me == 0) fence_proxy_async_smem();  // the work area is about to be overwritten by asynchronous copies
    if (has_second_producer(MODE)) asm volatile("bar.sync 3, 64;" ::: "memory");  // the rewritten descriptors are in global memory
    if (smid >= (uint32_t)ARD_TM_SM_MAX) {  // more SMs than the scratch was laid out for: refuse rather than share a slot
      if (lane == 0) { *abort_flag = 1; atomicMax(p.status, (int)ARD_ERR_UNSUPPORTED); }
    } else if (lane == 0) {
      // only the rewritten copies live in global memory and need the tensor-map proxy's acquire; a descriptor
      // used as encoded is read from the kernel's parameters
      auto acquire = [&](const CUtensorMap* m, int mi) {
        if (m != &p.maps[mi].tm) tensormap_acquire(m);
      };
      acquire(mapA, 0);
      acquire(mapB, 1);
      if (is_lstm_mode(MODE)) {
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          if (MODE == M_LSTM_BWD_DATA || MODE == M_LSTM_BWD_WEIGHT) acquire(mapA4[g], 2 + g);
          if (MODE == M_LSTM_FWD || MODE == M_LSTM_BWD_DATA) acquire(mapB4[g], 6 + g);
        }
      }
      int stage = 0;
      uint32_t phase = 0;
      int turn = 0;  // whose block this is: blocks alternate between the two producers over all tiles
      bool ok = true;
      Unit un;
      for (int i = 0; ok && sch.unit(w0, i, un); ++i) {
        const TileInfo ti = sch.template tile<PLAIN>(p, un.t);
        const int kb_begin = un.kb0, kb_end = un.kb1 < 0 ? ti.nkb : un.kb1;
        const uint32_t stage_tx = (uint32_t)(L::A_BYTES + ti.nbox * 64 * BK * 2) * CTAS;  // bytes of the whole pair
        // walk of the kept-block list: entry li, 64-wide piece `sub` of that pattern tile
        int li = 0, sub = 0;
        int kbase = (ti.klist != nullptr && ti.nkb > 0) ? ti.klist[0] * p.ts : 0;
        if (!TWO && me == 1) break;  // one producer only
        for (int kb = kb_begin; kb < kb_end; ++kb, turn ^= TWO ? 1 : 0) {
          if (turn != me) {
            // the other producer's block: only the walk moves on
            if (ti.klist != nullptr && ++sub == ti.kper) {
              sub = 0;
              ++li;
              if (kb + 1 < ti.nkb) kbase = ti.klist[li] * p.ts;
            }
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            continue;
          }
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
          const uint32_t sA = base + stage * L::STAGE_BYTES;
          const uint32_t sB = sA + L::A_BYTES;
          // In a pair every load reports to the leader's barrier, which expects the bytes of both CTAs.
          const uint32_t fbar = (CTAS == 2) ? mapa_u32(full_bar(stage), 0u) : full_bar(stage);
          if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), stage_tx);
          auto load = [&](uint32_t dst, const CUtensorMap* map, int x, int y) {
            if (CTAS == 2) tma_load_2d_pair(dst, map, fbar, x, y);
            else tma_load_2d(dst, map, fbar, x, y);
          };
          // contraction coordinate of this block
          int kx;
          if (ti.klist != nullptr) {
            kx = kbase + sub * BK;
            if (++sub == ti.kper) {
              sub = 0;
              ++li;
              if (kb + 1 < ti.nkb) kbase = ti.klist[li] * p.ts;  // used by the next block, not this one
            }
          } else {
            kx = kb * BK;
          }
          const CUtensorMap* mapBk = mapB;
          if (MODE == M_LSTM_BWD_DATA) {
            // contraction runs gate by gate over the kept units: block kb = (gate, 64 kept units)
            const int nkg = ti.nkb >> 2;
            const int g = kb / nkg;
            kx = (kb - g * nkg) * BK;
            mapBk = mapB4[g];
            load(sA, mapA4[g], kx, ti.m0);
          } else if (!A_MN) {
            load(sA, mapA, kx, ti.m0);  // [BM rows][64 k]
          } else {
#pragma unroll
            for (int i = 0; i < BM / 64; ++i)  // [64 k rows][64 m] per box
              load(sA + i * (64 * BK * 2), MODE == M_LSTM_BWD_WEIGHT ? sel_map(mapA4, ti.gate) : mapA, ti.ax[i], kx);
          }
          // B always moves in 64-wide boxes: K-major [64 rows][64 k] stacked, MN-major [64 k][64 n].
          // In a pair this CTA stages the second half of the tile's B boxes if its rank is 1.
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            if (i < ti.nbox) {
              if (MODE == M_LSTM_FWD) load(sB + i * (64 * BK * 2), mapB4[i], kx, ti.bx[i]);
              else if (!B_MN) load(sB + i * (64 * BK * 2), mapBk, kx, ti.bx[i]);
              else load(sB + i * (64 * BK * 2), mapBk, ti.bx[i], kx);
            }
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0 && rank == 0) {
      // descriptors without the start address: K-major (LBO unused, SBO 1024) or MN-major (LBO 8 KiB, SBO 1024)
      const uint64_t desc_a_hi = A_MN ? make_desc(0, 64 * BK * 2, 1024) : make_desc(0, 16, 1024);
      const uint64_t desc_b_hi = B_MN ? make_desc(0, 64 * BK * 2, 1024) : make_desc(0, 16, 1024);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      Unit un;
      int nacc = 0;  // tiles that used an accumulator so far (a tile without contraction blocks uses none)
      for (; ok && sch.unit(w0, it, un); ++it) {
        const TileInfo ti = sch.template tile<PLAIN>(p, un.t);
        const int kb_begin = un.kb0, kb_end = un.kb1 < 0 ? ti.nkb : un.kb1;
        if (kb_end <= kb_begin) continue;  // nothing to multiply: the epilogue warps write the zeros on their own
        const uint32_t idesc = make_idesc(ti.bn, A_MN, B_MN, BM * CTAS);
        const int acc = nacc & 1;
        const uint32_t acc_phase = (uint32_t)(nacc >> 1) & 1u;
        ++nacc;
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = kb_begin; kb < kb_end; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status)) { ok = false; break; }
          if (MODE == M_ROWS_BWD_WEIGHT) {
            // the gathered operands were written by ordinary asynchronous copies (generic proxy)
            fence_proxy_async_smem();
            tc_fence_after();
          }
          // This thread's instruction stream is what feeds the tensor pipe: the descriptors of a block are
          // the stage's descriptor plus a constant per 16-deep step (the start-address field counts 16-byte
          // units: K-major 32 bytes = 2 per step, MN-major 16 k-rows = 2048 bytes = 128 per step).
          const uint32_t sA = base + stage * L::STAGE_BYTES;
          const uint64_t ad0 = desc_a_hi | (uint64_t)((sA & 0x3FFFFu) >> 4);
          const uint64_t bd0 = desc_b_hi | (uint64_t)(((sA + L::A_BYTES) & 0x3FFFFu) >> 4);
#pragma unroll
          for (int s = 0; s < BK / 16; ++s) {
            const uint64_t ad = ad0 + (uint64_t)(s * (A_MN ? 128 : 2));
            const uint64_t bd = bd0 + (uint64_t)(s * (B_MN ? 128 : 2));
            const uint32_t accum = (kb != kb_begin || s != 0) ? 1u : 0u;
            if (CTAS == 2) tc_mma_bf16_pair(d_tmem, ad, bd, idesc, accum);
            else tc_mma_bf16(d_tmem, ad, bd, idesc, accum);
          }
          // frees the stage (in both CTAs of a pair) once these MMAs have read it
          if (CTAS == 2) tc_commit2(empty_bar(stage), (uint16_t)3);
          else tc_commit(empty_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        if (CTAS == 2) tc_commit2(tfull_bar(acc), (uint16_t)3);
        else tc_commit(tfull_bar(acc));
      }
    }
  } else {
    // ===================== epilogue (warps 2..9) =====================
    const int q = warp & 3;                 // TMEM lane quadrant this warp may read
    const int half = (warp - 2) >> 2;       // which half of the tile's columns
    const int row_in_tile = q * 32 + lane;  // accumulator row owned by this thread
    float* stg = reinterpret_cast<float*>(smem + L::STG_OFF) + (warp - 2) * (32 * 33);
    const int dp = sch.dp, bb = sch.b - 1;
    const uint32_t magic_dp = (uint32_t)(0x100000000ull / (unsigned)dp) + 1u;  // exact x/dp for x < 2^16
    int it = 0, nacc = 0;
    bool ok = true;
    Unit un;
    for (; ok && sch.unit(w0, it, un); ++it) {
      const TileInfo ti = sch.template tile<PLAIN>(p, un.t);
      // An empty contraction leaves zeros: such a tile has no accumulator and no barrier traffic, these warps
      // just write it (the same way as any other tile, from zeros instead of the accumulator).
      const bool has_acc = (un.kb1 < 0 ? ti.nkb : un.kb1) > un.kb0;
      const int acc = nacc & 1;
      const uint32_t acc_phase = (uint32_t)(nacc >> 1) & 1u;
      if (has_acc) {
        ++nacc;
        if (!mbar_wait(tfull_bar(acc), acc_phase, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
      }
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN);
      const int m = ti.m0 + row_in_tile;
      const int nch = ti.bn / 32;  // 32-column chunks in this tile, split between the two warps of a quadrant
      const int ch_lo = half * (nch / 2), ch_hi = (half == 0) ? nch / 2 : nch;

      // Output row and validity by mode.
      bool row_ok;
      long long out_row;
      if (MODE == M_ROW_BWD_WEIGHT || MODE == M_LSTM_BWD_WEIGHT) {
        row_ok = m < sch.M_gemm;
        out_row = (long long)bb + (long long)m * dp;
        if (FUSED && MODE == M_ROW_BWD_WEIGHT && p.hdr_in != nullptr) out_row = m;  // packed gradient rows
        if (MODE == M_LSTM_BWD_WEIGHT) out_row += ti.out_row0;
      } else if (MODE == M_ROWS_FWD || MODE == M_ROWS_BWD_DATA) {
        row_ok = m < sch.M_gemm;
        out_row = row_ok ? (long long)p.ridx[m] : 0;  // the results go back to the rows they came from
      } else if (MODE == M_TILE_BWD_WEIGHT) {
        row_ok = row_in_tile < ti.rows_valid && m < sch.M_gemm;
        out_row = m;
      } else if (MODE == M_TILEC_BWD_WEIGHT) {
        const int orow = (row_in_tile >> 6) ? ti.orow[1] : ti.orow[0];
        out_row = orow + (row_in_tile & 63);
        row_ok = orow >= 0 && out_row < sch.M_gemm;
      } else {
        row_ok = m < sch.M_gemm;
        out_row = m;
        // compact operand of a row list: the results go back to the rows the operand was gathered from
        if (FUSED && (MODE == M_ROW_FWD || MODE == M_ROW_BWD_DATA) && p.ridx != nullptr && row_ok) out_row = p.ridx[m];
      }

      // The values of one 32-column chunk of this thread's accumulator row (already loaded into r[]), whose
      // first output column is n: rescale, and for the layer-step kernels bias / activation / ReLU adjoint.
      auto values = [&](const uint32_t (&r)[32], int n, float (&v)[32]) {
        if (FUSED && MODE == M_ROW_FWD) {
          // layer step: bias of the original neuron, activation, rescale (Sec. 3.2, last paragraph).
          // Lane l fetches the bias of column n + l once; the row loop takes it from there by shuffle (32
          // loads per thread and chunk otherwise, all of them on the critical path of a single-wave launch).
          float bl = 0.f;
          if (p.bias != nullptr && n + lane < sch.n_keep) bl = __ldg(p.bias + bb + (n + lane) * dp);
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            float z = (has_acc ? __uint_as_float(r[i]) : 0.f) + __shfl_sync(0xffffffffu, bl, i);
            if (p.relu) z = fmaxf(z, 0.f);
            v[i] = p.alpha * z;
          }
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = has_acc ? p.alpha * __uint_as_float(r[i]) : 0.f;
        }
        if (FUSED && MODE == M_ROW_BWD_DATA && p.act != nullptr && row_ok) {
          // adjoint of the producing layer's ReLU: zero where its (saved) output was not positive
          const __nv_bfloat16* arow = reinterpret_cast<const __nv_bfloat16*>(p.act) + (size_t)m * p.ldact + n;
          const int na = min(32, sch.N_gemm - n);
          if (na >= 32) {
#pragma unroll
            for (int q8 = 0; q8 < 4; ++q8) {
              const uint4 a = reinterpret_cast<const uint4*>(arow)[q8];
              const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
              for (int h = 0; h < 8; ++h) {
                // bf16 > 0: sign bit clear and magnitude non-zero
                const uint32_t bits = (w[h >> 1] >> ((h & 1) * 16)) & 0xFFFFu;
                if ((bits & 0x8000u) || (bits & 0x7FFFu) == 0u || (bits & 0x7FFFu) > 0x7F80u) v[q8 * 8 + h] = 0.f;
              }
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (i < na && !(__bfloat162float(arow[i]) > 0.f)) v[i] = 0.f;
          }
        }

      };

      // One 32-column chunk of this thread's accumulator row, already loaded into r[].
      auto emit = [&](const uint32_t (&r)[32], int ch) {
        const int oc = sel4(ti.ocol, ch >> 1);
        if (oc < 0) return;                    // padding of a class tile
        const int n = oc + (ch & 1) * 32;      // output column of this chunk
        float v[32];
        values(r, n, v);

        if (MODE == M_ROW_FWD && p.scatter && dp > 1) {
          // Full-width rows: compact column j -> column b-1 + j*dp, zeros everywhere else
          // (Sec. 3.1: dropped outputs are zero).  The 32x32 block is staged through shared memory.
          // The 32 x (32*dp) output block is written in 16-byte pieces; a lane keeps the same piece of
          // the row (or, for narrow blocks, the same piece of a few rows) for the whole block, so where
          // the kept columns fall inside its piece (Eq. 1) is worked out once and each row then costs
          // a shared-memory read, a shift and one store.  Consecutive lanes write consecutive pieces.
          if (n < sch.n_keep) {
#pragma unroll
            for (int i = 0; i < 32; ++i) stg[lane * 33 + i] = v[i];
            __syncwarp();
            const int nv = min(32, sch.n_keep - n);  // kept columns in this chunk
            const int cs = n * dp;
            const bool last = n + 32 >= sch.n_keep;
            const int width = (last ? p.N : (n + 32) * dp) - cs;  // the last chunk also owns the dropped tail
            const int G = (width + 7) >> 3;                        // 16-byte pieces per output row
            const int rows_here = min(32, sch.M_gemm - (ti.m0 + q * 32));
            __nv_bfloat16* obase = reinterpret_cast<__nv_bfloat16*>(p.out) + (size_t)(ti.m0 + q * 32) * p.ldo + cs;
            int rpp = 1, rsub = 0, g = lane, gstep = 32;  // rows per pass, this lane's row in a pass, its piece
            if (G < 32) {
              rpp = 32 / G;
              rsub = lane / G;
              g = lane - rsub * G;
              gstep = G;
              if (rsub >= rpp) g = G;  // no work for this lane
            }
            for (; g < G; g += gstep) {
              // first kept column j0 (relative to n) at or after the piece's first column, and its
              // position inside the piece; further kept columns follow dp positions apart
              const int rel = 8 * g - bb;
              int j0 = 0, pos0 = -rel;
              if (rel > 0) {
                j0 = (int)__umulhi((uint32_t)(rel + dp - 1), magic_dp);
                pos0 = j0 * dp - rel;
              }
              const int nleft = width - 8 * g;  // < 8 only for the last piece of a ragged row
              const float* src = stg + rsub * 33 + j0;
              __nv_bfloat16* dst = obase + (size_t)rsub * p.ldo + 8 * g;
              const size_t dstep = (size_t)rpp * p.ldo;
              for (int rr = rsub; rr < rows_here; rr += rpp, src += rpp * 33, dst += dstep) {
                uint32_t w0 = 0u, w1 = 0u, w2 = 0u, w3 = 0u;
                if (dp >= 8) {
                  if (pos0 < 8 && j0 < nv) {  // at most one kept column per piece
                    const uint32_t u = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(src[0])) << ((pos0 & 1) * 16);
                    const int wd = pos0 >> 1;
                    w0 = wd == 0 ? u : 0u;
                    w1 = wd == 1 ? u : 0u;
                    w2 = wd == 2 ? u : 0u;
                    w3 = wd == 3 ? u : 0u;
                  }
                } else {
#pragma unroll
                  for (int m = 0; m < 4; ++m) {
                    const int pos = pos0 + m * dp;
                    if (pos < 8 && j0 + m < nv) {
                      const uint32_t u = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(src[m])) << ((pos & 1) * 16);
                      const int wd = pos >> 1;
                      w0 |= wd == 0 ? u : 0u;
                      w1 |= wd == 1 ? u : 0u;
                      w2 |= wd == 2 ? u : 0u;
                      w3 |= wd == 3 ? u : 0u;
                    }
                  }
                }
                if (nleft >= 8) {
                  *reinterpret_cast<uint4*>(dst) = make_uint4(w0, w1, w2, w3);
                } else {
                  const uint32_t w[4] = {w0, w1, w2, w3};
#pragma unroll
                  for (int pos = 0; pos < 8; ++pos)
                    if (pos < nleft)
                      dst[pos] = __ushort_as_bfloat16((unsigned short)(w[pos >> 1] >> ((pos & 1) * 16)));
                }
              }
            }
            __syncwarp();
          }
        } else {
          const int nvalid = (is_class_mode(MODE) && !PLAIN) ? 32
                             : (MODE == M_LSTM_FWD ? min(32, sch.n_keep - (ti.n0 + (ch & 1) * 32))
                                                   : min(32, sch.N_gemm - n));
          if (row_ok && nvalid > 0) {
            store_row32(p.out, (size_t)out_row * p.ldo, n, v, nvalid, p.out_is_f32, p.accumulate);
            if ((MODE == M_ROW_BWD_WEIGHT || MODE == M_LSTM_BWD_WEIGHT) && p.zero_fill) {
              // Compact row m owns output rows [m*dp, (m+1)*dp); the last one also owns the tail.
              const long long goff = (MODE == M_LSTM_BWD_WEIGHT) ? ti.out_row0 : 0;  // the gate's block of rows
              const long long first = goff + (long long)m * dp;
              const long long lastrow = goff + ((m == sch.M_gemm - 1) ? (long long)p.N - 1
                                                                     : min((long long)(m + 1) * dp - 1, (long long)p.N - 1));
              for (long long rz = first; rz <= lastrow; ++rz)
                if (rz != out_row) zero_row32(p.out, (size_t)rz * p.ldo, n, nvalid, p.out_is_f32);
            }
          }
        }
      };

      if (Sched<BN, MODE, CTAS, SHARE>::SK_MODE && un.sk_tile >= 0) {
        // A share of a shared tile.  The raw fp32 partial sums are parked in global memory; the warp that
        // arrives last for this 32-row block of the tile adds the shares in contraction order (so the
        // result does not depend on who is last) and runs the normal epilogue.  Nobody waits.
        constexpr int WSLOTS = EPI_WARPS * CTAS;
        const int wslot = (int)rank * EPI_WARPS + (warp - 2);
        float4* mine = p.sk_ws + (size_t)((w0 * 2 + un.slot) * WSLOTS + wslot) * SK_SLOT_F4 + lane;
        uint32_t r[32];
#pragma unroll 1
        for (int ch = ch_lo; ch < ch_hi; ++ch) {
          tmem_ld32(t_row + (uint32_t)(ch * 32), r);
          tmem_ld_wait();
          float4* dst = mine + (ch - ch_lo) * 256;
#pragma unroll
          for (int q8 = 0; q8 < 8; ++q8)
            __stcg(dst + q8 * 32, make_float4(__uint_as_float(r[4 * q8]), __uint_as_float(r[4 * q8 + 1]),
                                              __uint_as_float(r[4 * q8 + 2]), __uint_as_float(r[4 * q8 + 3])));
        }
        __threadfence();
        __syncwarp();
        int* cnt = p.sk_cnt + un.sk_tile * WSLOTS + wslot;
        int arrived = 0;
        if (lane == 0) arrived = atomicAdd(cnt, 1);
        arrived = __shfl_sync(0xffffffffu, arrived, 0);
        if (arrived == un.nsplit - 1) {
          if (lane == 0) *cnt = 0;  // armed again for the next launch
          __threadfence();
          // Two 32-column chunks per round, so that 16 loads per thread are in flight for each share.
#pragma unroll 1
          for (int ch = ch_lo; ch < ch_hi; ch += 2) {
            const bool two = ch + 1 < ch_hi;
            float sum0[32], sum1[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) sum0[i] = sum1[i] = 0.f;
#pragma unroll 1
            for (int j = un.jfirst; j < un.jfirst + un.nsplit; ++j) {
              if (j == w0) {
                tmem_ld32(t_row + (uint32_t)(ch * 32), r);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) sum0[i] += __uint_as_float(r[i]);
                if (two) {
                  tmem_ld32(t_row + (uint32_t)((ch + 1) * 32), r);
                  tmem_ld_wait();
#pragma unroll
                  for (int i = 0; i < 32; ++i) sum1[i] += __uint_as_float(r[i]);
                }
              } else {
                const int slot_j = un.sk_tile - sch.share_start(j) / sch.KT;
                const float4* src =
                    p.sk_ws + (size_t)((j * 2 + slot_j) * WSLOTS + wslot) * SK_SLOT_F4 + lane + (ch - ch_lo) * 256;
                float4 x0[8], x1[8];
#pragma unroll
                for (int q8 = 0; q8 < 8; ++q8) x0[q8] = __ldcg(src + q8 * 32);
#pragma unroll
                for (int q8 = 0; q8 < 8; ++q8) x1[q8] = two ? __ldcg(src + 256 + q8 * 32) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int q8 = 0; q8 < 8; ++q8) {
                  sum0[4 * q8] += x0[q8].x;
                  sum0[4 * q8 + 1] += x0[q8].y;
                  sum0[4 * q8 + 2] += x0[q8].z;
                  sum0[4 * q8 + 3] += x0[q8].w;
                }
#pragma unroll
                for (int q8 = 0; q8 < 8; ++q8) {
                  sum1[4 * q8] += x1[q8].x;
                  sum1[4 * q8 + 1] += x1[q8].y;
                  sum1[4 * q8 + 2] += x1[q8].z;
                  sum1[4 * q8 + 3] += x1[q8].w;
                }
              }
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(sum0[i]);
            emit(r, ch);
            if (two) {
#pragma unroll
              for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(sum1[i]);
              emit(r, ch + 1);
            }
          }
        }
      } else {
        // Software pipeline over this warp's chunks: the TMEM load of chunk i+1 is in flight while
        // chunk i is converted and stored.
        // bf16 rows written plainly go out two chunks at a time through the warp's staging block, so that a
        // store instruction writes four whole 128-byte lines (eight lanes per row) instead of 16 bytes in each
        // of 32 rows: with a short contraction the epilogue is what a tile waits for, and the scattered form
        // kept it at 6.4 us per 256 x 256 tile where the products and loads need 4.1.
        constexpr bool PAIR_MODES = MODE == M_ROW_FWD || MODE == M_ROW_BWD_DATA || MODE == M_ROW_BWD_WEIGHT ||
                                    (is_class_mode(MODE) && PLAIN);
        const bool pair_ok = PAIR_MODES && !p.out_is_f32 && !p.accumulate && !(MODE == M_ROW_FWD && p.scatter && dp > 1) &&
                             !(MODE == M_ROW_BWD_WEIGHT && p.zero_fill);
        const unsigned okmask = __ballot_sync(0xffffffffu, row_ok);
        // The class tiling keeps its list in the first part of the staging area: its warps stage one chunk
        // (32 rows x 17 words) behind it and write 64-byte row segments, four lanes per row.
        constexpr bool CLASS_LIST = is_class_mode(MODE) && !PLAIN;
        constexpr int SW = CLASS_LIST ? 17 : 33;  // words per staged row
        uint32_t* stw = CLASS_LIST ? reinterpret_cast<uint32_t*>(smem + L::STG_OFF + CLASS_LIST_BYTES) + (warp - 2) * (32 * 17)
                                   : reinterpret_cast<uint32_t*>(stg);
        const bool one_ok = CLASS_LIST && !p.out_is_f32 && !p.accumulate;
        auto stage_half = [&](const uint32_t (&r)[32], int n, int half2) {
          float v[32];
          values(r, n, v);
          uint32_t* sw = stw + lane * SW + half2 * 16;
#pragma unroll
          for (int i = 0; i < 16; ++i) sw[i] = pack_bf16(v[2 * i], v[2 * i + 1]);
        };
        auto flush_one = [&](int n) {  // 32 rows x 32 columns starting at output column n
          __syncwarp();
          const int piece = lane & 3;
#pragma unroll
          for (int it4 = 0; it4 < 4; ++it4) {
            const int rr = it4 * 8 + (lane >> 2);
            const long long orow = __shfl_sync(0xffffffffu, out_row, rr);
            const uint32_t* q = stw + rr * SW + piece * 4;
            const uint4 w = make_uint4(q[0], q[1], q[2], q[3]);
            if ((okmask >> rr) & 1u)
              *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + (size_t)orow * p.ldo + n + piece * 8) = w;
          }
          __syncwarp();
        };
        // one chunk of a class tile: staged and written in row segments, or the per-thread form
        auto emit_class = [&](const uint32_t (&r)[32], int ch) {
          const int oc1 = sel4(ti.ocol, ch >> 1);
          if (one_ok && oc1 >= 0) {
            const int n = oc1 + (ch & 1) * 32;
            stage_half(r, n, 0);
            flush_one(n);
          } else {
            emit(r, ch);
          }
        };
        auto flush_pair = [&](int n) {  // 32 rows x 64 columns starting at output column n
          __syncwarp();
          const int piece = lane & 7;
#pragma unroll
          for (int it8 = 0; it8 < 8; ++it8) {
            const int rr = it8 * 4 + (lane >> 3);
            const long long orow = __shfl_sync(0xffffffffu, out_row, rr);
            const uint32_t* q = stw + rr * SW + piece * 4;
            const uint4 w = make_uint4(q[0], q[1], q[2], q[3]);
            if ((okmask >> rr) & 1u)
              *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + (size_t)orow * p.ldo + n + piece * 8) = w;
          }
          __syncwarp();
        };
        uint32_t ra[32], rb[32];
        if (has_acc && ch_lo < ch_hi) tmem_ld32(t_row + (uint32_t)(ch_lo * 32), ra);
#pragma unroll 1
        for (int ch = ch_lo; ch < ch_hi; ch += 2) {
          if (has_acc) {
            tmem_ld_wait();
            if (ch + 1 < ch_hi) tmem_ld32(t_row + (uint32_t)((ch + 1) * 32), rb);
          }
          const int oc = sel4(ti.ocol, ch >> 1);
          const bool paired = pair_ok && (ch & 1) == 0 && ch + 1 < ch_hi && oc >= 0 && oc + 64 <= sch.N_gemm;
          if (paired) stage_half(ra, oc, 0);
          else if (CLASS_LIST) emit_class(ra, ch);
          else emit(ra, ch);
          if (ch + 1 < ch_hi) {
            if (has_acc) {
              tmem_ld_wait();
              if (ch + 2 < ch_hi) tmem_ld32(t_row + (uint32_t)((ch + 2) * 32), ra);
            }
            if (paired) {
              stage_half(rb, oc + 32, 1);
              flush_pair(oc);
            } else if (CLASS_LIST) {
              emit_class(rb, ch + 1);
            } else {
              emit(rb, ch + 1);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0 && has_acc) {
        if (CTAS == 2) mbar_arrive_cluster(mapa_u32(tempty_bar(acc), 0u));  // the leader's barrier
        else mbar_arrive(tempty_bar(acc));
      }
    }
  }
  };
  if (is_class_mode(MODE) && sch.dense) roles(std::true_type{});
  else roles(std::false_type{});

  // ---- teardown ----
  tc_fence_before();
  __syncwarp();  // lanes that left their role's loop one by one arrive at the block-wide barrier together
  if (CTAS == 2) cluster_sync_all();  // neither CTA may leave while its peer can still touch its memory
  else __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if (CTAS == 2) tmem_dealloc2(tmem_base, TMEM_COLS);
    else tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// max_tiles: tile count of the densest pattern
template <int BN, int MODE, int CTAS, bool SHARE = false, bool FUSED = false>
ard_status launch_mode(ard_ctx* ctx, const TcParams& p, const TcMap* maps, int max_tiles, cudaStream_t s) {
  using L = SmemLayout<BN, CTAS>;
  static bool attr_done[64] = {};
  static int max_clusters[64] = {};
  auto kern = ard_gemm_tc_kernel<BN, MODE, CTAS, SHARE, FUSED>;
  const int dev = ctx->device & 63;
  if (!attr_done[dev]) {
    ARD_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::TOTAL));
    attr_done[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(tc_threads(MODE));
  cfg.dynamicSmemBytes = L::TOTAL;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  int workers = ctx->sm_count / CTAS;
  cfg.attrs = attr;
  cfg.numAttrs = 0;
  if (CTAS == 2) {
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.numAttrs = 1;
    if (max_clusters[dev] == 0) {
      // how many CTA pairs the device can hold at once (SM pairs must share a TPC)
      cfg.gridDim = dim3(ctx->sm_count / 2 * 2);
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n < 1) n = ctx->sm_count / 2;
      max_clusters[dev] = n;
    }
    workers = max_clusters[dev];
  }
  if (max_tiles < workers) workers = max_tiles;
  if (workers < 1) workers = 1;
  if (workers * CTAS > ctx->sm_count) return ARD_ERR_UNSUPPORTED;  // the partial-sum scratch is sized per SM
  cfg.gridDim = dim3(workers * CTAS);
  if (ard_pdl_allowed(ctx, s)) {
    attr[cfg.numAttrs].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[cfg.numAttrs].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs++;
  }
  TcParamsT<nmaps(MODE)> pc;
  static_cast<TcParams&>(pc) = p;
  pc.tm_slots = ctx->d_tm_slots;
  for (int i = 0; i < nmaps(MODE); ++i) pc.maps[i] = maps[i];
  ARD_CUDA_OK(cudaLaunchKernelEx(&cfg, kern, pc));
  ctx->launches++;
  ARD_CUDA_OK(cudaGetLastError());
  return ARD_OK;
}

inline int cdiv(int a, int b) { return (a + b - 1) / b; }

}  // namespace

// N extent of the output tile.
//   Row patterns: 0 = chosen on the device from the sampled n_keep, or the value forced by ard_set_tile_n.
//   Tile patterns: 0 = class form (256-wide tiles gathered from pattern tiles of one class), available for
//   pattern tiles of 64 / 128 (forward and backward-data also 256) and periods up to 64; otherwise a fixed
//   width that divides the pattern tile.
int tc_pick_bn(ard_ctx* ctx, ard_kind kind, GemmOp op, int dp_bound, int ts) {
  const int f = ctx->force_bn;
  if (kind == ARD_TILE) {
    const bool class_ok = dp_bound <= 64 && (ts == 64 || ts == 128 || (ts == 256 && op != OP_BWD_WEIGHT));
    if (f == 0 && class_ok) return 0;
    if (f && ts % f == 0 && (op == OP_BWD_WEIGHT || f <= 128)) return f;
    if (op == OP_BWD_WEIGHT) return ts % 256 == 0 ? 256 : (ts % 128 == 0 ? 128 : 64);
    return ts % 128 == 0 ? 128 : 64;
  }
  return f;
}

ard_status launch_gemm_tc(ard_ctx* ctx, ard_kind kind, GemmOp op, const TcArgs& a, cudaStream_t s) {
  TcParams p = {};
  const TcMap maps[2] = {a.mapA, a.mapB};
  p.mapA_indexed = a.mapA_indexed;
  p.mapB_indexed = a.mapB_indexed;
  p.hdr = a.g.hdr;
  p.idx = a.g.idx;
  p.col_ptr = a.g.col_ptr;
  p.col_idx = a.g.col_idx;
  p.row_ptr = a.g.row_ptr;
  p.row_idx = a.g.row_idx;
  p.B = a.g.B;
  p.K = a.g.K;
  p.N = a.g.N;
  p.ts = a.ts;
  p.alpha = a.g.alpha;
  p.out = a.g.out;
  p.ldo = a.g.ldo;
  p.out_is_f32 = a.g.out_is_f32;
  p.scatter = (kind == ARD_ROW && op == OP_FWD && a.g.flag0 == ARD_OUT_SCATTER_ZEROFILL) ? 1 : 0;
  p.zero_fill = (op == OP_BWD_WEIGHT) ? a.g.flag1 : 0;
  p.status = a.g.status;
  p.force_bn = (kind == ARD_ROW) ? a.bn : 0;
  p.accumulate = a.g.accumulate;
  p.band_m = ctx->band_m;
  const bool share = kind == ARD_ROW && ctx->stream_k && ctx->d_sk_ws != nullptr;
  p.sk_ws = share ? reinterpret_cast<float4*>(ctx->d_sk_ws) : nullptr;
  p.sk_cnt = ctx->d_sk_cnt;
  p.sk_min_blocks = ctx->sk_min_blocks;
  p.sk_min_gain = ctx->sk_min_gain;
  p.hdr_in = a.g.hdr_in;
  p.bias = a.g.bias;
  p.relu = a.g.relu;
  p.act = a.g.act;
  p.ldact = a.g.ldact;
  p.ext_mode = a.g.ext_mode;
  p.ridx = a.g.ridx;
  // the layer-step variants are separate instantiations, so that the plain products carry none of their code
  const bool fused = kind == ARD_ROW && (p.hdr_in != nullptr || p.bias != nullptr || p.relu != 0 || p.act != nullptr ||
                                         p.ext_mode != 0);
  const int bn = (kind == ARD_ROW) ? 256 : a.bn;
  if (kind == ARD_ROW && op == OP_BWD_WEIGHT && p.ext_mode == 2 && ctx->use_pairs && p.N > BM &&
      (p.force_bn == 0 || p.force_bn >= 128) && ctx->d_sk_ws != nullptr) {
    // Weight gradient over a row list's compact operands: few output tiles (channels x fan-in) and a contraction
    // as long as the list, so the tiles are always cut along the contraction and shared by all SMs.
    p.sk_ws = reinterpret_cast<float4*>(ctx->d_sk_ws);
    p.sk_any = 1;
    return launch_mode<256, M_ROW_BWD_WEIGHT, 2, true, true>(ctx, p, maps, 1 << 30, s);  // every SM takes a share
  }

#define ARD_TC_CASE(BN_, MODE_, TILES_) \
  if (bn == BN_) return launch_mode<BN_, MODE_, 1>(ctx, p, maps, (TILES_), s);
#define ARD_TC_ROW(MODE_, TILES_)                                                      \
  if (fused) return launch_mode<256, MODE_, 1, false, true>(ctx, p, maps, (TILES_), s);      \
  return share ? launch_mode<256, MODE_, 1, true>(ctx, p, maps, (TILES_), s) : launch_mode<256, MODE_, 1, false>(ctx, p, maps, (TILES_), s);
  // Row patterns with at least two 128-row tiles of output use CTA pairs (256-row tiles).
#define ARD_TC_PAIR(MODE_, MROWS_, NCOLS_)                                                      \
  if (ctx->use_pairs && (MROWS_) > BM && (p.force_bn == 0 || p.force_bn >= 128) && fused)       \
    return launch_mode<256, MODE_, 2, false, true>(ctx, p, maps, cdiv((MROWS_), 2 * BM) * cdiv((NCOLS_), 128), s);         \
  if (ctx->use_pairs && (MROWS_) > BM && (p.force_bn == 0 || p.force_bn >= 128))                \
    return share ? launch_mode<256, MODE_, 2, true>(ctx, p, maps, cdiv((MROWS_), 2 * BM) * cdiv((NCOLS_), 128), s)         \
                 : launch_mode<256, MODE_, 2, false>(ctx, p, maps, cdiv((MROWS_), 2 * BM) * cdiv((NCOLS_), 128), s);

  if (kind == ARD_ROW) {
    if (op == OP_FWD) {
      const int mt = cdiv(p.B, BM);
      ARD_TC_PAIR(M_ROW_FWD, p.B, p.N)
      ARD_TC_ROW(M_ROW_FWD, mt * cdiv(p.N, 64))
    } else if (op == OP_BWD_DATA) {
      const int mt = cdiv(p.B, BM);
      ARD_TC_PAIR(M_ROW_BWD_DATA, p.B, p.K)
      ARD_TC_ROW(M_ROW_BWD_DATA, mt * cdiv(p.K, 64))
    } else {
      const int mt = cdiv(p.N, BM);
      ARD_TC_PAIR(M_ROW_BWD_WEIGHT, p.N, p.K)
      ARD_TC_ROW(M_ROW_BWD_WEIGHT, mt * cdiv(p.K, 64))
    }
  } else if (bn == 0) {
    // class form of the tile pattern; the grid covers all SMs, CTAs without tiles leave at once
    const int many = 1 << 30;
    const int rows = (op == OP_BWD_WEIGHT) ? p.N : p.B;
    const bool pairs = ctx->use_pairs && rows > BM;
    if (op == OP_FWD)
      return pairs ? launch_mode<256, M_TILEC_FWD, 2>(ctx, p, maps, many, s) : launch_mode<256, M_TILEC_FWD, 1>(ctx, p, maps, many, s);
    if (op == OP_BWD_DATA)
      return pairs ? launch_mode<256, M_TILEC_BWD_DATA, 2>(ctx, p, maps, many, s)
                   : launch_mode<256, M_TILEC_BWD_DATA, 1>(ctx, p, maps, many, s);
    return pairs ? launch_mode<256, M_TILEC_BWD_WEIGHT, 2>(ctx, p, maps, many, s)
                 : launch_mode<256, M_TILEC_BWD_WEIGHT, 1>(ctx, p, maps, many, s);
  } else {
    // List form with at least two 128-row tiles of output and 128-wide pattern tiles: CTA pairs (256 x 128
    // tiles; each CTA stages half of the kept block, the instruction is the wide one).
    const bool pairs = ctx->use_pairs && p.B > BM && bn == 128;
    if (op == OP_FWD) {
      const int mt = cdiv(p.B, BM);
      if (pairs) return launch_mode<128, M_TILE_FWD, 2>(ctx, p, maps, cdiv(p.B, 2 * BM) * cdiv(p.N, 128), s);
      ARD_TC_CASE(128, M_TILE_FWD, mt * cdiv(p.N, 128))
      ARD_TC_CASE(64, M_TILE_FWD, mt * cdiv(p.N, 64))
    } else if (op == OP_BWD_DATA) {
      const int mt = cdiv(p.B, BM);
      if (pairs) return launch_mode<128, M_TILE_BWD_DATA, 2>(ctx, p, maps, cdiv(p.B, 2 * BM) * cdiv(p.K, 128), s);
      ARD_TC_CASE(128, M_TILE_BWD_DATA, mt * cdiv(p.K, 128))
      ARD_TC_CASE(64, M_TILE_BWD_DATA, mt * cdiv(p.K, 64))
    } else {
      const int tiles = (p.K / p.ts) * (p.N / p.ts) * cdiv(p.ts, BM) * (p.ts / bn);
      ARD_TC_CASE(256, M_TILE_BWD_WEIGHT, tiles)
      ARD_TC_CASE(128, M_TILE_BWD_WEIGHT, tiles)
      ARD_TC_CASE(64, M_TILE_BWD_WEIGHT, tiles)
    }
  }
#undef ARD_TC_CASE
#undef ARD_TC_ROW
#undef ARD_TC_PAIR
  return ARD_ERR_UNSUPPORTED;
}

// Products over a list of kept rows (Sec. 5.2.1).  Single-CTA tiles.
ard_status launch_rows_tc(ard_ctx* ctx, GemmOp op, const TcArgs& a, const int32_t* ridx, const void* gA, int ldgA,
                          const void* gB, int ldgB, cudaStream_t s) {
  TcParams p = {};
  // forward, backward-data: mapA the gathered operand (one-row boxes), mapB the weight (64 x 64 boxes); the weight
  // gradient takes its operands as plain pointers (gA = dY, gB = A) and uses neither
  const TcMap maps[2] = {a.mapA, a.mapB};
  p.hdr = a.g.hdr;
  p.B = a.g.B;
  p.K = a.g.K;
  p.N = a.g.N;
  p.alpha = a.g.alpha;
  p.out = a.g.out;
  p.ldo = a.g.ldo;
  p.out_is_f32 = a.g.out_is_f32;
  p.status = a.g.status;
  p.force_bn = a.bn;
  p.band_m = ctx->band_m;
  p.sk_min_blocks = 16;
  p.sk_min_gain = 1;
  p.ridx = ridx;
  p.gA = reinterpret_cast<const __nv_bfloat16*>(gA);
  p.ldgA = ldgA;
  p.gB = reinterpret_cast<const __nv_bfloat16*>(gB);
  p.ldgB = ldgB;
  if (op == OP_FWD) return launch_mode<256, M_ROWS_FWD, 1>(ctx, p, maps, cdiv(p.B, BM) * cdiv(p.N, 64), s);
  if (op == OP_BWD_DATA) return launch_mode<256, M_ROWS_BWD_DATA, 1>(ctx, p, maps, cdiv(p.B, BM) * cdiv(p.K, 64), s);
  return launch_mode<256, M_ROWS_BWD_WEIGHT, 1>(ctx, p, maps, cdiv(p.N, BM) * cdiv(p.K, 64), s);
}

// LSTM gate products (single CTA per tile; the batch of a recurrent step is small).
ard_status launch_lstm_tc(ard_ctx* ctx, int backward, const TcArgs& a, cudaStream_t s) {
  TcParams p = {};
  TcMap maps[10];
  maps[0] = a.mapA;
  maps[1] = a.mapB;
  for (int g = 0; g < 4; ++g) { maps[2 + g] = a.mapA4[g]; maps[6 + g] = a.mapB4[g]; }
  // the per-gate descriptors carry the pattern; A and B themselves are used only where they are plain
  p.mapA_indexed = 0;
  p.mapB_indexed = 0;
  p.hdr = a.g.hdr;
  p.idx = a.g.idx;
  p.col_ptr = p.col_idx = p.row_ptr = p.row_idx = nullptr;
  p.B = a.g.B;
  p.K = a.g.K;
  p.N = a.g.N;
  p.ts = a.ts;  // forward: gate block width of Z
  p.alpha = a.g.alpha;
  p.out = a.g.out;
  p.ldo = a.g.ldo;
  p.out_is_f32 = a.g.out_is_f32;
  p.scatter = 0;
  p.zero_fill = 0;
  p.status = a.g.status;
  p.force_bn = a.bn;
  p.accumulate = a.g.accumulate;
  p.band_m = 0;
  p.sk_ws = nullptr;
  p.sk_cnt = nullptr;
  p.sk_min_blocks = 16;
  p.sk_min_gain = 1;
  p.hdr_in = nullptr;
  p.bias = nullptr;
  p.relu = 0;
  p.act = nullptr;
  p.ldact = 0;
  const int mt = cdiv(p.B, BM);
  if (!backward) return launch_mode<256, M_LSTM_FWD, 1>(ctx, p, maps, mt * cdiv(p.N, 64), s);
  if (backward == 2) {
    // weight gradient of the four gate blocks: p.B = rows summed over, p.N = H units per gate
    p.zero_fill = a.g.flag1;
    if (ctx->use_pairs && p.N > BM && (p.force_bn == 0 || p.force_bn >= 128))
      return launch_mode<256, M_LSTM_BWD_WEIGHT, 2>(ctx, p, maps, 4 * cdiv(p.N, 2 * BM) * cdiv(p.K, 128), s);
    return launch_mode<256, M_LSTM_BWD_WEIGHT, 1>(ctx, p, maps, 4 * cdiv(p.N, BM) * cdiv(p.K, 64), s);
  }
  return launch_mode<256, M_LSTM_BWD_DATA, 1>(ctx, p, maps, mt * cdiv(p.K, 64), s);
}
