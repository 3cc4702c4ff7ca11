// Internal declarations shared by the translation units of libard.so.
#pragma once

#include <cuda_runtime.h>
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>
#include <stdint.h>

#include <vector>

#include "ard.h"

// ---- device-resident pattern --------------------------------------------------------------------
// One int32 allocation: a 16-word header followed by the index lists.
enum {
  HDR_KIND = 0,
  HDR_DP = 1,
  HDR_B = 2,
  HDR_NKEEP = 3,   // kept neurons (row) or kept tiles (tile)
  HDR_UNITS = 4,
  HDR_TR = 5,
  HDR_TC = 6,
  HDR_TS = 7,
  HDR_MAPIDX = 8,  // dp*(dp-1)/2 + (b-1): the pattern's number among all (dp, b) pairs
  HDR_WORDS = 16
};

struct ard_pattern {
  ard_ctx* ctx;
  ard_kind kind;
  int K_dim, N_dim, ts, Tr, Tc, units;
  int dp_bound;        // largest dp the last sample/set call can have produced
  unsigned long long generation;  // bumped by every sample / set call
  int32_t* d_hdr;      // device: header
  int32_t* d_idx;      // device: kept list (row: neuron index; tile: t-1), capacity `units`
  int32_t* d_col_ptr;  // tile only: [Tc+1]
  int32_t* d_col_idx;  // tile only: [units]
  int32_t* d_row_ptr;  // tile only: [Tr+1]
  int32_t* d_row_idx;  // tile only: [units]
};

// Device-resident list of the kept rows of an input matrix with M rows (Sec. 5.2.1) and the per-region
// dropout probabilities it is drawn from (Sec. 5.1).  d_hdr mimics a pattern header (dp = b = 1, n_keep).
struct ard_rows {
  ard_ctx* ctx;
  int M, x, regions;
  int32_t* d_hdr;    // HDR_WORDS
  int32_t* d_idx;    // kept rows, ascending, capacity M
  int32_t* d_stage;  // sampler scratch: the kept rows of every 2048-row slice, compacted per slice
  int32_t* d_counts; // sampler scratch: kept rows per slice
  uint8_t* d_flag;   // 1 = kept, per row
  uint32_t* d_P;     // per region: dropped iff the row's random word is below this
};

struct ArdDistribution {
  int ndp = 0;
  unsigned long long* d_cdf = nullptr;  // device: ndp entries
  std::vector<unsigned long long> h_cdf;
};

enum MapVariant {
  MAP_PLAIN = 0,         // the descriptor as encoded: [rows][cols], pitch ld
  MAP_STRIDED_ROWS = 1,  // per pattern: rows b-1, b-1+dp, ... (n_keep of them), all cols
  MAP_COMPACT_COLS = 2   // per pattern: all rows, cols 0..n_keep-1 of a compact matrix
};

// A TMA descriptor handed to a kernel BY VALUE (a kernel parameter), with what the kernel needs to turn it into
// the descriptor of the sampled pattern.  The host encodes the descriptor of the whole matrix and never learns
// the pattern; the producer warp of the kernel rewrites the address, one extent and the row pitch for the (dp, b)
// it reads from the pattern header (tensormap_specialise in sm100_ptx.h) and publishes the result in a slot of
// the context's descriptor scratch that belongs to its SM.  Nothing is cached, allocated or copied per call.
struct alignas(64) TcMap {
  CUtensorMap tm;          // [rows][cols] of `base`, pitch ld: also what a dense pattern (dp = 1) reads
  const void* base;
  const void* dense_base;  // MAP_COMPACT_COLS: the matrix a dense pattern reads instead of `base` (nullptr: base)
  int ld, dense_ld;        // elements
  int variant;             // MapVariant
  int pad_;
};

// Descriptor scratch of a context: one group of 128-byte slots per SM for the kernels that own their SM (the
// tcgen05 product kernels: their shared memory leaves no room for a second block), and one group per block for the
// whole-sequence LSTM kernels (cooperative launches of at most ARD_TM_LSTM_BLOCKS blocks, one at a time per
// context).
constexpr int ARD_TM_SM_MAX = 256;
constexpr int ARD_TM_SLOTS = 16;
constexpr int ARD_TM_LSTM_BLOCKS = 512;
constexpr int ARD_TM_LSTM_SLOTS = 8;
// Two buffers of 128 batch rows by (8 units per block x ARD_TM_LSTM_BLOCKS) bf16 columns.
constexpr int ARD_LSTM_HC_LD = 8 * ARD_TM_LSTM_BLOCKS;
static inline size_t lstm_hc_bytes() { return (size_t)2 * 128 * ARD_LSTM_HC_LD * 2; }
static inline size_t tm_slots_bytes() {
  return ((size_t)ARD_TM_SM_MAX * ARD_TM_SLOTS + (size_t)ARD_TM_LSTM_BLOCKS * ARD_TM_LSTM_SLOTS) * sizeof(CUtensorMap);
}

constexpr int ARD_MLP_EVENTS = 104;  // fork, forward done, two joins, and three per layer (up to 32 layers)

struct ard_ctx {
  int device;
  int sm_count;
  ard_path path;
  int force_bn;
  int use_pairs;      // tensor-core row kernels: CTA pairs (cta_group::2) when the output has >= 2 row tiles
  int band_m;         // raster band height of the tensor-core kernels, in 128-row tiles
  int reuse_compact;  // opt-in: consecutive backward calls share one compacted dY
  int lstm_persistent; // ard_lstm_forward: one cooperative kernel for the whole sequence when the layer fits
  unsigned int* d_grid_bar;  // arrival counter of that kernel's grid-wide barrier
  float* d_lstm_partial;     // partial sums of the whole-sequence BPTT kernel, lstm_bwd_partial_bytes(sm_count)
  void* d_lstm_hc;           // compact copies of h_{t-1} and h_t of the whole-sequence forward kernel, lstm_hc_bytes()
  int lstm_compact_h;        // ... which contracts over the kept units of h alone under a pattern
  int use_pdl;        // launch kernels with programmatic stream serialization (see ard_launch)
  int pdl_in_capture; // ... also while the stream is being captured into a CUDA graph
  int stream_k;       // tensor-core row kernels: share the last, partial wave of tiles along the contraction
  int sk_min_blocks;  // fewest 64-wide contraction blocks worth a separate share
  int sk_min_gain;    // fewest blocks the sharing must save per worker to be used
  void* d_sk_ws;      // partial accumulators of the shared tail, sk_ws_bytes(sm_count)
  int* d_sk_cnt;      // arrival counters, zero between launches
  struct { const void* src; int ld, B, N; const ard_pattern* pat; unsigned long long gen; cudaStream_t stream; } last_gather;
  size_t workspace_bytes;
  void* d_workspace;
  int* d_status;
  ArdDistribution dist[ARD_MAX_DISTRIBUTIONS];
  CUtensorMap* d_tm_slots;  // descriptor scratch, tm_slots_bytes()
  unsigned long long launches;
  void* encode_fn;  // cuTensorMapEncodeTiled, resolved at run time
  // ard_mlp_step: the weight-side work of an iteration (weight compaction, weight and bias gradients) runs on
  // a second stream, forked from and joined back into the caller's stream with these events
  int mlp_two_streams;
  int mlp_persistent;  // ard_mlp_step: the whole iteration in one cooperative kernel when the stack fits it
  cudaStream_t side_stream;
  cudaStream_t aux_stream;  // expansion of the weight gradients and bias gradients
  cudaEvent_t ev[ARD_MLP_EVENTS];
  int n_ev;  // events created so far (0: none yet)
};

// Shared tail of the tensor-core row kernels: every CTA owns two slots, each holding the fp32 partial
// sums of its 128 rows x 256 columns of a tile; one arrival counter per (tail tile, epilogue warp),
// fewer tail tiles than CTAs, 8 epilogue warps per CTA.
static inline size_t sk_ws_bytes(int sm_count) { return (size_t)sm_count * 2 * 128 * 256 * sizeof(float); }
static inline size_t sk_cnt_bytes(int sm_count) { return (size_t)sm_count * 8 * sizeof(int); }

// max(1, ceil(t * s)) with the product taken exactly (Sec. 5.1, step 3: "at least t% of the sampled values").
// t * s as a double is off by at most half a unit in the last place, which only matters when the rounded product
// is an integer; the fused multiply-add gives the sign of what the rounding dropped.  Needs s < 2^31, 0 <= t <= 1.
static inline long long ard_exact_need(double t, long long s) {
  const double prod = t * (double)s;
  const double err = fma(t, (double)s, -prod);
  double c = ceil(prod);
  if (c == prod && err > 0.0) c += 1.0;
  return c < 1.0 ? 1 : (long long)c;
}

// Creates the context's second and third stream and their events on first use; false if they do not exist
// and cannot be created now (`main` is being captured into a graph: nothing may be created then).
bool ard_side_streams(ard_ctx* ctx, cudaStream_t main);

// The shared tail of the row kernels parks partial sums in ONE scratch per context, so it must stay off while
// products of the same context run side by side on several streams: calls that fork hold one of these.
struct SharedTailOff {
  ard_ctx* ctx;
  int saved;
  SharedTailOff(ard_ctx* c, bool forked) : ctx(c), saved(c->stream_k) { if (forked) c->stream_k = 0; }
  ~SharedTailOff() { ctx->stream_k = saved; }
};

// ---- launchers implemented in the .cu files -----------------------------------------------------
// One whole-matrix descriptor (see TcMap): [rows][cols] bf16 at `base`, pitch ld, boxes of box_rows x box_cols.
ard_status ard_encode_tcmap(ard_ctx* ctx, const void* base, int rows, int cols, int ld, int units, int variant,
                            int box_rows, int box_cols, TcMap* out);
// The iteration of ard_mlp_step in one cooperative kernel; ARD_ERR_UNSUPPORTED (nothing enqueued) when the
// stack does not fit it.
ard_status launch_mlp_persistent(ard_ctx* ctx, const ard_mlp_layer* layers, int n_layers, int B, const void* X, int ldx,
                                 const void* dOut, int lddout, void* dX, int lddx, int dist_id, uint64_t seed,
                                 uint64_t iteration_base, uint64_t* iteration_counter, cudaStream_t s);
ard_status launch_sampler(ard_ctx* ctx, ard_pattern* pat, const unsigned long long* d_cdf, int ndp,
                          uint64_t seed, uint64_t iteration, uint32_t stream_id, int forced_dp, int forced_b,
                          cudaStream_t s, unsigned long long* d_counter = nullptr, int advance = 0);

struct GemmArgs {
  const int32_t* hdr;
  const int32_t* idx;
  const int32_t* col_ptr;
  const int32_t* col_idx;
  const int32_t* row_ptr;
  const int32_t* row_idx;
  int B, K, N;
  float alpha;
  const void* A0;  // X or dY
  int lda0;
  const void* A1;  // W or X
  int lda1;
  void* out;
  int ldo;
  int flag0;       // fwd: outmode; bwd: dy_is_compact
  int flag1;       // bwd_weight: zero_fill_dropped
  int out_is_f32;
  int accumulate;  // add to the existing output instead of overwriting it
  int* status;
  // Fused layer step (row patterns).  hdr_in: header of the row pattern of the layer that produced the
  // input; the input matrix and the weight then hold only that layer's kept columns (n_in of them), so
  // the fan-in extent of the product is n_in instead of K.
  const int32_t* hdr_in;
  const float* bias;  // forward: added before the activation, indexed by the original neuron
  int relu;           // forward: max(., 0) before the rescale
  const void* act;    // backward-data: the output is zeroed where act <= 0 (operand element type, layout of dX)
  int ldact;
  // Row-list products on compact operands (Sec. 5.2.1): hdr is the row list's header, the layer is dense.
  // ext_mode 1: hdr's count is the row extent of A and of the output, output row m goes to row ridx[m];
  // ext_mode 2: hdr's count is the length of the contraction (weight gradient).
  int ext_mode;
  const int32_t* ridx;
};

enum GemmOp { OP_FWD = 0, OP_BWD_DATA = 1, OP_BWD_WEIGHT = 2 };

// CUDA-core family (fp32 or bf16 operands, fp32 accumulate).
ard_status launch_gemm_cc(ard_ctx* ctx, ard_kind kind, GemmOp op, ard_dtype dtype, const GemmArgs& a, int ts,
                          cudaStream_t s);

// tcgen05 family (bf16 operands, fp32 accumulate in TMEM).
struct TcArgs {
  TcMap mapA;
  TcMap mapB;
  TcMap mapA4[4];  // LSTM gate products: one descriptor per gate
  TcMap mapB4[4];
  int mapA_indexed, mapB_indexed;  // 0: used as encoded, 1: specialised to the pattern, 2: to the input pattern
  GemmArgs g;
  int ts;
  int bn;  // N tile: 64, 128 or 256
};
int tc_pick_bn(ard_ctx* ctx, ard_kind kind, GemmOp op, int dp_bound, int ts);
ard_status launch_gemm_tc(ard_ctx* ctx, ard_kind kind, GemmOp op, const TcArgs& a, cudaStream_t s);
ard_status launch_lstm_tc(ard_ctx* ctx, int backward, const TcArgs& a, cudaStream_t s);
ard_status launch_rows_tc(ard_ctx* ctx, GemmOp op, const TcArgs& a, const int32_t* ridx, const void* gA, int ldgA,
                          const void* gB, int ldgB, cudaStream_t s);

// Whole-sequence LSTM kernels (lstm_persistent.cu).
size_t lstm_bwd_partial_bytes(int sm_count);
bool lstm_persistent_bwd_fits(ard_ctx* ctx, int B, int H);
ard_status launch_lstm_backward_persistent(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H, float alpha,
                                           const TcMap mapDZ[4], const TcMap mapW[4], const void* W, int ldw,
                                           const float* C, const float* G, const float* dH_last, float* D, float* dc,
                                           void* DZ, cudaStream_t s);
bool lstm_persistent_fits(ard_ctx* ctx, int B, int klen, int H);
ard_status launch_lstm_forward_persistent(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H,
                                          int kx0, int klen, int add_zx, float alpha, const TcMap& mapXH, const TcMap mapW[4],
                                          const TcMap* mapHc, const void* W, int ldw,
                                          void* XH, const float* bias, float* C, float* G, cudaStream_t s);

ard_status launch_gather_cols(ard_ctx* ctx, const int32_t* hdr, const int32_t* idx, const void* src, int ld_src,
                              void* dst, int ld_dst, int rows, int elem_bytes, int max_cols, int skip_dense,
                              cudaStream_t s);

ard_status launch_expand_cols(ard_ctx* ctx, const int32_t* hdr, const void* src, int ld_src, int src_is_bf16, float* dst,
                              int ld_dst, int rows, int N, float alpha, cudaStream_t s);

// Sensitivity-aware row dropout (rows.cu).
ard_status launch_sensitivity(ard_ctx* ctx, ard_rows* rows, ard_dtype dtype, const void* A, int lda, int Kc, int c,
                              int n_runs, int need, float threshold, uint32_t P_sens, uint32_t P_insens, uint64_t seed,
                              uint64_t iteration, uint32_t stream_id, cudaStream_t s);
ard_status launch_fill_probability(ard_ctx* ctx, ard_rows* rows, uint32_t P, cudaStream_t s);
ard_status launch_rows_sample(ard_ctx* ctx, ard_rows* rows, uint64_t seed, uint64_t iteration, uint32_t stream_id,
                              cudaStream_t s);
ard_status launch_rows_gather(ard_ctx* ctx, const ard_rows* rows, const void* src, int ld_src_bytes, void* dst,
                              int ld_dst_bytes, int row_bytes, cudaStream_t s);
ard_status launch_zero_dropped_rows(ard_ctx* ctx, const ard_rows* rows, void* out, int ld_bytes, int row_bytes,
                                    cudaStream_t s);

ard_status launch_zero_dropped_tiles(ard_ctx* ctx, const ard_pattern* pat, void* dW, int lddw, int elem_bytes,
                                     cudaStream_t s);

// Layer-step helpers (aux_kernels.cu); elem_bytes 2 or 4.
ard_status launch_compact_weight_cols(ard_ctx* ctx, const int32_t* hdr, const int32_t* hdr_in, const void* W, int ldw,
                                      void* Wk, int ldwk, int N, int K, int elem_bytes, cudaStream_t s);
ard_status launch_expand_weight_grad_cols(ard_ctx* ctx, const int32_t* hdr, const int32_t* hdr_in, const void* dWk,
                                          int lddwk, void* dW, int lddw, int N, int K, int elem_bytes, int zero_fill,
                                          cudaStream_t s);
ard_status launch_bias_grad(ard_ctx* ctx, const int32_t* hdr, const void* dZ, int lddz, int dz_is_compact,
                            int elem_bytes_is_bf16, int B, int N, float* db, int zero_fill, cudaStream_t s);

ard_status launch_lstm_gates(ard_ctx* ctx, const ard_pattern* pat, ard_dtype h_dtype, int B, int H, float alpha,
                             const float* Z, int ldz_gate, const float* bias, const float* c_prev, int ldc, float* c,
                             void* h, int ldh, int h_scatter, float* gates_saved, cudaStream_t s);
ard_status launch_lstm_gates_bwd(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dz_dtype, int B, int H, float alpha,
                                 const float* gates_saved, const float* c_prev, const float* c, int ldc,
                                 const float* dh, int lddh, int dh_scatter, float* dc_inout, void* dZ, int ldz_gate,
                                 cudaStream_t s);

// ---- programmatic dependent launch ----------------------------------------------------------------
// Every kernel of the library is launched so that its blocks may become resident while the previous
// kernel of the stream is still draining: the block set-up (barriers, tensor memory, index arithmetic)
// and the launch latency then overlap the tail of that kernel.  In return every kernel (1) lets its own
// successor start early with pdl_launch_dependents() and (2) calls pdl_wait_prior_grids() before its
// first access to global memory; that call returns once all earlier kernels of the stream have
// completed and their writes are visible.  Both are no-ops for a kernel launched the ordinary way.
// (3) Nothing an earlier kernel of the stream writes (pattern headers and lists, activations, gradients)
// is read through the read-only data path (const __restrict__ parameters, __ldg): a block can be
// resident long before its wait returns, and that path is not made coherent by the wait: a block of the
// kernel that followed the sampler was seen to read the previous iteration's pattern header that way.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_prior_grids() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// The attribute is also kept while a stream is being captured into a CUDA graph (the nodes are then joined
// by programmatic edges); ard_set_option(ctx, ARD_OPT_PDL_IN_CAPTURE, 0) launches the ordinary way during a capture.
inline bool ard_pdl_allowed(const ard_ctx* ctx, cudaStream_t s) {
  if (!ctx->use_pdl) return false;
  if (ctx->pdl_in_capture) return true;
  cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &st) != cudaSuccess) return false;
  return st == cudaStreamCaptureStatusNone;
}

template <typename... P, typename... A>
inline cudaError_t ard_launch(const ard_ctx* ctx, void (*kern)(P...), dim3 grid, dim3 block, size_t smem,
                              cudaStream_t s, A... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  if (ard_pdl_allowed(ctx, s)) {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  }
  return cudaLaunchKernelEx(&cfg, kern, P(args)...);
}

#define ARD_CUDA_OK(expr)                       \
  do {                                          \
    cudaError_t e__ = (expr);                   \
    if (e__ != cudaSuccess) return ARD_ERR_CUDA; \
  } while (0)
