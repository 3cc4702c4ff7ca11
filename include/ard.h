/*
 * ard.h -- C ABI of the Approximate Random Dropout (ARD) hot path for NVIDIA B200 (sm_100a).
 *
 * Method: "DNN Training Acceleration via Exploring GPGPU Friendly Sparsity" (arXiv 2203.05705),
 * Sec. 3: every training iteration one regular dropout pattern (period dp, bias b) is drawn from a
 * distribution K over periods; a row pattern drops whole neurons, a tile pattern drops weight tiles
 * (DropConnect-like); the dropped rows / tiles are never fetched or multiplied.
 *
 * Conventions shared by every call
 *   - Every pointer named X, W, Y, dY, dX, dW, Z, c, h ... is a DEVICE pointer owned by the caller.
 *     Pointers named K, and every `int32_t* out`-style argument of ard_pattern_to_host /
 *     ard_pattern_tile_lists_to_host, are HOST pointers.
 *   - Matrices are row-major.  The weight is stored NEURON-MAJOR: W[N][K] with leading dimension
 *     ldw (elements); row n holds the K fan-in weights of output neuron n.  This is the transpose
 *     of the math orientation W[K x N] in Y = X W.  dW has the same layout.
 *   - `cuda_stream` is a cudaStream_t passed as void*.  Calls only enqueue work; they do not
 *     synchronise unless stated.  The pattern lives on the device: nothing about it returns to the
 *     host unless ard_pattern_to_host is called.
 *   - The library allocates device memory only in its create calls (ard_create, ard_pattern_create,
 *     ard_rows_create, ard_blocks_create) and frees it in the matching destroy call.  No product call
 *     allocates, copies descriptors or synchronises: the TMA descriptors of the bf16 tensor-core path
 *     are encoded on the host per call, travel as kernel parameters and are fitted to the sampled pattern
 *     by the kernel itself, so operands may sit at a new address in every call.
 *   - A context's scratch memory and status word are shared by its calls: work enqueued through one
 *     context must be ordered (one stream, or streams ordered by events).  Use one context per
 *     concurrently running stream.
 *   - Every call returns an ard_status.  Problems the host can see (NULL, sizes, leading
 *     dimensions, alignment, distribution) are rejected before anything is launched.  Problems only
 *     the device can see (a wait inside a kernel that ran out of patience) set a sticky device
 *     status word, read with ard_last_device_status; the kernel then exits normally and the output
 *     of that call is unspecified.  Nothing aborts or traps.
 *   - Arithmetic: ARD_F32 operands are multiplied and accumulated in fp32 on the CUDA cores;
 *     ARD_BF16 operands are multiplied on the tensor cores with fp32 accumulation.
 *   - There is no CPU fallback.
 */
#ifndef ARD_H_
#define ARD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ard_ctx ard_ctx;         /* owns distributions, workspace, descriptor cache, status word */
typedef struct ard_pattern ard_pattern; /* handle of a device-resident pattern (header + index lists)   */
typedef struct ard_rows ard_rows;       /* handle of a device-resident list of kept input-matrix rows   */
typedef struct ard_blocks ard_blocks;   /* handle of a device-resident set of kept input-matrix blocks  */

typedef enum {
  ARD_OK = 0,
  ARD_ERR_INVALID_ARG = 1,   /* NULL pointer, negative size, unknown enum value            */
  ARD_ERR_SHAPE = 2,         /* sizes inconsistent with the pattern, ld < extent, tile size */
  ARD_ERR_ALIGNMENT = 3,     /* pointer or leading dimension not aligned as the path needs  */
  ARD_ERR_DISTRIBUTION = 4,  /* K negative / not summing to 1 / longer than the unit count  */
  ARD_ERR_UNSUPPORTED = 5,
  ARD_ERR_CUDA = 6,          /* a CUDA runtime or driver call failed                        */
  ARD_ERR_TIMEOUT = 7,       /* a bounded wait inside a kernel expired (device status)      */
  ARD_ERR_NOMEM = 8          /* workspace too small or allocation failed                    */
} ard_status;

typedef enum { ARD_F32 = 0, ARD_BF16 = 1 } ard_dtype;
typedef enum { ARD_ROW = 0, ARD_TILE = 1 } ard_kind;
typedef enum { ARD_OUT_COMPACT = 0, ARD_OUT_SCATTER_ZEROFILL = 1 } ard_outmode;
/* Flags that may be OR-ed into the `outmode` argument of ard_fwd and into the `dy_is_compact`
 * argument of ard_bwd_data (whose bit 0 keeps its meaning): */
#define ARD_FLAG_OUT_F32 0x10    /* bf16 operands: write the result as fp32 (leading dimension in fp32 elements) */
#define ARD_FLAG_ACCUMULATE 0x20 /* add the product to the existing output; not with ARD_OUT_SCATTER_ZEROFILL   */
#define ARD_FLAG_RELU 0x40       /* ard_layer_fwd only: apply max(., 0) before the rescale                      */

/* Selects the kernel family for ARD_BF16 calls.  AUTO picks the tcgen05 path when the shape and
 * alignment allow it and the CUDA-core path otherwise; the other two force one family (FORCE_TC
 * returns ARD_ERR_ALIGNMENT / ARD_ERR_UNSUPPORTED instead of falling back). */
typedef enum { ARD_PATH_AUTO = 0, ARD_PATH_CUDA_CORE = 1, ARD_PATH_TENSOR_CORE = 2 } ard_path;

#define ARD_MAX_DISTRIBUTIONS 16
#define ARD_MAX_NDP 4096      /* longest distribution accepted                                  */
#define ARD_MAX_NDP_TC 32     /* longest distribution the tensor-core path takes (longer ones: CUDA cores)  */

/* ---- context -------------------------------------------------------------------------------- */

/* Creates a context on CUDA device `device` with `workspace_bytes` of device scratch memory (used
 * to compact a full-width dY for the tensor-core backward GEMMs; 2*B*N bytes suffice for one
 * layer).  Synchronous. */
ard_status ard_create(ard_ctx** ctx, int device, size_t workspace_bytes);
ard_status ard_destroy(ard_ctx* ctx);
ard_status ard_set_path(ard_ctx* ctx, ard_path path);
/* Tuning switches of a context (host state only; nothing is read from the environment).  Defaults in brackets.
 *   ARD_OPT_PDL [1]               launch kernels with programmatic stream serialization
 *   ARD_OPT_PDL_IN_CAPTURE [1]    ... also while the stream is being captured into a CUDA graph
 *   ARD_OPT_SIDE_STREAMS [1]      ard_layer_products / ard_rows_products / ard_blocks_products / ard_mlp_step may
 *                                 fork onto the context's own streams (0: everything on the caller's stream)
 *   ARD_OPT_CTA_PAIRS [1]         tensor-core products with more than 128 output rows use pairs of SMs
 *   ARD_OPT_BAND_ROWS [16]        raster band of the tensor-core tile order, in 128-row tiles (0: one band)
 *   ARD_OPT_MLP_PERSISTENT [1]    ard_mlp_step runs the whole iteration in one cooperative kernel when the stack
 *                                 fits it (see ard_mlp_step); 0: always call by call
 *   ARD_OPT_LSTM_COMPACT_H [1]    the whole-sequence kernels of ard_lstm_forward / ard_lstm_backward contract over
 *                                 the kept units alone when the pattern drops any: forward over a compact copy of
 *                                 h_{t-1} in context scratch, BPTT (at most 256 kept units) with every block of
 *                                 dz_{t+1} in one CTA and one grid-wide barrier per step (0: forward over all H
 *                                 columns, the dropped ones being zero, BPTT always cut along the contraction
 *                                 with partial sums); same results up to the order of fp32 additions
 * Errors: ARD_ERR_INVALID_ARG (unknown option, negative value). */
typedef enum { ARD_OPT_PDL = 0, ARD_OPT_PDL_IN_CAPTURE = 1, ARD_OPT_SIDE_STREAMS = 2, ARD_OPT_CTA_PAIRS = 3,
               ARD_OPT_BAND_ROWS = 4, ARD_OPT_MLP_PERSISTENT = 5, ARD_OPT_LSTM_COMPACT_H = 6 } ard_option;
ard_status ard_set_option(ard_ctx* ctx, ard_option option, int value);
/* Opt-in for training loops.  The tensor-core backward GEMMs of a row pattern read a compacted copy
 * of a full-width dY (kept columns only) that the library makes in the context workspace.  With
 * enable != 0, a backward call whose dY pointer, leading dimension, batch size, pattern sample and
 * stream equal those of the previous backward call on this context reuses that copy instead of
 * gathering again (ard_bwd_data followed by ard_bwd_weight of the same layer then gather once).
 * Enable only if dY is not written between such calls.  Default: off. */
ard_status ard_set_compact_reuse(ard_ctx* ctx, int enable);
/* Tuning / test knob of the tensor-core path: forces the N extent of the output tile (a multiple of
 * 32 from 64 to 256; 0 restores the built-in choice, which for row patterns picks the width with the
 * fewest waves x time per tile on the device).  A forced value a product cannot use is ignored for
 * it. */
ard_status ard_set_tile_n(ard_ctx* ctx, int bn);
/* Optional schedule of the tensor-core path for row patterns.  The output tiles of a product are
 * dealt to the SMs (or SM pairs) in waves.  With enable != 0, when the tile count leaves a partial
 * wave after at least one complete wave, the left-over tiles are computed first, cut along the
 * contraction dimension and shared by all workers, which park fp32 partial sums in context
 * scratch; the share that arrives last adds them in contraction order (so the result does not
 * depend on the arrival order and is the same from launch to launch) and writes the tile.
 * min_blocks: fewest 64-wide contraction blocks worth a separate share (default 16).
 * min_gain_blocks: used only if it shortens the work of every worker by at least this many blocks
 * (default 24).  0 keeps the current value of either.
 * Default: disabled.  On a B200 the parked partial sums and the later start of the shared tiles'
 * epilogues cost about what the better balance saves (a few percent either way, depending on the
 * period), and the forward product with zero fill gets slower.
 * The partial sums live in one scratch per context, so the schedule needs the context's row products to run
 * one after the other: the calls that enqueue several products side by side (ard_layer_products,
 * ard_rows_products, ard_mlp_step on several streams) switch it off for their own launches. */
ard_status ard_set_shared_tail(ard_ctx* ctx, int enable, int min_blocks, int min_gain_blocks);

/* Sec. 3.3: the distribution K = {k_i}, i = 1..ndp, over the periods dp, sum k_i = 1.
 * K: HOST array of ndp doubles, k_i >= 0, |sum - 1| <= 1e-9, 1 <= ndp <= ARD_MAX_NDP.
 * K is quantised to an integer cumulative table on a 2^32 grid (c_i = floor(s_i 2^32 + 1/2) from
 * sequential prefix sums s_i, clamped to be non-decreasing, last entry 2^32), which is the
 * distribution the sampler realises exactly.  Synchronous (small copy).  dist_id in
 * [0, ARD_MAX_DISTRIBUTIONS). */
ard_status ard_set_distribution(ard_ctx* ctx, int dist_id, const double* K, int ndp);
/* The quantisation alone, on the host (no context or GPU needed): validates K as above and writes the
 * ndp cumulative entries to cdf_out (HOST uint64). */
ard_status ard_quantise_distribution(const double* K, int ndp, uint64_t* cdf_out);
/* Sec. 3.3, Algorithm 1: finds K for a target global dropout rate p by gradient descent, on the host
 * in fp64 (no context or GPU needed).  v (length ndp) starts at zero, d = softmax(v) is the
 * distribution, p_u = {(i-1)/i}; the loss (d.p_u - p)^2 + lambda * sum_i d_i ln d_i is reduced by
 * steps v <- v - step * dloss/dv until it changes by less than tol or max_iter steps were taken.
 * (The paper's listing is not printed; squared difference, lambda, the start and the stopping rule are
 * this library's reading of the text.)  At convergence ln k_i is affine in (i-1)/i and
 * K.p_u - p = -lambda*beta/2 with beta its slope, so a small lambda meets the rate closely:
 * lambda = 1e-3, step = 10, tol = 1e-16 reaches |K.p_u - p| ~ 1e-3 in ~2e4 steps for ndp = 16.
 * K_out: HOST array of ndp doubles, summing to 1 within rounding (pass it to ard_set_distribution).
 * iterations_out (may be NULL): steps taken.  Errors: ARD_ERR_INVALID_ARG (NULL, ndp out of range,
 * p outside [0,1), non-positive lambda / step, negative tol), ARD_ERR_DISTRIBUTION (p above the
 * reachable (ndp-1)/ndp, or the iteration diverged because step is too large). */
ard_status ard_search_distribution(double p, int ndp, double lambda, double step, int max_iter, double tol,
                                   double* K_out, int* iterations_out);
/* Copies the quantised cumulative table (ndp entries, HOST uint64) back, for tests. */
ard_status ard_get_distribution_cdf(ard_ctx* ctx, int dist_id, uint64_t* cdf_out, int capacity, int* ndp_out);

/* ---- pattern --------------------------------------------------------------------------------- */

/* A pattern object for a weight of math shape [K_dim x N_dim].
 *   ARD_ROW  (Sec. 3.1): units = the N_dim output neurons; `tile` must be 0.
 *   ARD_TILE (Sec. 3.2): units = the (K_dim/tile) x (N_dim/tile) weight tiles, numbered row-major
 *                        from 1 over (r, c) with r along K and c along N; tile must divide both. */
ard_status ard_pattern_create(ard_ctx* ctx, ard_pattern** pat, ard_kind kind, int K_dim, int N_dim, int tile);
ard_status ard_pattern_destroy(ard_pattern* pat);

/* Sec. 3.4: draws dp from distribution `dist_id`, then b uniformly from {1..dp}, and writes the
 * kept-unit lists (Eq. 1: unit i, 1-based, is kept iff (i - b) mod dp == 0) into the pattern, all
 * on the device, asynchronously on `cuda_stream`.
 * Randomness: Philox4x32-10 with key (seed low, seed high) and counter (iteration low, iteration
 * high, stream_id, 0); word 0 selects dp as the smallest i with word0 < c_i, word 1 selects
 * b = 1 + floor(word1 * dp / 2^32).  The result is a pure function of (table, seed, iteration,
 * stream_id, shape).  Returns ARD_ERR_DISTRIBUTION if the distribution is unset or longer than
 * the pattern's unit count. */
ard_status ard_sample_pattern(ard_ctx* ctx, ard_pattern* pat, int dist_id, uint64_t seed,
                              uint64_t iteration, uint32_t stream_id, void* cuda_stream);

/* Sets (dp, b) explicitly (1 <= b <= dp <= units) and emits the same lists; for tests and for
 * running a layer dense (dp = 1).  Asynchronous. */
ard_status ard_pattern_set(ard_ctx* ctx, ard_pattern* pat, int dp, int b, void* cuda_stream);

/* Test / debug: synchronises the stream and copies dp, b, the number of kept units and the kept
 * list (row: 0-based neuron indices; tile: 0-based linear tile indices t-1, ascending) to HOST
 * buffers.  idx may be NULL; at most idx_capacity entries are written. */
ard_status ard_pattern_to_host(const ard_pattern* pat, int32_t* dp, int32_t* b, int32_t* n_keep,
                               int32_t* idx, size_t idx_capacity, void* cuda_stream);
/* Tile patterns only: the kept tiles grouped by tile-column (col_ptr[Tc+1], col_idx = tile-rows
 * ascending) and by tile-row (row_ptr[Tr+1], row_idx = tile-columns ascending).  HOST buffers;
 * col_idx / row_idx need room for Tr*Tc entries.  Synchronises. */
ard_status ard_pattern_tile_lists_to_host(const ard_pattern* pat, int32_t* col_ptr, int32_t* col_idx,
                                          int32_t* row_ptr, int32_t* row_idx, void* cuda_stream);

/* ---- the three GEMMs (Sec. 3.1 / 3.2: only kept rows / tiles are fetched and multiplied) ------ */

/* Forward:  Y = alpha * X * (W .* Mask(pattern)).
 *   X [B][K] (ldx), W [N][K] neuron-major (ldw).
 *   Row pattern, ARD_OUT_SCATTER_ZEROFILL: Y [B][N] (ldy), dropped columns written as zero.
 *   Row pattern, ARD_OUT_COMPACT: Y [B][n_keep] (ldy >= N so that any pattern fits): column j holds
 *     kept neuron j; columns >= n_keep are not written.
 *   Tile pattern: Y [B][N] always full (outmode ignored).
 *   alpha is the rescale the caller wants fused (1/(1-p) for inverted dropout). */
ard_status ard_fwd(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, int B, int K, int N, float alpha,
                   const void* X, int ldx, const void* W, int ldw, void* Y, int ldy, ard_outmode outmode,
                   void* cuda_stream);

/* Backward-data:  dX = alpha * dY * (W .* Mask)^T,  dX [B][K] (lddx).
 *   dy_is_compact = 0: dY [B][N] full width, dropped columns are ignored (never read as values).
 *   dy_is_compact = 1 (row pattern only): dY [B][n_keep] with column j belonging to kept neuron j. */
ard_status ard_bwd_data(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, int B, int K, int N, float alpha,
                        const void* dY, int lddy, int dy_is_compact, const void* W, int ldw, void* dX, int lddx,
                        void* cuda_stream);

/* Backward-data without any allocation (the paper has no counterpart: this is a deployment
 * variant of ard_bwd_data, same result).  For callers that are not allowed to allocate device
 * memory when they run the layer: a process whose memory plan was frozen after start-up, a plug-in
 * inside an application that owns the allocator, or anyone who must avoid the device-wide
 * synchronisation of cudaMalloc / cudaFree.  ard_bwd_data compacts dY into the workspace that
 * ard_create allocated (and fails with ARD_ERR_NOMEM when that workspace is too small); this call needs no
 * workspace at all, and calls neither cudaMalloc / cudaFree nor any allocating library routine.
 *   Row patterns only, full-width dY [B][N] (lddy), W [N][K] (ldw), dX [B][K] (lddx); runs on the
 *   CUDA cores (fp32 accumulate) for both dtypes.  The compacted copy of dY is kept in a fixed
 *   array inside the library image: ARD_STATIC_SCRATCH_BYTES per GPU that loads the library, held
 *   until the process exits.  B*N*sizeof(element) must not exceed that size, otherwise the call
 *   returns ARD_ERR_NOMEM and launches nothing.
 *   The first call on each device looks up the array's device address; make that first call before
 *   starting any stream capture.  Every call on a device shares the one array, which keeps the
 *   previous call's contents (all entries that are read are rewritten first; nothing needs
 *   clearing).  Calls that overlap on the GPU (other streams, other host threads) race on it:
 *   serialise them.  The looked-up address is cached per device in a plain host array without a lock: host
 *   threads that make the first call at the same time all store the same value, which is harmless. */
#define ARD_STATIC_SCRATCH_BYTES (8u << 20)
ard_status ard_bwd_data_static_scratch(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, int B, int K, int N,
                                       float alpha, const void* dY, int lddy, const void* W, int ldw, void* dX,
                                       int lddx, void* cuda_stream);

/* Backward-weight:  dW = alpha * (X^T dY) .* Mask, stored neuron-major dW [N][K] (lddw), element
 *   type dW_dtype (fp32 or bf16; an ARD_F32 layer requires ARD_F32).  Only kept rows (row pattern)
 *   or kept tiles (tile pattern) are computed and written; if zero_fill_dropped != 0 the dropped
 *   rows / tiles are written as zero, otherwise they are left untouched. */
ard_status ard_bwd_weight(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, ard_dtype dW_dtype, int B, int K,
                          int N, float alpha, const void* X, int ldx, const void* dY, int lddy, int dy_is_compact,
                          void* dW, int lddw, int zero_fill_dropped, void* cuda_stream);

/* The three products of one layer in one iteration behind one call: the same results as ard_fwd, ard_bwd_data
 * (full-width dY) and ard_bwd_weight (full-width dY) with these arguments, but enqueued so that they may run
 * side by side: the forward product on the caller's stream, the backward products on streams the context
 * owns (a tile pattern: one each; a row pattern: both on one, sharing the compact copy of dY), joined back
 * into the caller's stream before the call returns.  The products depend only on X, W, dY and the pattern
 * (Sec. 3.1, 3.2), and on small layers one of them leaves most SMs idle.  The first call on a context creates
 * the streams (make it before any stream capture); the call itself can be captured into a CUDA graph.
 * Inputs must not be written, and outputs not read, by other work until the caller's stream has passed the
 * call.  After ard_set_option(ctx, ARD_OPT_SIDE_STREAMS, 0) everything stays on the caller's stream.  Asynchronous. */
ard_status ard_layer_products(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, ard_dtype dW_dtype, int B, int K,
                              int N, float alpha, const void* X, int ldx, const void* W, int ldw, const void* dY,
                              int lddy, void* Y, int ldy, ard_outmode outmode, void* dX, int lddx, void* dW, int lddw,
                              int zero_fill_dropped, void* cuda_stream);

/* ---- fused layer step (row patterns) ----------------------------------------------------------
 * Sec. 3.2, last paragraph: a layer of a training iteration is the fully connected product, the
 * activation and the dropout mask; under a pattern the mask disappears into the product.  Sec. 3.1:
 * a dropped neuron also removes its column from the input matrix of the layer it feeds and the
 * matching fan-in weights of that layer, so BOTH matrices of that layer's product are compact.
 * (The paper prints no formula for the step; ReLU with relu'(0) = 0, a bias per neuron and the
 * rescale after the activation are this library's reading.)
 *
 * For a layer with row pattern `pat` (N neurons, n kept) fed by a layer with row pattern `in_pat`
 * (its N_dim == this layer's K; n_in kept), or by a full-width input (in_pat == NULL, n_in = K):
 *
 *   forward        A[:, j]  = alpha * act( sum_i X[:, i] * Wk[keep[j]][i] + bias[keep[j]] )     j < n
 *   backward-data  dX[:, i] = alpha * sum_j dZ[:, j] * Wk[keep[j]][i]  (0 where act_prev[:, i] <= 0)  i < n_in
 *   backward-weight dWk[keep[j]][i] = alpha * sum_r dZ[r][j] * X[r][i]                           i < n_in
 *
 * where, with in_pat, X [B][n_in], act_prev [B][n_in] and dX [B][n_in] are COMPACT over the feeding
 * layer's kept neurons (column i = its i-th kept neuron; leading dimensions >= K so that any pattern
 * fits) and Wk / dWk are PACKED in both dimensions: row j holds the j-th kept neuron of `pat`, column i
 * the weight from the i-th kept neuron of the feeding layer (buffers of [N][K-wide rows] so that any
 * pair of patterns fits): Wk is made from W by ard_compact_weight_cols once per iteration, dWk is
 * expanded into dW by ard_expand_weight_grad_cols; in the formulas above read Wk[j][i] for
 * Wk[keep[j]][i].  Without in_pat, Wk = W, dWk = dW (rows at the neurons' own positions) and X is full
 * width.  dZ is the gradient of the pre-activations Z = X Wk + bias (compact [B][n] when the compact
 * bit is set).  To chain layers, call ard_layer_bwd_data of layer l+1 with alpha = alpha_l and
 * act_prev = A_l: its result is dZ_l, compact, which layer l's backward calls take with alpha = 1.
 * bias (fp32 [N], indexed by the original neuron) and act_prev may be NULL.  act_prev has the
 * operand element type.  The output modes and flags are those of ard_fwd / ard_bwd_data /
 * ard_bwd_weight (ARD_OUT_COMPACT, ARD_OUT_SCATTER_ZEROFILL, ARD_FLAG_OUT_F32; ARD_FLAG_RELU selects
 * act = ReLU, otherwise the identity); ARD_FLAG_ACCUMULATE cannot be combined with bias, ReLU or
 * act_prev.  zero_fill_dropped applies without in_pat only (a packed dWk has no rows of dropped neurons:
 * ARD_ERR_INVALID_ARG if both are given; the expansion writes the zeros of dW).  Tensor-core path: bf16, aligned as for ard_fwd, act_prev 16-byte
 * aligned with ldact % 8 == 0; otherwise (and for ARD_F32) the CUDA-core path runs the same step. */
ard_status ard_layer_fwd(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, ard_dtype dtype, int B, int K,
                         int N, float alpha, const void* X, int ldx, const void* Wk, int ldw, const float* bias,
                         void* A, int lda, int outmode_and_flags, void* cuda_stream);
ard_status ard_layer_bwd_data(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, ard_dtype dtype, int B,
                              int K, int N, float alpha, const void* dZ, int lddz, int dz_is_compact_and_flags,
                              const void* Wk, int ldw, const void* act_prev, int ldact, void* dX, int lddx,
                              void* cuda_stream);
ard_status ard_layer_bwd_weight(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, ard_dtype dtype,
                                ard_dtype dW_dtype, int B, int K, int N, float alpha, const void* X, int ldx,
                                const void* dZ, int lddz, int dz_is_compact, void* dWk, int lddw,
                                int zero_fill_dropped, void* cuda_stream);
/* Wk[j][i] = W[keep[j]][keep_in[i]] for j < n, i < n_in; columns n_in up to the next multiple of 64
 * (bounded by ldwk) and rows n up to the next multiple of 64 (bounded by N) are written as zero, nothing
 * else is touched.  W, Wk [N][K-wide rows] of element type `dtype`, ldw, ldwk >= K, W != Wk. */
ard_status ard_compact_weight_cols(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, ard_dtype dtype,
                                   int K, int N, const void* W, int ldw, void* Wk, int ldwk, void* cuda_stream);
/* dW[keep[j]][keep_in[i]] = dWk[j][i] for j < n and i < n_in.  zero_fill != 0: every other entry
 * of dW [N][K] (dropped neurons, dropped inputs) is written as zero; otherwise it is left untouched. */
ard_status ard_expand_weight_grad_cols(ard_ctx* ctx, const ard_pattern* pat, const ard_pattern* in_pat, ard_dtype dtype,
                                       int K, int N, const void* dWk, int lddwk, void* dW, int lddw, int zero_fill,
                                       void* cuda_stream);
/* db[keep[j]] = sum over the B rows of dZ[:, j] (fp32, rows added in a fixed order); dZ of element type
 * `dtype`, compact [B][n] or full width [B][N]; zero_fill_dropped != 0 zeroes db at dropped neurons. */
ard_status ard_bias_grad(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, int B, int N, const void* dZ, int lddz,
                         int dz_is_compact, float* db, int zero_fill_dropped, void* cuda_stream);
/* ard_sample_pattern with the iteration taken from device memory: the pattern is drawn for iteration
 * iteration_base + *iteration_counter (DEVICE uint64, owned by the caller, read when the kernel runs);
 * with advance != 0 the kernel then adds one to the counter.  A training step captured once into a CUDA
 * graph therefore draws a new pattern at every replay: let the last sampling call of the step advance. */
ard_status ard_sample_pattern_counter(ard_ctx* ctx, ard_pattern* pat, int dist_id, uint64_t seed,
                                      uint64_t iteration_base, uint64_t* iteration_counter, int advance,
                                      uint32_t stream_id, void* cuda_stream);

/* One training iteration of a stack of bf16 layers as one native call: draws the pattern of every layer
 * that asks for one (stream id = layer index + 1, iteration = iteration_base + *iteration_counter, the
 * last draw advances the counter), runs the forward chain with ard_layer_fwd and the backward chain with
 * ard_layer_bwd_weight / ard_bias_grad / ard_layer_bwd_data.  A layer with compact_out != 0 writes its
 * activations compact and the layer after it multiplies compact matrices on both sides (its weight is
 * compacted into Wk first, its gradient expanded from dWk into dW); with compact_out == 0 activations and
 * gradients between the two layers are full width.  The last layer must have compact_out == 0; dOut
 * [B][N_last] is the gradient with respect to its output A (for a linear last layer: relu = 0, alpha = 1,
 * pattern set dense with ard_pattern_set(1, 1) and sample = 0).  On return: layers[l].dW (dropped rows
 * and columns zero), layers[l].db if not NULL, dX [B][K_0] if not NULL; A and dZ of every layer hold what
 * the step computed.  `layers` is a HOST array; all pointers inside are DEVICE pointers owned by the caller;
 * dimensions must satisfy the alignment rules of ard_fwd or the slower CUDA-core kernels run.  Enqueues
 * only; allocates nothing after the context's first forking call (which creates two internal streams
 * and their events), so it can be captured into a CUDA graph after one ordinary call.  When every hidden
 * layer has compact_out != 0 the weight compactions, weight gradients, gradient expansions and bias
 * gradients are enqueued on two streams owned by the context, forked from `cuda_stream` after the patterns
 * are drawn and joined back into it before the call returns: to the caller (and to a capture) all work of
 * the call is ordered on `cuda_stream`, but the buffers of `layers` must not be touched by other streams
 * while the iteration runs.
 * A small stack runs as ONE cooperative kernel instead (a memset of 4 bytes and one launch per iteration;
 * same results up to the order of fp32 additions, same patterns, same counter, the same bits from launch to
 * launch): 2 to 4 layers, 1 <= B <= 128, every hidden layer a row pattern with compact_out != 0, N a multiple
 * of 64 and K, ldw multiples of 8, the last layer at most 16 neurons wide, dense and not sampled, all
 * pointers 16-byte aligned, ldx and lddx multiples of 8, a distribution of at most 64 periods, and a device
 * that can hold one block per SM at once.  Anything else, ARD_PATH_CUDA_CORE, or
 * ard_set_option(ctx, ARD_OPT_MLP_PERSISTENT, 0) takes the call-by-call path above.  In the one-kernel form
 * Wk holds the packed weights as before, dWk is not used, and the kernel shares the context's grid-barrier
 * counter and descriptor scratch with the whole-sequence LSTM kernels: one such kernel at a time per context. */
typedef struct ard_mlp_layer {
  int K, N;          /* fan-in and neurons; K of layer l+1 == N of layer l                                  */
  ard_pattern* pat;  /* row pattern over the N neurons (created with K_dim = K, N_dim = N)                  */
  int sample;        /* != 0: draw a new pattern this iteration; 0: keep the one the pattern holds          */
  int relu;          /* != 0: ReLU between the product and the rescale                                      */
  int compact_out;   /* != 0: compact activations, compact matrices in the next layer                       */
  int dW_is_f32;     /* element type of dW and dWk: fp32 (!= 0) or bf16                                      */
  float alpha;       /* rescale of this layer's output, e.g. 1/(1-p)                                        */
  int ldw;           /* leading dimension of W, Wk, dW, dWk (>= K)                                           */
  const void* W;     /* bf16 [N][ldw]                                                                        */
  const float* bias; /* fp32 [N] or NULL                                                                     */
  void* Wk;          /* bf16 [N][ldw] scratch, needed when the previous layer has compact_out               */
  void* A;           /* bf16 [B][N] activations (compact: columns 0..n-1)                                    */
  void* dZ;          /* bf16 [B][N] gradient of the pre-activations, written by the layer above; not needed
                        for the last layer                                                                   */
  void* dWk;         /* [N][ldw] scratch of dW's type, needed when the previous layer has compact_out       */
  void* dW;          /* [N][ldw] weight gradient                                                             */
  float* db;         /* fp32 [N] bias gradient or NULL                                                       */
} ard_mlp_layer;
ard_status ard_mlp_step(ard_ctx* ctx, const ard_mlp_layer* layers, int n_layers, int B, const void* X, int ldx,
                        const void* dOut, int lddout, void* dX, int lddx, int dist_id, uint64_t seed,
                        uint64_t iteration_base, uint64_t* iteration_counter, void* cuda_stream);

/* ---- row-based sensitivity-aware dropout of a convolution layer's input matrix (Sec. 5.1, 5.2.1) ----
 * The layer is the product Y = A W of its input matrix A [M][Kc] (im2col of the input feature map: M
 * output positions, Kc = C*k*k; making A is a library routine outside this interface) with the filters
 * W [N][Kc] (neuron-major as everywhere here).  Sec. 5.1 predicts per region of A whether it is sensitive
 * and gives it a low (sensitive) or a high dropout probability; Sec. 5.2.1 draws, per iteration, which rows
 * of A are dropped, multiplies only the kept rows and fills the results back into the same rows of Y.
 * The paper fixes neither the region shape nor which values are sampled nor any constant; this library's
 * reading: regions of `region_rows` consecutive rows by the whole width; the random k_frac of a region's values
 * is drawn in runs of c = run_len neighbouring values of a row.  run_len = 1 is the text's statement: every
 * sampled value is drawn on its own, one random word per value.  A larger run_len (it must divide Kc;
 * gcd(Kc, 32) makes a run what one memory transaction delivers) is a departure from Sec. 5.1 that the caller
 * asks for by name: neighbouring values of an im2col matrix are correlated, so the clustered sample is a
 * different statistic, but it costs a fraction of the memory traffic.  Of the region's Cn = region_rows*Kc/c
 * runs, n_c = max(1, floor(k_frac*Cn + 1/2)) are drawn with replacement; run d of region g is chosen by word
 * (d mod 4) of the Philox4x32-10 block with key (seed) and counter (iteration low, iteration high, g,
 * stream_id * 65536 + d div 4) as run number floor(word * Cn / 2^32), runs numbered row-major (runs below the
 * last row of A count as not exceeding); s = n_c*c samples; sensitive iff at least max(1, ceil(t_frac * s))
 * sampled values are > threshold, the product taken exactly (t_frac is the binary fraction the double holds,
 * so 0.3 of 10 samples needs 3 and 0.1 of 10 needs 2); a probability p
 * is the integer min(floor(p 2^32), 2^32 - 1); row r is dropped iff word 0 of the block with counter
 * (iteration low, iteration high, r, stream_id * 65536 + 65535) is below its region's integer.
 * stream_id < 65536.  Everything stays on the device; ard_rows_to_host is for tests. */
ard_status ard_rows_create(ard_ctx* ctx, ard_rows** rows, int M, int region_rows);
ard_status ard_rows_destroy(ard_rows* rows);
/* Sec. 5.1: writes the dropout probability of every region (m_prob if sensitive, else n_prob).
 * A [M][Kc] (lda) of element type dtype.  run_len: see above (1 = independent values).  Errors:
 * ARD_ERR_INVALID_ARG (run_len < 1 or not a divisor of Kc, fractions outside their ranges, stream_id >= 65536),
 * ARD_ERR_UNSUPPORTED (more than 262140 runs per region).  Asynchronous. */
ard_status ard_sensitivity_predict(ard_ctx* ctx, ard_rows* rows, ard_dtype dtype, const void* A, int lda, int Kc,
                                   double k_frac, int run_len, double t_frac, float threshold, double m_prob,
                                   double n_prob, uint64_t seed, uint64_t iteration, uint32_t stream_id,
                                   void* cuda_stream);
/* The same probability for every region (tests; p = 0 keeps every row).  Asynchronous. */
ard_status ard_rows_set_probability(ard_ctx* ctx, ard_rows* rows, double p, void* cuda_stream);
/* Sec. 5.2.1: draws the dropped rows and writes the ascending list of kept rows.  Asynchronous. */
ard_status ard_rows_sample(ard_ctx* ctx, ard_rows* rows, uint64_t seed, uint64_t iteration, uint32_t stream_id,
                           void* cuda_stream);
/* The three products over the kept rows (bf16 operands on the tensor cores, fp32 accumulation), with
 * keep = the list drawn by ard_rows_sample, A [M][K] (lda; K = Kc), W [N][K] (ldw), Y / dY [M][N], dA [M][K]:
 *   ard_rows_fwd         Y[r, :]  = alpha * A[r, :] W^T   for kept rows r, zero for dropped rows
 *   ard_rows_bwd_data    dA[r, :] = alpha * dY[r, :] W    for kept rows r, zero for dropped rows
 *   ard_rows_bwd_weight  dW = alpha * sum over kept rows r of dY[r, :]^T A[r, :]   (dW [N][K], dW_dtype)
 * Only the kept rows of A / dY are fetched: the loading warp of the kernel follows the list with 16-byte
 * asynchronous copies (an index list has no stride a TMA box could follow).  Requires 16-byte aligned
 * pointers, leading dimensions that are multiples of 8 elements and K, N multiples of 8
 * (ARD_ERR_ALIGNMENT otherwise: there is no second kernel family for this part).  M must equal the M of
 * `rows`.  Asynchronous. */
ard_status ard_rows_fwd(ard_ctx* ctx, const ard_rows* rows, int M, int K, int N, float alpha, const void* A, int lda,
                        const void* W, int ldw, void* Y, int ldy, void* cuda_stream);
ard_status ard_rows_bwd_data(ard_ctx* ctx, const ard_rows* rows, int M, int K, int N, float alpha, const void* dY,
                             int lddy, const void* W, int ldw, void* dA, int ldda, void* cuda_stream);
ard_status ard_rows_bwd_weight(ard_ctx* ctx, const ard_rows* rows, ard_dtype dW_dtype, int M, int K, int N, float alpha,
                               const void* A, int lda, const void* dY, int lddy, void* dW, int lddw,
                               void* cuda_stream);
/* The same products through the dense, small matrices of Sec. 5.2.1 (step 2), for layers large enough that an
 * extra pass over the kept rows pays: ard_rows_gather copies the kept rows of src [M][width] (ld_src) to the top
 * of dst (ld_dst): row j of dst is row keep[j] of src, and the rows from n_keep up to the next multiple of 64 are
 * zero.  dst must hold ceil(M / 64) * 64 rows (any list fits); bf16 elements, width a multiple of 8, 16-byte
 * aligned pointers, leading dimensions multiples of 8.  The products then read their row operands (Ak = gathered
 * A, dYk = gathered dY, both [ceil(M/64)*64][.]) with TMA like any dense matrix, take the number of rows from the
 * list on the device and write forward / backward-data results back to rows keep[j] of Y / dA (dropped rows
 * zero); the weight gradient's contraction runs over the list's rows and, having few output tiles and a long
 * contraction, is cut along the contraction and shared by all SMs (fp32 partial sums added in a fixed order).
 * A compact copy made for the forward product serves the weight gradient of the same iteration.  Results equal
 * those of ard_rows_fwd / _bwd_data / _bwd_weight.  Same argument rules; asynchronous. */
ard_status ard_rows_gather(ard_ctx* ctx, const ard_rows* rows, int M, int width, const void* src, int ld_src, void* dst,
                           int ld_dst, void* cuda_stream);
ard_status ard_rows_fwd_compact(ard_ctx* ctx, const ard_rows* rows, int M, int K, int N, float alpha, const void* Ak,
                                int ldak, const void* W, int ldw, void* Y, int ldy, void* cuda_stream);
ard_status ard_rows_bwd_data_compact(ard_ctx* ctx, const ard_rows* rows, int M, int K, int N, float alpha,
                                     const void* dYk, int lddyk, const void* W, int ldw, void* dA, int ldda,
                                     void* cuda_stream);
ard_status ard_rows_bwd_weight_compact(ard_ctx* ctx, const ard_rows* rows, ard_dtype dW_dtype, int M, int K, int N,
                                       float alpha, const void* Ak, int ldak, const void* dYk, int lddyk, void* dW,
                                       int lddw, void* cuda_stream);
/* Both gathers and the three products of one iteration in one call: Ak and dYk (ceil(M/64)*64 rows each) are
 * written, then Y, dA and dW as by the three calls above.  The output-gradient half (gather of dY,
 * backward-data) runs on a stream the context owns beside the input half (gather of A, forward) on the caller's
 * stream; the weight gradient waits for both gathered matrices; everything is joined into the caller's stream
 * before the call returns.  The first call on a context creates the stream (make it before any stream
 * capture); after ard_set_option(ctx, ARD_OPT_SIDE_STREAMS, 0) everything stays on the caller's stream.
 * Asynchronous. */
ard_status ard_rows_products(ard_ctx* ctx, const ard_rows* rows, ard_dtype dW_dtype, int M, int K, int N, float alpha,
                             const void* A, int lda, const void* W, int ldw, const void* dY, int lddy, void* Ak,
                             int ldak, void* dYk, int lddyk, void* Y, int ldy, void* dA, int ldda, void* dW, int lddw,
                             void* cuda_stream);
/* Test / debug: synchronises; n_keep, the kept rows (at most idx_capacity) and the per-region integers
 * (ceil(M / region_rows) entries) to HOST buffers; idx and region_probability may be NULL. */
ard_status ard_rows_to_host(const ard_rows* rows, int32_t* n_keep, int32_t* idx, size_t idx_capacity,
                            uint32_t* region_probability, void* cuda_stream);

/* Sec. 5.3, Eq. 12-14: the dropout probability of every training epoch, on the host in fp64 (no context or GPU
 * needed): low at the start, rising, lower again towards the end, with the shape of the skew-normal density
 *   f(y) = (2/sigma) phi((y-mu)/sigma) Phi(lambda (y-mu)/sigma)                                     (Eq. 12)
 * whose parameters follow from a prescribed expectation and variance through
 *   E = mu + mu0 sigma, mu0 = sqrt(2/pi) lambda / sqrt(1+lambda^2);  D = (1 - mu0^2) sigma^2       (Eq. 13, 14).
 * The paper does not say what the axis or the scale of the curve are; this library's reading: the axis is the
 * epoch number e = 0..n_epochs-1, mean_epoch and var_epoch are E and D along it, and
 *   p_out[e] = min(p_max, p_total * n_epochs * f(e) / sum_e' f(e')),
 * so the mean over the epochs is p_total unless an entry was clipped.  A training loop passes p_out[e] (or a
 * pair of values derived from it) as the probabilities of ard_sensitivity_predict / ard_blocks_sample.
 * p_out: HOST array of n_epochs doubles.  Errors: ARD_ERR_INVALID_ARG (NULL, n_epochs < 1, probabilities
 * outside [0,1], var_epoch <= 0, non-finite arguments), ARD_ERR_UNSUPPORTED (the curve underflows to zero on
 * every epoch). */
ard_status ard_dropout_schedule(int n_epochs, double p_total, double mean_epoch, double var_epoch, double lambda,
                                double p_max, double* p_out);

/* ---- block-based sensitivity-aware dropout of a convolution layer's input matrix (Sec. 5.1, 5.2.2) ----
 * The input matrix A [M][Kc] is cut into ts x ts blocks; the Q = Kc/ts blocks that share their rows are a
 * group, there are G = M/ts groups (ts divides M and Kc; the tensor-core products need ts a multiple of 64).
 * A block is the dropout granularity.  Sec. 5.2.2 bounds the number of sensitive blocks per group so that
 * all groups keep nearly the same amount of work.  The paper fixes no constant, and the figure that shows the
 * balancing is not available; this library's reading: the prediction of Sec. 5.1 with one block as the
 * region, its random k_frac of the values drawn in runs of c = run_len neighbouring values of a row (run_len = 1,
 * every value on its own, is the text's statement; a larger run_len, a divisor of ts, is the departure described
 * for ard_sensitivity_predict): of the block's Cn = ts*ts/c runs, n_c = max(1, floor(k_frac*Cn + 1/2))
 * are drawn with replacement, s = n_c*c values are looked at; run d of block g*Q + j is chosen by word
 * (d mod 4) of the Philox4x32-10 block with key (seed) and counter (iteration low, iteration high, g*Q + j,
 * stream_id * 65536 + d div 4) as run number floor(word * Cn / 2^32), runs numbered row-major; a block passes
 * iff at least max(1, ceil(t_frac * s)) sampled values are > threshold, the product taken exactly); of a
 * group's passing blocks the
 * `cap` with the highest counts are sensitive (equal counts: lower j first); block g*Q + j is dropped iff
 * word 0 of the Philox block with counter (iteration low, iteration high, g*Q + j, stream_id * 65536 + 65535)
 * is below min(floor(p 2^32), 2^32 - 1), p = m_prob for a sensitive block, n_prob otherwise.
 * stream_id < 65536.  Everything stays on the device; ard_blocks_to_host is for tests. */
ard_status ard_blocks_create(ard_ctx* ctx, ard_blocks** blocks, int M, int Kc, int ts);
ard_status ard_blocks_destroy(ard_blocks* blocks);
/* Counts and labels of all blocks.  A [M][Kc] (lda) on the device, element type dtype.  Asynchronous. */
ard_status ard_blocks_predict(ard_ctx* ctx, ard_blocks* blocks, ard_dtype dtype, const void* A, int lda, double k_frac,
                              int run_len, double t_frac, float threshold, int cap, uint64_t seed, uint64_t iteration,
                              uint32_t stream_id, void* cuda_stream);
/* The same label for every block (tests; with ard_blocks_sample(m_prob = n_prob = 0) everything is kept). */
ard_status ard_blocks_set_label(ard_ctx* ctx, ard_blocks* blocks, int sensitive, void* cuda_stream);
/* Draws the dropped blocks and writes the kept blocks' index lists (those of a tile pattern over [Kc x M]
 * with tile (r, c) = (block j, group g), all ascending).  Asynchronous. */
ard_status ard_blocks_sample(ard_ctx* ctx, ard_blocks* blocks, double m_prob, double n_prob, uint64_t seed,
                             uint64_t iteration, uint32_t stream_id, void* cuda_stream);
/* The three products over the kept blocks (bf16 operands on the tensor cores, fp32 accumulation; only kept
 * blocks of A are fetched).  W [N][Kc] (ldw) are the filters, neuron-major as everywhere here.  The output
 * matrix and its gradient are held TRANSPOSED, Yt / dYt [N][M] (one row per output channel, the layout of
 * the layer's output feature map), because the products are the tile-pattern products of Sec. 3.2 with the
 * filters as the batch operand and A as the masked matrix:
 *   ard_blocks_fwd         Yt = alpha * W (A .* mask)^T
 *   ard_blocks_bwd_weight  dW = alpha * dYt (A .* mask)                       dW [N][Kc] (lddw), bf16
 *   ard_blocks_bwd_input   dA = alpha * (dYt^T W) .* mask                     dA [M][Kc] (ldda), dA_dtype;
 *                          dropped blocks are written as zero if zero_fill_dropped != 0, else left untouched
 * Requires 16-byte aligned pointers, leading dimensions that are multiples of 8 elements, N >= 1
 * (ARD_ERR_ALIGNMENT / ARD_ERR_UNSUPPORTED otherwise: there is no second kernel family for this part).
 * Asynchronous. */
ard_status ard_blocks_fwd(ard_ctx* ctx, const ard_blocks* blocks, int N, float alpha, const void* A, int lda,
                          const void* W, int ldw, void* Yt, int ldyt, void* cuda_stream);
ard_status ard_blocks_bwd_weight(ard_ctx* ctx, const ard_blocks* blocks, int N, float alpha, const void* A, int lda,
                                 const void* dYt, int lddyt, void* dW, int lddw, void* cuda_stream);
ard_status ard_blocks_bwd_input(ard_ctx* ctx, const ard_blocks* blocks, ard_dtype dA_dtype, int N, float alpha,
                                const void* dYt, int lddyt, const void* W, int ldw, void* dA, int ldda,
                                int zero_fill_dropped, void* cuda_stream);
/* The three products of one iteration behind one call, enqueued side by side on the context's streams as by
 * ard_layer_products (same first-call and capture rules), joined into the caller's stream before the call
 * returns; results as by the three calls above.  Asynchronous. */
ard_status ard_blocks_products(ard_ctx* ctx, const ard_blocks* blocks, ard_dtype dA_dtype, int N, float alpha,
                               const void* A, int lda, const void* W, int ldw, const void* dYt, int lddyt, void* Yt,
                               int ldyt, void* dW, int lddw, void* dA, int ldda, int zero_fill_dropped,
                               void* cuda_stream);
/* Test / debug: synchronises; per block g*Q + j its count, label and kept flag to HOST buffers of G*Q entries
 * (any may be NULL). */
ard_status ard_blocks_to_host(const ard_blocks* blocks, int32_t* counts, uint8_t* sensitive, uint8_t* keep,
                              void* cuda_stream);
/* The tile pattern that holds the lists (for ard_pattern_to_host / ard_pattern_tile_lists_to_host); owned by
 * `blocks`. */
const ard_pattern* ard_blocks_pattern(const ard_blocks* blocks);

/* ---- LSTM cell on the kept hidden units (Sec. 7: an LSTM step is again a matrix
 * product; one row pattern over the H hidden units serves every time step) -------------
 * Layouts are compact over kept units: with n = n_keep, Z [B][4*ldz_gate] holds the gate
 * pre-activations in four blocks i | f | g | o of width ldz_gate (>= n; block g starts at column
 * g*ldz_gate), bias [4][H] is indexed by the ORIGINAL unit (may be NULL), c_prev / c [B][ldc] and
 * gates_saved [B][4*ldc] are fp32, h [B][ldh] has element type h_dtype.
 *   i,f,o = sigmoid, g = tanh;  c = f*c_prev + i*g;  h = alpha * o * tanh(c)
 * h_scatter != 0 writes h full width [B][H] with zeros at dropped units (the layout the next
 * step's recurrent GEMM consumes), else compact [B][n]. */
ard_status ard_lstm_gates(ard_ctx* ctx, const ard_pattern* pat, ard_dtype h_dtype, int B, int H, float alpha,
                          const float* Z, int ldz_gate, const float* bias, const float* c_prev, int ldc, float* c,
                          void* h, int ldh, int h_scatter, float* gates_saved, void* cuda_stream);

/* Gate pre-activations of the kept hidden units for one time step, all four gate blocks in one call:
 *   Z[:, g*ldz_gate + j] = sum_k XH[:, k] * W[g*H + keep[j]][k],   g = 0..3 (i|f|g|o), j < n_keep.
 * XH [B][KH] bf16 (ldxh) is [x_t, h_{t-1}] side by side (KH = I + H; h full width, zeros at dropped
 * units), W [4H][KH] bf16 neuron-major (ldw), Z fp32 [B][4*ldz_gate] with ldz_gate >= H.  `pat` is a row
 * pattern created with K_dim = KH and N_dim = H (Sec. 3.1 applied to the hidden units, Sec. 7). */
ard_status ard_lstm_gate_gemm(ard_ctx* ctx, const ard_pattern* pat, int B, int KH, int H, const void* XH, int ldxh,
                              const void* W, int ldw, float* Z, int ldz_gate, void* cuda_stream);
/* Its adjoint with respect to XH:  dXH[:, k] (+)= sum_g sum_j dZ[:, g*ldz_gate + j] * W[g*H + keep[j]][k].
 * dZ bf16 compact [B][4*ldz_gate], dXH fp32 [B][KH] (lddxh); accumulate != 0 adds to dXH. */
ard_status ard_lstm_gate_gemm_bwd(ard_ctx* ctx, const ard_pattern* pat, int B, int KH, int H, const void* dZ,
                                  int ldz_gate, const void* W, int ldw, float* dXH, int lddxh, int accumulate,
                                  void* cuda_stream);

/* Whole-sequence forward: for t = 0..T-1, the gate product on XH[t] followed by the cell update, which writes
 * h_t into the h half of XH[t+1].  When the layer fits (B <= 128, the weight rows of 8 hidden units times
 * (I+H) columns fit in shared memory, H/8 <= number of SMs, operands aligned for the tensor-core path) this
 * is ONE cooperative kernel that keeps the weight in shared memory and the cell state in registers for the
 * whole sequence and synchronises the SMs once per step (every wait bounded, see ARD_ERR_TIMEOUT); Z is
 * then not used.  Otherwise, or after ard_set_lstm_persistent(ctx, 0), it is a loop in native code that
 * enqueues ard_lstm_gate_gemm and ard_lstm_gates per step.  Both give the same C, G and XH up to
 * summation order.  Under a pattern that drops units the kernel contracts over the kept units of h_{t-1} only
 * (ARD_OPT_LSTM_COMPACT_H): it keeps a compact copy of h in scratch of the context, next to the grid-barrier
 * counter the whole-sequence kernels share, so one whole-sequence call at a time per context.
 *   XH [T+1][B][I+H] bf16: the caller fills the x halves of XH[0..T-1] and the h half of XH[0] (h_0, zeros at
 *   dropped units); C [T+1][B][H] fp32 compact cell states, C[0] = c_0; G [T][B][4H] fp32 saved gates;
 *   Z [B][4H] fp32 scratch; W [4H][I+H] bf16 (ldw); bias [4][H] or NULL. */
ard_status ard_set_lstm_persistent(ard_ctx* ctx, int enable); /* default: enabled */
ard_status ard_lstm_forward(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H, float alpha, void* XH,
                            const void* W, int ldw, const float* bias, float* C, float* G, float* Z,
                            void* cuda_stream);
/* Whole-sequence BPTT of ard_lstm_forward.  D [T][B][I+H] fp32 must hold, on entry, zeros in the x halves and
 * the upstream gradient of h_{t-1} in the h half of D[t] (t >= 1); on return its x halves hold dx_t and the h
 * half of D[0] the gradient of h_0.  dH_last [B][H] fp32 is the gradient of h_{T-1}; dc [B][H] fp32 must be
 * zero on entry (or hold the gradient of c_T) and returns the gradient of c_0; DZ [T][B][4H] bf16 scratch;
 * dW [4H][I+H] fp32 receives the weight gradient (dropped units' rows zero).
 * When the layer fits (B <= 128, H <= 1024, 8*ceil(H/64) <= number of SMs, operands aligned) and
 * ard_set_lstm_persistent is on, the recurrence dh_{t-1} = upstream + dz_t W_h with the cell adjoint is ONE
 * cooperative kernel (weight slices resident in shared memory, dc in registers, two bounded grid-wide
 * synchronisations per step; one, and no partial sums, when the drawn pattern keeps at most 256 units, see
 * ARD_OPT_LSTM_COMPACT_H) and the x halves come from one product over all T*B rows; otherwise a loop
 * in native code enqueues ard_lstm_gates_bwd and ard_lstm_gate_gemm_bwd per step.  In both cases the h
 * halves of D[1..T-1] are overwritten (kept units: the total gradient of h_{t-1}; dropped units:
 * unspecified), and the h half of D[0] is meaningful at kept units only. */
ard_status ard_lstm_backward(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H, float alpha,
                             const void* XH, const void* W, int ldw, const float* C, const float* G,
                             const float* dH_last, float* D, float* dc, void* DZ, float* dW, void* cuda_stream);

/* ---- stacked LSTM with dropout on the layer OUTPUTS only (second reading of the LSTM experiment of Sec. 7) ----
 * The paper prints no LSTM equations; its LSTM networks are stacks of two and three layers.  In this reading every
 * unit of a layer is computed at every step, the recurrent path is left alone, and a row pattern (Sec. 3.1, Eq. 1),
 * one per layer and iteration, masks what the layer hands to its consumer:
 *     y_t = alpha * m .* h_t.
 * A dropped unit multiplies its fan-in row of the consumer's weight by zero (Sec. 3.1: the matching rows of the
 * next layer's weight matrix), so the consumer contracts over kept units only: the layer's output leaves as the
 * compact matrix Yc [T*B][n_keep] (ard_compact_cols of the h halves of XH), the input half of the next layer's gate
 * product is ard_layer_fwd over Yc with that pattern as in_pat and the weight packed by ard_compact_weight_cols,
 * and the recurrence runs from those pre-activations (ard_lstm_forward_from_gates).  Backward: the gradient of Yc
 * is expanded to full width with the rescale (ard_expand_cols) into D / dH_last, ard_lstm_backward_recurrent gives
 * the gate gradients DZ and the weight gradient of the recurrent half, and the input half is
 * ard_layer_bwd_data / ard_layer_bwd_weight over the same compact operands.  The layers themselves use a pattern
 * that stays dense (never sampled).  paper_2203_05705_b200/lstm.py (LstmStack) holds the buffers and the order of
 * the calls.
 *
 * ard_lstm_forward_from_gates: ard_lstm_forward whose input half is already done: on entry G [T][B][4H] holds
 *   x-part pre-activations of every step (fp32, e.g. written by ard_layer_fwd with ARD_FLAG_OUT_F32); the x halves
 *   of XH are not read.  Only the one-kernel recurrence exists for this form: ARD_ERR_UNSUPPORTED when the layer
 *   does not fit it (see ard_lstm_forward) or I < 1.
 * ard_lstm_backward_recurrent: ard_lstm_backward without the input half: computes DZ and dW[:, I : I+H] (all 4H
 *   rows; columns 0 .. I-1 of dW and the x halves of D are left untouched).  ARD_ERR_UNSUPPORTED when the layer
 *   does not fit the one-kernel recurrence. */
ard_status ard_lstm_forward_from_gates(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H, float alpha,
                                       void* XH, const void* W, int ldw, const float* bias, float* C, float* G,
                                       void* cuda_stream);
ard_status ard_lstm_backward_recurrent(ard_ctx* ctx, const ard_pattern* pat, int T, int B, int I, int H, float alpha,
                                       const void* XH, const void* W, int ldw, const float* C, const float* G,
                                       const float* dH_last, float* D, float* dc, void* DZ, float* dW,
                                       void* cuda_stream);
/* Eq. 1 applied to the columns of a matrix.  ard_compact_cols: dst[r][j] = src[r][keep[j]], j < n_keep (the kept
 * columns side by side; element type dtype).  ard_expand_cols, its adjoint with a rescale:
 * dst[r][keep[j]] = alpha * src[r][j], every other column of dst [rows][N] zero (src of type src_dtype, dst fp32).
 * pat: a row pattern over N units.  Errors: ARD_ERR_INVALID_ARG, ARD_ERR_SHAPE (N differs from the pattern's, leading
 * dimensions too small).  Asynchronous. */
ard_status ard_compact_cols(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dtype, int rows, int N, const void* src,
                            int ld_src, void* dst, int ld_dst, void* cuda_stream);
ard_status ard_expand_cols(ard_ctx* ctx, const ard_pattern* pat, ard_dtype src_dtype, int rows, int N, float alpha,
                           const void* src, int ld_src, float* dst, int ld_dst, void* cuda_stream);

/* Adjoint of ard_lstm_gates.  dh [B][lddh] (fp32; compact, or full width if dh_scatter != 0, in
 * which case only kept columns are read), dc_inout [B][ldc]: in = gradient arriving at c from the
 * next step, out = gradient w.r.t. c_prev.  dZ [B][4*ldz_gate] compact like Z, element type
 * dz_dtype. */
ard_status ard_lstm_gates_bwd(ard_ctx* ctx, const ard_pattern* pat, ard_dtype dz_dtype, int B, int H, float alpha,
                              const float* gates_saved, const float* c_prev, const float* c, int ldc,
                              const float* dh, int lddh, int dh_scatter, float* dc_inout, void* dZ, int ldz_gate,
                              void* cuda_stream);

/* ---- status ---------------------------------------------------------------------------------- */

/* Synchronises `cuda_stream`, returns the sticky device status word (ARD_OK if no kernel reported
 * a problem) and clears it. */
ard_status ard_last_device_status(ard_ctx* ctx, void* cuda_stream);
const char* ard_status_string(ard_status s);
/* Number of kernels this library has launched on behalf of `ctx` since creation. */
uint64_t ard_launch_count(const ard_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* ARD_H_ */
