// One training iteration of a stack of fully connected layers under row patterns, as a sequence of the
// library's own calls (Sec. 3.2, last paragraph: product -> activation -> dropout per layer; Sec. 3.1: a
// layer fed by a dropped layer multiplies compact matrices on both sides; Sec. 3.4: a new pattern per
// iteration).  Host code only: the order of the calls is all that lives here, every step runs in the
// kernels behind them.  Nothing here synchronises or allocates, so the whole iteration can be captured
// into a CUDA graph (after one ordinary call, in which the context creates the streams it forks onto).
#include "ard_internal.h"


extern "C" ard_status ard_mlp_step(ard_ctx* ctx, const ard_mlp_layer* layers, int n_layers, int B, const void* X,
                                   int ldx, const void* dOut, int lddout, void* dX, int lddx, int dist_id,
                                   uint64_t seed, uint64_t iteration_base, uint64_t* iteration_counter,
                                   void* cuda_stream) {
  if (!ctx || !layers || n_layers < 1 || B < 0 || !X || !dOut) return ARD_ERR_INVALID_ARG;
  const ard_dtype dt = ARD_BF16;
  int last_sampled = -1;
  for (int l = 0; l < n_layers; ++l) {
    const ard_mlp_layer& y = layers[l];
    if (!y.pat || !y.W || !y.A || !y.dW || y.K < 1 || y.N < 1) return ARD_ERR_INVALID_ARG;
    if (l > 0 && layers[l - 1].N != y.K) return ARD_ERR_SHAPE;
    if (l > 0 && layers[l - 1].compact_out && (!y.Wk || !y.dWk)) return ARD_ERR_INVALID_ARG;
    if (l + 1 < n_layers && !y.dZ) return ARD_ERR_INVALID_ARG;
    if (y.sample) last_sampled = l;
  }
  if (layers[n_layers - 1].compact_out) return ARD_ERR_INVALID_ARG;  // dOut is full width
  if (last_sampled >= 0 && !iteration_counter) return ARD_ERR_INVALID_ARG;
  ard_status st;
  cudaStream_t main_s = (cudaStream_t)cuda_stream;
  // A small stack (batch of at most 128 rows, a narrow output layer) runs as one cooperative kernel.
  if (ctx->mlp_persistent && ctx->path != ARD_PATH_CUDA_CORE) {
    st = launch_mlp_persistent(ctx, layers, n_layers, B, X, ldx, dOut, lddout, dX, lddx, dist_id, seed, iteration_base,
                               iteration_counter, main_s);
    if (st != ARD_ERR_UNSUPPORTED) return st;
  }
  // Three streams: everything the activations and their gradients wait for stays on the caller's stream;
  // weight compaction and the weight gradients, which nothing downstream of them in the iteration reads,
  // run beside it on the context's second stream, the expansion of those gradients and the bias gradients
  // on a third (forked after the patterns are drawn, joined at the end: the caller sees one ordered stream).  Needs compact matrices between all hidden layers: the
  // full-width form gathers through the context workspace, which the two streams would share.
  bool two = ctx->mlp_two_streams && n_layers >= 2 && n_layers <= 32;
  for (int l = 0; l + 1 < n_layers && two; ++l) two = layers[l].compact_out != 0;
  if (two && !ard_side_streams(ctx, main_s)) two = false;
  SharedTailOff tail_guard(ctx, two);
  cudaStream_t side_s = two ? ctx->side_stream : main_s;
  cudaStream_t aux_s = two ? ctx->aux_stream : main_s;
  void* side = (void*)side_s;
  void* aux = (void*)aux_s;
  // event slots: 0 fork, 1 forward done, 2 join, 3 + l weight of layer l compacted, 35 + l dZ of layer l ready,
  // 67 join of the third stream, 68 + l compact weight gradient of layer l ready
  auto after = [&](cudaStream_t waiter, cudaStream_t producer, int slot) -> bool {
    if (!two) return true;
    return cudaEventRecord(ctx->ev[slot], producer) == cudaSuccess &&
           cudaStreamWaitEvent(waiter, ctx->ev[slot], 0) == cudaSuccess;
  };
  // ---- patterns of this iteration (stream id = layer index + 1) ----
  // With several streams only the first layer's pattern is drawn on the caller's stream (its product is the
  // first thing that stream runs); the others are drawn on the second stream, ahead of the compactions that
  // need them.  The draws stay ordered (they share the iteration counter, the last one advances it).
  for (int l = 0; l < n_layers; ++l) {
    if (!layers[l].sample || (two && l > 0)) continue;
    st = ard_sample_pattern_counter(ctx, layers[l].pat, dist_id, seed, iteration_base, iteration_counter,
                                    l == last_sampled, (uint32_t)(l + 1), cuda_stream);
    if (st != ARD_OK) return st;
  }
  // ---- forward ----
  if (!after(side_s, main_s, 0)) return ARD_ERR_CUDA;  // fork: the second stream starts behind the first sampler
  if (two) {
    for (int l = 1; l < n_layers; ++l) {
      if (!layers[l].sample) continue;
      st = ard_sample_pattern_counter(ctx, layers[l].pat, dist_id, seed, iteration_base, iteration_counter,
                                      l == last_sampled, (uint32_t)(l + 1), side);
      if (st != ARD_OK) return st;
    }
    for (int l = 1; l < n_layers; ++l) {  // all weight compactions, beside the first layer's product
      const ard_mlp_layer& y = layers[l];
      st = ard_compact_weight_cols(ctx, y.pat, layers[l - 1].pat, dt, y.K, y.N, y.W, y.ldw, y.Wk, y.ldw, side);
      if (st != ARD_OK) return st;
      if (cudaEventRecord(ctx->ev[3 + l], side_s) != cudaSuccess) return ARD_ERR_CUDA;
    }
  }
  for (int l = 0; l < n_layers; ++l) {
    const ard_mlp_layer& y = layers[l];
    const ard_pattern* in = (l > 0 && layers[l - 1].compact_out) ? layers[l - 1].pat : nullptr;
    const void* in_act = l == 0 ? X : layers[l - 1].A;
    const int ld_in = l == 0 ? ldx : layers[l - 1].N;
    if (in && two) {
      if (cudaStreamWaitEvent(main_s, ctx->ev[3 + l], 0) != cudaSuccess) return ARD_ERR_CUDA;
    } else if (in) {
      st = ard_compact_weight_cols(ctx, y.pat, in, dt, y.K, y.N, y.W, y.ldw, y.Wk, y.ldw, cuda_stream);
      if (st != ARD_OK) return st;
    }
    const int mode = (y.compact_out ? ARD_OUT_COMPACT : ARD_OUT_SCATTER_ZEROFILL) | (y.relu ? ARD_FLAG_RELU : 0);
    st = ard_layer_fwd(ctx, y.pat, in, dt, B, y.K, y.N, y.alpha, in_act, ld_in, in ? y.Wk : y.W, y.ldw, y.bias, y.A, y.N,
                       mode, cuda_stream);
    if (st != ARD_OK) return st;
  }
  // ---- backward ----
  if (!after(side_s, main_s, 1)) return ARD_ERR_CUDA;  // the other streams read the activations from here on
  if (two && cudaStreamWaitEvent(aux_s, ctx->ev[1], 0) != cudaSuccess) return ARD_ERR_CUDA;
  for (int l = n_layers - 1; l >= 0; --l) {
    const ard_mlp_layer& y = layers[l];
    const ard_pattern* in = (l > 0 && layers[l - 1].compact_out) ? layers[l - 1].pat : nullptr;
    const void* in_act = l == 0 ? X : layers[l - 1].A;
    const int ld_in = l == 0 ? ldx : layers[l - 1].N;
    const void* dZ = l == n_layers - 1 ? dOut : y.dZ;
    const int lddz = l == n_layers - 1 ? lddout : y.N;
    const int dz_compact = (l == n_layers - 1) ? 0 : (y.compact_out ? 1 : 0);
    const ard_dtype dwt = y.dW_is_f32 ? ARD_F32 : ARD_BF16;
    // the expansion writes every entry of dW, so the compact gradient needs no zeros of its own
    // weight side (second stream when there are two): needs dZ of this layer, which the layer above wrote.
    // (The last layer's dOut is full width: if its pattern is not dense, both its backward products compact
    // it into the context workspace, each on its own stream; they write the same values from the same
    // source, so the overlap is harmless.)
    if (two && l < n_layers - 1 && cudaStreamWaitEvent(side_s, ctx->ev[35 + l], 0) != cudaSuccess) return ARD_ERR_CUDA;
    st = ard_layer_bwd_weight(ctx, y.pat, in, dt, dwt, B, y.K, y.N, 1.0f, in_act, ld_in, dZ, lddz, dz_compact,
                              in ? y.dWk : y.dW, y.ldw, in ? 0 : 1, side);
    if (st != ARD_OK) return st;
    // third stream: expansion of this layer's gradient and its bias gradient (both off everybody's path)
    if (in) {
      if (!after(aux_s, side_s, 68 + l)) return ARD_ERR_CUDA;
      st = ard_expand_weight_grad_cols(ctx, y.pat, in, dwt, y.K, y.N, y.dWk, y.ldw, y.dW, y.ldw, 1, aux);
      if (st != ARD_OK) return st;
    }
    if (y.db) {
      if (two && l < n_layers - 1 && cudaStreamWaitEvent(aux_s, ctx->ev[35 + l], 0) != cudaSuccess) return ARD_ERR_CUDA;
      st = ard_bias_grad(ctx, y.pat, dt, B, y.N, dZ, lddz, dz_compact, y.db, 1, aux);
      if (st != ARD_OK) return st;
    }
    if (l > 0) {
      const ard_mlp_layer& prev = layers[l - 1];
      st = ard_layer_bwd_data(ctx, y.pat, in, dt, B, y.K, y.N, prev.alpha, dZ, lddz, dz_compact, in ? y.Wk : y.W, y.ldw,
                              prev.relu ? prev.A : nullptr, prev.N, prev.dZ, prev.N, cuda_stream);
      if (st != ARD_OK) return st;
      if (two && cudaEventRecord(ctx->ev[35 + l - 1], main_s) != cudaSuccess) return ARD_ERR_CUDA;
    } else if (dX) {
      st = ard_bwd_data(ctx, y.pat, dt, B, y.K, y.N, 1.0f, dZ, lddz, dz_compact, y.W, y.ldw, dX, lddx, cuda_stream);
      if (st != ARD_OK) return st;
    }
  }
  if (!after(main_s, side_s, 2)) return ARD_ERR_CUDA;  // join
  if (!after(main_s, aux_s, 67)) return ARD_ERR_CUDA;
  return ARD_OK;
}
