"""CPU oracle for Approximate Random Dropout (ARD): TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 statement of what the hot path computes: the dropout
pattern (Sec. 3.1 Eq. 1, Sec. 3.2, Sec. 3.4) expanded to a dense 0/1 mask and
applied to full-size matrix products.  It shares no code with the CUDA path and
must never be imported by the product package; only the tests, the smoke check
and the CPU-baseline leg of the benchmark may call it.

Pins (each lives in tests/test_oracle_*.py):
  pattern.philox4x32_10    known-answer vectors of the published generator
  pattern.quantise_K       exact integer sum 2^32; zero-probability entries never drawn
  pattern.draw             Monte-Carlo per-neuron drop rate vs Eq. 2-3; chi^2 of dp; b uniform
  pattern.row_keep         worked example of Sec. 3.1 (dp=3, b=1); kept fraction 1/dp
  pattern.tile_keep        worked example of Sec. 3.2 (dp=4, b=1); kept fraction 1/dp
  gemm.*                   scalar triple loops on tiny shapes; dp=1 == numpy matmul; adjoint identity
  lstm.*                   dp=1 == torch.nn.LSTM (fp64, forward and autograd gradients);
                           kept sub-network == torch.nn.LSTM of hidden size n_k; finite differences
  lstm_stack.*             torch.nn.LSTM modules (fp64) with the mask applied between them, forward and autograd
                           gradients; central differences; dropped units' fan-in rows of the next layer get no gradient
  mlp_chain.*              finite differences of the scalar <dZ3, Z3>
  mlp.*                    torch autograd (fp64) on the same network written with library ops; central
                           differences; == mlp_chain without bias; compact-matrix form == masked full width
  cnn.*                    decisions that do not depend on the sample; binomial law of the region decision; single
                           values drawn independently by default (variance and joint law of two positions);
                           drop rates of the row sampler; worked row example of Sec. 5.2.1; masked product ==
                           product of the dense small matrix; brute force; adjoint identities
  cnn_blocks.*             block decisions that do not depend on the sample; one block per group == the row
                           variant's region; binomial law of a block's count; the bound on sensitive blocks per
                           group; drop rates of the two labels; loops over kept blocks; all kept == plain product;
                           adjoint identities
  schedule.*               Eq. 12 == the library's skew-normal density, integrates to one; Eq. 13-14 by numerical
                           integration; shape 0 == normal; prescribed mean of the scaled curve; one maximum
  search.*                 gradient vs central differences; stationary points lie in the Gibbs family
                           ln k_i = beta (i-1)/i + c with beta = -2 (k.p_u - p)/lambda; small-lambda limit ==
                           the maximum-entropy distribution at rate p; Eq. 2-3 in exact rationals

Parity unpinned (the paper fixes no value to compare with): the constants of the
distribution search (the body of Algorithm 1 is not printed: loss form, lambda, step size, start and
stopping rule are a reading, see search.py) and therefore the authors' own K, the tile
linearisation order beyond the first tile of the worked example, every constant of the
sensitivity prediction (region shape, which values are sampled, k, t, threshold, m, n: see cnn.py; the balancing rule of the block variant: see cnn_blocks.py; axis and scale of the dropout-probability curve over the
epochs: see schedule.py), the LSTM
reading (which units are dropped, gate order) and the rescale convention.
"""
