// Dropout probability per training epoch (Sec. 5.3, Eq. 12-14).  Host code, fp64; nothing here touches
// the GPU.  A training loop calls it once and passes entry e as the probabilities of the sensitivity-aware
// dropout calls of epoch e.
//
// The paper gives the curve's shape (a skew-normal density over the epochs: low at first, rising, lower
// again at the end) and says that its two parameters follow from a prescribed expectation and variance.
// Open choices made here: the axis is the epoch number; the expectation and variance are those of the curve
// along that axis; the curve is scaled so that its mean over the epochs is the overall probability, then
// clipped to [0, p_max].
#include <math.h>

#include <vector>

#include "ard.h"

extern "C" ard_status ard_dropout_schedule(int n_epochs, double p_total, double mean_epoch, double var_epoch,
                                           double lambda, double p_max, double* p_out) {
  if (!p_out || n_epochs < 1) return ARD_ERR_INVALID_ARG;
  if (!(p_total >= 0.0 && p_total <= 1.0) || !(p_max >= 0.0 && p_max <= 1.0)) return ARD_ERR_INVALID_ARG;
  if (!(var_epoch > 0.0) || !isfinite(mean_epoch) || !isfinite(lambda) || !isfinite(var_epoch)) return ARD_ERR_INVALID_ARG;
  const double pi = 3.14159265358979323846;
  // Eq. 13-14 solved for the density's parameters
  const double m0 = sqrt(2.0 / pi) * lambda / sqrt(1.0 + lambda * lambda);
  const double s0sq = 1.0 - (2.0 / pi) * lambda * lambda / (1.0 + lambda * lambda);
  const double sigma = sqrt(var_epoch / s0sq);
  const double mu = mean_epoch - m0 * sigma;
  std::vector<double> f(n_epochs);
  double total = 0.0;
  for (int e = 0; e < n_epochs; ++e) {
    // Eq. 12
    const double z = ((double)e - mu) / sigma;
    const double phi = exp(-0.5 * z * z) / sqrt(2.0 * pi);
    const double Phi = 0.5 * erfc(-lambda * z / sqrt(2.0));
    f[e] = 2.0 / sigma * phi * Phi;
    total += f[e];
  }
  if (!(total > 0.0)) return ARD_ERR_UNSUPPORTED;  // the curve lies entirely outside the epochs
  for (int e = 0; e < n_epochs; ++e) {
    const double v = p_total * (double)n_epochs * f[e] / total;
    p_out[e] = v < p_max ? v : p_max;
  }
  return ARD_OK;
}
