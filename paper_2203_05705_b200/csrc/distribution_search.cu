// Search for the distribution K over the pattern periods (Sec. 3.3, Algorithm 1).  Host code, fp64;
// nothing here touches the GPU.
//
// The listing's body is not printed in the paper; the text fixes the ingredients: v of length N,
// d = softmax(v), p_u = {(i-1)/i}, objective = difference between d . p_u and the target rate p, plus
// the negative entropy of d, gradient updates of v, stop when the loss is stuck.  Open choices made
// here: squared difference, weight lambda on the negative entropy, v starts at zero (uniform d), full
// gradient steps of fixed size, stop when the loss changes by less than `tol`.
#include <math.h>

#include <vector>

#include "ard.h"

extern "C" ard_status ard_search_distribution(double p, int ndp, double lambda, double step, int max_iter,
                                              double tol, double* K_out, int* iterations_out) {
  if (!K_out || ndp < 1 || ndp > ARD_MAX_NDP || max_iter < 1) return ARD_ERR_INVALID_ARG;
  if (!(p >= 0.0 && p < 1.0) || !(lambda > 0.0) || !(step > 0.0) || !(tol >= 0.0)) return ARD_ERR_INVALID_ARG;
  // the largest global rate any distribution over 1..ndp can reach is (ndp-1)/ndp
  if (p > (double)(ndp - 1) / (double)ndp) return ARD_ERR_DISTRIBUTION;
  const int n = ndp;
  std::vector<double> v(n, 0.0), d(n), pu(n), gd(n);
  for (int i = 0; i < n; ++i) pu[i] = (double)i / (double)(i + 1);
  double prev = 0.0;
  int it = 0;
  for (it = 1; it <= max_iter; ++it) {
    // d = softmax(v)
    double vmax = v[0];
    for (int i = 1; i < n; ++i) vmax = v[i] > vmax ? v[i] : vmax;
    double sum = 0.0;
    for (int i = 0; i < n; ++i) { d[i] = exp(v[i] - vmax); sum += d[i]; }
    for (int i = 0; i < n; ++i) d[i] /= sum;
    // loss = (d . p_u - p)^2 + lambda * sum d ln d
    double rate = 0.0, negent = 0.0;
    for (int i = 0; i < n; ++i) { rate += d[i] * pu[i]; negent += d[i] * log(d[i]); }
    const double e = rate - p;
    const double loss = e * e + lambda * negent;
    if (it > 1 && fabs(prev - loss) < tol) break;
    prev = loss;
    // gradient with respect to d, then through the softmax
    double dot = 0.0;
    for (int i = 0; i < n; ++i) { gd[i] = 2.0 * e * pu[i] + lambda * (log(d[i]) + 1.0); dot += d[i] * gd[i]; }
    for (int i = 0; i < n; ++i) v[i] -= step * d[i] * (gd[i] - dot);
  }
  if (it > max_iter) it = max_iter;
  for (int i = 0; i < n; ++i) {
    if (!isfinite(d[i])) return ARD_ERR_DISTRIBUTION;  // the step was too large for this problem
    K_out[i] = d[i];
  }
  if (iterations_out) *iterations_out = it;
  return ARD_OK;
}
