// qb_sensitivity_bits: per-layer sensitivity from Hessian top-eigenvalue samples and the bit widths that
// follow from its ranking (Section 3.2, Eq. 2 and the paragraph after it).  Host code only: the inputs
// are a few hundred doubles that the caller's Hessian analysis produced, and the result (one bit width
// per encoder layer) is what qb_layer_linears takes per descriptor.
#include <algorithm>
#include <cmath>
#include <numeric>
#include <vector>

#include "common.cuh"

extern "C" qb_status qb_sensitivity_bits(const double* lambda, int32_t layers, int32_t samples,
                                         const int32_t* budget_bits, int32_t reverse, double* omega_out,
                                         int32_t* order_out, int32_t* bits_out) {
  if (!lambda || !budget_bits || !bits_out || layers < 1 || samples < 1) {
    qb::set_last_error("qb_sensitivity_bits: null pointer or layers/samples < 1 (layers=%d samples=%d)", layers,
                       samples);
    return QB_ERR_INVALID;
  }
  for (int32_t r = 0; r < layers; ++r)
    if (!qb::valid_bits(budget_bits[r])) {
      qb::set_last_error("qb_sensitivity_bits: budget_bits[%d] = %d is not one of 2, 3, 4, 8", r, budget_bits[r]);
      return QB_ERR_INVALID;
    }
  std::vector<double> omega(layers);
  for (int32_t i = 0; i < layers; ++i) {
    const double* row = lambda + (size_t)i * samples;
    double total = 0.0;
    for (int32_t s = 0; s < samples; ++s) {
      if (!std::isfinite(row[s])) {
        qb::set_last_error("qb_sensitivity_bits: lambda[%d][%d] is not finite", i, s);
        return QB_ERR_NONFINITE;
      }
      total += row[s];
    }
    const double mu = total / (double)samples;
    double ss = 0.0;
    for (int32_t s = 0; s < samples; ++s) ss += (row[s] - mu) * (row[s] - mu);
    // standard deviation of the empirical distribution of the samples (divisor: samples)
    omega[i] = std::fabs(mu) + std::sqrt(ss / (double)samples);
  }
  std::vector<int32_t> order(layers);
  std::iota(order.begin(), order.end(), 0);
  // descending in Omega; layers with equal Omega stay in index order
  std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return omega[a] > omega[b]; });
  for (int32_t r = 0; r < layers; ++r) bits_out[order[r]] = budget_bits[reverse ? layers - 1 - r : r];
  if (omega_out) std::copy(omega.begin(), omega.end(), omega_out);
  if (order_out) std::copy(order.begin(), order.end(), order_out);
  return QB_OK;
}
