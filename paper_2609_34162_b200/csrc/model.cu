// libslidedp: the step-time model of the host-resident step (host arithmetic only).
// See include/slidedp.h for the contract of every entry point.
#include "internal.h"

extern "C" {

int slidedp_model_stream_step(int64_t n_total, int R, int64_t chunk_elems, int nbuf,
                              const slidedp_rates* rates, double* lower_bound_ms,
                              double* predicted_ms) {
  if (n_total < 0 || R < 1 || R > SLIDEDP_MAX_RANKS || chunk_elems <= 0 || nbuf < 1 || !rates ||
      !lower_bound_ms || !predicted_ms)
    return SLIDEDP_ERR_INVALID_ARG;
  if (!(rates->h2d_gbs > 0.0) || !(rates->d2h_gbs > 0.0) || !(rates->update_gparams_s > 0.0) ||
      !(rates->norm_gbs >= 0.0) || !(rates->per_copy_us >= 0.0))
    return SLIDEDP_ERR_INVALID_ARG;
  const int64_t nchunks = n_total == 0 ? 0 : (n_total + chunk_elems - 1) / chunk_elems;
  const double norm_ms =
      rates->norm_gbs > 0.0 ? 2.0 * R * (double)n_total / (rates->norm_gbs * 1e6) : 0.0;
  const double copy_fixed_ms = 3.0 * rates->per_copy_us * 1e-3;
  // resource demand: W_j / beta_j per lane
  const double in_ms = 12.0 * (double)n_total / (rates->h2d_gbs * 1e6) + nchunks * copy_fixed_ms;
  const double out_ms = 12.0 * (double)n_total / (rates->d2h_gbs * 1e6) + nchunks * copy_fixed_ms;
  const double compute_ms = norm_ms + (double)n_total / (rates->update_gparams_s * 1e6);
  double bound = in_ms > out_ms ? in_ms : out_ms;
  if (compute_ms > bound) bound = compute_ms;
  *lower_bound_ms = bound;
  // execution dependencies: completion times, chunk by chunk; the last nbuf copy-outs are kept
  std::vector<double> out_done((size_t)nbuf, 0.0);
  double f_in = 0.0, f_k = norm_ms, f_out = 0.0;
  for (int64_t c = 0; c < nchunks; ++c) {
    const int64_t len = n_total - c * chunk_elems < chunk_elems ? n_total - c * chunk_elems
                                                                 : chunk_elems;
    const double d_in = 12.0 * (double)len / (rates->h2d_gbs * 1e6) + copy_fixed_ms;
    const double d_k = (double)len / (rates->update_gparams_s * 1e6);
    const double d_out = 12.0 * (double)len / (rates->d2h_gbs * 1e6) + copy_fixed_ms;
    const double slot_free = c >= nbuf ? out_done[(size_t)(c % nbuf)] : 0.0;
    f_in = d_in + (f_in > slot_free ? f_in : slot_free);
    f_k = d_k + (f_k > f_in ? f_k : f_in);
    f_out = d_out + (f_out > f_k ? f_out : f_k);
    out_done[(size_t)(c % nbuf)] = f_out;
  }
  *predicted_ms = f_out > f_k ? f_out : f_k;
  return SLIDEDP_OK;
}

}  // extern "C"
