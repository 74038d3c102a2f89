/*
 * slidedp_oracle.c -- plain C restatement of the SlideDP reduce + AdamW step.
 * TEST INFRASTRUCTURE ONLY; see slidedp_oracle.h for what each function follows.
 *
 * Build with -ffp-contract=off and without -ffast-math: every float operation
 * below is one IEEE round-to-nearest-even operation, every double operation one
 * IEEE double operation, in the order written.
 */
#include "slidedp_oracle.h"

#include <math.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- Table 1: bytes of state per parameter -------------------------------- */
size_t oracle_state_bytes(int64_t n, int out5[5]) {
  const int bytes[5] = {2 /* BF16 compute weight */, 2 /* BF16 gradient */,
                        4 /* FP32 master */, 4 /* FP32 m */, 4 /* FP32 v */};
  size_t per_param = 0;
  for (int k = 0; k < 5; ++k) {
    per_param += (size_t)bytes[k];
    if (out5) out5[k] = bytes[k];
  }
  return n < 0 ? 0 : per_param * (size_t)n;
}

/* ---- BF16 <-> FP32 --------------------------------------------------------- */
float oracle_bf16_to_f32(uint16_t b) {
  uint32_t u = (uint32_t)b << 16; /* BF16 is the top half of an FP32 */
  float f;
  memcpy(&f, &u, sizeof f);
  return f;
}

uint16_t oracle_f32_to_bf16(float x) {
  uint32_t u;
  memcpy(&u, &x, sizeof u);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) /* NaN: keep the sign, force a quiet payload */
    return (uint16_t)((u >> 16) | 0x0040u);
  /* Round to nearest, ties to even: the 16 dropped bits are compared with one
   * half (0x8000); on a tie the kept mantissa's last bit decides. */
  uint32_t kept = u >> 16, dropped = u & 0xFFFFu;
  if (dropped > 0x8000u || (dropped == 0x8000u && (kept & 1u))) kept += 1u;
  return (uint16_t)kept; /* a carry into the exponent gives the next binade or inf */
}

/* ---- Sec. 3.2 "Gradient return": sum over ranks, then average ------------- */
static float mean_of_ranks(const uint16_t* const* grads, int R, int64_t i, float inv_R32) {
  float s = oracle_bf16_to_f32(grads[0][i]);
  for (int r = 1; r < R; ++r) s = s + oracle_bf16_to_f32(grads[r][i]); /* FP32 add */
  return s * inv_R32;                                                    /* FP32 mul */
}

void oracle_reduce_mean(const uint16_t* const* grads, int R, int64_t n, double inv_R,
                        float* gbar) {
  const float inv_R32 = (float)inv_R;
  for (int64_t i = 0; i < n; ++i) gbar[i] = mean_of_ranks(grads, R, i, inv_R32);
}

void oracle_reduce_mean_bf16(const uint16_t* const* grads, int R, int64_t n, double inv_R,
                             uint16_t* out) {
  const float inv_R32 = (float)inv_R;
  for (int64_t i = 0; i < n; ++i) out[i] = oracle_f32_to_bf16(mean_of_ranks(grads, R, i, inv_R32));
}

/* ---- global L2 norm of the averaged gradient (not in the paper) ----------- */
double oracle_grad_sumsq(const uint16_t* const* grads, int R, int64_t n, double inv_R,
                         int nthreads) {
  const float inv_R32 = (float)inv_R;
  if (nthreads <= 1) {
    double S = 0.0;
    for (int64_t i = 0; i < n; ++i) {
      double g = (double)mean_of_ranks(grads, R, i, inv_R32);
      S += g * g;
    }
    return S;
  }
  double partial[256];
  if (nthreads > 256) nthreads = 256;
  for (int b = 0; b < nthreads; ++b) partial[b] = 0.0;
#ifdef _OPENMP
#pragma omp parallel for schedule(static, 1) num_threads(nthreads)
#endif
  for (int b = 0; b < nthreads; ++b) {
    int64_t lo = n / nthreads * b + (b < n % nthreads ? b : n % nthreads);
    int64_t hi = lo + n / nthreads + (b < n % nthreads ? 1 : 0);
    double S = 0.0;
    for (int64_t i = lo; i < hi; ++i) {
      double g = (double)mean_of_ranks(grads, R, i, inv_R32);
      S += g * g;
    }
    partial[b] = S;
  }
  double S = 0.0;
  for (int b = 0; b < nthreads; ++b) S += partial[b];
  return S;
}

double oracle_clip_coef(double sumsq, double max_norm, double* norm_out) {
  double norm = sqrt(sumsq);
  if (norm_out) *norm_out = norm;
  if (!(max_norm > 0.0)) return 1.0;
  double c = max_norm / (norm + 1e-6);
  if (c != c) return c; /* NaN norm: propagate */
  return c < 1.0 ? c : 1.0;
}

/* ---- the update: Adam moments, bias correction, decoupled decay, BF16 copy - */
int oracle_reduce_adamw_chunk(const uint16_t* const* grads, int R, int64_t n,
                              float* master, float* m, float* v, uint16_t* param_bf16,
                              const oracle_hparams* hp, double clip_coef, int nthreads) {
  if (!grads || !hp || R < 1 || n < 0 || hp->step < 1) return -1;
  if (n > 0 && (!master || !m || !v || !param_bf16)) return -1;
  const float inv_R32 = (float)hp->inv_R;
  const double lr = hp->lr, beta1 = hp->beta1, beta2 = hp->beta2, eps = hp->eps,
               wd = hp->weight_decay;
  const double bc1 = 1.0 - pow(beta1, (double)hp->step); /* bias corrections */
  const double bc2 = 1.0 - pow(beta2, (double)hp->step);
  (void)nthreads;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(nthreads > 1 ? nthreads : 1)
#endif
  for (int64_t i = 0; i < n; ++i) {
    double g = (double)mean_of_ranks(grads, R, i, inv_R32) * clip_coef;
    double w = (double)master[i];
    double m1 = beta1 * (double)m[i] + (1.0 - beta1) * g;
    double v1 = beta2 * (double)v[i] + (1.0 - beta2) * g * g;
    double mhat = m1 / bc1;
    double vhat = v1 / bc2;
    double u = mhat / (sqrt(vhat) + eps);
    double w1 = w - lr * (u + wd * w);
    m[i] = (float)m1; /* one rounding each, double -> FP32, nearest-even */
    v[i] = (float)v1;
    master[i] = (float)w1;
    param_bf16[i] = oracle_f32_to_bf16(master[i]); /* from the ROUNDED master */
  }
  return 0;
}

int oracle_step(const uint16_t* const* grads, int R, int64_t n_total,
                float* master, float* m, float* v, uint16_t* param_bf16,
                int64_t chunk_elems, const oracle_hparams* hp,
                double* norm_out, double* coef_out, int nthreads) {
  if (!grads || !hp || R < 1 || R > 64 || n_total < 0) return -1;
  double c = 1.0, norm = 0.0;
  if (hp->max_norm > 0.0) {
    /* the norm covers every parameter of the step, before any update */
    double S = oracle_grad_sumsq(grads, R, n_total, hp->inv_R, nthreads);
    c = oracle_clip_coef(S, hp->max_norm, &norm);
  }
  if (norm_out) *norm_out = norm;
  if (coef_out) *coef_out = c;
  if (chunk_elems <= 0) chunk_elems = n_total > 0 ? n_total : 1;
  for (int64_t off = 0; off < n_total; off += chunk_elems) {
    int64_t len = n_total - off < chunk_elems ? n_total - off : chunk_elems;
    const uint16_t* gp[64];
    for (int r = 0; r < R; ++r) gp[r] = grads[r] + off;
    int rc = oracle_reduce_adamw_chunk(gp, R, len, master + off, m + off, v + off,
                                       param_bf16 + off, hp, c, nthreads);
    if (rc) return rc;
  }
  return 0;
}

void oracle_cast_master_to_bf16(const float* master, int64_t n, uint16_t* param_bf16) {
  for (int64_t i = 0; i < n; ++i) param_bf16[i] = oracle_f32_to_bf16(master[i]);
}

int oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
