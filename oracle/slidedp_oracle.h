/*
 * slidedp_oracle.h -- plain CPU oracle for the SlideDP reduce + AdamW step.
 *
 * TEST INFRASTRUCTURE ONLY. This is the slow, obviously-correct restatement of
 * the step that the CUDA library is checked against. It shares no code, header,
 * constant or helper with the CUDA path, and the product never calls it: only
 * the tests, the smoke check and the benchmark's cpu_baseline / reference arm do.
 *
 * What it computes, for N flat parameters and R rank gradients:
 *   state      16 bytes per parameter: BF16 parameter, BF16 gradient, FP32 master,
 *              FP32 first and second Adam moments (paper Sec. 2.1, Table 1).
 *   reduction  the rank-local gradients are summed, then averaged, giving ONE
 *              gradient per layer (paper Sec. 3.2 "Gradient return"). Reading
 *              taken here: left-to-right over ranks 0..R-1 with FP32 round-to-
 *              nearest-even adds, then one FP32 multiply by (float)(1/R); the
 *              average is NOT rounded back to BF16.
 *   update     one Adam update of the single authoritative FP32 master/m/v per
 *              iteration (paper Sec. 3.2, shared host state), evaluated in
 *              double from the stored FP32 state with one rounding per output.
 *              The paper says only "mixed-precision Adam"; decoupled weight
 *              decay, bias correction and eps outside the root follow
 *              Kingma & Ba Alg. 1 / Loshchilov & Hutter Alg. 2.
 *   emission   the BF16 parameter copy is a round-to-nearest-even cast of the
 *              rounded FP32 master (paper Sec. 3.3 "Overlap within a layer").
 *   clipping   not in the paper: global L2 norm of the averaged gradient over
 *              all parameters of the step, coefficient min(1, max/(norm+1e-6)).
 *              The 1e-6 constant and the left-to-right rank order are
 *              definitions fixed by this library (parity unpinned by the paper);
 *              everything else is pinned by the CPU tests.
 *
 * All pointers are host pointers. BF16 values travel as uint16_t bit patterns.
 * nthreads <= 1 runs every loop sequentially in index order; nthreads > 1 splits
 * the index range into nthreads contiguous blocks (OpenMP static). The update is
 * elementwise, so threading cannot change it; the sum of squares adds the
 * per-block partials in block order.
 */
#ifndef SLIDEDP_ORACLE_H
#define SLIDEDP_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  double lr, beta1, beta2, eps, weight_decay;
  double inv_R;     /* the FP32 rank sum is multiplied by (float)inv_R           */
  double max_norm;  /* <= 0: clipping off                                        */
  int64_t step;     /* 1-based index of the update being performed               */
} oracle_hparams;

/* Table 1: 2N + 2N + 4N + 8N = 16N bytes. out5 (nullable) receives the five
 * per-parameter byte counts {bf16 param, bf16 grad, fp32 master, fp32 m, fp32 v}. */
size_t oracle_state_bytes(int64_t n, int out5[5]);

/* BF16 <-> FP32. Widening is exact; narrowing is round-to-nearest-even, NaN stays
 * NaN (quiet), +-inf stays. */
float oracle_bf16_to_f32(uint16_t b);
uint16_t oracle_f32_to_bf16(float x);

/* gbar[i] = fl32( (((g_0[i] + g_1[i]) + ...) + g_{R-1}[i]) * fl32(inv_R) ). */
void oracle_reduce_mean(const uint16_t* const* grads, int R, int64_t n, double inv_R,
                        float* gbar);

/* The paper's GPU-reduction route returns ONE BF16 gradient per layer to the host (Sec. 3.2
 * "Gradient return"): out[i] = round-to-nearest-even BF16 of gbar[i] as defined above. */
void oracle_reduce_mean_bf16(const uint16_t* const* grads, int R, int64_t n, double inv_R,
                             uint16_t* out);

/* Sum over i of double(gbar[i])^2 for the averaged gradient of one chunk. */
double oracle_grad_sumsq(const uint16_t* const* grads, int R, int64_t n, double inv_R,
                         int nthreads);

/* norm = sqrt(sumsq); returns c = (max_norm > 0) ? min(1, max_norm/(norm+1e-6)) : 1.
 * A NaN norm gives a NaN coefficient. */
double oracle_clip_coef(double sumsq, double max_norm, double* norm_out);

/* One update of a chunk, in place on master/m/v, writing the BF16 copy. clip_coef
 * is the step's coefficient (1.0 when clipping is off); hp->max_norm is ignored
 * here. Returns 0, or -1 on a bad argument. */
int oracle_reduce_adamw_chunk(const uint16_t* const* grads, int R, int64_t n,
                              float* master, float* m, float* v, uint16_t* param_bf16,
                              const oracle_hparams* hp, double clip_coef, int nthreads);

/* A whole step over N parameters: norm over everything first (if hp->max_norm > 0),
 * then the update chunk by chunk (chunk_elems <= 0: one chunk). norm_out and
 * coef_out are nullable. */
int oracle_step(const uint16_t* const* grads, int R, int64_t n_total,
                float* master, float* m, float* v, uint16_t* param_bf16,
                int64_t chunk_elems, const oracle_hparams* hp,
                double* norm_out, double* coef_out, int nthreads);

/* Parameter delivery (paper Sec. 3.3 "Overlap within a layer": the FP32 master is cast to BF16
 * for the next delivery): p[i] = round-to-nearest-even BF16 of master[i]. */
void oracle_cast_master_to_bf16(const float* master, int64_t n, uint16_t* param_bf16);

/* Threads an nthreads > 1 call would really use (1 when built without OpenMP). */
int oracle_max_threads(void);

#ifdef __cplusplus
}
#endif
#endif
