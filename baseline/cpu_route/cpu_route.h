/*
 * cpu_route.h -- the paper's OWN data path for the update step, as a timed baseline.
 *
 * NOT part of libslidedp and not used by it; it shares no code with libslidedp or with the test
 * oracle. It exists so that this repository can say, on the same box, what the route the paper
 * describes costs beside the fused GPU path:
 *
 *   gradient return (paper Sec. 3.2): either the GPUs reduce and ONE BF16 gradient of G_l bytes
 *     is copied to the host ("GPU reduction"), or all R rank gradients are copied, R G_l bytes,
 *     and the host sums them ("CPU reduction");
 *   update (Sec. 3.2 / 3.3, Reduce -> D2H -> Adam): a multi-threaded, vectorised CPU Adam over the
 *     single FP32 master / m / v in host memory, chunk by chunk as the D2H copies land;
 *   delivery (Sec. 3.3 "Overlap within a layer"): the CPU casts the FP32 master to BF16 into
 *     aligned page-locked staging with non-temporal stores while DMA moves the previous chunk
 *     (2 bytes per parameter over the link; sent once, "sharded", or R times, "replicated").
 *
 * Arithmetic: FP32 throughout, as a vectorised CPU Adam would be (the paper says only
 * "mixed-precision Adam"); the hyper-parameter constants are formed in double and rounded once.
 * Same formulas as libslidedp otherwise (AdamW, bias correction, eps outside the root, decoupled
 * decay, left-to-right FP32 rank sum times (float)(1/R)). Results therefore agree with the FP64
 * oracle only to FP32 rounding; tests state the tolerance.
 *
 * All functions return 0 on success, a negative value on a bad argument, a positive cudaError_t
 * when a CUDA runtime call failed, or CPUROUTE_TIMEOUT.
 */
#ifndef SLIDEDP_CPU_ROUTE_H
#define SLIDEDP_CPU_ROUTE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CPUROUTE_TIMEOUT 100001

typedef struct {
  double lr, beta1, beta2, eps, weight_decay;
  double inv_R;      /* the FP32 rank sum is multiplied by (float)inv_R (CPU reduction)   */
  double clip_coef;  /* the step's clip coefficient, computed elsewhere; 1.0 = no clip   */
  int64_t step;      /* 1-based                                                           */
} cpuroute_hparams;

/* Which code path the build and this CPU give: "avx512-bf16", "avx512f" or "scalar". */
const char* cpuroute_isa(void);
/* Selects a LOWER code path than the CPU's best (so that every path can be tested on one box):
 * one of the three names above. -2 if the CPU cannot run it, -1 for an unknown name. */
int cpuroute_limit_isa(const char* name);
int cpuroute_max_threads(void);

/* param_bf16[i] = round-to-nearest-even BF16 of master[i] (NaN stays NaN), n elements, written
 * with non-temporal (streaming) stores where dst is 64-byte aligned. nthreads >= 1. */
int cpuroute_cast_bf16(const float* master, int64_t n, uint16_t* param_bf16, int nthreads);

/* One AdamW update of n parameters in FP32 from R BF16 gradients on the HOST (R = 1: the
 * gradient the GPUs already reduced; R > 1: the host sums in rank order, FP32, then multiplies by
 * (float)inv_R). master / m / v in place; param_bf16 (nullable) receives the BF16 cast of the new
 * master with streaming stores (the cast fused into the update). */
int cpuroute_adamw(const uint16_t* const* grads_bf16, int R, int64_t n, float* master, float* m,
                   float* v, uint16_t* param_bf16, const cpuroute_hparams* hp, int nthreads);

/* What one pipelined step measured (ms; wall clock on the host unless stated). */
typedef struct {
  double ms_total;        /* first D2H enqueue to last H2D complete                          */
  double ms_wait_d2h;     /* time the update worker sat waiting for gradient copies           */
  double ms_update;       /* time inside the CPU update (sum over chunks)                     */
  double ms_d2h_lane;     /* CUDA-event span of the D2H copies                                */
  double ms_h2d_lane;     /* CUDA-event span of the H2D copies                                */
  int64_t d2h_bytes, h2d_bytes, chunks;
} cpuroute_stats;

/* The paper's pipeline for one layer on one GPU:
 *   for every chunk: D2H of the chunk of each of the R_host device gradients (BF16) into pinned
 *   staging (all copies queued up front on one stream, an event per chunk); as each chunk lands
 *   the update worker (nthreads OpenMP threads) runs cpuroute_adamw on it, writing the BF16 cast
 *   into pinned parameter staging; the chunk's BF16 parameters are then copied H2D to each of the
 *   `copies` device parameter buffers (delivery to `copies` ranks).
 * dev_grads: R_host device pointers (n BF16 each). R_host = 1 is GPU reduction (the caller has
 * reduced already), R_host = R is CPU reduction. host_grad_staging: R_host pinned buffers of n
 * BF16. host master / m / v: n floats (any host memory; pinned not required, the CPU touches
 * them). host_param_staging: pinned, n BF16. dev_params: `copies` device pointers, n BF16 each.
 * chunk_elems: parameters per chunk (multiple of 32). */
int cpuroute_step(const void* const* dev_grads, int R_host, int64_t n, uint16_t* const* host_grad_staging,
                  float* master, float* m, float* v, uint16_t* host_param_staging,
                  void* const* dev_params, int copies, int64_t chunk_elems,
                  const cpuroute_hparams* hp, int nthreads, cpuroute_stats* stats);

/* Delivery alone (Sec. 3.3): CPU cast of chunk k+1 with non-temporal stores into pinned staging
 * while DMA moves chunk k, 2 bytes per parameter over the link. Stats: ms_total, ms_update
 * (time inside the cast), ms_h2d_lane, h2d_bytes, chunks. */
int cpuroute_deliver(const float* master, int64_t n, uint16_t* host_param_staging, void* dev_params,
                     int64_t chunk_elems, int nthreads, cpuroute_stats* stats);

#ifdef __cplusplus
}
#endif
#endif
