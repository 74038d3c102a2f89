// libslidedp: the device-resident path: kernel launchers, the global norm, the fused update, the
// rank reduction alone and the norm variant that allocates nothing.
// See include/slidedp.h for the contract of every entry point.
#include "internal.h"
#include "kernels.cuh"

#include <atomic>

using namespace slidedp;
using namespace slidedp::host;

namespace slidedp {
namespace host {

// Launch configuration for a kernel that may start being scheduled while the previous kernel
// of the stream is finishing (programmatic dependent launch; the kernel itself waits for that
// kernel's completion before touching memory). `early` = false is a plain launch.
struct LaunchCfg {
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[1];
  LaunchCfg(unsigned blocks, unsigned threads, cudaStream_t st, bool early) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3(blocks);
    cfg.blockDim = dim3(threads);
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = early ? 1 : 0;
  }
};

template <int R_T>
static void launch_update_t(const GradPtrs& gp, int /*R*/, int64_t n, float* w, float* m, float* v,
                     uint16_t* p, const UpdateConsts& k, const double* coef, cudaStream_t st,
                     bool early) {
  const int64_t groups = (n + kVec - 1) / kVec;
  const unsigned blocks = (unsigned)((groups + kUpdateThreads - 1) / kUpdateThreads);
  LaunchCfg lc(blocks, kUpdateThreads, st, early);
  (void)cudaLaunchKernelEx(&lc.cfg, reduce_adamw_kernel<R_T>, gp, n, w, m, v, p, k, coef);
}

int launch_update(slidedp_ctx* ctx, const GradPtrs& gp, int R, int64_t n, float* w, float* m,
                  float* v, uint16_t* p, const UpdateConsts& k, const double* coef,
                  cudaStream_t st, bool early) {
  if (n == 0) return SLIDEDP_OK;
  FAULT_POINT();
  // one instantiation per rank count: the R loads are fully unrolled (a runtime-R loop over a
  // 16-entry register array ran at 4.0 TB/s for R = 3 against 6.4+ TB/s unrolled)
  switch (R) {
#define SLIDEDP_CASE(r) case r: launch_update_t<r>(gp, R, n, w, m, v, p, k, coef, st, early); break;
    SLIDEDP_CASE(1) SLIDEDP_CASE(2) SLIDEDP_CASE(3) SLIDEDP_CASE(4) SLIDEDP_CASE(5) SLIDEDP_CASE(6)
    SLIDEDP_CASE(7) SLIDEDP_CASE(8) SLIDEDP_CASE(9) SLIDEDP_CASE(10) SLIDEDP_CASE(11)
    SLIDEDP_CASE(12) SLIDEDP_CASE(13) SLIDEDP_CASE(14) SLIDEDP_CASE(15) SLIDEDP_CASE(16)
#undef SLIDEDP_CASE
    default: return SLIDEDP_ERR_INVALID_ARG;
  }
  ctx->launches += 1;
  CU_AFTER_LAUNCH();
  return SLIDEDP_OK;
}

// The update with the BF16 copy stored into several buffers (sharded multi-GPU step).
static int launch_update_bcast(slidedp_ctx* ctx, const GradPtrs& gp, int R, int64_t n, float* w,
                               float* m, float* v, const ManyOuts& outs, const UpdateConsts& k,
                               const double* coef, cudaStream_t st) {
  if (n == 0) return SLIDEDP_OK;
  FAULT_POINT();
  const int64_t groups = (n + kVec - 1) / kVec;
  const unsigned blocks = (unsigned)((groups + kUpdateThreads - 1) / kUpdateThreads);
  switch (R) {
#define SLIDEDP_CASE(r)                                                                         \
  case r:                                                                                       \
    reduce_adamw_bcast_kernel<r><<<blocks, kUpdateThreads, 0, st>>>(gp, n, w, m, v, outs, k, coef); \
    break;
    SLIDEDP_CASE(1) SLIDEDP_CASE(2) SLIDEDP_CASE(3) SLIDEDP_CASE(4) SLIDEDP_CASE(5) SLIDEDP_CASE(6)
    SLIDEDP_CASE(7) SLIDEDP_CASE(8) SLIDEDP_CASE(9) SLIDEDP_CASE(10) SLIDEDP_CASE(11)
    SLIDEDP_CASE(12) SLIDEDP_CASE(13) SLIDEDP_CASE(14) SLIDEDP_CASE(15) SLIDEDP_CASE(16)
#undef SLIDEDP_CASE
    default: return SLIDEDP_ERR_INVALID_ARG;
  }
  ctx->launches += 1;
  CU_AFTER_LAUNCH();
  return SLIDEDP_OK;
}

// One instantiation per rank count (R is validated to 1..16 before this is reached). Queued so
// that the kernel can be scheduled while the previous kernel of the stream is finishing (it waits
// for that kernel itself before its first load).
void launch_sumsq(const GradPtrs& gp, int R, int64_t n, float inv_R, double* tile_sums,
                  unsigned blocks, cudaStream_t st) {
  if (R == 1) {   // single rank: two tiles per block, every load of a tile in flight (same bits)
    LaunchCfg lc((blocks + kDeepTiles - 1) / kDeepTiles, kNormThreads, st, /*early=*/true);
    (void)cudaLaunchKernelEx(&lc.cfg, grad_sumsq_tiles_r1_kernel, gp.p[0], n, inv_R, tile_sums);
    return;
  }
  LaunchCfg lc(blocks, kNormThreads, st, /*early=*/true);
  switch (R) {
#define SLIDEDP_CASE(r) \
  case r: (void)cudaLaunchKernelEx(&lc.cfg, grad_sumsq_tiles_kernel<r>, gp, n, inv_R, tile_sums); break;
    SLIDEDP_CASE(2) SLIDEDP_CASE(3) SLIDEDP_CASE(4) SLIDEDP_CASE(5) SLIDEDP_CASE(6)
    SLIDEDP_CASE(7) SLIDEDP_CASE(8) SLIDEDP_CASE(9) SLIDEDP_CASE(10) SLIDEDP_CASE(11)
    SLIDEDP_CASE(12) SLIDEDP_CASE(13) SLIDEDP_CASE(14) SLIDEDP_CASE(15) SLIDEDP_CASE(16)
#undef SLIDEDP_CASE
    default: break;
  }
}

static int ensure_partials(slidedp_ctx* ctx, int64_t need, cudaStream_t st) {
  if (need <= ctx->partials_cap) return SLIDEDP_OK;
  // Rare: a step of more than 17 G parameters. Growing keeps the tiles already written.
  int64_t cap = ctx->partials_cap;
  while (cap < need) cap *= 2;
  double* bigger = nullptr;
  CU(cudaMalloc(&bigger, (size_t)cap * sizeof(double)));
  cudaError_t e = cudaMemcpyAsync(bigger, ctx->partials, (size_t)ctx->partials_used * sizeof(double),
                                  cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess) {
    int rc = bounded_stream_wait(ctx, st, ctx->wait_seconds);
    if (rc != SLIDEDP_OK) { cudaFree(bigger); return rc; }
  } else {
    cudaFree(bigger);
    return cuda_fail(ctx, e);
  }
  cudaFree(ctx->partials);
  ctx->partials = bigger;
  ctx->partials_cap = cap;
  return SLIDEDP_OK;
}

int norm_chunk(slidedp_ctx* ctx, const GradPtrs& gp, int R, int64_t n, double inv_R,
               int first_chunk, cudaStream_t st) {
  if (first_chunk) ctx->partials_used = 0;
  if (n == 0) return SLIDEDP_OK;
  const int64_t ntiles = (n + kNormTile - 1) / kNormTile;
  int rc = ensure_partials(ctx, ctx->partials_used + ntiles, st);
  if (rc != SLIDEDP_OK) return rc;
  // one block per tile: the hardware scheduler balances them, a tail of one tile at most
  const unsigned blocks = (unsigned)ntiles;
  double* dst = ctx->partials + ctx->partials_used;
  const float inv = (float)inv_R;
  FAULT_POINT();
  launch_sumsq(gp, R, n, inv, dst, blocks, st);
  ctx->launches += 1;
  CU_AFTER_LAUNCH();
  ctx->partials_used += ntiles;
  return SLIDEDP_OK;
}

// The finish kernel is queued so that it can be scheduled while the tile kernel before it is
// still finishing (it waits for that kernel itself): hides its launch, 2-3 us per norm pass.
static void launch_finish(const double* partials, int64_t count, double max_norm, double* scalars,
                          cudaStream_t st) {
  LaunchCfg lc(1, kFinishThreads, st, /*early=*/true);
  (void)cudaLaunchKernelEx(&lc.cfg, grad_norm_finish_kernel, partials, count, max_norm, scalars);
}

int norm_finish(slidedp_ctx* ctx, double max_norm, cudaStream_t st) {
  FAULT_POINT();
  launch_finish(ctx->partials, ctx->partials_used, max_norm, ctx->scalars, st);
  ctx->launches += 1;
  CU_AFTER_LAUNCH();
  ctx->norm_issued = true;
  return SLIDEDP_OK;
}

// Copies the four scalars to the pinned mirror on `st` and waits (bounded) for them.
static int fetch_scalars(slidedp_ctx* ctx, cudaStream_t st) {
  CU(cudaMemcpyAsync(ctx->host_scalars, ctx->scalars, 4 * sizeof(double),
                     cudaMemcpyDeviceToHost, st));
  CU(cudaEventRecord(ctx->scalar_event, st));
  return bounded_event_wait(ctx, ctx->scalar_event, ctx->wait_seconds);
}


}  // namespace host
}  // namespace slidedp

extern "C" {

int slidedp_grad_norm(slidedp_ctx* ctx, const void* const* grads_bf16, int R, int64_t n,
                      double inv_R, int first_chunk, void* cuda_stream) {
  if (!ctx || n < 0 || inv_R != inv_R) return SLIDEDP_ERR_INVALID_ARG;
  GradPtrs gp;
  int rc = check_grads(grads_bf16, R, &gp);
  if (rc != SLIDEDP_OK) return rc;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  return norm_chunk(ctx, gp, R, n, inv_R, first_chunk, static_cast<cudaStream_t>(cuda_stream));
}

int slidedp_grad_norm_finish(slidedp_ctx* ctx, double max_norm, double* host_norm,
                             double* host_coef, void* cuda_stream) {
  if (!ctx || max_norm != max_norm) return SLIDEDP_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int rc = norm_finish(ctx, max_norm, st);
  if (rc != SLIDEDP_OK) return rc;
  if (host_norm || host_coef) {
    rc = fetch_scalars(ctx, st);
    if (rc != SLIDEDP_OK) return rc;
    if (host_norm) *host_norm = ctx->host_scalars[1];
    if (host_coef) *host_coef = ctx->host_scalars[2];
  }
  return SLIDEDP_OK;
}

int slidedp_grad_norm_tiles(slidedp_ctx* ctx, const void* const* grads_bf16, int R, int64_t n,
                            double inv_R, double* tile_sums_out, void* cuda_stream) {
  if (!ctx || n < 0 || inv_R != inv_R) return SLIDEDP_ERR_INVALID_ARG;
  GradPtrs gp;
  int rc = check_grads(grads_bf16, R, &gp);
  if (rc != SLIDEDP_OK) return rc;
  if (n == 0) return SLIDEDP_OK;
  if (!tile_sums_out) return SLIDEDP_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(tile_sums_out) & 7u) != 0) return SLIDEDP_ERR_MISALIGNED;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  const int64_t ntiles = (n + kNormTile - 1) / kNormTile;
  FAULT_POINT();
  launch_sumsq(gp, R, n, (float)inv_R, tile_sums_out, (unsigned)ntiles,
               static_cast<cudaStream_t>(cuda_stream));
  ctx->launches += 1;
  CU_AFTER_LAUNCH();
  return SLIDEDP_OK;
}

int slidedp_grad_norm_finish_from(slidedp_ctx* ctx, const double* tile_sums, int64_t count,
                                  double max_norm, double* host_norm, double* host_coef,
                                  void* cuda_stream) {
  if (!ctx || count < 0 || max_norm != max_norm || (count > 0 && !tile_sums))
    return SLIDEDP_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  FAULT_POINT();
  launch_finish(tile_sums, count, max_norm, ctx->scalars, st);
  ctx->launches += 1;
  CU_AFTER_LAUNCH();
  ctx->norm_issued = true;
  if (host_norm || host_coef) {
    int rc = fetch_scalars(ctx, st);
    if (rc != SLIDEDP_OK) return rc;
    if (host_norm) *host_norm = ctx->host_scalars[1];
    if (host_coef) *host_coef = ctx->host_scalars[2];
  }
  return SLIDEDP_OK;
}

int slidedp_reduce_adamw_chunk(slidedp_ctx* ctx, const void* const* grads_bf16, int R, int64_t n,
                               float* master, float* m, float* v, void* param_bf16_out,
                               const slidedp_hparams* hp, void* cuda_stream) {
  if (!ctx || n < 0) return SLIDEDP_ERR_INVALID_ARG;
  int rc = check_hparams(hp);
  if (rc != SLIDEDP_OK) return rc;
  GradPtrs gp;
  rc = check_grads(grads_bf16, R, &gp);
  if (rc != SLIDEDP_OK) return rc;
  if (n > 0 && (!master || !m || !v || !param_bf16_out)) return SLIDEDP_ERR_INVALID_ARG;
  if (!aligned16(master) || !aligned16(m) || !aligned16(v) || !aligned16(param_bf16_out))
    return SLIDEDP_ERR_MISALIGNED;
  const bool clip = hp->max_norm > 0.0;
  if (clip && !ctx->norm_issued) return SLIDEDP_ERR_NO_NORM;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  return launch_update(ctx, gp, R, n, master, m, v, static_cast<uint16_t*>(param_bf16_out),
                       make_consts(hp), clip ? ctx->scalars + 2 : nullptr,
                       static_cast<cudaStream_t>(cuda_stream), /*early=*/true);
}

int slidedp_scatter_tile_sums(slidedp_ctx* ctx, const double* tile_sums, int64_t count,
                              double* const* dsts, int n_dsts, void* cuda_stream) {
  if (!ctx || count < 0 || !dsts || n_dsts < 1 || n_dsts > SLIDEDP_MAX_RANKS)
    return SLIDEDP_ERR_INVALID_ARG;
  if (count > 0 && !tile_sums) return SLIDEDP_ERR_INVALID_ARG;
  F64Dsts d;
  for (int o = 0; o < kMaxRanks; ++o) d.p[o] = nullptr;
  for (int o = 0; o < n_dsts; ++o) {
    if (!dsts[o]) return SLIDEDP_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(dsts[o]) & 7u) != 0) return SLIDEDP_ERR_MISALIGNED;
    d.p[o] = dsts[o];
  }
  if ((reinterpret_cast<uintptr_t>(tile_sums) & 7u) != 0) return SLIDEDP_ERR_MISALIGNED;
  if (count == 0) return SLIDEDP_OK;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  FAULT_POINT();
  scatter_tile_sums_kernel<<<(unsigned)((count + 255) / 256), 256, 0,
                             static_cast<cudaStream_t>(cuda_stream)>>>(tile_sums, count, d, n_dsts);
  ctx->launches += 1;
  CU_AFTER_LAUNCH();
  return SLIDEDP_OK;
}

int slidedp_reduce_adamw_chunk_bcast(slidedp_ctx* ctx, const void* const* grads_bf16, int R,
                                     int64_t n, float* master, float* m, float* v,
                                     void* const* param_bf16_outs, int n_outs,
                                     const slidedp_hparams* hp, void* cuda_stream) {
  if (!ctx || n < 0) return SLIDEDP_ERR_INVALID_ARG;
  int rc = check_hparams(hp);
  if (rc != SLIDEDP_OK) return rc;
  GradPtrs gp;
  rc = check_grads(grads_bf16, R, &gp);
  if (rc != SLIDEDP_OK) return rc;
  if (!param_bf16_outs || n_outs < 1 || n_outs > SLIDEDP_MAX_RANKS) return SLIDEDP_ERR_INVALID_ARG;
  if (n > 0 && (!master || !m || !v)) return SLIDEDP_ERR_INVALID_ARG;
  if (!aligned16(master) || !aligned16(m) || !aligned16(v)) return SLIDEDP_ERR_MISALIGNED;
  ManyOuts outs;
  outs.count = n_outs;
  for (int o = 0; o < kMaxRanks; ++o) outs.p[o] = nullptr;
  for (int o = 0; o < n_outs; ++o) {
    if (!param_bf16_outs[o]) return SLIDEDP_ERR_INVALID_ARG;
    if (!aligned16(param_bf16_outs[o])) return SLIDEDP_ERR_MISALIGNED;
    outs.p[o] = static_cast<uint16_t*>(param_bf16_outs[o]);
  }
  const bool clip = hp->max_norm > 0.0;
  if (clip && !ctx->norm_issued) return SLIDEDP_ERR_NO_NORM;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  return launch_update_bcast(ctx, gp, R, n, master, m, v, outs, make_consts(hp),
                             clip ? ctx->scalars + 2 : nullptr,
                             static_cast<cudaStream_t>(cuda_stream));
}

int slidedp_hbm_mix_probe(slidedp_ctx* ctx, const void* const* grads_bf16, int R, int64_t n,
                          float* master, float* m, float* v, void* scratch_bf16_out, int reps,
                          double* best_gbs, void* cuda_stream) {
  if (!ctx || n < kVec || reps < 1 || !best_gbs) return SLIDEDP_ERR_INVALID_ARG;
  GradPtrs gp;
  int rc = check_grads(grads_bf16, R, &gp);
  if (rc != SLIDEDP_OK) return rc;
  if (!master || !m || !v || !scratch_bf16_out) return SLIDEDP_ERR_INVALID_ARG;
  if (!aligned16(master) || !aligned16(m) || !aligned16(v) || !aligned16(scratch_bf16_out))
    return SLIDEDP_ERR_MISALIGNED;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int64_t groups = n / kVec;
  const unsigned blocks = (unsigned)((groups + kUpdateThreads - 1) / kUpdateThreads);
  uint16_t* out = static_cast<uint16_t*>(scratch_bf16_out);
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  CU(cudaEventCreate(&e0));
  if (cudaEventCreate(&e1) != cudaSuccess) { cudaEventDestroy(e0); return cuda_fail(ctx, cudaErrorUnknown); }
  double best = 0.0;
  for (int rep = 0; rep < reps + 2 && rc == SLIDEDP_OK; ++rep) {      // two warm-up launches
    cudaError_t e = cudaEventRecord(e0, st);
    if (e == cudaSuccess) {
      switch (R) {
#define SLIDEDP_CASE(r) \
  case r: traffic_mix_kernel<r><<<blocks, kUpdateThreads, 0, st>>>(gp, n, master, m, v, out); break;
        SLIDEDP_CASE(1) SLIDEDP_CASE(2) SLIDEDP_CASE(3) SLIDEDP_CASE(4) SLIDEDP_CASE(5) SLIDEDP_CASE(6)
        SLIDEDP_CASE(7) SLIDEDP_CASE(8) SLIDEDP_CASE(9) SLIDEDP_CASE(10) SLIDEDP_CASE(11)
        SLIDEDP_CASE(12) SLIDEDP_CASE(13) SLIDEDP_CASE(14) SLIDEDP_CASE(15) SLIDEDP_CASE(16)
#undef SLIDEDP_CASE
        default: break;
      }
      ctx->launches += 1;
      e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaEventRecord(e1, st);
    if (e != cudaSuccess) { rc = cuda_fail(ctx, e); break; }
    rc = bounded_event_wait(ctx, e1, ctx->wait_seconds);
    if (rc != SLIDEDP_OK) break;
    float ms = 0.f;
    if (rep >= 2 && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess && ms > 0.f) {
      const double gbs = (double)(26 + 2 * R) * (double)(groups * kVec) / ((double)ms * 1e6);
      if (gbs > best) best = gbs;
    }
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (rc == SLIDEDP_OK) *best_gbs = best;
  return rc;
}

int slidedp_reduce_mean_bf16(slidedp_ctx* ctx, const void* const* grads_bf16, int R, int64_t n,
                             double inv_R, void* out_bf16, void* cuda_stream) {
  if (!ctx || n < 0 || inv_R != inv_R) return SLIDEDP_ERR_INVALID_ARG;
  GradPtrs gp;
  int rc = check_grads(grads_bf16, R, &gp);
  if (rc != SLIDEDP_OK) return rc;
  if (n > 0 && !out_bf16) return SLIDEDP_ERR_INVALID_ARG;
  if (!aligned16(out_bf16)) return SLIDEDP_ERR_MISALIGNED;
  if (n == 0) return SLIDEDP_OK;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int64_t per_block = (R == 1 ? 16 : 8) * (int64_t)kReduceThreads;   // elements per block
  const unsigned blocks = (unsigned)((n + per_block - 1) / per_block);
  uint16_t* out = static_cast<uint16_t*>(out_bf16);
  const float inv = (float)inv_R;
  FAULT_POINT();
  switch (R) {
#define SLIDEDP_CASE(r) \
  case r: reduce_mean_bf16_kernel<r><<<blocks, kReduceThreads, 0, st>>>(gp, n, inv, out); break;
    SLIDEDP_CASE(1) SLIDEDP_CASE(2) SLIDEDP_CASE(3) SLIDEDP_CASE(4) SLIDEDP_CASE(5) SLIDEDP_CASE(6)
    SLIDEDP_CASE(7) SLIDEDP_CASE(8) SLIDEDP_CASE(9) SLIDEDP_CASE(10) SLIDEDP_CASE(11)
    SLIDEDP_CASE(12) SLIDEDP_CASE(13) SLIDEDP_CASE(14) SLIDEDP_CASE(15) SLIDEDP_CASE(16)
#undef SLIDEDP_CASE
    default: return SLIDEDP_ERR_INVALID_ARG;
  }
  ctx->launches += 1;
  CU_AFTER_LAUNCH();
  return SLIDEDP_OK;
}

// ---- norm without allocation ---------------------------------------------------------------
//
// Scratch for callers that cannot allocate: the per-tile sums live in an array that is part
// of the library's device image. In HOST code the name `noalloc_tile_sums` is only a handle
// for the symbol, not a device address; the address each device gave it is looked up once
// per device with cudaGetSymbolAddress (with that device current) and cached here.
constexpr int64_t kNoallocMaxTiles = SLIDEDP_NOALLOC_MAX_ELEMS / kNormTile;   // 65536
static __device__ __align__(256) double noalloc_tile_sums[kNoallocMaxTiles];

// One slot per device, written once. Atomic so that two host threads making their first call
// at the same time both end up with the same (identical) address and no data race.
constexpr int kNoallocMaxDevices = 64;
static std::atomic<double*> noalloc_scratch_addr[kNoallocMaxDevices];   // zero-initialised

int slidedp_grad_norm_noalloc(const void* const* grads_bf16, int R, int64_t n, double inv_R,
                              double max_norm, double* out4, void* cuda_stream) {
  if (n < 0 || !out4 || inv_R != inv_R || max_norm != max_norm) return SLIDEDP_ERR_INVALID_ARG;
  GradPtrs gp;
  int rc = check_grads(grads_bf16, R, &gp);
  if (rc != SLIDEDP_OK) return rc;
  if (!aligned16(out4)) return SLIDEDP_ERR_MISALIGNED;
  if (n > SLIDEDP_NOALLOC_MAX_ELEMS) return SLIDEDP_ERR_TOO_LARGE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return SLIDEDP_ERR_CUDA; }
  if (dev < 0 || dev >= kNoallocMaxDevices) return SLIDEDP_ERR_INVALID_ARG;
  double* scratch = noalloc_scratch_addr[dev].load(std::memory_order_acquire);
  if (!scratch) {
    // one-time set-up for this device (current right now): resolve the symbol's address. With
    // lazy module loading this is also where the driver loads the library's device image,
    // array included, which is why the header asks for this call at start-up.
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, noalloc_tile_sums) != cudaSuccess || !p) {
      (void)cudaGetLastError();
      return SLIDEDP_ERR_CUDA;
    }
    scratch = static_cast<double*>(p);
    noalloc_scratch_addr[dev].store(scratch, std::memory_order_release);
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int64_t ntiles = (n + kNormTile - 1) / kNormTile;
  if (ntiles > 0) {
    const unsigned blocks = (unsigned)ntiles;
    const float inv = (float)inv_R;
    launch_sumsq(gp, R, n, inv, scratch, blocks, st);
    if (cudaGetLastError() != cudaSuccess) return SLIDEDP_ERR_CUDA;
  }
  // reads tiles [0, ntiles) only: whatever an earlier call left beyond them is never seen
  grad_norm_finish_kernel<<<1, kFinishThreads, 0, st>>>(scratch, ntiles, max_norm, out4);
  if (cudaGetLastError() != cudaSuccess) return SLIDEDP_ERR_CUDA;
  return SLIDEDP_OK;
}

}  // extern "C"
