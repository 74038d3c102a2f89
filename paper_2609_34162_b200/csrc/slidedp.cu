// libslidedp: C ABI over the sm_100a kernels in kernels.cuh. See include/slidedp.h for
// the contract of every entry point. Host code here only validates arguments, prepares the
// per-step constants in double, launches kernels and drives the host-resident slot ring.
#include "slidedp.h"

#include <cuda_runtime.h>
#include <math.h>
#include <string.h>
#include <time.h>

#include <new>
#include <vector>

#include "kernels.cuh"

using namespace slidedp;

namespace {

constexpr double kWaitSeconds = 300.0;       // bound on every host-side wait
constexpr int64_t kInitialPartials = 1 << 20;  // 8 MB: 2^20 tiles = 17 G parameters

// Timing events of ONE kernel (the first chunk's). Per-chunk timing events, on the copy
// streams or the compute stream, sit on the chunk's H2D -> kernel -> D2H chain and cost
// several percent of link bandwidth at 16 MiB chunks, so a step records a fixed handful.
struct ChunkEvents {
  cudaEvent_t k_start, k_end;
};

}  // namespace

struct slidedp_ctx {
  int device = 0;
  size_t budget = 0;
  int last_cuda = 0;
  int64_t launches = 0;
  // norm workspace
  double* partials = nullptr;
  int64_t partials_cap = 0;
  int64_t partials_used = 0;
  double* scalars = nullptr;        // device: sumsq, norm, coef, nonfinite
  double* host_scalars = nullptr;   // pinned mirror
  bool norm_issued = false;
  cudaEvent_t scalar_event = nullptr;
  // host-resident streaming
  cudaStream_t s_in = nullptr, s_compute = nullptr, s_out = nullptr;
  float* slots = nullptr;
  size_t slot_bytes = 0;            // bytes currently allocated for all slots
  int64_t ring_cap = 0;             // floats per state array per slot in the current layout
  int ring_nbuf = 0;
  int64_t ring_next = 0;            // running chunk count: the next chunk's slot is this mod nbuf
  bool ring_busy = false;           // streaming work may still be in flight
  cudaEvent_t ev_loaded[3] = {nullptr, nullptr, nullptr};
  cudaEvent_t ev_updated[3] = {nullptr, nullptr, nullptr};
  cudaEvent_t ev_free[3] = {nullptr, nullptr, nullptr};
  cudaEvent_t ev_begin = nullptr, ev_norm_done = nullptr, ev_end = nullptr;
  cudaEvent_t ev_in_first = nullptr, ev_in_last = nullptr, ev_out_first = nullptr, ev_out_last = nullptr;
  std::vector<ChunkEvents> timing;  // grown on demand, reused
};

namespace {

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

int cuda_fail(slidedp_ctx* ctx, cudaError_t e) {
  if (ctx) ctx->last_cuda = (int)e;
  (void)cudaGetLastError();
  return SLIDEDP_ERR_CUDA;
}

#define CU(call)                                            \
  do {                                                      \
    cudaError_t e_ = (call);                                \
    if (e_ != cudaSuccess) return cuda_fail(ctx, e_);       \
  } while (0)

double now_seconds() {
  timespec ts;
  clock_gettime(CLOCK_MONOTONIC, &ts);
  return (double)ts.tv_sec + 1e-9 * (double)ts.tv_nsec;
}

// Waits for an event without ever blocking unboundedly inside the driver.
int bounded_event_wait(slidedp_ctx* ctx, cudaEvent_t ev, double seconds) {
  const double deadline = now_seconds() + seconds;
  for (;;) {
    cudaError_t e = cudaEventQuery(ev);
    if (e == cudaSuccess) return SLIDEDP_OK;
    if (e != cudaErrorNotReady) return cuda_fail(ctx, e);
    if (now_seconds() > deadline) return SLIDEDP_ERR_TIMEOUT;
    timespec nap = {0, 20000};
    nanosleep(&nap, nullptr);
  }
}

int bounded_stream_wait(slidedp_ctx* ctx, cudaStream_t s, double seconds) {
  const double deadline = now_seconds() + seconds;
  for (;;) {
    cudaError_t e = cudaStreamQuery(s);
    if (e == cudaSuccess) return SLIDEDP_OK;
    if (e != cudaErrorNotReady) return cuda_fail(ctx, e);
    if (now_seconds() > deadline) return SLIDEDP_ERR_TIMEOUT;
    timespec nap = {0, 20000};
    nanosleep(&nap, nullptr);
  }
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_grads(const void* const* grads, int R, GradPtrs* out) {
  if (!grads || R < 1 || R > SLIDEDP_MAX_RANKS) return SLIDEDP_ERR_INVALID_ARG;
  for (int r = 0; r < kMaxRanks; ++r) out->p[r] = nullptr;
  for (int r = 0; r < R; ++r) {
    if (!grads[r]) return SLIDEDP_ERR_INVALID_ARG;
    if (!aligned16(grads[r])) return SLIDEDP_ERR_MISALIGNED;
    out->p[r] = static_cast<const uint16_t*>(grads[r]);
  }
  return SLIDEDP_OK;
}

int check_hparams(const slidedp_hparams* hp) {
  if (!hp) return SLIDEDP_ERR_INVALID_ARG;
  if (hp->step < 1) return SLIDEDP_ERR_INVALID_ARG;
  if (!(hp->beta1 >= 0.0 && hp->beta1 < 1.0)) return SLIDEDP_ERR_INVALID_ARG;
  if (!(hp->beta2 >= 0.0 && hp->beta2 < 1.0)) return SLIDEDP_ERR_INVALID_ARG;
  if (!(hp->eps >= 0.0) || hp->lr != hp->lr || hp->weight_decay != hp->weight_decay ||
      hp->inv_R != hp->inv_R)
    return SLIDEDP_ERR_INVALID_ARG;
  return SLIDEDP_OK;
}

UpdateConsts make_consts(const slidedp_hparams* hp) {
  UpdateConsts k;
  const double bc1 = 1.0 - pow(hp->beta1, (double)hp->step);
  const double bc2 = 1.0 - pow(hp->beta2, (double)hp->step);
  k.beta1 = hp->beta1;
  k.beta2 = hp->beta2;
  k.omb1 = 1.0 - hp->beta1;
  k.omb2 = 1.0 - hp->beta2;
  k.rsqrt_bc2 = 1.0 / sqrt(bc2);
  k.eps = hp->eps;
  k.neg_lr_over_bc1 = -hp->lr / bc1;
  k.decay = 1.0 - hp->lr * hp->weight_decay;
  k.inv_R = (float)hp->inv_R;
  return k;
}

template <int R_T>
void launch_update_t(const GradPtrs& gp, int /*R*/, int64_t n, float* w, float* m, float* v,
                     uint16_t* p, const UpdateConsts& k, const double* coef, cudaStream_t st) {
  const int64_t groups = (n + kVec - 1) / kVec;
  const unsigned blocks = (unsigned)((groups + kUpdateThreads - 1) / kUpdateThreads);
  reduce_adamw_kernel<R_T><<<blocks, kUpdateThreads, 0, st>>>(gp, n, w, m, v, p, k, coef);
}

int launch_update(slidedp_ctx* ctx, const GradPtrs& gp, int R, int64_t n, float* w, float* m,
                  float* v, uint16_t* p, const UpdateConsts& k, const double* coef,
                  cudaStream_t st) {
  if (n == 0) return SLIDEDP_OK;
  // one instantiation per rank count: the R loads are fully unrolled (a runtime-R loop over a
  // 16-entry register array ran at 4.0 TB/s for R = 3 against 6.4+ TB/s unrolled)
  switch (R) {
#define SLIDEDP_CASE(r) case r: launch_update_t<r>(gp, R, n, w, m, v, p, k, coef, st); break;
    SLIDEDP_CASE(1) SLIDEDP_CASE(2) SLIDEDP_CASE(3) SLIDEDP_CASE(4) SLIDEDP_CASE(5) SLIDEDP_CASE(6)
    SLIDEDP_CASE(7) SLIDEDP_CASE(8) SLIDEDP_CASE(9) SLIDEDP_CASE(10) SLIDEDP_CASE(11)
    SLIDEDP_CASE(12) SLIDEDP_CASE(13) SLIDEDP_CASE(14) SLIDEDP_CASE(15) SLIDEDP_CASE(16)
#undef SLIDEDP_CASE
    default: return SLIDEDP_ERR_INVALID_ARG;
  }
  ctx->launches += 1;
  CU(cudaGetLastError());
  return SLIDEDP_OK;
}

// One instantiation per rank count (R is validated to 1..16 before this is reached).
void launch_sumsq(const GradPtrs& gp, int R, int64_t n, float inv_R, double* tile_sums,
                  unsigned blocks, cudaStream_t st) {
  switch (R) {
#define SLIDEDP_CASE(r) \
  case r: grad_sumsq_tiles_kernel<r><<<blocks, kNormThreads, 0, st>>>(gp, n, inv_R, tile_sums); break;
    SLIDEDP_CASE(1) SLIDEDP_CASE(2) SLIDEDP_CASE(3) SLIDEDP_CASE(4) SLIDEDP_CASE(5) SLIDEDP_CASE(6)
    SLIDEDP_CASE(7) SLIDEDP_CASE(8) SLIDEDP_CASE(9) SLIDEDP_CASE(10) SLIDEDP_CASE(11)
    SLIDEDP_CASE(12) SLIDEDP_CASE(13) SLIDEDP_CASE(14) SLIDEDP_CASE(15) SLIDEDP_CASE(16)
#undef SLIDEDP_CASE
    default: break;
  }
}

int ensure_partials(slidedp_ctx* ctx, int64_t need, cudaStream_t st) {
  if (need <= ctx->partials_cap) return SLIDEDP_OK;
  // Rare: a step of more than 17 G parameters. Growing keeps the tiles already written.
  int64_t cap = ctx->partials_cap;
  while (cap < need) cap *= 2;
  double* bigger = nullptr;
  CU(cudaMalloc(&bigger, (size_t)cap * sizeof(double)));
  cudaError_t e = cudaMemcpyAsync(bigger, ctx->partials, (size_t)ctx->partials_used * sizeof(double),
                                  cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess) {
    int rc = bounded_stream_wait(ctx, st, kWaitSeconds);
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
  launch_sumsq(gp, R, n, inv, dst, blocks, st);
  ctx->launches += 1;
  CU(cudaGetLastError());
  ctx->partials_used += ntiles;
  return SLIDEDP_OK;
}

int norm_finish(slidedp_ctx* ctx, double max_norm, cudaStream_t st) {
  grad_norm_finish_kernel<<<1, kFinishThreads, 0, st>>>(ctx->partials, ctx->partials_used,
                                                        max_norm, ctx->scalars);
  ctx->launches += 1;
  CU(cudaGetLastError());
  ctx->norm_issued = true;
  return SLIDEDP_OK;
}

// Copies the four scalars to the pinned mirror on `st` and waits (bounded) for them.
int fetch_scalars(slidedp_ctx* ctx, cudaStream_t st) {
  CU(cudaMemcpyAsync(ctx->host_scalars, ctx->scalars, 4 * sizeof(double),
                     cudaMemcpyDeviceToHost, st));
  CU(cudaEventRecord(ctx->scalar_event, st));
  return bounded_event_wait(ctx, ctx->scalar_event, kWaitSeconds);
}

// Grows the slot allocation to `need` bytes if the budget allows (checked before any work).
int ensure_slots(slidedp_ctx* ctx, size_t need) {
  if (ctx->budget && need > ctx->budget) return SLIDEDP_ERR_BUDGET;
  if (need > ctx->slot_bytes) {
    if (ctx->slots) { CU(cudaFree(ctx->slots)); ctx->slots = nullptr; ctx->slot_bytes = 0; }
    CU(cudaMalloc(&ctx->slots, need));
    ctx->slot_bytes = need;
  }
  return SLIDEDP_OK;
}

int is_pinned(slidedp_ctx* ctx, const void* p, bool* pinned) {
  cudaPointerAttributes a;
  cudaError_t e = cudaPointerGetAttributes(&a, p);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    *pinned = false;
    if (e == cudaErrorInvalidValue) return SLIDEDP_OK;  // plain pageable memory on old drivers
    return cuda_fail(ctx, e);
  }
  *pinned = (a.type == cudaMemoryTypeHost);
  return SLIDEDP_OK;
}

// Waits (bounded) until nothing queued on the context's three streams is left running.
int drain_streams(slidedp_ctx* ctx) {
  for (cudaStream_t st : {ctx->s_out, ctx->s_compute, ctx->s_in}) {
    int rc = bounded_stream_wait(ctx, st, kWaitSeconds);
    if (rc != SLIDEDP_OK) return rc;
  }
  ctx->ring_busy = false;
  return SLIDEDP_OK;
}

// Validates and enqueues one host-resident step on the context's streams. The slot ring
// carries over from call to call (slot index = running chunk count mod nbuf, every copy-in
// waits for the slot's last copy-out), so consecutive calls overlap like the chunks of one
// call; a call with another slot layout first drains what is queued.
int enqueue_stream_step(slidedp_ctx* ctx, const void* const* grads_bf16, int R, int64_t n_total,
                        float* host_master, float* host_m, float* host_v, void* param_bf16_out,
                        int64_t chunk_elems, int nbuf, int norm_ready, const slidedp_hparams* hp,
                        bool synchronous, bool timed, int64_t* nchunks_out) {
  if (!ctx || n_total < 0) return SLIDEDP_ERR_INVALID_ARG;
  int rc = check_hparams(hp);
  if (rc != SLIDEDP_OK) return rc;
  GradPtrs gp;
  rc = check_grads(grads_bf16, R, &gp);
  if (rc != SLIDEDP_OK) return rc;
  if (nbuf < 2 || nbuf > 3 || chunk_elems <= 0 || (chunk_elems % 8) != 0)
    return SLIDEDP_ERR_INVALID_ARG;
  if (n_total > 0 && (!host_master || !host_m || !host_v || !param_bf16_out))
    return SLIDEDP_ERR_INVALID_ARG;
  if (!aligned16(host_master) || !aligned16(host_m) || !aligned16(host_v) ||
      !aligned16(param_bf16_out))
    return SLIDEDP_ERR_MISALIGNED;
  const bool clip = hp->max_norm > 0.0;
  if (clip && norm_ready && !ctx->norm_issued) return SLIDEDP_ERR_NO_NORM;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  if (n_total > 0) {
    const float* hs[3] = {host_master, host_m, host_v};
    for (const float* h : hs) {
      bool pinned = false;
      rc = is_pinned(ctx, h, &pinned);
      if (rc != SLIDEDP_OK) return rc;
      if (!pinned) return SLIDEDP_ERR_NOT_PINNED;
    }
  }

  // slots: nbuf x {master, m, v} x cap floats
  const int64_t cap = chunk_elems < n_total ? chunk_elems : ((n_total + 7) / 8) * 8;
  const size_t need = (size_t)nbuf * 3 * (size_t)cap * sizeof(float);
  if (ctx->budget && need > ctx->budget) return SLIDEDP_ERR_BUDGET;
  const bool relayout = cap != ctx->ring_cap || nbuf != ctx->ring_nbuf || need > ctx->slot_bytes;
  if (relayout && ctx->ring_busy) {
    rc = drain_streams(ctx);
    if (rc != SLIDEDP_OK) return rc;
  }
  rc = ensure_slots(ctx, need);
  if (rc != SLIDEDP_OK) return rc;
  if (relayout) {
    ctx->ring_cap = cap;
    ctx->ring_nbuf = nbuf;
    ctx->ring_next = 0;
  }
  const int64_t nchunks = n_total == 0 ? 0 : (n_total + chunk_elems - 1) / chunk_elems;
  *nchunks_out = nchunks;
  if (timed) {
    while (ctx->timing.empty() && nchunks > 0) {
      ChunkEvents c;
      CU(cudaEventCreate(&c.k_start));
      CU(cudaEventCreate(&c.k_end));
      ctx->timing.push_back(c);
    }
  }

  ctx->ring_busy = true;
  if (synchronous) {
    CU(cudaEventRecord(ctx->ev_begin, ctx->s_compute));
    CU(cudaStreamWaitEvent(ctx->s_in, ctx->ev_begin, 0));
    CU(cudaStreamWaitEvent(ctx->s_out, ctx->ev_begin, 0));
  }
  if (clip && !norm_ready) {
    rc = norm_chunk(ctx, gp, R, n_total, hp->inv_R, 1, ctx->s_compute);
    if (rc != SLIDEDP_OK) return rc;
    rc = norm_finish(ctx, hp->max_norm, ctx->s_compute);
    if (rc != SLIDEDP_OK) return rc;
  }
  if (synchronous) CU(cudaEventRecord(ctx->ev_norm_done, ctx->s_compute));

  const UpdateConsts k = make_consts(hp);
  const double* coef = clip ? ctx->scalars + 2 : nullptr;
  uint16_t* pout = static_cast<uint16_t*>(param_bf16_out);
  for (int64_t c = 0; c < nchunks; ++c) {
    const int slot = (int)((ctx->ring_next + c) % nbuf);
    const int64_t off = c * chunk_elems;
    const int64_t len = n_total - off < chunk_elems ? n_total - off : chunk_elems;
    const size_t bytes = (size_t)len * sizeof(float);
    float* sw = ctx->slots + (size_t)slot * 3 * cap;
    float* sm = sw + cap;
    float* sv = sm + cap;
    ChunkEvents* te = (timed && c == 0) ? &ctx->timing[0] : nullptr;
    // copy-in: the slot must have been drained by the copy-out that last used it (a no-op
    // for an event that was never recorded or has completed)
    CU(cudaStreamWaitEvent(ctx->s_in, ctx->ev_free[slot], 0));
    if (timed && c == 0) CU(cudaEventRecord(ctx->ev_in_first, ctx->s_in));
    CU(cudaMemcpyAsync(sw, host_master + off, bytes, cudaMemcpyHostToDevice, ctx->s_in));
    CU(cudaMemcpyAsync(sm, host_m + off, bytes, cudaMemcpyHostToDevice, ctx->s_in));
    CU(cudaMemcpyAsync(sv, host_v + off, bytes, cudaMemcpyHostToDevice, ctx->s_in));
    if (timed && c == nchunks - 1) CU(cudaEventRecord(ctx->ev_in_last, ctx->s_in));
    CU(cudaEventRecord(ctx->ev_loaded[slot], ctx->s_in));
    // update
    CU(cudaStreamWaitEvent(ctx->s_compute, ctx->ev_loaded[slot], 0));
    if (te) CU(cudaEventRecord(te->k_start, ctx->s_compute));
    GradPtrs gc = gp;
    for (int r = 0; r < R; ++r) gc.p[r] = gp.p[r] + off;
    rc = launch_update(ctx, gc, R, len, sw, sm, sv, pout + off, k, coef, ctx->s_compute);
    if (rc != SLIDEDP_OK) return rc;
    if (te) CU(cudaEventRecord(te->k_end, ctx->s_compute));
    CU(cudaEventRecord(ctx->ev_updated[slot], ctx->s_compute));
    // copy-out
    CU(cudaStreamWaitEvent(ctx->s_out, ctx->ev_updated[slot], 0));
    if (timed && c == 0) CU(cudaEventRecord(ctx->ev_out_first, ctx->s_out));
    CU(cudaMemcpyAsync(host_master + off, sw, bytes, cudaMemcpyDeviceToHost, ctx->s_out));
    CU(cudaMemcpyAsync(host_m + off, sm, bytes, cudaMemcpyDeviceToHost, ctx->s_out));
    CU(cudaMemcpyAsync(host_v + off, sv, bytes, cudaMemcpyDeviceToHost, ctx->s_out));
    if (timed && c == nchunks - 1) CU(cudaEventRecord(ctx->ev_out_last, ctx->s_out));
    CU(cudaEventRecord(ctx->ev_free[slot], ctx->s_out));
  }
  ctx->ring_next += nchunks;
  if (synchronous) {
    // the step ends when the compute stream (norm, even with no chunks) and the last
    // copy-out are both done
    CU(cudaStreamWaitEvent(ctx->s_out, ctx->ev_norm_done, 0));
    if (clip) CU(cudaMemcpyAsync(ctx->host_scalars, ctx->scalars, 4 * sizeof(double),
                                 cudaMemcpyDeviceToHost, ctx->s_out));
    CU(cudaEventRecord(ctx->ev_end, ctx->s_out));
  }
  return SLIDEDP_OK;
}

}  // namespace

// ---------------------------------------------------------------------------------------
extern "C" {

const char* slidedp_strerror(int status) {
  switch (status) {
    case SLIDEDP_OK: return "ok";
    case SLIDEDP_ERR_INVALID_ARG: return "invalid argument";
    case SLIDEDP_ERR_MISALIGNED: return "a base pointer is not 16-byte aligned";
    case SLIDEDP_ERR_BUDGET: return "streaming slots exceed the GPU memory budget";
    case SLIDEDP_ERR_NOT_PINNED: return "host state pointer is not page-locked";
    case SLIDEDP_ERR_CUDA: return "a CUDA call failed";
    case SLIDEDP_ERR_TIMEOUT: return "a bounded wait expired";
    case SLIDEDP_ERR_NO_NORM: return "clipping requested before any norm was finished";
    case SLIDEDP_ERR_TOO_LARGE: return "n exceeds the fixed capacity of the no-allocation entry point";
    default: return "unknown status";
  }
}

size_t slidedp_state_bytes(int64_t n) {
  // BF16 parameter + BF16 gradient + FP32 master + FP32 m + FP32 v
  return n < 0 ? 0 : (size_t)n * (2 + 2 + 4 + 4 + 4);
}

int slidedp_last_cuda_error(const slidedp_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }
int64_t slidedp_kernel_launches(const slidedp_ctx* ctx) { return ctx ? ctx->launches : 0; }

int slidedp_create(slidedp_ctx** out, int device, size_t gpu_budget_bytes) {
  if (!out) return SLIDEDP_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess) { (void)cudaGetLastError(); return SLIDEDP_ERR_CUDA; }
  if (device < 0 || device >= count) return SLIDEDP_ERR_INVALID_ARG;
  DeviceGuard guard(device);
  if (!guard.ok) return SLIDEDP_ERR_CUDA;
  slidedp_ctx* ctx = new (std::nothrow) slidedp_ctx();
  if (!ctx) return SLIDEDP_ERR_INVALID_ARG;
  ctx->device = device;
  ctx->budget = gpu_budget_bytes;
  cudaError_t e = cudaSuccess;
  auto step = [&](cudaError_t r) { if (e == cudaSuccess) e = r; };
  step(cudaMalloc(&ctx->partials, (size_t)kInitialPartials * sizeof(double)));
  ctx->partials_cap = kInitialPartials;
  step(cudaMalloc(&ctx->scalars, 4 * sizeof(double)));
  step(cudaMallocHost(&ctx->host_scalars, 4 * sizeof(double)));
  step(cudaStreamCreateWithFlags(&ctx->s_in, cudaStreamNonBlocking));
  step(cudaStreamCreateWithFlags(&ctx->s_compute, cudaStreamNonBlocking));
  step(cudaStreamCreateWithFlags(&ctx->s_out, cudaStreamNonBlocking));
  step(cudaEventCreateWithFlags(&ctx->scalar_event, cudaEventDisableTiming));
  for (int i = 0; i < 3; ++i) {
    step(cudaEventCreateWithFlags(&ctx->ev_loaded[i], cudaEventDisableTiming));
    step(cudaEventCreateWithFlags(&ctx->ev_updated[i], cudaEventDisableTiming));
    step(cudaEventCreateWithFlags(&ctx->ev_free[i], cudaEventDisableTiming));
  }
  step(cudaEventCreate(&ctx->ev_begin));
  step(cudaEventCreate(&ctx->ev_norm_done));
  step(cudaEventCreate(&ctx->ev_end));
  step(cudaEventCreate(&ctx->ev_in_first));
  step(cudaEventCreate(&ctx->ev_in_last));
  step(cudaEventCreate(&ctx->ev_out_first));
  step(cudaEventCreate(&ctx->ev_out_last));
  if (e == cudaSuccess) {
    const double init[4] = {0.0, 0.0, 1.0, 0.0};
    step(cudaMemcpy(ctx->scalars, init, sizeof init, cudaMemcpyHostToDevice));
  }
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    slidedp_destroy(ctx);
    return SLIDEDP_ERR_CUDA;
  }
  *out = ctx;
  return SLIDEDP_OK;
}

int slidedp_destroy(slidedp_ctx* ctx) {
  if (!ctx) return SLIDEDP_OK;
  DeviceGuard guard(ctx->device);
  int rc = SLIDEDP_OK;
  cudaStream_t own[3] = {ctx->s_in, ctx->s_compute, ctx->s_out};
  for (cudaStream_t s : own)
    if (s) {
      int r = bounded_stream_wait(ctx, s, kWaitSeconds);
      if (r != SLIDEDP_OK && rc == SLIDEDP_OK) rc = r;
    }
  for (cudaStream_t s : own) if (s) cudaStreamDestroy(s);
  auto kill = [](cudaEvent_t ev) { if (ev) cudaEventDestroy(ev); };
  kill(ctx->scalar_event); kill(ctx->ev_begin); kill(ctx->ev_norm_done); kill(ctx->ev_end);
  kill(ctx->ev_in_first); kill(ctx->ev_in_last); kill(ctx->ev_out_first); kill(ctx->ev_out_last);
  for (int i = 0; i < 3; ++i) { kill(ctx->ev_loaded[i]); kill(ctx->ev_updated[i]); kill(ctx->ev_free[i]); }
  for (ChunkEvents& c : ctx->timing) { kill(c.k_start); kill(c.k_end); }
  if (ctx->slots) cudaFree(ctx->slots);
  if (ctx->partials) cudaFree(ctx->partials);
  if (ctx->scalars) cudaFree(ctx->scalars);
  if (ctx->host_scalars) cudaFreeHost(ctx->host_scalars);
  (void)cudaGetLastError();
  delete ctx;
  return rc;
}

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
                       static_cast<cudaStream_t>(cuda_stream));
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
  const unsigned blocks = (unsigned)((n + 8 * kReduceThreads - 1) / (8 * kReduceThreads));
  uint16_t* out = static_cast<uint16_t*>(out_bf16);
  const float inv = (float)inv_R;
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
  CU(cudaGetLastError());
  return SLIDEDP_OK;
}

int slidedp_stream_step(slidedp_ctx* ctx, const void* const* grads_bf16, int R, int64_t n_total,
                        float* host_master, float* host_m, float* host_v, void* param_bf16_out,
                        int64_t chunk_elems, int nbuf, int norm_ready,
                        const slidedp_hparams* hp, slidedp_stats* stats) {
  if (stats) {
    memset(stats, 0, sizeof *stats);
    stats->clip_coef = 1.0;
  }
  int64_t nchunks = 0;
  int rc = enqueue_stream_step(ctx, grads_bf16, R, n_total, host_master, host_m, host_v,
                               param_bf16_out, chunk_elems, nbuf, norm_ready, hp,
                               /*synchronous=*/true, stats != nullptr, &nchunks);
  if (rc != SLIDEDP_OK) return rc;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  rc = bounded_event_wait(ctx, ctx->ev_end, kWaitSeconds);
  if (rc != SLIDEDP_OK) return rc;
  rc = drain_streams(ctx);
  if (rc != SLIDEDP_OK) return rc;

  if (stats) {
    const bool clip = hp->max_norm > 0.0;
    float ms = 0.f;
    CU(cudaEventElapsedTime(&ms, ctx->ev_begin, ctx->ev_end));
    stats->ms_total = ms;
    CU(cudaEventElapsedTime(&ms, ctx->ev_begin, ctx->ev_norm_done));
    stats->ms_norm = (clip && !norm_ready) ? ms : 0.0;
    stats->chunks = nchunks;
    if (nchunks > 0) {
      const ChunkEvents& te = ctx->timing[0];
      const int64_t first_len = n_total < chunk_elems ? n_total : chunk_elems;
      CU(cudaEventElapsedTime(&ms, te.k_start, te.k_end));
      stats->ms_kernel = (double)ms * ((double)n_total / (double)first_len);
      CU(cudaEventElapsedTime(&ms, ctx->ev_in_first, ctx->ev_in_last));
      stats->ms_h2d = ms;
      CU(cudaEventElapsedTime(&ms, ctx->ev_out_first, ctx->ev_out_last));
      stats->ms_d2h = ms;
    }
    const double link_bytes = 12.0 * (double)n_total;
    if (stats->ms_h2d > 0) stats->gbs_h2d = link_bytes / (stats->ms_h2d * 1e6);
    if (stats->ms_d2h > 0) stats->gbs_d2h = link_bytes / (stats->ms_d2h * 1e6);
    if (clip) {
      stats->norm = ctx->host_scalars[1];
      stats->clip_coef = ctx->host_scalars[2];
      stats->nonfinite = ctx->host_scalars[3] != 0.0;
    }
  }
  return SLIDEDP_OK;
}

int slidedp_stream_step_async(slidedp_ctx* ctx, const void* const* grads_bf16, int R,
                              int64_t n_total, float* host_master, float* host_m, float* host_v,
                              void* param_bf16_out, int64_t chunk_elems, int nbuf, int norm_ready,
                              const slidedp_hparams* hp) {
  int64_t nchunks = 0;
  return enqueue_stream_step(ctx, grads_bf16, R, n_total, host_master, host_m, host_v,
                             param_bf16_out, chunk_elems, nbuf, norm_ready, hp,
                             /*synchronous=*/false, /*timed=*/false, &nchunks);
}

int slidedp_stream_wait(slidedp_ctx* ctx) {
  if (!ctx) return SLIDEDP_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  return drain_streams(ctx);
}

int slidedp_deliver_params(slidedp_ctx* ctx, const float* host_master, int64_t n_total,
                           void* param_bf16_out, int64_t chunk_elems, int nbuf,
                           slidedp_stats* stats) {
  if (!ctx || n_total < 0) return SLIDEDP_ERR_INVALID_ARG;
  if (nbuf < 2 || nbuf > 3 || chunk_elems <= 0 || (chunk_elems % 8) != 0)
    return SLIDEDP_ERR_INVALID_ARG;
  if (n_total > 0 && (!host_master || !param_bf16_out)) return SLIDEDP_ERR_INVALID_ARG;
  if (!aligned16(host_master) || !aligned16(param_bf16_out)) return SLIDEDP_ERR_MISALIGNED;
  if (stats) {
    memset(stats, 0, sizeof *stats);
    stats->clip_coef = 1.0;
  }
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  int rc = SLIDEDP_OK;
  if (n_total > 0) {
    bool pinned = false;
    rc = is_pinned(ctx, host_master, &pinned);
    if (rc != SLIDEDP_OK) return rc;
    if (!pinned) return SLIDEDP_ERR_NOT_PINNED;
  }
  const int64_t cap = chunk_elems < n_total ? chunk_elems : ((n_total + 7) / 8) * 8;
  const size_t need = (size_t)nbuf * (size_t)cap * sizeof(float);
  if (ctx->budget && need > ctx->budget) return SLIDEDP_ERR_BUDGET;
  // the slots are laid out differently here: let queued streaming steps finish first
  rc = drain_streams(ctx);
  if (rc != SLIDEDP_OK) return rc;
  ctx->ring_cap = 0;
  ctx->ring_nbuf = 0;
  rc = ensure_slots(ctx, need);
  if (rc != SLIDEDP_OK) return rc;
  const int64_t nchunks = n_total == 0 ? 0 : (n_total + chunk_elems - 1) / chunk_elems;
  uint16_t* pout = static_cast<uint16_t*>(param_bf16_out);

  CU(cudaEventRecord(ctx->ev_begin, ctx->s_compute));
  CU(cudaStreamWaitEvent(ctx->s_in, ctx->ev_begin, 0));
  for (int64_t c = 0; c < nchunks; ++c) {
    const int slot = (int)(c % nbuf);
    const int64_t off = c * chunk_elems;
    const int64_t len = n_total - off < chunk_elems ? n_total - off : chunk_elems;
    float* sw = ctx->slots + (size_t)slot * cap;
    // copy-in: the slot must have been read by the cast of chunk c - nbuf
    if (c >= nbuf) CU(cudaStreamWaitEvent(ctx->s_in, ctx->ev_free[slot], 0));
    if (stats && c == 0) CU(cudaEventRecord(ctx->ev_in_first, ctx->s_in));
    CU(cudaMemcpyAsync(sw, host_master + off, (size_t)len * sizeof(float),
                       cudaMemcpyHostToDevice, ctx->s_in));
    if (stats && c == nchunks - 1) CU(cudaEventRecord(ctx->ev_in_last, ctx->s_in));
    CU(cudaEventRecord(ctx->ev_loaded[slot], ctx->s_in));
    // cast
    CU(cudaStreamWaitEvent(ctx->s_compute, ctx->ev_loaded[slot], 0));
    const unsigned blocks = (unsigned)((len + 8 * kCastThreads - 1) / (8 * kCastThreads));
    cast_master_to_bf16_kernel<<<blocks, kCastThreads, 0, ctx->s_compute>>>(sw, len, pout + off);
    ctx->launches += 1;
    CU(cudaGetLastError());
    CU(cudaEventRecord(ctx->ev_free[slot], ctx->s_compute));
  }
  CU(cudaEventRecord(ctx->ev_end, ctx->s_compute));
  rc = bounded_event_wait(ctx, ctx->ev_end, kWaitSeconds);
  if (rc != SLIDEDP_OK) return rc;
  rc = bounded_stream_wait(ctx, ctx->s_in, kWaitSeconds);
  if (rc != SLIDEDP_OK) return rc;
  if (stats) {
    float ms = 0.f;
    CU(cudaEventElapsedTime(&ms, ctx->ev_begin, ctx->ev_end));
    stats->ms_total = ms;
    stats->chunks = nchunks;
    if (nchunks > 0) {
      CU(cudaEventElapsedTime(&ms, ctx->ev_in_first, ctx->ev_in_last));
      stats->ms_h2d = ms;
      if (ms > 0) stats->gbs_h2d = 4.0 * (double)n_total / (ms * 1e6);
    }
  }
  return SLIDEDP_OK;
}

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

int slidedp_link_probe(slidedp_ctx* ctx, void* host_a, void* host_b, void* dev_a, void* dev_b,
                       size_t bytes, size_t copy_bytes, int reps, double out4[4]) {
  if (!ctx || !host_a || !host_b || !dev_a || !dev_b || !out4 || bytes == 0 || copy_bytes == 0 ||
      reps < 1)
    return SLIDEDP_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  for (void* h : {host_a, host_b}) {
    bool pinned = false;
    int rc = is_pinned(ctx, h, &pinned);
    if (rc != SLIDEDP_OK) return rc;
    if (!pinned) return SLIDEDP_ERR_NOT_PINNED;
  }
  cudaEvent_t a0, a1, b0, b1;
  CU(cudaEventCreate(&a0)); CU(cudaEventCreate(&a1)); CU(cudaEventCreate(&b0)); CU(cudaEventCreate(&b1));
  int rc = SLIDEDP_OK;
  auto pieces = [&](bool h2d, cudaStream_t st) -> cudaError_t {
    for (size_t off = 0; off < bytes; off += copy_bytes) {
      const size_t len = bytes - off < copy_bytes ? bytes - off : copy_bytes;
      cudaError_t e = h2d ? cudaMemcpyAsync((char*)dev_a + off, (char*)host_a + off, len,
                                            cudaMemcpyHostToDevice, st)
                          : cudaMemcpyAsync((char*)host_b + off, (char*)dev_b + off, len,
                                            cudaMemcpyDeviceToHost, st);
      if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
  };
  // mode 0: H2D alone; 1: D2H alone; 2: both at once
  for (int mode = 0; mode < 3 && rc == SLIDEDP_OK; ++mode) {
    double best_in = 0.0, best_out = 0.0;
    for (int rep = 0; rep < reps + 1 && rc == SLIDEDP_OK; ++rep) {  // first pass warms up
      cudaError_t e = cudaSuccess;
      if (mode != 1) {
        e = cudaEventRecord(a0, ctx->s_in);
        if (e == cudaSuccess) e = pieces(true, ctx->s_in);
        if (e == cudaSuccess) e = cudaEventRecord(a1, ctx->s_in);
      }
      if (e == cudaSuccess && mode != 0) {
        e = cudaEventRecord(b0, ctx->s_out);
        if (e == cudaSuccess) e = pieces(false, ctx->s_out);
        if (e == cudaSuccess) e = cudaEventRecord(b1, ctx->s_out);
      }
      if (e != cudaSuccess) { rc = cuda_fail(ctx, e); break; }
      if (mode != 1) rc = bounded_event_wait(ctx, a1, kWaitSeconds);
      if (rc == SLIDEDP_OK && mode != 0) rc = bounded_event_wait(ctx, b1, kWaitSeconds);
      if (rc != SLIDEDP_OK) break;
      float ms = 0.f;
      if (mode != 1 && cudaEventElapsedTime(&ms, a0, a1) == cudaSuccess && rep > 0 && ms > 0) {
        const double g = (double)bytes / (ms * 1e6);
        if (g > best_in) best_in = g;
      }
      if (mode != 0 && cudaEventElapsedTime(&ms, b0, b1) == cudaSuccess && rep > 0 && ms > 0) {
        const double g = (double)bytes / (ms * 1e6);
        if (g > best_out) best_out = g;
      }
    }
    if (mode == 0) out4[0] = best_in;
    if (mode == 1) out4[1] = best_out;
    if (mode == 2) { out4[2] = best_in; out4[3] = best_out; }
  }
  cudaEventDestroy(a0); cudaEventDestroy(a1); cudaEventDestroy(b0); cudaEventDestroy(b1);
  return rc;
}

// ---- norm without allocation ---------------------------------------------------------------
//
// Scratch for callers that cannot allocate: the per-tile sums live in an array that is part
// of the library's device image. In HOST code the name `noalloc_tile_sums` is only a handle
// for the symbol, not a device address; the address each device gave it is looked up once
// per device with cudaGetSymbolAddress (with that device current) and cached here.
constexpr int64_t kNoallocMaxTiles = SLIDEDP_NOALLOC_MAX_ELEMS / kNormTile;   // 65536
static __device__ __align__(256) double noalloc_tile_sums[kNoallocMaxTiles];

constexpr int kNoallocMaxDevices = 64;
static double* noalloc_scratch_addr[kNoallocMaxDevices];   // zero-initialised: not looked up yet

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
  double* scratch = noalloc_scratch_addr[dev];
  if (!scratch) {
    // one-time set-up for this device (current right now): resolve the symbol's address
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, noalloc_tile_sums) != cudaSuccess || !p) {
      (void)cudaGetLastError();
      return SLIDEDP_ERR_CUDA;
    }
    scratch = static_cast<double*>(p);
    noalloc_scratch_addr[dev] = scratch;
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
