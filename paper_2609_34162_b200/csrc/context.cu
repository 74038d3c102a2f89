// libslidedp: context life cycle and the entry points that need no GPU work.
// See include/slidedp.h for the contract of every entry point.
#include "internal.h"

#include <new>

using namespace slidedp;
using namespace slidedp::host;

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

int slidedp_set_wait_seconds(slidedp_ctx* ctx, double seconds) {
  if (!ctx || !(seconds > 0.0) || seconds > 86400.0) return SLIDEDP_ERR_INVALID_ARG;
  ctx->wait_seconds = seconds;
  return SLIDEDP_OK;
}

int slidedp_test_fail_nth_call(slidedp_ctx* ctx, int64_t nth) {
  if (!ctx) return SLIDEDP_ERR_INVALID_ARG;
  ctx->fail_countdown = nth > 0 ? nth : 0;
  return SLIDEDP_OK;
}

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
  ctx->fail_countdown = 0;
  int rc = SLIDEDP_OK;
  cudaStream_t own[3] = {ctx->s_in, ctx->s_compute, ctx->s_out};
  for (cudaStream_t s : own)
    if (s) {
      int r = bounded_stream_wait(ctx, s, ctx->wait_seconds);
      if (r != SLIDEDP_OK && rc == SLIDEDP_OK) rc = r;
    }
  for (cudaStream_t s : own) if (s) cudaStreamDestroy(s);
  auto kill = [](cudaEvent_t ev) { if (ev) cudaEventDestroy(ev); };
  kill(ctx->scalar_event); kill(ctx->ev_begin); kill(ctx->ev_norm_done); kill(ctx->ev_end);
  kill(ctx->ev_in_first); kill(ctx->ev_in_last); kill(ctx->ev_out_first); kill(ctx->ev_out_last);
  for (int i = 0; i < 3; ++i) { kill(ctx->ev_loaded[i]); kill(ctx->ev_updated[i]); kill(ctx->ev_free[i]); }
  for (ChunkEvents& c : ctx->timing) { kill(c.k_start); kill(c.k_end); }
  for (slidedp::host::IpcMapping& m : ctx->ipc) cudaIpcCloseMemHandle(m.base);
  ctx->ipc.clear();
  if (ctx->slots) cudaFree(ctx->slots);
  if (ctx->partials) cudaFree(ctx->partials);
  if (ctx->scalars) cudaFree(ctx->scalars);
  if (ctx->host_scalars) cudaFreeHost(ctx->host_scalars);
  (void)cudaGetLastError();
  delete ctx;
  return rc;
}

}  // extern "C"
