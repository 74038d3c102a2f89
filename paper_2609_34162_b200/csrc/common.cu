// libslidedp: helpers shared by every entry point (bounded waits, argument checks, the
// per-step constants prepared in double on the host).
#include "internal.h"

#include <math.h>
#include <time.h>

namespace slidedp {
namespace host {

int cuda_fail(slidedp_ctx* ctx, cudaError_t e) {
  if (ctx) ctx->last_cuda = (int)e;
  (void)cudaGetLastError();
  return SLIDEDP_ERR_CUDA;
}

static double now_seconds() {
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
  // eps, lr, weight decay and 1/R must be finite numbers (NaN fails every comparison below)
  const double big = 1.7976931348623157e308;
  if (!(hp->eps >= 0.0 && hp->eps <= big)) return SLIDEDP_ERR_INVALID_ARG;
  if (!(hp->lr >= -big && hp->lr <= big)) return SLIDEDP_ERR_INVALID_ARG;
  if (!(hp->weight_decay >= -big && hp->weight_decay <= big)) return SLIDEDP_ERR_INVALID_ARG;
  if (!(hp->inv_R >= -big && hp->inv_R <= big)) return SLIDEDP_ERR_INVALID_ARG;
  if (hp->max_norm != hp->max_norm) return SLIDEDP_ERR_INVALID_ARG;
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

}  // namespace host
}  // namespace slidedp
