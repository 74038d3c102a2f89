// Internal declarations shared by the translation units of libslidedp (not installed).
#pragma once

#include "slidedp.h"

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "types.h"

namespace slidedp {
namespace host {

constexpr double kDefaultWaitSeconds = 300.0;  // default bound on every host-side wait
constexpr int64_t kInitialPartials = 1 << 20;  // 8 MB: 2^20 tiles = 17 G parameters


// Timing events of ONE kernel (the middle chunk's). Per-chunk timing events, on the copy
// streams or the compute stream, sit on the chunk's H2D -> kernel -> D2H chain and cost
// several percent of link bandwidth at 16 MiB chunks, so a step records a fixed handful.
struct ChunkEvents {
  cudaEvent_t k_start, k_end;
};

// A peer process's allocation mapped into this process (slidedp_ipc_open).
struct IpcMapping {
  unsigned char opaque[64];
  char* base;
  size_t bytes;
  int refs;
};

}  // namespace host
}  // namespace slidedp

struct slidedp_ctx {
  int device = 0;
  size_t budget = 0;
  int last_cuda = 0;
  int64_t launches = 0;
  double wait_seconds = slidedp::host::kDefaultWaitSeconds;   // slidedp_set_wait_seconds
  // host-side fault injection (slidedp_test_fail_nth_call): the countdown-th guarded runtime
  // call from now is not issued and reports cudaErrorUnknown; <= 0: off
  int64_t fail_countdown = 0;
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
  std::vector<slidedp::host::ChunkEvents> timing;  // grown on demand, reused
  std::vector<slidedp::host::IpcMapping> ipc;      // peer allocations mapped by slidedp_ipc_open
};

namespace slidedp {
namespace host {

// Makes `dev` current for the lifetime of the guard and restores the previous device.
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

int cuda_fail(slidedp_ctx* ctx, cudaError_t e);

// True when the host-side fault injection of `ctx` says that the next guarded call must fail.
inline bool injected_failure(slidedp_ctx* ctx) {
  return ctx && ctx->fail_countdown > 0 && --ctx->fail_countdown == 0;
}

// Returns SLIDEDP_ERR_CUDA (recording the error in ctx) when a runtime call fails. Under fault
// injection the call is NOT issued and counts as failed with cudaErrorUnknown.
#define CU(call)                                                                              \
  do {                                                                                        \
    cudaError_t e_ = slidedp::host::injected_failure(ctx) ? cudaErrorUnknown : (call);        \
    if (e_ != cudaSuccess) return slidedp::host::cuda_fail(ctx, e_);                          \
  } while (0)
// A guarded point with no call of its own: placed before a kernel launch, so that an injected
// failure stops the entry point before the kernel could change any state.
#define FAULT_POINT() CU(cudaSuccess)
// The check after a kernel launch: never injected (the kernel has been queued already).
#define CU_AFTER_LAUNCH()                                                                     \
  do {                                                                                        \
    cudaError_t e_ = cudaGetLastError();                                                      \
    if (e_ != cudaSuccess) return slidedp::host::cuda_fail(ctx, e_);                          \
  } while (0)

// Bounded host-side waits: polls, never an unbounded block inside the driver.
int bounded_event_wait(slidedp_ctx* ctx, cudaEvent_t ev, double seconds);
int bounded_stream_wait(slidedp_ctx* ctx, cudaStream_t s, double seconds);

// Argument checks and per-step constants.
bool aligned16(const void* p);
int check_grads(const void* const* grads, int R, GradPtrs* out);
int check_hparams(const slidedp_hparams* hp);
UpdateConsts make_consts(const slidedp_hparams* hp);

// Kernel launchers (update.cu), used by the device-resident entry points and the slot ring.
int launch_update(slidedp_ctx* ctx, const GradPtrs& gp, int R, int64_t n, float* w, float* m,
                  float* v, uint16_t* p, const UpdateConsts& k, const double* coef,
                  cudaStream_t st, bool early);
void launch_sumsq(const GradPtrs& gp, int R, int64_t n, float inv_R, double* tile_sums,
                  unsigned blocks, cudaStream_t st);
int norm_chunk(slidedp_ctx* ctx, const GradPtrs& gp, int R, int64_t n, double inv_R,
               int first_chunk, cudaStream_t st);
int norm_finish(slidedp_ctx* ctx, double max_norm, cudaStream_t st);

}  // namespace host
}  // namespace slidedp
