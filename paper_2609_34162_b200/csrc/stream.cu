// libslidedp: the host-resident path: the slot ring over three streams, parameter delivery and the
// host-link probe.
// See include/slidedp.h for the contract of every entry point.
#include "internal.h"
#include "cast_kernel.cuh"

#include <string.h>

using namespace slidedp;
using namespace slidedp::host;

namespace {

// Which timing events an enqueue records: the first chunk's copies, the last chunk's copies, one
// (middle) chunk's kernel.
constexpr int kMarkFirst = 1, kMarkLast = 2, kMarkKernel = 4;


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
    int rc = bounded_stream_wait(ctx, st, ctx->wait_seconds);
    if (rc != SLIDEDP_OK) return rc;
  }
  ctx->ring_busy = false;
  return SLIDEDP_OK;
}

// After an entry point failed midway through enqueuing: wait (bounded) for whatever it did queue,
// so that no copy still touches the caller's memory once the error is returned, and restart the
// slot ring from a clean state. The original status is what the caller gets; if even the drain
// times out the ring stays marked busy and a later slidedp_stream_wait finishes the job.
int abandon_queued(slidedp_ctx* ctx, int status) {
  const int64_t keep = ctx->fail_countdown;
  ctx->fail_countdown = 0;                 // the clean-up itself is never a fault point
  const int last = ctx->last_cuda;
  if (drain_streams(ctx) == SLIDEDP_OK) {
    ctx->ring_next = 0;
    ctx->ring_cap = 0;                     // forces a fresh layout (and event state) next time
    ctx->ring_nbuf = 0;
  }
  ctx->last_cuda = last;
  ctx->fail_countdown = keep;
  return status;
}

// Validates and enqueues one host-resident step on the context's streams. The slot ring
// carries over from call to call (slot index = running chunk count mod nbuf, every copy-in
// waits for the slot's last copy-out), so consecutive calls overlap like the chunks of one
// call; a call with another slot layout first drains what is queued.
int enqueue_chunks(slidedp_ctx* ctx, const GradPtrs& gp, int R, int64_t n_total, float* host_master,
                   float* host_m, float* host_v, void* param_bf16_out, int64_t chunk_elems,
                   int nbuf, int64_t cap, int norm_ready, const slidedp_hparams* hp,
                   bool synchronous, int marks, int64_t nchunks);

int enqueue_stream_step(slidedp_ctx* ctx, const void* const* grads_bf16, int R, int64_t n_total,
                        float* host_master, float* host_m, float* host_v, void* param_bf16_out,
                        int64_t chunk_elems, int nbuf, int norm_ready, const slidedp_hparams* hp,
                        bool synchronous, int marks, int64_t* nchunks_out, int64_t cap_hint = 0) {
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
  // (a multi-layer call passes the slot capacity of its largest layer, so that small layers do
  // not force a new layout and a drain in the middle of the step)
  const int64_t own_cap = chunk_elems < n_total ? chunk_elems : ((n_total + 7) / 8) * 8;
  const int64_t cap = cap_hint > own_cap ? cap_hint : own_cap;
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
  if (marks & kMarkKernel) {
    while (ctx->timing.empty() && nchunks > 0) {
      ChunkEvents c;
      CU(cudaEventCreate(&c.k_start));
      CU(cudaEventCreate(&c.k_end));
      ctx->timing.push_back(c);
    }
  }

  ctx->ring_busy = true;
  rc = enqueue_chunks(ctx, gp, R, n_total, host_master, host_m, host_v, param_bf16_out,
                      chunk_elems, nbuf, cap, norm_ready, hp, synchronous, marks, nchunks);
  if (rc != SLIDEDP_OK) return abandon_queued(ctx, rc);
  return SLIDEDP_OK;
}

// The enqueue proper (everything after the checks and the slot allocation). Any failure in
// here leaves work queued; the caller cleans up with abandon_queued.
int enqueue_chunks(slidedp_ctx* ctx, const GradPtrs& gp, int R, int64_t n_total, float* host_master,
                   float* host_m, float* host_v, void* param_bf16_out, int64_t chunk_elems,
                   int nbuf, int64_t cap, int norm_ready, const slidedp_hparams* hp,
                   bool synchronous, int marks, int64_t nchunks) {
  const bool clip = hp->max_norm > 0.0;
  int rc = SLIDEDP_OK;
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
    ChunkEvents* te = ((marks & kMarkKernel) && c == (nchunks - 1) / 2) ? &ctx->timing[0] : nullptr;
    // copy-in: the slot must have been drained by the copy-out that last used it (a no-op
    // for an event that was never recorded or has completed)
    CU(cudaStreamWaitEvent(ctx->s_in, ctx->ev_free[slot], 0));
    if ((marks & kMarkFirst) && c == 0) CU(cudaEventRecord(ctx->ev_in_first, ctx->s_in));
    CU(cudaMemcpyAsync(sw, host_master + off, bytes, cudaMemcpyHostToDevice, ctx->s_in));
    CU(cudaMemcpyAsync(sm, host_m + off, bytes, cudaMemcpyHostToDevice, ctx->s_in));
    CU(cudaMemcpyAsync(sv, host_v + off, bytes, cudaMemcpyHostToDevice, ctx->s_in));
    if ((marks & kMarkLast) && c == nchunks - 1) CU(cudaEventRecord(ctx->ev_in_last, ctx->s_in));
    CU(cudaEventRecord(ctx->ev_loaded[slot], ctx->s_in));
    // update
    CU(cudaStreamWaitEvent(ctx->s_compute, ctx->ev_loaded[slot], 0));
    if (te) CU(cudaEventRecord(te->k_start, ctx->s_compute));
    GradPtrs gc = gp;
    for (int r = 0; r < R; ++r) gc.p[r] = gp.p[r] + off;
    rc = launch_update(ctx, gc, R, len, sw, sm, sv, pout + off, k, coef, ctx->s_compute,
                       /*early=*/false);
    if (rc != SLIDEDP_OK) return rc;
    if (te) CU(cudaEventRecord(te->k_end, ctx->s_compute));
    CU(cudaEventRecord(ctx->ev_updated[slot], ctx->s_compute));
    // copy-out
    CU(cudaStreamWaitEvent(ctx->s_out, ctx->ev_updated[slot], 0));
    if ((marks & kMarkFirst) && c == 0) CU(cudaEventRecord(ctx->ev_out_first, ctx->s_out));
    CU(cudaMemcpyAsync(host_master + off, sw, bytes, cudaMemcpyDeviceToHost, ctx->s_out));
    CU(cudaMemcpyAsync(host_m + off, sm, bytes, cudaMemcpyDeviceToHost, ctx->s_out));
    CU(cudaMemcpyAsync(host_v + off, sv, bytes, cudaMemcpyDeviceToHost, ctx->s_out));
    if ((marks & kMarkLast) && c == nchunks - 1) CU(cudaEventRecord(ctx->ev_out_last, ctx->s_out));
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

extern "C" {

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
                               /*synchronous=*/true, stats ? (kMarkFirst | kMarkLast | kMarkKernel) : 0, &nchunks);
  if (rc != SLIDEDP_OK) return rc;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  rc = bounded_event_wait(ctx, ctx->ev_end, ctx->wait_seconds);
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
      // the timed kernel is the middle chunk's (warm, with copies running on both sides)
      const int64_t mid_off = ((nchunks - 1) / 2) * chunk_elems;
      const int64_t mid_len = n_total - mid_off < chunk_elems ? n_total - mid_off : chunk_elems;
      CU(cudaEventElapsedTime(&ms, te.k_start, te.k_end));
      stats->ms_kernel = (double)ms * ((double)n_total / (double)mid_len);
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
                             /*synchronous=*/false, /*marks=*/0, &nchunks);
}

int slidedp_stream_layers(slidedp_ctx* ctx, const slidedp_layer* layers, int num_layers, int R,
                          int64_t chunk_elems, int nbuf, const slidedp_hparams* hp,
                          slidedp_stats* stats) {
  if (stats) {
    memset(stats, 0, sizeof *stats);
    stats->clip_coef = 1.0;
  }
  if (!ctx || num_layers < 0 || (num_layers > 0 && !layers)) return SLIDEDP_ERR_INVALID_ARG;
  int rc = check_hparams(hp);
  if (rc != SLIDEDP_OK) return rc;
  const bool clip = hp->max_norm > 0.0;
  // every layer's arguments are checked before anything is queued
  int first = -1, last = -1;
  for (int l = 0; l < num_layers; ++l) {
    const slidedp_layer& L = layers[l];
    GradPtrs gp;
    if (L.n < 0) return SLIDEDP_ERR_INVALID_ARG;
    rc = check_grads(L.grads_bf16, R, &gp);
    if (rc != SLIDEDP_OK) return rc;
    if (L.n > 0 && (!L.host_master || !L.host_m || !L.host_v || !L.param_bf16_out))
      return SLIDEDP_ERR_INVALID_ARG;
    if (!aligned16(L.host_master) || !aligned16(L.host_m) || !aligned16(L.host_v) ||
        !aligned16(L.param_bf16_out))
      return SLIDEDP_ERR_MISALIGNED;
    if (L.n > 0) { if (first < 0) first = l; last = l; }
  }
  if (nbuf < 2 || nbuf > 3 || chunk_elems <= 0 || (chunk_elems % 8) != 0)
    return SLIDEDP_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  for (int l = 0; l < num_layers; ++l) {
    if (layers[l].n == 0) continue;
    for (const float* h : {layers[l].host_master, layers[l].host_m, layers[l].host_v}) {
      bool pinned = false;
      rc = is_pinned(ctx, h, &pinned);
      if (rc != SLIDEDP_OK) return rc;
      if (!pinned) return SLIDEDP_ERR_NOT_PINNED;
    }
  }
  int64_t biggest = 0;
  for (int l = 0; l < num_layers; ++l) if (layers[l].n > biggest) biggest = layers[l].n;
  const int64_t cap_all = chunk_elems < biggest ? chunk_elems : ((biggest + 7) / 8) * 8;
  if (ctx->budget && (size_t)nbuf * 3 * (size_t)cap_all * sizeof(float) > ctx->budget)
    return SLIDEDP_ERR_BUDGET;

  int64_t chunks = 0;
  ctx->ring_busy = true;
  auto enqueue = [&]() -> int {
    CU(cudaEventRecord(ctx->ev_begin, ctx->s_compute));
    CU(cudaStreamWaitEvent(ctx->s_in, ctx->ev_begin, 0));
    CU(cudaStreamWaitEvent(ctx->s_out, ctx->ev_begin, 0));
    if (clip) {
      // the norm covers every layer of the step before any update (tile sums in layer order)
      for (int l = 0; l < num_layers; ++l) {
        GradPtrs gp;
        check_grads(layers[l].grads_bf16, R, &gp);
        int r2 = norm_chunk(ctx, gp, R, layers[l].n, hp->inv_R, l == 0, ctx->s_compute);
        if (r2 != SLIDEDP_OK) return r2;
      }
      if (num_layers == 0) ctx->partials_used = 0;
      int r2 = norm_finish(ctx, hp->max_norm, ctx->s_compute);
      if (r2 != SLIDEDP_OK) return r2;
    }
    CU(cudaEventRecord(ctx->ev_norm_done, ctx->s_compute));
    for (int l = 0; l < num_layers; ++l) {
      const slidedp_layer& L = layers[l];
      if (L.n == 0) continue;                  // nothing to stream (and no slot re-layout for it)
      int64_t nchunks = 0;
      const int marks = stats ? ((l == first ? kMarkFirst : 0) | (l == last ? kMarkLast : 0)) : 0;
      int r2 = enqueue_stream_step(ctx, L.grads_bf16, R, L.n, L.host_master, L.host_m, L.host_v,
                                   L.param_bf16_out, chunk_elems, nbuf, /*norm_ready=*/1, hp,
                                   /*synchronous=*/false, marks, &nchunks, cap_all);
      if (r2 != SLIDEDP_OK) return r2;
      chunks += nchunks;
    }
    CU(cudaStreamWaitEvent(ctx->s_out, ctx->ev_norm_done, 0));
    if (clip) CU(cudaMemcpyAsync(ctx->host_scalars, ctx->scalars, 4 * sizeof(double),
                                 cudaMemcpyDeviceToHost, ctx->s_out));
    CU(cudaEventRecord(ctx->ev_end, ctx->s_out));
    return SLIDEDP_OK;
  };
  rc = enqueue();
  if (rc != SLIDEDP_OK) return abandon_queued(ctx, rc);
  rc = bounded_event_wait(ctx, ctx->ev_end, ctx->wait_seconds);
  if (rc != SLIDEDP_OK) return rc;
  rc = drain_streams(ctx);
  if (rc != SLIDEDP_OK) return rc;
  if (stats) {
    float ms = 0.f;
    int64_t total = 0;
    for (int l = 0; l < num_layers; ++l) total += layers[l].n;
    CU(cudaEventElapsedTime(&ms, ctx->ev_begin, ctx->ev_end));
    stats->ms_total = ms;
    CU(cudaEventElapsedTime(&ms, ctx->ev_begin, ctx->ev_norm_done));
    stats->ms_norm = clip ? ms : 0.0;
    stats->chunks = chunks;
    if (first >= 0) {
      CU(cudaEventElapsedTime(&ms, ctx->ev_in_first, ctx->ev_in_last));
      stats->ms_h2d = ms;
      CU(cudaEventElapsedTime(&ms, ctx->ev_out_first, ctx->ev_out_last));
      stats->ms_d2h = ms;
      if (stats->ms_h2d > 0) stats->gbs_h2d = 12.0 * (double)total / (stats->ms_h2d * 1e6);
      if (stats->ms_d2h > 0) stats->gbs_d2h = 12.0 * (double)total / (stats->ms_d2h * 1e6);
    }
    if (clip) {
      stats->norm = ctx->host_scalars[1];
      stats->clip_coef = ctx->host_scalars[2];
      stats->nonfinite = ctx->host_scalars[3] != 0.0;
    }
  }
  return SLIDEDP_OK;
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

  ctx->ring_busy = true;
  auto enqueue = [&]() -> int {
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
    FAULT_POINT();
    cast_master_to_bf16_kernel<<<blocks, kCastThreads, 0, ctx->s_compute>>>(sw, len, pout + off);
    ctx->launches += 1;
    CU_AFTER_LAUNCH();
    CU(cudaEventRecord(ctx->ev_free[slot], ctx->s_compute));
  }
  CU(cudaEventRecord(ctx->ev_end, ctx->s_compute));
  return SLIDEDP_OK;
  };
  rc = enqueue();
  if (rc != SLIDEDP_OK) return abandon_queued(ctx, rc);
  rc = bounded_event_wait(ctx, ctx->ev_end, ctx->wait_seconds);
  if (rc != SLIDEDP_OK) return rc;
  rc = bounded_stream_wait(ctx, ctx->s_in, ctx->wait_seconds);
  if (rc != SLIDEDP_OK) return rc;
  ctx->ring_busy = false;
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
  cudaEvent_t a0 = nullptr, a1 = nullptr, b0 = nullptr, b1 = nullptr;
  auto destroy_events = [&]() {
    for (cudaEvent_t ev : {a0, a1, b0, b1}) if (ev) cudaEventDestroy(ev);
  };
  for (cudaEvent_t* ev : {&a0, &a1, &b0, &b1}) {
    const cudaError_t e = injected_failure(ctx) ? cudaErrorUnknown : cudaEventCreate(ev);
    if (e != cudaSuccess) { destroy_events(); return cuda_fail(ctx, e); }
  }
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
      cudaError_t e = injected_failure(ctx) ? cudaErrorUnknown : cudaSuccess;
      if (e == cudaSuccess && mode != 1) {
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
      if (mode != 1) rc = bounded_event_wait(ctx, a1, ctx->wait_seconds);
      if (rc == SLIDEDP_OK && mode != 0) rc = bounded_event_wait(ctx, b1, ctx->wait_seconds);
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
  if (rc != SLIDEDP_OK) {
    // leave nothing running on the caller's buffers (bounded; the status stays the first one)
    const int last = ctx->last_cuda;
    bounded_stream_wait(ctx, ctx->s_in, ctx->wait_seconds);
    bounded_stream_wait(ctx, ctx->s_out, ctx->wait_seconds);
    ctx->last_cuda = last;
  }
  destroy_events();
  return rc;
}

}  // extern "C"
