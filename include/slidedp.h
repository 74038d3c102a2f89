/*
 * slidedp.h -- C ABI of libslidedp: the data-parallel hot path of SlideDP's synchronous
 * step on one B200 (sm_100a).
 *
 * For each flat parameter chunk the library sums R rank-gradient BF16 buffers in a fixed
 * rank order with FP32 accumulation, scales by 1/R, optionally applies a deterministic
 * global-L2-norm clip, runs AdamW over the single authoritative FP32 master / m / v state
 * and emits the BF16 parameter copy for the next delivery. The paper runs this step on
 * host CPUs (Sec. 3.2 "Gradient return", Sec. 3.3 Reduce -> D2H -> Adam); here it is one
 * fused streaming kernel per chunk, with the state either resident in HBM or resident in
 * pinned host memory and streamed through a small ring of device slots.
 *
 * State per parameter (paper Sec. 2.1, Table 1): BF16 parameter 2 B, BF16 gradient 2 B,
 * FP32 master 4 B, FP32 m 4 B, FP32 v 4 B = 16 B.
 *
 * Conventions
 *  - Every function returns SLIDEDP_OK (0) or a negative slidedp_status; nothing throws,
 *    aborts or exits. slidedp_strerror() names a status; slidedp_last_cuda_error() gives
 *    the cudaError_t behind SLIDEDP_ERR_CUDA.
 *  - The caller owns every data buffer and passes raw pointers; "device" pointers are
 *    cudaMalloc'd (or torch) addresses on the context's device, "host" pointers are plain
 *    host addresses, "pinned" pointers are page-locked host addresses. The library
 *    allocates only inside slidedp_ctx (norm partials, scalars, streaming slots, streams,
 *    events) and keeps nothing else between calls.
 *  - BF16 buffers are arrays of 16-bit patterns. Every gradient / state / output base
 *    pointer must be 16-byte aligned (SLIDEDP_ERR_MISALIGNED otherwise); n may be any
 *    non-negative count (a ragged tail is handled element by element; n = 0 is a no-op).
 *  - cuda_stream arguments are cudaStream_t handles passed as void* (NULL = legacy
 *    default stream). Device-resident calls only enqueue work on that stream and return.
 *  - master / m / v are updated in place; gradients are read-only; param_bf16_out must
 *    not overlap any other argument.
 *  - A context is not thread-safe: use one per host thread, or serialise the calls on it. All
 *    device pointers passed with a context must live on that context's device.
 */
#ifndef SLIDEDP_H
#define SLIDEDP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SLIDEDP_MAX_RANKS 16

#if defined(__GNUC__)
#define SLIDEDP_API __attribute__((visibility("default")))
#else
#define SLIDEDP_API
#endif

typedef enum {
  SLIDEDP_OK = 0,
  SLIDEDP_ERR_INVALID_ARG = -1, /* null pointer, R outside 1..16, n < 0, step < 1, beta outside [0,1),
                                   non-finite lr / eps / weight decay / 1/R, ...                        */
  SLIDEDP_ERR_MISALIGNED = -2,  /* a base pointer is not 16-byte aligned                               */
  SLIDEDP_ERR_BUDGET = -3,      /* the streaming slots would not fit the context's GPU memory budget   */
  SLIDEDP_ERR_NOT_PINNED = -4,  /* a host state pointer of slidedp_stream_step is not page-locked      */
  SLIDEDP_ERR_CUDA = -5,        /* a CUDA runtime call failed; see slidedp_last_cuda_error()            */
  SLIDEDP_ERR_TIMEOUT = -6,     /* a bounded wait for queued work expired                               */
  SLIDEDP_ERR_NO_NORM = -7,     /* clipping requested but no finished norm is held by the context      */
  SLIDEDP_ERR_TOO_LARGE = -8    /* n exceeds the fixed capacity of slidedp_grad_norm_noalloc            */
} slidedp_status;

typedef struct slidedp_ctx slidedp_ctx;

/* Hyper-parameters of one update. All doubles: float-typed constants alone (0.9f, 1-0.9f)
 * already break a 1e-6 relative tolerance on m. */
typedef struct {
  double lr, beta1, beta2, eps, weight_decay;
  double inv_R;    /* the FP32 rank sum is multiplied by (float)inv_R                        */
  double max_norm; /* > 0: scale the averaged gradient by the context's clip coefficient      */
  int64_t step;    /* 1-based index of the update being performed (bias correction uses it)  */
} slidedp_hparams;

/* What slidedp_stream_step measured (CUDA events; times in ms, rates in GB/s = 1e9 B/s). */
typedef struct {
  double norm, clip_coef; /* the step's global norm and coefficient (0 and 1 if clipping off) */
  double ms_total;        /* first enqueue to last D2H complete                                */
  double ms_norm;         /* the norm pass when it ran inside the call                         */
  double ms_h2d;          /* copy-in lane: start of its first copy to end of its last copy    */
  double ms_kernel;       /* update kernels: the middle chunk's kernel time scaled to n_total  */
  double ms_d2h;          /* copy-out lane: start of its first copy to end of its last copy   */
  double gbs_h2d, gbs_d2h;/* bytes moved / that lane's span                                    */
  int64_t chunks;
  int32_t nonfinite;      /* 1 if the norm was inf or NaN                                      */
  int32_t reserved;
} slidedp_stats;

/* ---- context ------------------------------------------------------------------------ */

/* Creates a context on `device`. gpu_budget_bytes caps what slidedp_stream_step may allocate
 * for its slots (0 = no cap). Allocates the norm workspace (a few MB) and three streams. */
SLIDEDP_API int slidedp_create(slidedp_ctx** out, int device, size_t gpu_budget_bytes);
/* Waits (bounded) for the context's own streams, frees everything. NULL is a no-op. */
SLIDEDP_API int slidedp_destroy(slidedp_ctx* ctx);

/* ---- failure handling ------------------------------------------------------------------
 *
 * (Paper Sec. 3.3 "Completion and buffer reuse" is the only related passage: a buffer is reused
 * only after the work that reads it completed, and a stalled consumer exerts backpressure. The
 * library adds a bound on every host-side wait so that a stalled device never blocks a caller
 * for ever.)
 *
 * Every host-side wait of the library is a poll with a deadline of `wait_seconds` (default 300;
 * slidedp_set_wait_seconds changes it for this context, 0 < seconds <= 86400). When a wait runs
 * out the entry point returns SLIDEDP_ERR_TIMEOUT. Nothing is cancelled: the queued copies and
 * kernels keep running, the caller's buffers must stay valid, and a later slidedp_stream_wait
 * (after raising the bound or simply later) returns SLIDEDP_OK once they are done, after which
 * the context is as usable as before and the step's results are complete.
 *
 * SLIDEDP_ERR_CUDA from a streaming entry point (slidedp_stream_step, _async, slidedp_stream_layers,
 * slidedp_deliver_params, slidedp_link_probe) means a runtime call failed midway through enqueuing. Before returning, the
 * entry point waits (bounded) for the part it had already queued, so no copy touches the
 * caller's memory after the return, and restarts its slot ring; the context stays usable. The
 * host state is then partly updated: chunks queued before the failure carry the new values, the
 * others the old ones, so the caller must restore its own copy of the step's inputs before
 * retrying. From a device-resident entry point SLIDEDP_ERR_CUDA from a failed launch means the
 * kernel was not queued and the state is untouched.
 *
 * slidedp_test_fail_nth_call is a HOST-SIDE test hook (nothing on the GPU is made to fail): the
 * nth guarded CUDA runtime call (or kernel launch) that the context issues from now on is not
 * issued at all and is reported as failed with cudaErrorUnknown, so that every error path above
 * can be exercised; nth <= 0 switches the hook off. The countdown stops at the failure.
 */
SLIDEDP_API int slidedp_set_wait_seconds(slidedp_ctx* ctx, double seconds);
SLIDEDP_API int slidedp_test_fail_nth_call(slidedp_ctx* ctx, int64_t nth);
SLIDEDP_API const char* slidedp_strerror(int status);
SLIDEDP_API int slidedp_last_cuda_error(const slidedp_ctx* ctx);

/* Paper Sec. 2.1 / Table 1: bytes of persistent state for n parameters = 16 n. */
SLIDEDP_API size_t slidedp_state_bytes(int64_t n);

/* ---- global L2 norm of the averaged gradient (clipping; not part of the paper) --------
 *
 * slidedp_grad_norm adds, for one chunk, the sum over i of gbar_i^2 to the context's
 * accumulator, where gbar_i = fl32(fl32-sum over ranks in order 0..R-1 of g_r[i]) * (float)inv_R
 * as in Sec. 3.2 "Gradient return" (sum, then average). Squares and sums are FP64. The chunk
 * is cut into fixed tiles of 16384 elements; each tile is summed by a fixed tree into its
 * own slot, so the result does not depend on the launch shape, and a step cut into chunks
 * at multiples of 16384 elements gives bit-identical results to the uncut step.
 * first_chunk != 0 restarts the accumulation. Call the chunks of a step in a fixed order on
 * ONE stream (or order the streams yourself).
 *
 * slidedp_grad_norm_finish folds the tile sums in a fixed order and leaves, in device
 * memory owned by the context, sumsq, norm = sqrt(sumsq) and
 * coef = max_norm > 0 ? min(1, max_norm / (norm + 1e-6)) : 1. If host_norm / host_coef is
 * non-NULL the call also waits (bounded) for the stream and returns the values.
 */
SLIDEDP_API int slidedp_grad_norm(slidedp_ctx* ctx, const void* const* grads_bf16 /* host array of R device ptrs */,
                      int R, int64_t n, double inv_R, int first_chunk, void* cuda_stream);
SLIDEDP_API int slidedp_grad_norm_finish(slidedp_ctx* ctx, double max_norm, double* host_norm /* nullable */,
                             double* host_coef /* nullable */, void* cuda_stream);

/* The two halves of the norm with the tile sums in CALLER memory, for a step whose parameters are
 * sharded over several GPUs (each GPU updates a contiguous shard and reads its slice of every
 * rank's gradient, Sec. 3.2 "Parameter dispatch" / "Gradient return"): each GPU computes the tile
 * sums of its shard with slidedp_grad_norm_tiles, the shards' sums are gathered in shard order
 * into one array (an all-gather of 8 bytes per 16384 parameters), and every GPU folds that array
 * with slidedp_grad_norm_finish_from. If the shard bounds are multiples of SLIDEDP_NORM_TILE
 * elements the gathered array equals the tile sums of the unsharded step, so every GPU obtains
 * bit for bit the coefficient of the single-GPU step.
 * tile_sums_out: device, ceil(n / SLIDEDP_NORM_TILE) doubles. tile_sums: device, count doubles.
 * slidedp_grad_norm_finish_from leaves norm and coefficient in the context exactly like
 * slidedp_grad_norm_finish (same host_norm / host_coef behaviour). */
#define SLIDEDP_NORM_TILE 16384
SLIDEDP_API int slidedp_grad_norm_tiles(slidedp_ctx* ctx, const void* const* grads_bf16, int R, int64_t n,
                            double inv_R, double* tile_sums_out, void* cuda_stream);
SLIDEDP_API int slidedp_grad_norm_finish_from(slidedp_ctx* ctx, const double* tile_sums, int64_t count,
                                  double max_norm, double* host_norm /* nullable */,
                                  double* host_coef /* nullable */, void* cuda_stream);

/* ---- device-resident update: one fused kernel per chunk -------------------------------
 *
 * For i in [0, n):   (Sec. 3.2: one update of the authoritative FP32 state per iteration
 *                     from the rank-averaged gradient; Sec. 3.3: the BF16 copy is a cast
 *                     of the FP32 master)
 *   gbar = fl32( ((g_0[i] + g_1[i]) + ... + g_{R-1}[i]) in FP32 ) * (float)inv_R
 *   g    = gbar * c          c = context's clip coefficient if hp->max_norm > 0, else 1
 *   m'   = beta1 m + (1-beta1) g          v' = beta2 v + (1-beta2) g^2
 *   w'   = w - lr * ( (m'/(1-beta1^t)) / (sqrt(v'/(1-beta2^t)) + eps) + weight_decay * w )
 *   master[i], m[i], v[i] = fl32(w'), fl32(m'), fl32(v')      (FP64 arithmetic, one rounding)
 *   param_bf16_out[i] = bf16_round_to_nearest_even(master[i])
 * grads_bf16: host array of R device pointers to n BF16 values each; a pointer may also address
 * a peer GPU's buffer with peer access enabled (the kernel reads gradients with plain global
 * loads in rank order, which is what fuses the cross-rank reduction into the update: plain
 * global loads only). master, m, v: device,
 * n floats, in place. param_bf16_out: device, n BF16 values. When hp->max_norm > 0 a
 * slidedp_grad_norm_finish must have been enqueued earlier on the same stream
 * (SLIDEDP_ERR_NO_NORM if none was ever issued on this context).
 * Asynchronous on cuda_stream; traffic is 26 + 2R bytes per parameter.
 * master, m and v may also be PINNED HOST pointers (unified addressing): the kernel then reads and
 * writes host memory directly, with no device slots at all. That needs no GPU memory budget but
 * reaches less of the host link than slidedp_stream_step (measured 40 vs 47 GB/s each way).
 */
SLIDEDP_API int slidedp_reduce_adamw_chunk(slidedp_ctx* ctx, const void* const* grads_bf16, int R, int64_t n,
                               float* master, float* m, float* v, void* param_bf16_out,
                               const slidedp_hparams* hp, void* cuda_stream);

/* ---- the sharded multi-GPU step: buffers shared between processes, BF16 copy to every GPU ----
 *
 * With real ranks (one process per GPU, each holding its rank-local BF16 gradient of the whole
 * layer) the step shards over the flat parameter space (paper Sec. 3.2: "Gradient return" sums
 * the rank-local gradients and returns one result; "Parameter dispatch", sharded delivery, has
 * every rank hold P_l/R of the layer and reconstructs it with an all-gather). GPU s owns the
 * contiguous shard [lo_s, hi_s) of master / m / v and
 *   1. reads slice [lo_s, hi_s) of EVERY rank's gradient through pointers mapped from the peers
 *      (the kernels above read gradients with plain global loads in rank order, so the
 *      cross-rank reduction is fused into the norm and update kernels and crosses the GPU
 *      interconnect exactly once);
 *   2. computes the tile sums of its shard (slidedp_grad_norm_tiles); the shards' sums are
 *      gathered in shard order (8 bytes per 16384 parameters; slidedp_scatter_tile_sums stores
 *      them straight into every GPU's gathered array) and folded by every GPU with
 *      slidedp_grad_norm_finish_from, giving the coefficient of the unsharded step bit for bit
 *      when the shard bounds are multiples of SLIDEDP_NORM_TILE;
 *   3. updates its shard with slidedp_reduce_adamw_chunk_bcast, which is
 *      slidedp_reduce_adamw_chunk with the BF16 copy stored into n_outs buffers instead of one:
 *      the position of the shard in this GPU's BF16 parameter buffer and in every peer's
 *      (mapped). The all-gather of the BF16 parameters is thus done by the update kernel's own
 *      stores. param_bf16_outs: host array of n_outs (1..16) device pointers, each to n BF16
 *      values, 16-byte aligned, none overlapping any other argument. Every other argument,
 *      check, status and the arithmetic are those of slidedp_reduce_adamw_chunk (same bits).
 * Ordering between GPUs is the caller's: a peer's buffer may be read (gradients) only after
 * that peer has produced it, and written (BF16 copy) only when that peer no longer reads the
 * previous copy; a peer sees the new copy after this GPU's stream has completed (a host-side
 * barrier around the step does all three). paper_2609_34162_b200/sharded.py is the reference
 * orchestration over torch.distributed.
 *
 * slidedp_ipc_export fills `out` for a caller-owned device buffer (any address inside a
 * cudaMalloc'd allocation, e.g. a torch tensor of the default allocator; memory from
 * virtual-memory-management allocators cannot be exported); the 80 bytes are plain data to send
 * to the peer process by any means. slidedp_ipc_open maps a peer's handle into this process and
 * returns the device address that corresponds to the exported one (valid on this context's
 * device, peer access enabled on demand; a handle cannot be opened by the process that
 * exported it). slidedp_ipc_close unmaps it (the context also unmaps what is left at destroy).
 * The exporting process must keep the buffer allocated while a peer has it mapped.
 */
typedef struct {
  unsigned char opaque[64]; /* the CUDA inter-process handle of the containing allocation */
  uint64_t offset;          /* of the exported address inside that allocation             */
  uint64_t bytes;           /* from the exported address to the end of the allocation     */
} slidedp_ipc_handle;
SLIDEDP_API int slidedp_ipc_export(slidedp_ctx* ctx, const void* dev_ptr, slidedp_ipc_handle* out);
SLIDEDP_API int slidedp_ipc_open(slidedp_ctx* ctx, const slidedp_ipc_handle* handle, void** dev_ptr_out);
SLIDEDP_API int slidedp_ipc_close(slidedp_ctx* ctx, void* dev_ptr);
/* Step 2's gather without a collective library: stores this GPU's `count` tile sums
 * (device, as written by slidedp_grad_norm_tiles) at dsts[0..n_dsts), each a device pointer to the
 * position of this shard inside a GPU's gathered array (this GPU's own and the peers', mapped).
 * Plain stores from one small kernel; asynchronous on cuda_stream. */
SLIDEDP_API int slidedp_scatter_tile_sums(slidedp_ctx* ctx, const double* tile_sums, int64_t count,
                              double* const* dsts, int n_dsts, void* cuda_stream);
SLIDEDP_API int slidedp_reduce_adamw_chunk_bcast(slidedp_ctx* ctx, const void* const* grads_bf16, int R,
                                     int64_t n, float* master, float* m, float* v,
                                     void* const* param_bf16_outs, int n_outs,
                                     const slidedp_hparams* hp, void* cuda_stream);

/* ---- rank reduction alone ---------------------------------------------------------------------
 *
 * The paper's GPU-reduction route (Sec. 3.2 "Gradient return"): the rank-local gradients are summed,
 * averaged, and ONE gradient of the layer's size is returned for the copy to the host, where the
 * paper's CPU update consumes it. For callers that keep that route:
 *   out_bf16[i] = bf16_rne( fl32( ((g_0[i] + g_1[i]) + ... + g_{R-1}[i]) in FP32 ) * (float)inv_R )
 * (the fused update above does NOT round the average to BF16; this entry point exists for the
 * paper's data path, not for slidedp_reduce_adamw_chunk). grads_bf16: host array of R device
 * pointers; out_bf16: device, n BF16 values, 16-byte aligned, may not overlap the inputs.
 * Asynchronous on cuda_stream; traffic 2R + 2 bytes per parameter.
 */
SLIDEDP_API int slidedp_reduce_mean_bf16(slidedp_ctx* ctx, const void* const* grads_bf16, int R, int64_t n,
                             double inv_R, void* out_bf16, void* cuda_stream);

/* ---- host-resident update: state in pinned host memory, streamed chunk by chunk -------
 *
 * host_master / host_m / host_v: PINNED host arrays of n_total floats, updated in place.
 * grads_bf16 (R device pointers, n_total each) and param_bf16_out (device, n_total) stay on
 * the device. The step is cut every chunk_elems parameters (a multiple of 8; the last chunk
 * may be short). Chunk k uses slot k mod nbuf (nbuf = 2 or 3): its three state arrays are
 * copied H2D on a copy-in stream, updated by the fused kernel on a compute stream and copied
 * back D2H on a copy-out stream, so that copy-in, kernel and copy-out of different chunks
 * overlap (Sec. 3.3 "Overlap within a layer"); a slot is reused only after its copy-out has
 * completed (Sec. 3.3 "Completion and buffer reuse"). Slots take nbuf * 3 * chunk_elems * 4
 * bytes of device memory inside the context and must fit its budget (SLIDEDP_ERR_BUDGET,
 * before any work). If hp->max_norm > 0 and norm_ready == 0 the call first computes the
 * global norm over these n_total gradients; with norm_ready != 0 it uses the coefficient
 * already held by the context (a step that spans several calls: run slidedp_grad_norm over
 * every layer and slidedp_grad_norm_finish first). Synchronous: returns after the last
 * copy-out completed (bounded wait, SLIDEDP_ERR_TIMEOUT). stats is nullable.
 * The call runs on the context's own non-blocking streams and does not order itself after
 * any stream of the caller: whatever produced the gradients, and with norm_ready the
 * slidedp_grad_norm_finish, must have completed (synchronise that stream first).
 * Link traffic is 12 bytes per parameter in each direction.
 */
SLIDEDP_API int slidedp_stream_step(slidedp_ctx* ctx, const void* const* grads_bf16, int R, int64_t n_total,
                        float* host_master, float* host_m, float* host_v,
                        void* param_bf16_out, int64_t chunk_elems, int nbuf, int norm_ready,
                        const slidedp_hparams* hp, slidedp_stats* stats);

/* The same step without the final wait, for callers that stream several layers back to back
 * (Sec. 3.3: completed layers release their updates while other work continues). The call only
 * enqueues; consecutive calls share the slot ring, so the copy-out of one layer's last chunk runs
 * beside the copy-in of the next layer's first chunk instead of draining the pipeline per
 * layer. The host arrays, gradients and output must stay valid, and the context's clip
 * coefficient unchanged, until slidedp_stream_wait returns; that call waits (bounded) for
 * everything queued. A call whose slot layout differs (chunk_elems, nbuf) first drains. */
SLIDEDP_API int slidedp_stream_step_async(slidedp_ctx* ctx, const void* const* grads_bf16, int R,
                              int64_t n_total, float* host_master, float* host_m, float* host_v,
                              void* param_bf16_out, int64_t chunk_elems, int nbuf, int norm_ready,
                              const slidedp_hparams* hp);
SLIDEDP_API int slidedp_stream_wait(slidedp_ctx* ctx);

/* A whole multi-layer step in one call (paper Sec. 3.3: layers are the unit the update is
 * released in, and completed layers release their updates while other work continues): when
 * hp->max_norm > 0 the global norm is taken over the gradients of ALL layers, in layer order,
 * before any update; then every layer is streamed like slidedp_stream_step_async with that
 * coefficient, the layers sharing the slot ring back to back; the call returns after the last
 * copy-out (bounded wait). Every layer's arguments are checked before anything is queued.
 * layers[l]: grads_bf16 = host array of R device pointers to n BF16 values each; host_master /
 * host_m / host_v = PINNED, n floats, updated in place; param_bf16_out = device, n BF16. The
 * result is bit-identical to slidedp_grad_norm over the layers + slidedp_grad_norm_finish + one
 * slidedp_stream_step(norm_ready = 1) per layer. stats (nullable): norm, clip_coef, ms_total,
 * ms_norm, the two copy lanes over the whole step, chunks (sum); ms_kernel is not measured. */
typedef struct {
  const void* const* grads_bf16;
  int64_t n;
  float *host_master, *host_m, *host_v;
  void* param_bf16_out;
} slidedp_layer;
SLIDEDP_API int slidedp_stream_layers(slidedp_ctx* ctx, const slidedp_layer* layers, int num_layers, int R,
                          int64_t chunk_elems, int nbuf, const slidedp_hparams* hp,
                          slidedp_stats* stats);

/* ---- parameter delivery: BF16 copy of a host-resident FP32 master -------------------------
 *
 * The step BEFORE the update path (paper Sec. 3.3 "Overlap within a layer": on parameter
 * delivery chunk k+1 is cast to BF16 while DMA transfers chunk k; Sec. 3.2 "Parameter
 * dispatch"). The paper casts on the CPU and moves BF16 (2 bytes per parameter); here the
 * pinned FP32 master is copied H2D chunk by chunk (4 bytes per parameter) into the context's
 * slots and cast on the GPU, copy of chunk k+1 overlapping the cast of chunk k, so no host core
 * and no host DRAM bandwidth beyond the DMA read is spent:
 *   param_bf16_out[i] = bf16_round_to_nearest_even(host_master[i])        for i in [0, n_total)
 * host_master: PINNED, n_total floats, read-only. param_bf16_out: device, n_total BF16.
 * chunk_elems: multiple of 8; nbuf 2 or 3; slots take nbuf * chunk_elems * 4 bytes under the
 * context's budget (SLIDEDP_ERR_BUDGET). Synchronous (bounded wait); runs on the context's own
 * streams like slidedp_stream_step. stats (nullable): ms_total, ms_h2d / gbs_h2d (copy lane
 * span and 4 n_total bytes over it), chunks; the other fields are zero.
 */
SLIDEDP_API int slidedp_deliver_params(slidedp_ctx* ctx, const float* host_master, int64_t n_total,
                           void* param_bf16_out, int64_t chunk_elems, int nbuf,
                           slidedp_stats* stats);

/* ---- step-time model of the host-resident step (host arithmetic only, no GPU work) --------
 *
 * The paper's dependency model (Sec. 3.4 "Modeling Shared-Host Scaling") applied to
 * slidedp_stream_step. Resource demand gives the lower bound  T >= max_j W_j / beta_j  over the
 * copy-in lane, the copy-out lane and the compute lane; execution dependencies give each
 * operation's completion  f(v) = d_v + max({a_v} U {f(u) : u in P(v)})  with
 *   copy-in  of chunk k after copy-in  of k-1 (stream order) and copy-out of k-nbuf (buffer),
 *   kernel   of chunk k after copy-in  of k   (data) and kernel of k-1 (stream; the norm pass
 *            precedes kernel 0),
 *   copy-out of chunk k after kernel   of k   (data) and copy-out of k-1 (stream).
 * d_v = bytes / rate (+ per_copy_us for each of a chunk's three copies); all release times
 * a_v are 0. Rates are what slidedp_link_probe and the kernel benchmarks measured.
 * Writes the bound and the predicted completion of the last copy-out, in ms.
 */
typedef struct {
  double h2d_gbs, d2h_gbs;      /* link rates while both directions are busy (GB/s)         */
  double update_gparams_s;      /* fused update kernel rate on device slots (G-params/s)    */
  double norm_gbs;              /* norm pass rate over the gradients (GB/s); 0: no norm pass */
  double per_copy_us;           /* fixed cost of one cudaMemcpyAsync on its lane (us)        */
} slidedp_rates;
SLIDEDP_API int slidedp_model_stream_step(int64_t n_total, int R, int64_t chunk_elems, int nbuf,
                              const slidedp_rates* rates, double* lower_bound_ms,
                              double* predicted_ms);

/* ---- host-link probe: the roofline of the host-resident mode ---------------------------
 *
 * Copies `bytes` between a pinned host buffer and a device buffer in pieces of copy_bytes,
 * reps times, and reports GB/s: out4[0] H2D alone, out4[1] D2H alone, out4[2] / out4[3] H2D
 * and D2H while both run at once on two streams. host_a/host_b pinned, dev_a/dev_b device,
 * each at least `bytes` long. Synchronous (bounded waits).
 */
SLIDEDP_API int slidedp_link_probe(slidedp_ctx* ctx, void* host_a, void* host_b, void* dev_a, void* dev_b,
                       size_t bytes, size_t copy_bytes, int reps, double out4[4]);

/* ---- HBM probe with the update kernel's access mix: a roofline for the fused kernel -------
 *
 * Runs, reps times after two warm-up launches, a kernel with exactly the loads and stores of
 * slidedp_reduce_adamw_chunk at this R (12 + 2R bytes read, 14 written per parameter, same
 * launch shape and cache hints) and NO arithmetic, and reports the best rate in GB/s counted
 * with the same 26 + 2R bytes per parameter. master / m / v are read and written back unchanged;
 * scratch_bf16_out (device, n BF16) is overwritten. Synchronous (bounded waits) on cuda_stream.
 * Arguments and checks as for slidedp_reduce_adamw_chunk; n >= 4. (No counterpart in the paper:
 * measurement support, like slidedp_link_probe.)
 */
SLIDEDP_API int slidedp_hbm_mix_probe(slidedp_ctx* ctx, const void* const* grads_bf16, int R, int64_t n,
                          float* master, float* m, float* v, void* scratch_bf16_out, int reps,
                          double* best_gbs, void* cuda_stream);

/* ---- global norm for callers that cannot allocate ---------------------------------------
 *
 * (No counterpart in the paper: this entry point exists for deployment reasons only.)
 * Some callers may not allocate device memory at the moment they need the norm, or ever: code
 * running inside a memory-pool or allocator callback, a host process whose memory budget is
 * fixed and fully handed out at start-up, or a plug-in that is only given pointers. Such
 * callers cannot use slidedp_create (it allocates the workspace of slidedp_grad_norm).
 * slidedp_grad_norm_noalloc computes the same quantity as slidedp_grad_norm followed by
 * slidedp_grad_norm_finish for ONE chunk, with the same kernels, tiling and summation tree
 * (so the same bits), but keeps its tile sums in a fixed array compiled into the library's
 * device image instead of allocated memory. It takes no context and calls no cudaMalloc,
 * cudaFree or any allocating routine.
 *
 * grads_bf16: host array of R device pointers (16-byte aligned) to n BF16 values each, on the
 * CURRENT device. out4: device pointer (16-byte aligned) to four doubles that receive sumsq,
 * norm, coef = max_norm > 0 ? min(1, max_norm/(norm + 1e-6)) : 1, and 1.0 if the norm is not
 * finite (else 0.0). Asynchronous on cuda_stream.
 *
 * Limits and sharing: n <= SLIDEDP_NOALLOC_MAX_ELEMS (2^30); more gives
 * SLIDEDP_ERR_TOO_LARGE and nothing is launched. The array (512 KiB) is part of the library's
 * device image: every GPU on which the library's device code gets loaded holds it until the
 * process exits. All calls on a device share it: two calls whose kernels may overlap on the GPU
 * (different streams without ordering) race on it; calls ordered on one stream are safe. It
 * keeps the previous call's tile sums, and nothing has to start at zero: each call overwrites
 * the tiles it then reads and reads no others.
 *
 * The FIRST call on each device is a set-up call: with that device current it looks up the
 * array's device address. Under CUDA's default lazy module loading that look-up can be the
 * moment the driver loads the library's device image (array included) onto the GPU, which
 * takes device memory inside the driver. So make one call per device at start-up (n = 0 is
 * enough), OUTSIDE any region in which allocation is forbidden and before any stream capture;
 * every later call on that device allocates nothing (a GPU test checks that free device memory
 * does not move across later calls). The look-up is cached per device in an atomic, so first
 * calls from several host threads at once are safe.
 */
#define SLIDEDP_NOALLOC_MAX_ELEMS ((int64_t)1 << 30)
SLIDEDP_API int slidedp_grad_norm_noalloc(const void* const* grads_bf16, int R, int64_t n, double inv_R,
                              double max_norm, double* out4, void* cuda_stream);

/* Number of kernels this library has launched on the context since creation. */
SLIDEDP_API int64_t slidedp_kernel_launches(const slidedp_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif
