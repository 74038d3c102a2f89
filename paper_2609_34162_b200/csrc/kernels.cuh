// Device kernels of libslidedp (sm_100a): the fused rank-reduce + AdamW + BF16-emit
// streaming kernel, and the two-pass fixed-tree sum of squares behind the global norm.
//
// The path is elementwise and HBM-bound (26 + 2R bytes per parameter), so there are no
// tensor cores here: each thread owns a few consecutive parameters, moves them with
// vector accesses, keeps everything in registers and stores each output once.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "device_utils.cuh"
#include "types.h"

namespace slidedp {

constexpr int kVec = 4;                 // parameters per thread in the update kernel
constexpr int kUpdateThreads = 128;
constexpr int kNormVec = 8;             // elements per thread per load in the norm kernel
constexpr int kNormThreads = 256;
constexpr int kNormIters = 8;
constexpr int kNormTile = kNormThreads * kNormVec * kNormIters;   // 16384 elements per partial
constexpr int kFinishThreads = 1024;

// Hardware seeds for FP64 reciprocal square root and reciprocal (about 20 good bits; the
// full double exponent range). One Newton step each below brings them to ~1e-12.
__device__ __forceinline__ double rsqrt_seed(double x) {
  double r;
  asm("rsqrt.approx.ftz.f64 %0, %1;" : "=d"(r) : "d"(x));
  return r;
}
__device__ __forceinline__ double rcp_seed(double x) {
  double r;
  asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(r) : "d"(x));
  return r;
}

// One parameter's AdamW update in FP64 from the FP32 state. k1 = (1-beta1) c and
// k2 = (1-beta2) c^2 carry the clip coefficient c.
//
// The common path has no FP64 compares: sqrt(v1) and m1/d come from the hardware seeds plus
// one Newton step each (~1e-12 relative). v1 == 0 (zero gradient on zero state) is caught by an
// integer test of the double's high word, because the rsqrt seed of 0 is +inf. Everything else
// that the seeds cannot carry (v1 = +inf, d = 0 when eps = 0, NaN or inf operands) makes the
// result non-finite, and only then the update is redone with IEEE sqrt and division, so those
// cases follow the plain formulas exactly (e.g. v1 = inf gives u = 0, a finite decay-only step).
__device__ __forceinline__ void adamw_element(float gbar, float& w, float& m, float& v,
                                              const UpdateConsts& k, double k1, double k2) {
  const double g = (double)gbar;
  const double w0 = (double)w;
  const double m1 = fma(k.beta1, (double)m, k1 * g);
  const double v1 = fma(k.beta2, (double)v, k2 * (g * g));     // g*g is exact in double
  const double r = (__double2hiint(v1) == 0) ? 0.0 : rsqrt_seed(v1);
  double s = v1 * r;
  s = fma(fma(-s, s, v1), 0.5 * r, s);                         // s = sqrt(v1)
  const double d = fma(s, k.rsqrt_bc2, k.eps);                 // sqrt(v1/bc2) + eps
  const double rc = rcp_seed(d);
  double q = m1 * rc;
  q = fma(fma(-q, d, m1), rc, q);                              // q = m1 / d
  double w1 = fma(k.neg_lr_over_bc1, q, k.decay * w0);
  if ((__double2hiint(w1) & 0x7ff00000) == 0x7ff00000) {       // inf or NaN: rare, exact path
    const double d2 = fma(sqrt(v1), k.rsqrt_bc2, k.eps);
    w1 = fma(k.neg_lr_over_bc1, m1 / d2, k.decay * w0);
  }
  m = __double2float_rn(m1);
  v = __double2float_rn(v1);
  w = __double2float_rn(w1);
}

// ---- fused update kernel -------------------------------------------------------------
//
// One thread owns kVec = 4 consecutive parameters: one 8-byte BF16 load per rank, one
// 16-byte load per FP32 array, all issued before the first use, then the FP64 update in
// registers and one store per output. Four parameters (not eight) per thread keeps the
// kernel at 64 registers, so eight 128-thread blocks (32 warps) stay resident per SM; that
// is what hides the FP64 dependency chains behind the loads of the other warps. Measured
// on B200 at R = 4: 6.8-6.9 TB/s against 5.6 TB/s for the eight-per-thread form and 6.4 TB/s
// for a bulk-copy (TMA) shared-memory ring.
// R is a template parameter (one instantiation per rank count 1..16): the R loads and the
// left-to-right FP32 adds are fully unrolled.
//
// Where the BF16 copy goes is a policy: OneOut stores it once (the single-GPU step); ManyOuts
// stores the same values into several buffers, which in a sharded multi-GPU step are this
// GPU's parameter buffer and every peer's, mapped into this process: the all-gather of the
// BF16 parameters then happens inside the update kernel as plain peer stores, tile by tile.
struct OneOut {
  uint16_t* p;
  __device__ __forceinline__ void vec(int64_t base, uint2 packed) const {
    __stcs(reinterpret_cast<uint2*>(p + base), packed);
  }
  __device__ __forceinline__ void one(int64_t i, uint16_t bits) const { p[i] = bits; }
};
struct ManyOuts {
  uint16_t* p[kMaxRanks];
  int count;
  __device__ __forceinline__ void vec(int64_t base, uint2 packed) const {
    for (int o = 0; o < count; ++o) __stcs(reinterpret_cast<uint2*>(p[o] + base), packed);
  }
  __device__ __forceinline__ void one(int64_t i, uint16_t bits) const {
    for (int o = 0; o < count; ++o) p[o][i] = bits;
  }
};

template <int R, class Out>
__device__ __forceinline__ void reduce_adamw_body(const GradPtrs& gp, int64_t n,
                                                  float* __restrict__ master,
                                                  float* __restrict__ mom1,
                                                  float* __restrict__ mom2, const Out& out,
                                                  const UpdateConsts& k,
                                                  const double* __restrict__ clip_coef) {
  const int64_t base = ((int64_t)blockIdx.x * kUpdateThreads + threadIdx.x) * kVec;
  if (base >= n) return;
  wait_for_previous_kernel();      // the clip coefficient and the state come from earlier kernels
  const double c = clip_coef ? *clip_coef : 1.0;
  const double k1 = k.omb1 * c, k2 = k.omb2 * c * c;

  if (base + kVec <= n) {
    uint2 graw[R];
#pragma unroll
    for (int r = 0; r < R; ++r) graw[r] = __ldcs(reinterpret_cast<const uint2*>(gp.p[r] + base));
    uint4 wq = ld_stream(master + base);
    uint4 mq = ld_stream(mom1 + base);
    uint4 vq = ld_stream(mom2 + base);
    float s[kVec] = {bf16_lo(graw[0].x), bf16_hi(graw[0].x), bf16_lo(graw[0].y), bf16_hi(graw[0].y)};
#pragma unroll
    for (int r = 1; r < R; ++r) {
      s[0] = __fadd_rn(s[0], bf16_lo(graw[r].x));
      s[1] = __fadd_rn(s[1], bf16_hi(graw[r].x));
      s[2] = __fadd_rn(s[2], bf16_lo(graw[r].y));
      s[3] = __fadd_rn(s[3], bf16_hi(graw[r].y));
    }
    float* wf = reinterpret_cast<float*>(&wq);
    float* mf = reinterpret_cast<float*>(&mq);
    float* vf = reinterpret_cast<float*>(&vq);
    uint32_t pk[kVec / 2];
#pragma unroll
    for (int j = 0; j < kVec; j += 2) {
      adamw_element(__fmul_rn(s[j], k.inv_R), wf[j], mf[j], vf[j], k, k1, k2);
      adamw_element(__fmul_rn(s[j + 1], k.inv_R), wf[j + 1], mf[j + 1], vf[j + 1], k, k1, k2);
      pk[j / 2] = f32_to_bf16_bits(wf[j]) | (f32_to_bf16_bits(wf[j + 1]) << 16);
    }
    st_stream(master + base, wq);
    st_stream(mom1 + base, mq);
    st_stream(mom2 + base, vq);
    out.vec(base, make_uint2(pk[0], pk[1]));
  } else {
    // ragged tail: fewer than kVec parameters left, one at a time
    for (int64_t i = base; i < n; ++i) {
      float s = __uint_as_float((uint32_t)gp.p[0][i] << 16);
      for (int r = 1; r < R; ++r) s = __fadd_rn(s, __uint_as_float((uint32_t)gp.p[r][i] << 16));
      float w = master[i], m = mom1[i], v = mom2[i];
      adamw_element(__fmul_rn(s, k.inv_R), w, m, v, k, k1, k2);
      master[i] = w; mom1[i] = m; mom2[i] = v;
      out.one(i, (uint16_t)f32_to_bf16_bits(w));
    }
  }
}

template <int R>
__global__ void __launch_bounds__(kUpdateThreads, 8)
reduce_adamw_kernel(GradPtrs gp, int64_t n, float* __restrict__ master,
                    float* __restrict__ mom1, float* __restrict__ mom2,
                    uint16_t* __restrict__ param_out, UpdateConsts k,
                    const double* __restrict__ clip_coef) {
  reduce_adamw_body<R>(gp, n, master, mom1, mom2, OneOut{param_out}, k, clip_coef);
}

// The same update with the BF16 copy stored into `outs.count` buffers (see ManyOuts).
template <int R>
__global__ void __launch_bounds__(kUpdateThreads, 8)
reduce_adamw_bcast_kernel(GradPtrs gp, int64_t n, float* __restrict__ master,
                          float* __restrict__ mom1, float* __restrict__ mom2, ManyOuts outs,
                          UpdateConsts k, const double* __restrict__ clip_coef) {
  reduce_adamw_body<R>(gp, n, master, mom1, mom2, outs, k, clip_coef);
}

// ---- the update kernel's memory traffic with no arithmetic (a roofline probe) ------------------
//
// Same launch shape, same loads and stores as reduce_adamw_kernel<R> (R 8-byte BF16 loads and
// three 16-byte FP32 loads per thread, three 16-byte stores and one 8-byte store), but the FP32
// state is written back unchanged and the BF16 output is an xor of the gradient words: what this
// access mix (12 + 2R bytes read, 14 written per parameter) can reach on the device when nothing
// is computed. Only whole groups of kVec parameters are touched.
template <int R>
__global__ void __launch_bounds__(kUpdateThreads, 8)
traffic_mix_kernel(GradPtrs gp, int64_t n, float* __restrict__ master, float* __restrict__ mom1,
                   float* __restrict__ mom2, uint16_t* __restrict__ out) {
  const int64_t base = ((int64_t)blockIdx.x * kUpdateThreads + threadIdx.x) * kVec;
  if (base + kVec > n) return;
  uint2 x = make_uint2(0u, 0u);
  uint2 graw[R];
#pragma unroll
  for (int r = 0; r < R; ++r) graw[r] = __ldcs(reinterpret_cast<const uint2*>(gp.p[r] + base));
  const uint4 wq = ld_stream(master + base);
  const uint4 mq = ld_stream(mom1 + base);
  const uint4 vq = ld_stream(mom2 + base);
#pragma unroll
  for (int r = 0; r < R; ++r) { x.x ^= graw[r].x; x.y ^= graw[r].y; }
  st_stream(master + base, wq);
  st_stream(mom1 + base, mq);
  st_stream(mom2 + base, vq);
  __stcs(reinterpret_cast<uint2*>(out + base), x);
}

// ---- sum of squares of the averaged gradient ----------------------------------------------
//
// Pass 1: one FP64 partial per fixed tile of kNormTile elements. Inside a tile thread t
// adds its 8 * kNormIters squares in index order, the warp folds by an xor butterfly
// (16, 8, 4, 2, 1), and thread 0 adds the 8 warp sums in warp order: the tree is fixed, so
// a tile's partial does not depend on which block computes it or on the grid size.
// Launched with one block per tile; the loads of UNROLL iterations are in flight together
// (measured best: 2 at R = 4, 1 at R = 8, where more unrolling costs occupancy).
template <int R, int UNROLL = (R >= 6) ? 1 : (R >= 3 ? 2 : 4)>
__global__ void __launch_bounds__(kNormThreads)
grad_sumsq_tiles_kernel(GradPtrs gp, int64_t n, float inv_R, double* __restrict__ partials) {
  __shared__ double warp_sum[kNormThreads / 32];
  wait_for_previous_kernel();      // the gradients (and the tile-sum slots) may come from it
  const int64_t ntiles = (n + kNormTile - 1) / kNormTile;
  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const int64_t tbase = tile * kNormTile + (int64_t)threadIdx.x * kNormVec;
    double acc = 0.0;
#pragma unroll UNROLL
    for (int it = 0; it < kNormIters; ++it) {
      const int64_t e = tbase + (int64_t)it * (kNormThreads * kNormVec);
      float s[kNormVec];
      if (e + kNormVec <= n) {
        uint4 graw[R];
#pragma unroll
        for (int r = 0; r < R; ++r) graw[r] = ld_stream(gp.p[r] + e);
        {
          const uint32_t* x = reinterpret_cast<const uint32_t*>(&graw[0]);
#pragma unroll
          for (int j = 0; j < 4; ++j) { s[2 * j] = bf16_lo(x[j]); s[2 * j + 1] = bf16_hi(x[j]); }
        }
#pragma unroll
        for (int r = 1; r < R; ++r) {
          const uint32_t* x = reinterpret_cast<const uint32_t*>(&graw[r]);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            s[2 * j] = __fadd_rn(s[2 * j], bf16_lo(x[j]));
            s[2 * j + 1] = __fadd_rn(s[2 * j + 1], bf16_hi(x[j]));
          }
        }
      } else {
#pragma unroll
        for (int j = 0; j < kNormVec; ++j) {
          s[j] = 0.0f;
          if (e + j < n) {
            float t = __uint_as_float((uint32_t)gp.p[0][e + j] << 16);
            for (int r = 1; r < R; ++r)
              t = __fadd_rn(t, __uint_as_float((uint32_t)gp.p[r][e + j] << 16));
            s[j] = t;
          }
        }
      }
#pragma unroll
      for (int j = 0; j < kNormVec; ++j) {
        const double g = (double)__fmul_rn(s[j], inv_R);
        acc = fma(g, g, acc);
      }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
    if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      double t = warp_sum[0];
#pragma unroll
      for (int w = 1; w < kNormThreads / 32; ++w) t += warp_sum[w];
      partials[tile] = t;
    }
    __syncthreads();
  }
}

// Pass 1 at R = 1: the same tiles, the same per-thread order of additions and the same tree (so
// the same bits as the kernel above), but a launch shape made for a stream of only 2 bytes per
// parameter: one block computes kDeepTiles = 2 consecutive tiles and has ALL of a tile's loads
// in flight at once (8 x 16 bytes per thread), the second tile's loads issued before the first
// tile's arithmetic and shuffle tree. With one short-lived block per 32 KB tile the single-rank
// pass was latency-bound (5.1 TB/s at 100 M parameters, 6.2 at 400 M); this form measured 5.7
// and 7.0 TB/s on the same buffers. At R >= 2 a tile already carries enough bytes per block and
// the generic kernel is as fast or faster, so only R = 1 takes this path.
constexpr int kDeepTiles = 2;
__device__ __forceinline__ double tile_thread_sum_r1(const uint4 (&raw)[kNormIters], float inv_R) {
  double acc = 0.0;
#pragma unroll
  for (int it = 0; it < kNormIters; ++it) {
    const uint32_t* x = reinterpret_cast<const uint32_t*>(&raw[it]);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const double a = (double)__fmul_rn(bf16_lo(x[j]), inv_R);
      acc = fma(a, a, acc);
      const double b = (double)__fmul_rn(bf16_hi(x[j]), inv_R);
      acc = fma(b, b, acc);
    }
  }
  return acc;
}
__global__ void __launch_bounds__(kNormThreads)
grad_sumsq_tiles_r1_kernel(const uint16_t* __restrict__ g, int64_t n, float inv_R,
                           double* __restrict__ partials) {
  __shared__ double warp_sum[kDeepTiles][kNormThreads / 32];
  wait_for_previous_kernel();
  const int64_t ntiles = (n + kNormTile - 1) / kNormTile;
  const int64_t first = (int64_t)blockIdx.x * kDeepTiles;
  uint4 raw[kDeepTiles][kNormIters];
  // a tile is "full" when every one of its 16-byte vectors lies inside [0, n)
  bool full[kDeepTiles];
#pragma unroll
  for (int t = 0; t < kDeepTiles; ++t) {
    const int64_t tile = first + t;
    full[t] = tile < ntiles && (tile + 1) * kNormTile <= n;
    if (full[t]) {
      const int64_t tb = tile * kNormTile + (int64_t)threadIdx.x * kNormVec;
#pragma unroll
      for (int it = 0; it < kNormIters; ++it)
        raw[t][it] = ld_stream(g + tb + (int64_t)it * (kNormThreads * kNormVec));
    }
  }
#pragma unroll
  for (int t = 0; t < kDeepTiles; ++t) {
    const int64_t tile = first + t;
    if (tile >= ntiles) break;                     // uniform over the block
    double acc = 0.0;
    if (full[t]) {
      acc = tile_thread_sum_r1(raw[t], inv_R);
    } else {
      // the step's last, ragged tile: element by element where a vector would cross n
      const int64_t tb = tile * kNormTile + (int64_t)threadIdx.x * kNormVec;
      for (int it = 0; it < kNormIters; ++it) {
        const int64_t e = tb + (int64_t)it * (kNormThreads * kNormVec);
#pragma unroll
        for (int j = 0; j < kNormVec; ++j) {
          float s = 0.0f;
          if (e + j < n) s = __uint_as_float((uint32_t)g[e + j] << 16);
          const double x = (double)__fmul_rn(s, inv_R);
          acc = fma(x, x, acc);
        }
      }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
    if ((threadIdx.x & 31) == 0) warp_sum[t][threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      double s = warp_sum[t][0];
#pragma unroll
      for (int w = 1; w < kNormThreads / 32; ++w) s += warp_sum[t][w];
      partials[tile] = s;
    }
  }
}

// Pass 2: one block folds `count` partials in a fixed order: thread t adds partials
// t, t + 1024, ... in that order, then the same warp butterfly and warp-order sum.
// Writes scalars[0] = sumsq, [1] = norm, [2] = clip coefficient, [3] = 1.0 if non-finite.
__global__ void __launch_bounds__(kFinishThreads)
grad_norm_finish_kernel(const double* __restrict__ partials, int64_t count, double max_norm,
                        double* __restrict__ scalars) {
  __shared__ double warp_sum[kFinishThreads / 32];
  wait_for_previous_kernel();      // the tile sums come from the kernel(s) before this one
  double acc = 0.0;
  for (int64_t i = threadIdx.x; i < count; i += kFinishThreads) acc += partials[i];
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
  if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = warp_sum[0];
    for (int w = 1; w < kFinishThreads / 32; ++w) t += warp_sum[w];
    const double norm = sqrt(t);
    double c = 1.0;
    if (max_norm > 0.0) {
      c = max_norm / (norm + 1e-6);
      if (c > 1.0) c = 1.0;      // a NaN coefficient stays NaN
    }
    scalars[0] = t;
    scalars[1] = norm;
    scalars[2] = c;
    scalars[3] = (norm - norm == 0.0) ? 0.0 : 1.0;
  }
}

// ---- tile sums of one shard written into every GPU's gathered array ---------------------------
//
// The all-gather of the norm's tile sums in a sharded step (8 bytes per 16384 parameters): this
// GPU's `count` sums are stored at the same offset of `ndst` arrays, its own and the peers'
// (mapped), with plain stores. Pure data movement.
struct F64Dsts {
  double* p[kMaxRanks];
};
__global__ void __launch_bounds__(256)
scatter_tile_sums_kernel(const double* __restrict__ src, int64_t count, F64Dsts dsts, int ndst) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= count) return;
  const double x = src[i];
  for (int o = 0; o < ndst; ++o) dsts.p[o][i] = x;
}

// ---- rank reduction alone: the averaged gradient as one BF16 buffer --------------------
//
// The paper's GPU-reduction route materialises ONE gradient of G_l bytes per layer for the copy
// to the host (Sec. 3.2 "Gradient return"). Same left-to-right FP32 sum and FP32 multiply by
// (float)1/R as the fused kernel, then one round-to-nearest-even to BF16. Eight elements per
// thread; 2R + 2 bytes of traffic per parameter.
constexpr int kReduceThreads = 256;
// U = 16-byte loads per rank in flight per thread: 1 for R >= 2; 2 at R = 1, where a thread's 8
// elements are only 16 bytes and the kernel was latency-bound (5.7 -> 6.4 TB/s at 100 M
// parameters; the 32-byte load form of the same shape measured the same, so plain 16-byte
// accesses are kept).
template <int R, int U = (R == 1) ? 2 : 1>
__global__ void __launch_bounds__(kReduceThreads)
reduce_mean_bf16_kernel(GradPtrs gp, int64_t n, float inv_R, uint16_t* __restrict__ out) {
  const int64_t base = ((int64_t)blockIdx.x * kReduceThreads + threadIdx.x) * (8 * U);
  if (base >= n) return;
  if (base + 8 * U <= n) {
    uint4 graw[U][R];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int r = 0; r < R; ++r) graw[u][r] = ld_stream(gp.p[r] + base + 8 * u);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float s[8];
      {
        const uint32_t* x = reinterpret_cast<const uint32_t*>(&graw[u][0]);
#pragma unroll
        for (int j = 0; j < 4; ++j) { s[2 * j] = bf16_lo(x[j]); s[2 * j + 1] = bf16_hi(x[j]); }
      }
#pragma unroll
      for (int r = 1; r < R; ++r) {
        const uint32_t* x = reinterpret_cast<const uint32_t*>(&graw[u][r]);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          s[2 * j] = __fadd_rn(s[2 * j], bf16_lo(x[j]));
          s[2 * j + 1] = __fadd_rn(s[2 * j + 1], bf16_hi(x[j]));
        }
      }
      uint32_t b[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) b[j] = f32_to_bf16_bits(__fmul_rn(s[j], inv_R));
      st_stream(out + base + 8 * u, make_uint4(b[0] | (b[1] << 16), b[2] | (b[3] << 16),
                                               b[4] | (b[5] << 16), b[6] | (b[7] << 16)));
    }
  } else {
    for (int64_t i = base; i < n; ++i) {
      float t = __uint_as_float((uint32_t)gp.p[0][i] << 16);
      for (int r = 1; r < R; ++r) t = __fadd_rn(t, __uint_as_float((uint32_t)gp.p[r][i] << 16));
      out[i] = (uint16_t)f32_to_bf16_bits(__fmul_rn(t, inv_R));
    }
  }
}

}  // namespace slidedp
