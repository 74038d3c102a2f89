// The paper's own data path for the update step (gradient D2H -> multi-threaded CPU Adam ->
// CPU cast with streaming stores -> BF16 H2D), as a timed baseline. See cpu_route.h.
// Not part of libslidedp; shares no code with it or with the test oracle.
#include "cpu_route.h"

#include <cuda_runtime.h>
#include <immintrin.h>
#include <math.h>
#include <string.h>
#include <time.h>

#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

double now_ms() {
  timespec ts;
  clock_gettime(CLOCK_MONOTONIC, &ts);
  return 1e3 * (double)ts.tv_sec + 1e-6 * (double)ts.tv_nsec;
}

// ---- ISA selection (decided once, at run time) -------------------------------------------
enum Isa { kScalar = 0, kAvx512 = 1, kAvx512Bf16 = 2 };
Isa detect() {
  __builtin_cpu_init();
  if (__builtin_cpu_supports("avx512f") && __builtin_cpu_supports("avx512bw") &&
      __builtin_cpu_supports("avx512vl")) {
#if defined(__GNUC__) && __GNUC__ >= 10
    if (__builtin_cpu_supports("avx512bf16")) return kAvx512Bf16;
#endif
    return kAvx512;
  }
  return kScalar;
}
Isa& isa_slot() {
  static Isa v = detect();
  return v;
}
Isa isa() { return isa_slot(); }

// ---- scalar pieces --------------------------------------------------------------------------
inline float bf16_to_f32(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}
inline uint16_t f32_to_bf16_rne(float x) {
  uint32_t u;
  memcpy(&u, &x, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);   // NaN stays NaN
  return (uint16_t)((u + 0x7fffu + ((u >> 16) & 1u)) >> 16);
}

// Per-step constants, formed in double and rounded once to FP32.
struct Consts {
  float beta1, beta2, k1, k2, inv_sqrt_bc2, eps, step_size, decay, inv_R;
};
Consts make_consts(const cpuroute_hparams* hp) {
  const double bc1 = 1.0 - pow(hp->beta1, (double)hp->step);
  const double bc2 = 1.0 - pow(hp->beta2, (double)hp->step);
  Consts c;
  c.beta1 = (float)hp->beta1;
  c.beta2 = (float)hp->beta2;
  c.k1 = (float)((1.0 - hp->beta1) * hp->clip_coef);
  c.k2 = (float)((1.0 - hp->beta2) * hp->clip_coef * hp->clip_coef);
  c.inv_sqrt_bc2 = (float)(1.0 / sqrt(bc2));
  c.eps = (float)hp->eps;
  c.step_size = (float)(hp->lr / bc1);
  c.decay = (float)(1.0 - hp->lr * hp->weight_decay);
  c.inv_R = (float)hp->inv_R;
  return c;
}

inline void adamw_scalar(const uint16_t* const* g, int R, int64_t i, float* w, float* m, float* v,
                         uint16_t* p, const Consts& c) {
  float s = bf16_to_f32(g[0][i]);
  for (int r = 1; r < R; ++r) s += bf16_to_f32(g[r][i]);
  if (R > 1) s *= c.inv_R;
  const float m1 = c.beta1 * m[i] + c.k1 * s;
  const float v1 = c.beta2 * v[i] + c.k2 * (s * s);
  const float d = sqrtf(v1) * c.inv_sqrt_bc2 + c.eps;
  const float w1 = c.decay * w[i] - c.step_size * (m1 / d);
  m[i] = m1; v[i] = v1; w[i] = w1;
  if (p) p[i] = f32_to_bf16_rne(w1);
}

// ---- AVX-512 pieces ----------------------------------------------------------------------
__attribute__((target("avx512f,avx512bw,avx512vl"))) inline __m512 load_bf16x16(const uint16_t* p) {
  const __m256i h = _mm256_loadu_si256((const __m256i*)p);
  return _mm512_castsi512_ps(_mm512_slli_epi32(_mm512_cvtepu16_epi32(h), 16));
}
// FP32 x16 -> BF16 x16, round to nearest even, NaN kept quiet: integer form
__attribute__((target("avx512f,avx512bw,avx512vl"))) inline __m256i to_bf16x16_int(__m512 x) {
  const __m512i u = _mm512_castps_si512(x);
  const __m512i lsb = _mm512_and_si512(_mm512_srli_epi32(u, 16), _mm512_set1_epi32(1));
  __m512i r = _mm512_srli_epi32(_mm512_add_epi32(u, _mm512_add_epi32(lsb, _mm512_set1_epi32(0x7fff))), 16);
  const __mmask16 nan = _mm512_cmp_ps_mask(x, x, _CMP_UNORD_Q);
  const __m512i q = _mm512_or_si512(_mm512_srli_epi32(u, 16), _mm512_set1_epi32(0x0040));
  r = _mm512_mask_mov_epi32(r, nan, q);
  return _mm512_cvtepi32_epi16(r);
}
#if defined(__GNUC__) && __GNUC__ >= 10
__attribute__((target("avx512f,avx512bw,avx512vl,avx512bf16"))) inline __m256i to_bf16x16_hw(__m512 x) {
  // vcvtneps2bf16 treats denormal inputs as zero; BF16 results of FP32 denormals are BF16
  // denormals, which round-to-nearest-even must keep, so those lanes take the integer form
  const __m512 ax = _mm512_castsi512_ps(_mm512_and_si512(_mm512_castps_si512(x), _mm512_set1_epi32(0x7fffffff)));
  const __mmask16 tiny = _mm512_cmp_ps_mask(ax, _mm512_castsi512_ps(_mm512_set1_epi32(0x00800000)), _CMP_LT_OQ);
  __m256i r = (__m256i)_mm512_cvtneps_pbh(x);
  if (tiny) r = _mm256_mask_mov_epi16(r, tiny, to_bf16x16_int(x));
  return r;
}
#endif

template <bool HW>
__attribute__((target("avx512f,avx512bw,avx512vl,avx512bf16"))) inline __m256i to_bf16x16(__m512 x) {
#if defined(__GNUC__) && __GNUC__ >= 10
  if (HW) return to_bf16x16_hw(x);
#endif
  return to_bf16x16_int(x);
}

template <bool HW>
__attribute__((target("avx512f,avx512bw,avx512vl,avx512bf16")))
void cast_range_avx512(const float* src, int64_t lo, int64_t hi, uint16_t* dst) {
  int64_t i = lo;
  // head: until dst is 64-byte aligned (two vectors of 16 make one 64-byte line of BF16)
  while (i < hi && ((uintptr_t)(dst + i) & 63u) != 0) { dst[i] = f32_to_bf16_rne(src[i]); ++i; }
  for (; i + 32 <= hi; i += 32) {
    const __m256i a = to_bf16x16<HW>(_mm512_loadu_ps(src + i));
    const __m256i b = to_bf16x16<HW>(_mm512_loadu_ps(src + i + 16));
    const __m512i line = _mm512_inserti64x4(_mm512_castsi256_si512(a), b, 1);
    _mm512_stream_si512((__m512i*)(dst + i), line);          // non-temporal: no cache pollution
  }
  for (; i < hi; ++i) dst[i] = f32_to_bf16_rne(src[i]);
}

template <bool HW>
__attribute__((target("avx512f,avx512bw,avx512vl,avx512bf16")))
void adamw_range_avx512(const uint16_t* const* g, int R, int64_t lo, int64_t hi, float* w, float* m,
                        float* v, uint16_t* p, const Consts& c) {
  const __m512 beta1 = _mm512_set1_ps(c.beta1), beta2 = _mm512_set1_ps(c.beta2);
  const __m512 k1 = _mm512_set1_ps(c.k1), k2 = _mm512_set1_ps(c.k2);
  const __m512 isb = _mm512_set1_ps(c.inv_sqrt_bc2), eps = _mm512_set1_ps(c.eps);
  const __m512 step = _mm512_set1_ps(c.step_size), decay = _mm512_set1_ps(c.decay);
  const __m512 invR = _mm512_set1_ps(c.inv_R);
  int64_t i = lo;
  if (p) while (i < hi && ((uintptr_t)(p + i) & 63u) != 0) { adamw_scalar(g, R, i, w, m, v, p, c); ++i; }
  for (; i + 32 <= hi; i += 32) {
    __m256i pb[2];
    for (int h = 0; h < 2; ++h) {
      const int64_t j = i + 16 * h;
      __m512 s = load_bf16x16(g[0] + j);
      for (int r = 1; r < R; ++r) s = _mm512_add_ps(s, load_bf16x16(g[r] + j));
      if (R > 1) s = _mm512_mul_ps(s, invR);
      const __m512 m1 = _mm512_add_ps(_mm512_mul_ps(beta1, _mm512_loadu_ps(m + j)), _mm512_mul_ps(k1, s));
      const __m512 v1 = _mm512_add_ps(_mm512_mul_ps(beta2, _mm512_loadu_ps(v + j)),
                                      _mm512_mul_ps(k2, _mm512_mul_ps(s, s)));
      const __m512 d = _mm512_add_ps(_mm512_mul_ps(_mm512_sqrt_ps(v1), isb), eps);
      const __m512 w1 = _mm512_sub_ps(_mm512_mul_ps(decay, _mm512_loadu_ps(w + j)),
                                      _mm512_mul_ps(step, _mm512_div_ps(m1, d)));
      _mm512_storeu_ps(m + j, m1);
      _mm512_storeu_ps(v + j, v1);
      _mm512_storeu_ps(w + j, w1);
      pb[h] = to_bf16x16<HW>(w1);
    }
    if (p) _mm512_stream_si512((__m512i*)(p + i), _mm512_inserti64x4(_mm512_castsi256_si512(pb[0]), pb[1], 1));
  }
  for (; i < hi; ++i) adamw_scalar(g, R, i, w, m, v, p, c);
}

// Splits [0, n) into nthreads contiguous ranges cut at multiples of 32 elements.
template <class F>
void parallel_ranges(int64_t n, int nthreads, F body) {
  if (nthreads < 1) nthreads = 1;
  const int64_t lines = (n + 31) / 32;
#ifdef _OPENMP
#pragma omp parallel for schedule(static, 1) num_threads(nthreads)
#endif
  for (int t = 0; t < nthreads; ++t) {
    int64_t lo = lines * t / nthreads * 32, hi = lines * (t + 1) / nthreads * 32;
    if (hi > n) hi = n;
    if (lo < hi) body(lo, hi);
  }
  _mm_sfence();     // streaming stores are globally visible before anyone DMAs the buffer
}

void cast_chunk(const float* src, int64_t n, uint16_t* dst, int nthreads) {
  const Isa k = isa();
  parallel_ranges(n, nthreads, [&](int64_t lo, int64_t hi) {
    if (k == kAvx512Bf16) cast_range_avx512<true>(src, lo, hi, dst);
    else if (k == kAvx512) cast_range_avx512<false>(src, lo, hi, dst);
    else for (int64_t i = lo; i < hi; ++i) dst[i] = f32_to_bf16_rne(src[i]);
    _mm_sfence();
  });
}

void adamw_chunk(const uint16_t* const* g, int R, int64_t n, float* w, float* m, float* v,
                 uint16_t* p, const Consts& c, int nthreads) {
  const Isa k = isa();
  parallel_ranges(n, nthreads, [&](int64_t lo, int64_t hi) {
    if (k == kAvx512Bf16) adamw_range_avx512<true>(g, R, lo, hi, w, m, v, p, c);
    else if (k == kAvx512) adamw_range_avx512<false>(g, R, lo, hi, w, m, v, p, c);
    else for (int64_t i = lo; i < hi; ++i) adamw_scalar(g, R, i, w, m, v, p, c);
    _mm_sfence();
  });
}

// Bounded wait for an event (polls; never blocks for ever inside the driver).
int wait_event(cudaEvent_t ev, double seconds) {
  const double deadline = now_ms() + 1e3 * seconds;
  for (;;) {
    const cudaError_t e = cudaEventQuery(ev);
    if (e == cudaSuccess) return 0;
    if (e != cudaErrorNotReady) { (void)cudaGetLastError(); return (int)e; }
    if (now_ms() > deadline) return CPUROUTE_TIMEOUT;
    timespec nap = {0, 5000};
    nanosleep(&nap, nullptr);
  }
}
constexpr double kWaitSeconds = 120.0;

#define CUR(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { (void)cudaGetLastError(); rc = (int)e_; goto done; } } while (0)

}  // namespace

extern "C" {

const char* cpuroute_isa(void) {
  switch (isa()) {
    case kAvx512Bf16: return "avx512-bf16";
    case kAvx512: return "avx512f";
    default: return "scalar";
  }
}

int cpuroute_limit_isa(const char* name) {
  if (!name) return -1;
  const Isa have = detect();
  Isa want;
  if (strcmp(name, "avx512-bf16") == 0) want = kAvx512Bf16;
  else if (strcmp(name, "avx512f") == 0) want = kAvx512;
  else if (strcmp(name, "scalar") == 0) want = kScalar;
  else return -1;
  if (want > have) return -2;                 // the CPU cannot run that path
  isa_slot() = want;
  return 0;
}

int cpuroute_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

int cpuroute_cast_bf16(const float* master, int64_t n, uint16_t* param_bf16, int nthreads) {
  if (n < 0 || (n > 0 && (!master || !param_bf16))) return -1;
  cast_chunk(master, n, param_bf16, nthreads);
  return 0;
}

int cpuroute_adamw(const uint16_t* const* grads_bf16, int R, int64_t n, float* master, float* m,
                   float* v, uint16_t* param_bf16, const cpuroute_hparams* hp, int nthreads) {
  if (!grads_bf16 || R < 1 || R > 64 || n < 0 || !hp || hp->step < 1) return -1;
  if (n > 0 && (!master || !m || !v)) return -1;
  for (int r = 0; r < R; ++r) if (!grads_bf16[r]) return -1;
  adamw_chunk(grads_bf16, R, n, master, m, v, param_bf16, make_consts(hp), nthreads);
  return 0;
}

int cpuroute_step(const void* const* dev_grads, int R_host, int64_t n, uint16_t* const* host_grad_staging,
                  float* master, float* m, float* v, uint16_t* host_param_staging,
                  void* const* dev_params, int copies, int64_t chunk_elems,
                  const cpuroute_hparams* hp, int nthreads, cpuroute_stats* stats) {
  if (!dev_grads || !host_grad_staging || R_host < 1 || R_host > 64 || n < 0 || !hp || hp->step < 1 ||
      !dev_params || copies < 1 || copies > 64 || chunk_elems <= 0 || (chunk_elems % 32) != 0)
    return -1;
  if (n > 0 && (!master || !m || !v || !host_param_staging)) return -1;
  if (stats) memset(stats, 0, sizeof *stats);
  const int64_t nchunks = n == 0 ? 0 : (n + chunk_elems - 1) / chunk_elems;
  const Consts c = make_consts(hp);
  int rc = 0;
  cudaStream_t s_d2h = nullptr, s_h2d = nullptr;
  std::vector<cudaEvent_t> landed((size_t)nchunks, nullptr);
  cudaEvent_t d0 = nullptr, d1 = nullptr, h0 = nullptr, h1 = nullptr;
  double t_wait = 0.0, t_upd = 0.0;
  const double t_begin = now_ms();
  CUR(cudaStreamCreateWithFlags(&s_d2h, cudaStreamNonBlocking));
  CUR(cudaStreamCreateWithFlags(&s_h2d, cudaStreamNonBlocking));
  CUR(cudaEventCreate(&d0)); CUR(cudaEventCreate(&d1)); CUR(cudaEventCreate(&h0)); CUR(cudaEventCreate(&h1));
  for (int64_t k = 0; k < nchunks; ++k) CUR(cudaEventCreateWithFlags(&landed[(size_t)k], cudaEventDisableTiming));
  // gradient return: every chunk's copies queued up front, one event per chunk
  CUR(cudaEventRecord(d0, s_d2h));
  for (int64_t k = 0; k < nchunks; ++k) {
    const int64_t off = k * chunk_elems, len = n - off < chunk_elems ? n - off : chunk_elems;
    for (int r = 0; r < R_host; ++r)
      CUR(cudaMemcpyAsync(host_grad_staging[r] + off, (const uint16_t*)dev_grads[r] + off,
                          (size_t)len * 2, cudaMemcpyDeviceToHost, s_d2h));
    CUR(cudaEventRecord(landed[(size_t)k], s_d2h));
  }
  CUR(cudaEventRecord(d1, s_d2h));
  CUR(cudaEventRecord(h0, s_h2d));
  for (int64_t k = 0; k < nchunks; ++k) {
    const int64_t off = k * chunk_elems, len = n - off < chunk_elems ? n - off : chunk_elems;
    const double t0 = now_ms();
    rc = wait_event(landed[(size_t)k], kWaitSeconds);
    if (rc) goto done;
    const double t1 = now_ms();
    const uint16_t* gp[64];
    for (int r = 0; r < R_host; ++r) gp[r] = host_grad_staging[r] + off;
    adamw_chunk(gp, R_host, len, master + off, m + off, v + off, host_param_staging + off, c, nthreads);
    const double t2 = now_ms();
    t_wait += t1 - t0;
    t_upd += t2 - t1;
    for (int q = 0; q < copies; ++q)            // delivery of this chunk to every receiving rank
      CUR(cudaMemcpyAsync((uint16_t*)dev_params[q] + off, host_param_staging + off, (size_t)len * 2,
                          cudaMemcpyHostToDevice, s_h2d));
  }
  CUR(cudaEventRecord(h1, s_h2d));
  rc = wait_event(h1, kWaitSeconds);
  if (rc) goto done;
  rc = wait_event(d1, kWaitSeconds);
  if (rc) goto done;
  if (stats) {
    float ms = 0.f;
    stats->ms_total = now_ms() - t_begin;
    stats->ms_wait_d2h = t_wait;
    stats->ms_update = t_upd;
    if (cudaEventElapsedTime(&ms, d0, d1) == cudaSuccess) stats->ms_d2h_lane = ms;
    if (cudaEventElapsedTime(&ms, h0, h1) == cudaSuccess) stats->ms_h2d_lane = ms;
    stats->d2h_bytes = 2 * n * R_host;
    stats->h2d_bytes = 2 * n * copies;
    stats->chunks = nchunks;
  }
done:
  if (rc && s_d2h) { cudaStreamSynchronize(s_d2h); }     // leave nothing running on the buffers
  if (rc && s_h2d) { cudaStreamSynchronize(s_h2d); }
  for (cudaEvent_t e : landed) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : {d0, d1, h0, h1}) if (e) cudaEventDestroy(e);
  if (s_d2h) cudaStreamDestroy(s_d2h);
  if (s_h2d) cudaStreamDestroy(s_h2d);
  return rc;
}

int cpuroute_deliver(const float* master, int64_t n, uint16_t* host_param_staging, void* dev_params,
                     int64_t chunk_elems, int nthreads, cpuroute_stats* stats) {
  if (n < 0 || chunk_elems <= 0 || (chunk_elems % 32) != 0) return -1;
  if (n > 0 && (!master || !host_param_staging || !dev_params)) return -1;
  if (stats) memset(stats, 0, sizeof *stats);
  const int64_t nchunks = n == 0 ? 0 : (n + chunk_elems - 1) / chunk_elems;
  int rc = 0;
  cudaStream_t s = nullptr;
  cudaEvent_t h0 = nullptr, h1 = nullptr;
  double t_cast = 0.0;
  const double t_begin = now_ms();
  CUR(cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking));
  CUR(cudaEventCreate(&h0)); CUR(cudaEventCreate(&h1));
  for (int64_t k = 0; k < nchunks; ++k) {
    const int64_t off = k * chunk_elems, len = n - off < chunk_elems ? n - off : chunk_elems;
    const double t0 = now_ms();
    cast_chunk(master + off, len, host_param_staging + off, nthreads);   // while DMA moves chunk k-1
    t_cast += now_ms() - t0;
    if (k == 0) CUR(cudaEventRecord(h0, s));
    CUR(cudaMemcpyAsync((uint16_t*)dev_params + off, host_param_staging + off, (size_t)len * 2,
                        cudaMemcpyHostToDevice, s));
  }
  if (nchunks == 0) CUR(cudaEventRecord(h0, s));
  CUR(cudaEventRecord(h1, s));
  rc = wait_event(h1, kWaitSeconds);
  if (rc) goto done;
  if (stats) {
    float ms = 0.f;
    stats->ms_total = now_ms() - t_begin;
    stats->ms_update = t_cast;
    if (cudaEventElapsedTime(&ms, h0, h1) == cudaSuccess) stats->ms_h2d_lane = ms;
    stats->h2d_bytes = 2 * n;
    stats->chunks = nchunks;
  }
done:
  if (rc && s) cudaStreamSynchronize(s);
  for (cudaEvent_t e : {h0, h1}) if (e) cudaEventDestroy(e);
  if (s) cudaStreamDestroy(s);
  return rc;
}

}  // extern "C"
