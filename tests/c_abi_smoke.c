/* The C ABI used from plain C, with no Python in between: one clipped step of a small chunk
 * through libslidedp (device-resident, then host-resident through pinned memory, then the BF16
 * delivery of the new master), compared with the C oracle under the benchmark's tolerances. Built and
 * run by tests/test_c_abi_program.py (gcc, links libslidedp, the oracle and the CUDA runtime).
 * Exit code 0 and a line starting with "PASS" on success. */
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "slidedp.h"
#include "slidedp_oracle.h"

#define CHECK_CUDA(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { \
  printf("FAIL cuda %s at line %d\n", cudaGetErrorString(e_), __LINE__); return 2; } } while (0)
#define CHECK_SD(x) do { int r_ = (x); if (r_ != SLIDEDP_OK) { \
  printf("FAIL libslidedp: %s at line %d\n", slidedp_strerror(r_), __LINE__); return 3; } } while (0)

static uint32_t lcg(uint32_t* s) { *s = *s * 1664525u + 1013904223u; return *s; }
static float uniform(uint32_t* s) { return (float)(lcg(s) >> 8) / 16777216.0f - 0.5f; }

int main(void) {
  enum { R = 3 };
  const int64_t n = 100003;
  uint32_t seed = 12345u;
  uint16_t* hg[R];
  float *hw = malloc(n * 4), *hm = malloc(n * 4), *hv = malloc(n * 4);
  uint16_t* hp = malloc(n * 2);
  for (int r = 0; r < R; ++r) {
    hg[r] = malloc(n * 2);
    for (int64_t i = 0; i < n; ++i) hg[r][i] = oracle_f32_to_bf16(4e-3f * uniform(&seed));
  }
  for (int64_t i = 0; i < n; ++i) {
    hw[i] = 0.05f * uniform(&seed);
    hm[i] = 1e-3f * uniform(&seed);
    hv[i] = 1e-6f * (uniform(&seed) + 0.5f);
  }
  slidedp_hparams hp_sd = {1e-5, 0.9, 0.95, 1e-8, 0.1, 1.0 / R, 0.05, 7};
  oracle_hparams hp_or = {1e-5, 0.9, 0.95, 1e-8, 0.1, 1.0 / R, 0.05, 7};

  /* device side */
  void* dg[R];
  float *dw, *dm, *dv;
  void* dp;
  for (int r = 0; r < R; ++r) {
    CHECK_CUDA(cudaMalloc(&dg[r], n * 2));
    CHECK_CUDA(cudaMemcpy(dg[r], hg[r], n * 2, cudaMemcpyHostToDevice));
  }
  CHECK_CUDA(cudaMalloc((void**)&dw, n * 4)); CHECK_CUDA(cudaMalloc((void**)&dm, n * 4));
  CHECK_CUDA(cudaMalloc((void**)&dv, n * 4)); CHECK_CUDA(cudaMalloc(&dp, n * 2));
  CHECK_CUDA(cudaMemcpy(dw, hw, n * 4, cudaMemcpyHostToDevice));
  CHECK_CUDA(cudaMemcpy(dm, hm, n * 4, cudaMemcpyHostToDevice));
  CHECK_CUDA(cudaMemcpy(dv, hv, n * 4, cudaMemcpyHostToDevice));
  slidedp_ctx* ctx = NULL;
  CHECK_SD(slidedp_create(&ctx, 0, 0));
  double norm = 0, coef = 0;
  CHECK_SD(slidedp_grad_norm(ctx, (const void* const*)dg, R, n, 1.0 / R, 1, NULL));
  CHECK_SD(slidedp_grad_norm_finish(ctx, hp_sd.max_norm, &norm, &coef, NULL));
  CHECK_SD(slidedp_reduce_adamw_chunk(ctx, (const void* const*)dg, R, n, dw, dm, dv, dp, &hp_sd, NULL));
  CHECK_CUDA(cudaDeviceSynchronize());
  float *gw = malloc(n * 4), *gm = malloc(n * 4), *gv = malloc(n * 4);
  uint16_t* gp = malloc(n * 2);
  CHECK_CUDA(cudaMemcpy(gw, dw, n * 4, cudaMemcpyDeviceToHost));
  CHECK_CUDA(cudaMemcpy(gm, dm, n * 4, cudaMemcpyDeviceToHost));
  CHECK_CUDA(cudaMemcpy(gv, dv, n * 4, cudaMemcpyDeviceToHost));
  CHECK_CUDA(cudaMemcpy(gp, dp, n * 2, cudaMemcpyDeviceToHost));
  const int64_t launches = slidedp_kernel_launches(ctx);

  /* host-resident: the same step with the FP32 state in page-locked host memory, streamed in
   * chunks of 8192 parameters through three slots; then the BF16 delivery of the new master */
  float *pw, *pm, *pv;
  void *dp2, *dp3;
  CHECK_CUDA(cudaMallocHost((void**)&pw, n * 4)); CHECK_CUDA(cudaMallocHost((void**)&pm, n * 4));
  CHECK_CUDA(cudaMallocHost((void**)&pv, n * 4));
  CHECK_CUDA(cudaMalloc(&dp2, n * 2)); CHECK_CUDA(cudaMalloc(&dp3, n * 2));
  memcpy(pw, hw, n * 4); memcpy(pm, hm, n * 4); memcpy(pv, hv, n * 4);
  slidedp_stats st;
  CHECK_SD(slidedp_stream_step(ctx, (const void* const*)dg, R, n, pw, pm, pv, dp2, 8192, 3, 0, &hp_sd, &st));
  slidedp_stats dst;
  CHECK_SD(slidedp_deliver_params(ctx, pw, n, dp3, 16384, 2, &dst));
  /* the same step once more, enqueued only and then waited for, on a second copy of the state;
   * and the host-link probe on the (now free) pinned buffers of that copy */
  float *qw, *qm, *qv;
  void* dp4;
  CHECK_CUDA(cudaMallocHost((void**)&qw, n * 4)); CHECK_CUDA(cudaMallocHost((void**)&qm, n * 4));
  CHECK_CUDA(cudaMallocHost((void**)&qv, n * 4)); CHECK_CUDA(cudaMalloc(&dp4, n * 2));
  memcpy(qw, hw, n * 4); memcpy(qm, hm, n * 4); memcpy(qv, hv, n * 4);
  CHECK_SD(slidedp_set_wait_seconds(ctx, 60.0));
  CHECK_SD(slidedp_stream_step_async(ctx, (const void* const*)dg, R, n, qw, qm, qv, dp4, 4096, 2, 1, &hp_sd));
  CHECK_SD(slidedp_stream_wait(ctx));
  const int async_same = memcmp(qw, pw, n * 4) == 0 && memcmp(qm, pm, n * 4) == 0 && memcmp(qv, pv, n * 4) == 0;
  /* the step once more as a two-layer call (the two halves of the chunk, one global norm) */
  float *rw, *rm, *rv;
  void* dp5;
  CHECK_CUDA(cudaMallocHost((void**)&rw, n * 4)); CHECK_CUDA(cudaMallocHost((void**)&rm, n * 4));
  CHECK_CUDA(cudaMallocHost((void**)&rv, n * 4)); CHECK_CUDA(cudaMalloc(&dp5, n * 2));
  memcpy(rw, hw, n * 4); memcpy(rm, hm, n * 4); memcpy(rv, hv, n * 4);
  const int64_t half = 50000;                       /* a multiple of 8: both halves stay aligned */
  const void* g0[R]; const void* g1[R];
  for (int r = 0; r < R; ++r) { g0[r] = dg[r]; g1[r] = (const uint16_t*)dg[r] + half; }
  slidedp_layer layers[2] = {{g0, half, rw, rm, rv, dp5},
                             {g1, n - half, rw + half, rm + half, rv + half, (uint16_t*)dp5 + half}};
  slidedp_stats lst;
  CHECK_SD(slidedp_stream_layers(ctx, layers, 2, R, 8192, 3, &hp_sd, &lst));
  /* the layer cut is not at a norm-tile boundary, so the norm agrees to rounding (not to the
   * bit) and the state is compared under the benchmark's tolerance */
  int64_t layers_bad = 0;
  const float *la[3] = {rw, rm, rv}, *lb[3] = {pw, pm, pv};
  for (int a = 0; a < 3; ++a)
    for (int64_t i = 0; i < n; ++i)
      if (!(fabs((double)la[a][i] - lb[a][i]) <= fmax(1e-6 * fabs((double)lb[a][i]), 1e-12))) ++layers_bad;
  const int layers_same = layers_bad == 0 && fabs(lst.norm - norm) <= 1e-12 * norm &&
                          lst.chunks == (half + 8191) / 8192 + (n - half + 8191) / 8192;
  slidedp_ipc_handle ih;
  CHECK_SD(slidedp_ipc_export(ctx, (const char*)dp5 + 64, &ih));
  double mix_gbs = 0;
  CHECK_SD(slidedp_hbm_mix_probe(ctx, (const void* const*)dg, R, n, dw, dm, dv, dp5, 2, &mix_gbs, NULL));
  double link[4] = {0, 0, 0, 0};
  CHECK_SD(slidedp_link_probe(ctx, qm, qv, dw, dm, (size_t)n * 4, 65536, 1, link));
  uint16_t *gp2 = malloc(n * 2), *gp3 = malloc(n * 2), *want3 = malloc(n * 2);
  CHECK_CUDA(cudaMemcpy(gp2, dp2, n * 2, cudaMemcpyDeviceToHost));
  CHECK_CUDA(cudaMemcpy(gp3, dp3, n * 2, cudaMemcpyDeviceToHost));
  CHECK_SD(slidedp_destroy(ctx));

  /* oracle side */
  double onorm = 0, ocoef = 0;
  if (oracle_step((const uint16_t* const*)hg, R, n, hw, hm, hv, hp, 0, &hp_or, &onorm, &ocoef, 1)) {
    printf("FAIL oracle_step\n");
    return 4;
  }
  int64_t bad = 0, bf16_differ = 0;
  const float* got[3] = {gw, gm, gv};
  const float* want[3] = {hw, hm, hv};
  for (int a = 0; a < 3; ++a)
    for (int64_t i = 0; i < n; ++i) {
      const double y = want[a][i], err = fabs((double)got[a][i] - y);
      const double allowed = fmax(1e-6 * fabs(y), 1e-12);
      if (!(err <= allowed)) ++bad;
    }
  for (int64_t i = 0; i < n; ++i) bf16_differ += gp[i] != hp[i];
  /* the host-resident state and BF16 copy equal the device-resident ones bit for bit, the
   * statistics carry the same norm, and the delivery is the oracle's cast of that master */
  int64_t host_differs = 0, delivery_differs = 0;
  const float* hgot[3] = {pw, pm, pv};
  for (int a = 0; a < 3; ++a) host_differs += memcmp(hgot[a], got[a], n * 4) != 0;
  host_differs += memcmp(gp2, gp, n * 2) != 0;
  oracle_cast_master_to_bf16(pw, n, want3);
  for (int64_t i = 0; i < n; ++i) delivery_differs += gp3[i] != want3[i];
  const int host_ok = layers_same && ih.offset >= 64 && mix_gbs > 0 && async_same && link[0] > 0 && link[1] > 0 && link[2] > 0 && link[3] > 0 &&
                      host_differs == 0 && delivery_differs == 0 && st.chunks == (n + 8191) / 8192 &&
                      st.norm == norm && st.clip_coef == coef && dst.chunks == (n + 16383) / 16384;
  const int ok = bad == 0 && bf16_differ <= n / 10000 && fabs(norm - onorm) <= 1e-6 * onorm &&
                 fabs(coef - ocoef) <= 1e-6 * ocoef && ocoef < 1.0 && launches == 3 && host_ok;
  printf("%s n=%lld R=%d norm=%.12g (oracle %.12g) coef=%.6f fp32_outside=%lld bf16_differ=%lld launches=%lld "
         "host_resident_differs=%lld delivery_differs=%lld chunks=%lld\n",
         ok ? "PASS" : "FAIL", (long long)n, R, norm, onorm, coef, (long long)bad,
         (long long)bf16_differ, (long long)launches, (long long)host_differs,
         (long long)delivery_differs, (long long)st.chunks);
  return ok ? 0 : 1;
}
