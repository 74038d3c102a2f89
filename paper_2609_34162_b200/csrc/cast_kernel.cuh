// The parameter-delivery cast kernel of libslidedp (sm_100a).
#pragma once

#include "device_utils.cuh"

namespace slidedp {

// Parameter delivery: FP32 master -> BF16 copy.
// Eight elements per thread: two 16-byte loads, one 16-byte store, round to nearest even.
// HBM traffic is 6 bytes per parameter, but the kernel always runs behind an H2D copy of the
// same chunk (4 bytes per parameter over the host link), which is the bound.
constexpr int kCastThreads = 256;
__global__ void __launch_bounds__(kCastThreads)
cast_master_to_bf16_kernel(const float* __restrict__ master, int64_t n,
                           uint16_t* __restrict__ param_out) {
  const int64_t base = ((int64_t)blockIdx.x * kCastThreads + threadIdx.x) * 8;
  if (base >= n) return;
  if (base + 8 <= n) {
    const uint4 a = ld_stream(master + base), b = ld_stream(master + base + 4);
    uint4 o;
    o.x = f32_to_bf16_bits(__uint_as_float(a.x)) | (f32_to_bf16_bits(__uint_as_float(a.y)) << 16);
    o.y = f32_to_bf16_bits(__uint_as_float(a.z)) | (f32_to_bf16_bits(__uint_as_float(a.w)) << 16);
    o.z = f32_to_bf16_bits(__uint_as_float(b.x)) | (f32_to_bf16_bits(__uint_as_float(b.y)) << 16);
    o.w = f32_to_bf16_bits(__uint_as_float(b.z)) | (f32_to_bf16_bits(__uint_as_float(b.w)) << 16);
    st_stream(param_out + base, o);
  } else {
    for (int64_t i = base; i < n; ++i) param_out[i] = (uint16_t)f32_to_bf16_bits(master[i]);
  }
}

}  // namespace slidedp
