// Small device helpers shared by the kernels of libslidedp: BF16 packing and streaming accesses.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace slidedp {

// ---- small helpers -----------------------------------------------------------------

__device__ __forceinline__ float bf16_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t x) { return __uint_as_float(x & 0xFFFF0000u); }

// FP32 -> BF16 bits, round to nearest even, NaN stays NaN.
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float x) {
  uint16_t r;
  asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(r) : "f"(x));
  return (uint32_t)r;
}

// Streaming (read-once / write-once) 128-bit accesses: keep them out of L1 and mark them
// evict-first in L2, since nothing on this path is ever re-read.
__device__ __forceinline__ uint4 ld_stream(const void* p) {
  return __ldcs(reinterpret_cast<const uint4*>(p));
}
__device__ __forceinline__ void st_stream(void* p, uint4 v) {
  __stcs(reinterpret_cast<uint4*>(p), v);
}

// Programmatic dependent launch: a kernel launched with the programmatic-stream-serialization
// attribute may be scheduled while the kernel before it in the stream is still finishing; this
// wait holds it until that kernel has completed and its writes are visible. Launched the plain
// way the instruction does nothing. Every kernel that can be launched that way executes it
// before its first global-memory access.
__device__ __forceinline__ void wait_for_previous_kernel() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

}  // namespace slidedp
