// libslidedp: sharing device buffers between the processes of a multi-rank step (one process per
// GPU): export a handle for a caller-owned device buffer, map a peer's handle, unmap it.
// See include/slidedp.h for the contract of every entry point.
//
// The mapped pointers are only ever handed to this library's own kernels, which read and write
// them with plain global loads and stores.
#include "internal.h"

#include <cuda.h>
#include <string.h>

using namespace slidedp;
using namespace slidedp::host;

namespace {

static_assert(sizeof(cudaIpcMemHandle_t) == 64, "handle layout");
static_assert(sizeof(slidedp_ipc_handle) == 80, "handle layout");

typedef CUresult (*mem_get_address_range_fn)(CUdeviceptr*, size_t*, CUdeviceptr);

// Base address and size of the allocation that contains `p`, through the driver entry point
// (the runtime has no call for it; the library does not link against the driver library).
int allocation_of(slidedp_ctx* ctx, const void* p, char** base, size_t* size) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult found = cudaDriverEntryPointSymbolNotFound;
  CU(cudaGetDriverEntryPoint("cuMemGetAddressRange", &fn, cudaEnableDefault, &found));
  if (!fn || found != cudaDriverEntryPointSuccess) return cuda_fail(ctx, cudaErrorNotSupported);
  CUdeviceptr b = 0;
  size_t s = 0;
  if (reinterpret_cast<mem_get_address_range_fn>(fn)(&b, &s, (CUdeviceptr)(uintptr_t)p) != CUDA_SUCCESS)
    return cuda_fail(ctx, cudaErrorInvalidValue);
  *base = reinterpret_cast<char*>((uintptr_t)b);
  *size = s;
  return SLIDEDP_OK;
}

}  // namespace

extern "C" {

int slidedp_ipc_export(slidedp_ctx* ctx, const void* dev_ptr, slidedp_ipc_handle* out) {
  if (!ctx || !dev_ptr || !out) return SLIDEDP_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  char* base = nullptr;
  size_t size = 0;
  int rc = allocation_of(ctx, dev_ptr, &base, &size);
  if (rc != SLIDEDP_OK) return rc;
  cudaIpcMemHandle_t h;
  CU(cudaIpcGetMemHandle(&h, base));
  memset(out, 0, sizeof *out);
  memcpy(out->opaque, &h, sizeof h);
  out->offset = (uint64_t)(static_cast<const char*>(dev_ptr) - base);
  out->bytes = (uint64_t)size - out->offset;
  return SLIDEDP_OK;
}

int slidedp_ipc_open(slidedp_ctx* ctx, const slidedp_ipc_handle* handle, void** dev_ptr_out) {
  if (!ctx || !handle || !dev_ptr_out) return SLIDEDP_ERR_INVALID_ARG;
  *dev_ptr_out = nullptr;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  // one mapping per exported allocation: a second buffer of the same allocation (a caching
  // allocator packs several into one) shares it and only counts a reference
  for (IpcMapping& m : ctx->ipc)
    if (memcmp(m.opaque, handle->opaque, sizeof m.opaque) == 0) {
      m.refs += 1;
      *dev_ptr_out = m.base + handle->offset;
      return SLIDEDP_OK;
    }
  cudaIpcMemHandle_t h;
  memcpy(&h, handle->opaque, sizeof h);
  void* base = nullptr;
  CU(cudaIpcOpenMemHandle(&base, h, cudaIpcMemLazyEnablePeerAccess));
  IpcMapping m;
  memcpy(m.opaque, handle->opaque, sizeof m.opaque);
  m.base = static_cast<char*>(base);
  m.bytes = handle->offset + handle->bytes;
  m.refs = 1;
  ctx->ipc.push_back(m);
  *dev_ptr_out = m.base + handle->offset;
  return SLIDEDP_OK;
}

int slidedp_ipc_close(slidedp_ctx* ctx, void* dev_ptr) {
  if (!ctx || !dev_ptr) return SLIDEDP_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return cuda_fail(ctx, cudaErrorInvalidDevice);
  const char* p = static_cast<const char*>(dev_ptr);
  for (size_t i = 0; i < ctx->ipc.size(); ++i) {
    IpcMapping& m = ctx->ipc[i];
    if (p < m.base || p >= m.base + m.bytes) continue;
    if (m.refs > 1) { m.refs -= 1; return SLIDEDP_OK; }
    CU(cudaIpcCloseMemHandle(m.base));       // on failure the mapping stays recorded
    ctx->ipc.erase(ctx->ipc.begin() + (long)i);
    return SLIDEDP_OK;
  }
  return SLIDEDP_ERR_INVALID_ARG;      // not a pointer this context mapped
}

}  // extern "C"
