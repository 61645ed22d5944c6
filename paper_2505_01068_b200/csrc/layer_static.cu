// gsit_im_layer_fwd_static: the IM encoder layer for callers that cannot hand over scratch memory.
//
// Some hosts of this library may not allocate device memory at all: a plug-in that runs inside another
// process's memory budget, a real-time loop in which an allocation could stall or synchronise the device, or
// code that runs after the application has frozen its memory pools.  gsit_im_layer_fwd needs a caller-provided
// workspace, which such a caller has no means to create, so this variant keeps the scratch in a fixed array that
// is part of the loaded library image.
#include <cuda_runtime.h>
#include <stdint.h>

#include "gsit.h"

namespace {

// The scratch itself.  It exists once per GPU that loads the library and is released only when the process
// exits; its contents survive from one call to the next.
static __device__ __align__(256) unsigned char g_static_layer_scratch[GSIT_STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
void* g_scratch_addr[MAX_DEVICES] = {};  // device address of the array on each GPU, looked up on first use

// In host code `g_static_layer_scratch` is only a handle; the address a kernel can use has to be asked for, with
// the GPU in question current.
cudaError_t scratch_address(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress((void**)&p, g_static_layer_scratch);
    if (e != cudaSuccess) return e;
    if (p == nullptr) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" gsit_status gsit_im_layer_fwd_static(const gsit_shape* shape, const gsit_layer_weights* weights,
                                                const float* x, int64_t x_row_stride, float* y,
                                                int64_t y_row_stride, gsit_stream stream) {
  if (shape == nullptr || weights == nullptr) return GSIT_ERR_INVALID_ARG;
  const size_t need = gsit_workspace_bytes(shape, GSIT_CALL_LAYER, weights->d_ff);
  if (need == (size_t)-1) return GSIT_ERR_INVALID_ARG;
  if (need > (size_t)GSIT_STATIC_SCRATCH_BYTES) return GSIT_ERR_WORKSPACE;  // problem too large for the fixed array
  void* scratch = nullptr;
  if (scratch_address(&scratch) != cudaSuccess) return GSIT_ERR_CUDA;
  // Every scratch row that contributes to a real output row is written before it is read, so nothing has to be
  // cleared even though the array still holds the previous call's intermediate results.  (Row tiles may read a few
  // stale rows past the last real one; what is computed from them is discarded.)
  return gsit_im_layer_fwd(shape, weights, x, x_row_stride, y, y_row_stride, scratch,
                           (size_t)GSIT_STATIC_SCRATCH_BYTES, stream);
}
