// caat_rowpar_forward_noalloc: the forward of one row-parallel layer for callers that
// cannot hand the library a workspace because they cannot allocate device memory at the
// time of the call.  Its scratch is a fixed array that lives in the library's device image.
#include <mutex>

#include "caat_internal.h"

namespace {

// Scratch of the forward (shared part of the layer output once, private part per rank).
// Every GPU that loads the library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[CAAT_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};   // device address of g_noalloc_scratch, per device ordinal

// In host code the array's name is only a handle: the address kernels must be given is the one
// cudaGetSymbolAddress returns for the CURRENT device.  Looked up once per device.
// (With lazy module loading that first lookup is also what makes the driver load this file's device
// image and reserve the array on the device: it can fail for lack of memory, and it is the reason
// the first call per device belongs at start-up.)
caat_status scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return caat::cuda_fail(e);
  if (dev < 0 || dev >= kMaxDevices) return caat::cuda_fail(cudaErrorInvalidDevice);
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return caat::cuda_fail(e);
    if (p == nullptr) return caat::cuda_fail(cudaErrorInvalidSymbol);
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return CAAT_OK;
}

}  // namespace

extern "C" caat_status caat_rowpar_forward_noalloc(const caat_ctx* ctx, caat_layer layer, int tokens, const void* Y,
                                                   const void* W, const void* R, const void* gamma,
                                                   const void* beta, void* Hn, void* X, float* rstd, float* mean,
                                                   void* cuda_stream) {
  if (!ctx) return CAAT_EINVAL;
  const size_t need = caat_workspace_bytes(ctx, layer, tokens, 0);
  if (need == 0) {
    // let the regular entry point name the argument error (it fails before any launch)
    return caat_rowpar_forward(ctx, layer, tokens, Y, W, R, gamma, beta, Hn, X, rstd, mean, nullptr, 0, cuda_stream);
  }
  if (need > (size_t)CAAT_NOALLOC_SCRATCH_BYTES) return CAAT_ELIMIT;
  void* scratch = nullptr;
  const caat_status s = scratch_address(&scratch);
  if (s != CAAT_OK) return s;
  // Nothing in this scratch has to start at zero: every element the row kernel reads was
  // written by the GEMM earlier in the same call, so the previous call's contents are harmless.
  return caat_rowpar_forward(ctx, layer, tokens, Y, W, R, gamma, beta, Hn, X, rstd, mean, scratch,
                             (size_t)CAAT_NOALLOC_SCRATCH_BYTES, cuda_stream);
}
