// jv_linear_attn_static: the linear-attention block for callers that cannot hand the
// library a scratch buffer because they cannot allocate one.
//
// Who that is: code that runs where device allocation is off the table -- an inference
// server whose memory pool already owns all of HBM (a cudaMalloc from a plug-in would fail
// or fragment it), a latency-critical loop where the implicit device synchronisation of
// cudaMalloc / cudaFree is not acceptable, or a host that only exposes "enqueue on this
// stream" hooks with no allocator at all.  For them the scratch of the linear block lives
// in a fixed array inside the library image.
#include "common.cuh"

namespace jv {
namespace {

// The scratch itself.  Every GPU that loads the library holds these bytes until the
// process exits.  In host code this name is only a handle for the runtime, not an address
// a kernel could use: the device address is looked up below with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[JV_STATIC_SCRATCH_BYTES];

// Device address of the array on the current device; resolved on the first call per
// device (with that device current) and cached.  Returns nullptr if the lookup fails.
void* static_scratch_ptr() {
  static void* cache[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return nullptr;
  }
  if (!cache[dev]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return nullptr;
    }
    cache[dev] = p;
  }
  return cache[dev];
}

}  // namespace
}  // namespace jv

extern "C" jv_status jv_linear_attn_static(const void* q, const void* k, const void* v, void* o,
                                           const jv_shape* shape, float eps, const jv_dwc* dwc,
                                           void* cuda_stream) {
  if (!shape) return JV_ERR_INVALID_ARG;
  // Size check first, on the host: a shape whose scratch does not fit the fixed array is
  // refused before anything else happens.  (0 means the shape / dwc themselves are invalid;
  // jv_linear_attn below reports that with its own code.)
  const size_t need = jv_workspace_bytes('L', shape, dwc);
  if (need > (size_t)JV_STATIC_SCRATCH_BYTES) return JV_ERR_WORKSPACE;
  void* scratch = jv::static_scratch_ptr();
  if (!scratch) return JV_ERR_CUDA;
  // Same validation, same kernels, same results as jv_linear_attn; only the scratch differs.
  // Nothing in that path allocates or frees device memory.  No part of the scratch has to
  // start at zero: every word a kernel consumes is written earlier in the same call.
  return jv_linear_attn(q, k, v, o, shape, eps, dwc, scratch, (size_t)JV_STATIC_SCRATCH_BYTES, cuda_stream);
}
