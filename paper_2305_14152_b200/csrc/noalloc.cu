// Scale gradient for callers that cannot provide scratch memory.
//
// peqa_qlinear_bwd needs a caller-allocated workspace for dS whenever a
// quantization group is wider than one 128-column piece (per-channel layers
// above all).  Some callers have no way to get one: code running where
// cudaMalloc is forbidden (inside a region that must not touch the allocator,
// a plugin that is only handed its input and output buffers, a process whose
// memory pool is owned and fully sized by another component).  For them the
// partial sums live in a fixed array that is part of this library's device
// image.  Every GPU that loads the library carries the array until the process
// exits.
#include <mutex>

#include "common.cuh"

namespace peqa {

namespace {

constexpr size_t kScratchFloats = (size_t)2 << 20;          // 2 Mi floats = 8 MiB per device
static __device__ __align__(256) float g_ds_scratch[kScratchFloats];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
float* g_scratch_ptr[kMaxDevices] = {nullptr};

// In host code `g_ds_scratch` is only a handle for the runtime, not an
// address the GPU can use; the device address has to be asked for, once per
// device, with that device current.
int scratch_for_current_device(float** out) {
  int dev = 0;
  PEQA_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return PEQA_ERR_TOO_LARGE;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    float* p = nullptr;
    PEQA_CUDA(cudaGetSymbolAddress((void**)&p, g_ds_scratch));
    if (!p) return cuda_fail(cudaErrorInvalidSymbol);
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return PEQA_OK;
}

}  // namespace

}  // namespace peqa

using namespace peqa;

extern "C" size_t peqa_bwd_ds_static_capacity_bytes(void) { return kScratchFloats * sizeof(float); }

extern "C" int peqa_qlinear_bwd_ds_static(const peqa_qweight_t* w, const void* X, const void* dY,
                                          int T, float* dS, void* stream) {
  int g = 0, G = 0;
  PEQA_TRY(check_qweight(w, &g, &G));
  if (!X || !dY || !dS) return PEQA_ERR_NULL;
  if (T <= 0 || w->in_features % 64 != 0 || w->out_features % 8 != 0) return PEQA_ERR_BAD_SHAPE;
  if (!aligned16(X) || !aligned16(dY) || !aligned16(dS)) return PEQA_ERR_ALIGNMENT;
  const size_t need = ds_workspace_bytes(w, g, T);
  if (need > kScratchFloats * sizeof(float)) return PEQA_ERR_TOO_LARGE;
  PEQA_TRY(check_arch());
  float* scratch = nullptr;
  if (need > 0) PEQA_TRY(scratch_for_current_device(&scratch));
  // Every partial sum the reduction reads is written by the gradient kernel of
  // the same call first, so nothing in the array has to start at zero.
  return launch_ds(w, nullptr, g, X, dY, T, dS, nullptr, nullptr, scratch, need, as_stream(stream));
}
