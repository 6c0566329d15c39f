// Measurement aid: a kernel that only reads a buffer, with the same partition
// as the decode kernels (one CTA per SM, each CTA one contiguous range).  Its
// time is the ceiling any kernel that has to stream that many bytes from HBM
// can reach under the same launch conditions, so decode times are reported
// next to it.
#include "common.cuh"

namespace peqa {

namespace {

constexpr int kProbeThreads = 1024;

__global__ void __launch_bounds__(kProbeThreads, 1)
read_probe_kernel(const uint4* __restrict__ src, size_t n16, uint32_t* __restrict__ sink) {
  const size_t per = (n16 + gridDim.x - 1) / gridDim.x;
  const size_t lo = (size_t)blockIdx.x * per;
  const size_t hi = lo + per < n16 ? lo + per : n16;
  uint32_t acc = 0;
  size_t i = lo + threadIdx.x;
  // four independent 16-byte loads in flight per thread
  for (; i + 3 * (size_t)kProbeThreads < hi; i += 4 * (size_t)kProbeThreads) {
    const uint4 a = __ldcs(src + i);
    const uint4 b = __ldcs(src + i + kProbeThreads);
    const uint4 c = __ldcs(src + i + 2 * kProbeThreads);
    const uint4 d = __ldcs(src + i + 3 * kProbeThreads);
    acc ^= a.x ^ a.y ^ a.z ^ a.w ^ b.x ^ b.y ^ b.z ^ b.w ^ c.x ^ c.y ^ c.z ^ c.w ^ d.x ^ d.y ^
           d.z ^ d.w;
  }
  for (; i < hi; i += kProbeThreads) {
    const uint4 a = __ldcs(src + i);
    acc ^= a.x ^ a.y ^ a.z ^ a.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
  __shared__ uint32_t warp_acc[kProbeThreads / 32];
  if ((threadIdx.x & 31) == 0) warp_acc[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t r = 0;
    for (int w = 0; w < kProbeThreads / 32; ++w) r ^= warp_acc[w];
    sink[blockIdx.x] = r;
  }
}

}  // namespace

}  // namespace peqa

using namespace peqa;

extern "C" int peqa_probe_read(const void* src, size_t bytes, uint32_t* sink, size_t sink_bytes,
                               void* stream) {
  if (!src || !sink) return PEQA_ERR_NULL;
  if (bytes == 0 || bytes % 16 != 0) return PEQA_ERR_BAD_SHAPE;
  if (!aligned16(src)) return PEQA_ERR_ALIGNMENT;
  int sms = 0, dev = 0;
  PEQA_CUDA(cudaGetDevice(&dev));
  PEQA_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  if (sink_bytes < (size_t)sms * sizeof(uint32_t)) return PEQA_ERR_WORKSPACE;
  read_probe_kernel<<<sms, kProbeThreads, 0, as_stream(stream)>>>(
      static_cast<const uint4*>(src), bytes / 16, sink);
  PEQA_CUDA(cudaGetLastError());
  return PEQA_OK;
}
