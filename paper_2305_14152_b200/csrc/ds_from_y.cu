// Per-channel scale gradient from the stored forward output.
//
// With one scale per output channel, Eq. 2 reads Y[t,i] = s[i] * u[t,i] with
// u = X (Q - z)^T, and the chain rule gives dS[i] = sum_t dY[t,i] u[t,i], that is
//   dS[i] = ( sum_t dY[t,i] * Y[t,i] ) / s[i].
// A layer that kept its bf16 output therefore needs no third contraction: the
// gradient is a column sum over two [T, N] tensors, bound by reading them once
// (4*T*N bytes), instead of 2*T*N*K flop.  What it costs is the bf16 rounding of
// Y (about 1e-3 relative on dS).
//
// Kernel 1: a thread owns 8 adjacent channels (one 16-byte load of each tensor
// per token) and a slice of the tokens; partial sums go to the workspace
// [slices][N].  Kernel 2 adds the slices in index order and divides by s.  No
// atomics: the result does not depend on timing.
#include <cuda_bf16.h>

#include "common.cuh"

namespace peqa {

namespace {

constexpr int kYThreads = 128;
constexpr int kYCols = kYThreads * 8;   // channels per CTA

__device__ __forceinline__ void fma_bf16x2(uint32_t a, uint32_t b, float& lo, float& hi) {
  lo = fmaf(__uint_as_float(a << 16), __uint_as_float(b << 16), lo);
  hi = fmaf(__uint_as_float(a & 0xFFFF0000u), __uint_as_float(b & 0xFFFF0000u), hi);
}

__global__ void __launch_bounds__(kYThreads)
ds_from_y_partial_kernel(const uint4* __restrict__ dY, const uint4* __restrict__ Y, int T, int N,
                         int tokens_per_slice, float* __restrict__ partial) {
  const int c8 = blockIdx.x * kYThreads + threadIdx.x;        // group of 8 channels
  if (c8 * 8 >= N) return;
  const int row16 = N >> 3;                                   // 16-byte units per token row
  const int t0 = blockIdx.y * tokens_per_slice;
  const int t1 = min(T, t0 + tokens_per_slice);
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  int t = t0;
  for (; t + 4 <= t1; t += 4) {
    uint4 a[4], b[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      a[u] = __ldg(dY + (size_t)(t + u) * row16 + c8);
      b[u] = __ldg(Y + (size_t)(t + u) * row16 + c8);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      fma_bf16x2(a[u].x, b[u].x, acc[0], acc[1]);
      fma_bf16x2(a[u].y, b[u].y, acc[2], acc[3]);
      fma_bf16x2(a[u].z, b[u].z, acc[4], acc[5]);
      fma_bf16x2(a[u].w, b[u].w, acc[6], acc[7]);
    }
  }
  for (; t < t1; ++t) {
    const uint4 a = __ldg(dY + (size_t)t * row16 + c8);
    const uint4 b = __ldg(Y + (size_t)t * row16 + c8);
    fma_bf16x2(a.x, b.x, acc[0], acc[1]);
    fma_bf16x2(a.y, b.y, acc[2], acc[3]);
    fma_bf16x2(a.z, b.z, acc[4], acc[5]);
    fma_bf16x2(a.w, b.w, acc[6], acc[7]);
  }
  float4* out = reinterpret_cast<float4*>(partial + (size_t)blockIdx.y * N + (size_t)c8 * 8);
  out[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
  out[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
}

__global__ void ds_from_y_finish_kernel(const float* __restrict__ partial, const float* __restrict__ scales,
                                        int N, int slices, float* __restrict__ dS) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  float acc = 0.0f;
  for (int q = 0; q < slices; ++q) acc += partial[(size_t)q * N + i];
  dS[i] = __fdiv_rn(acc, scales[i]);
}

// Token slices: enough CTAs for a few waves of the machine, at least 32 tokens each.
int ds_from_y_slices(int N, int T) {
  const int col_blocks = (N + kYCols - 1) / kYCols;
  int slices = (sm_count_or(148) * 8 + col_blocks - 1) / col_blocks;
  const int max_slices = (T + 31) / 32;
  if (slices > max_slices) slices = max_slices;
  if (slices < 1) slices = 1;
  return slices;
}

}  // namespace

size_t ds_from_y_workspace_bytes(const peqa_qweight_t* w, int T) {
  return (size_t)ds_from_y_slices(w->out_features, T) * (size_t)w->out_features * sizeof(float);
}

int launch_ds_from_y(const peqa_qweight_t* w, const void* dY, const void* Y, int T, float* dS,
                     void* workspace, cudaStream_t st) {
  const int N = w->out_features;
  const int slices = ds_from_y_slices(N, T);
  const int tokens_per_slice = (T + slices - 1) / slices;
  float* partial = static_cast<float*>(workspace);
  const dim3 grid((N + kYCols - 1) / kYCols, slices, 1);
  ds_from_y_partial_kernel<<<grid, kYThreads, 0, st>>>(static_cast<const uint4*>(dY),
                                                       static_cast<const uint4*>(Y), T, N,
                                                       tokens_per_slice, partial);
  PEQA_CUDA(cudaGetLastError());
  ds_from_y_finish_kernel<<<(N + 255) / 256, 256, 0, st>>>(partial, w->scales, N, slices, dS);
  PEQA_CUDA(cudaGetLastError());
  return PEQA_OK;
}

}  // namespace peqa
