// HBM-bound kernels of the PEQA path: RTN quantization (Eq. 1), the packed
// b-bit layout, and AdamW on the scales (App. A).
#include <math.h>

#include "common.cuh"

namespace peqa {

namespace {

constexpr int kQuantThreads = 256;
constexpr int kQuantWarps = kQuantThreads / 32;
constexpr int kMaxChunks = 2048;  // 32-column chunks per row -> K <= 65536

// Lane `lane` of a warp holds code c for column (32*chunk + lane).  The row is
// a little-endian bit string with column j at bits [bits*j, bits*j + bits), so
// the 32 codes of a chunk fill exactly `bits` consecutive words.  Each lane
// shifts its code to its place and the words are OR-reduced across the warp.
template <int BITS>
__device__ __forceinline__ void warp_pack_store(uint32_t code, int lane, uint32_t* dst) {
  const int pos = BITS * lane;
  const int word = pos >> 5;
  const int sh = pos & 31;
  const uint32_t lo = code << sh;
  const uint32_t hi = (sh + BITS > 32) ? (code >> (32 - sh)) : 0u;
#pragma unroll
  for (int wi = 0; wi < BITS; ++wi) {
    uint32_t contrib = (word == wi ? lo : 0u) | (word + 1 == wi ? hi : 0u);
    uint32_t v = __reduce_or_sync(0xffffffffu, contrib);
    if (lane == wi) dst[wi] = v;
  }
}

template <int BITS>
__device__ __forceinline__ uint32_t warp_unpack(const uint32_t* src, int lane) {
  const int pos = BITS * lane;
  const int word = pos >> 5;
  const int sh = pos & 31;
  uint32_t v = src[word] >> sh;
  if (sh + BITS > 32) v |= src[word + 1] << (32 - sh);
  return v & ((1u << BITS) - 1u);
}

// rint(fl(w / s)) with fl() the correctly rounded binary32 quotient.  The product
// w * (1/s) is within a few ulps of that quotient, so both round to the same
// integer unless the product sits within a few ulps of a half-integer; only then
// (or when the product is huge or not finite) is the IEEE division carried out.
__device__ __forceinline__ float rint_of_quotient(float w, float s, float rs) {
  const float t = __fmul_rn(w, rs);
  float k = rintf(t);
  const float dist = fabsf(__fsub_rn(fabsf(__fsub_rn(t, k)), 0.5f));
  if (!(fabsf(t) <= 4.0e6f) || dist <= __fmul_rn(fabsf(t), 2.0e-6f)) k = rintf(__fdiv_rn(w, s));
  return k;
}

// One CTA per output row; a thread works on runs of 8 consecutive columns, so
// a 32-column chunk is 4 adjacent lanes.  Pass 1: min/max per chunk.  Pass 2:
// per group (s, z) in strict binary32 (division and rounding as single IEEE
// operations, no FMA).  Pass 3: codes (second read of the row, served by L1/L2)
// and packing: eight 4-bit codes are exactly one word; eight 3-bit codes are 24
// bits, and lanes 0..2 of a 4-lane chunk assemble the three words from their
// own and their right neighbour's piece.
template <int BITS>
__global__ void __launch_bounds__(kQuantThreads)
quantize_rtn_kernel(const float* __restrict__ W, int K, int g, int cpg_shift,
                    uint32_t* __restrict__ qweight, uint8_t* __restrict__ zeros,
                    float* __restrict__ scales) {
  __shared__ float cmin[kMaxChunks];
  __shared__ float cmax[kMaxChunks];
  __shared__ float gscale[kMaxChunks];
  __shared__ float gzero[kMaxChunks];

  const int row = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunks = K >> 5;
  const int nv8 = K >> 3;
  const int G = K / g;
  const int cpg = g >> 5;  // chunks per group
  const float4* w4 = reinterpret_cast<const float4*>(W + (size_t)row * K);
  const float qmax = (float)((1 << BITS) - 1);

  // Every thread runs the same number of iterations (the shuffles name the whole
  // warp); runs past the end of the row are predicated off.  nv8 is a multiple of 4,
  // so the 4 lanes of a chunk are all in or all out.
  for (int vb = 0; vb < nv8; vb += kQuantThreads) {
    const int v = vb + threadIdx.x;
    const bool in = v < nv8;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    if (in) { a = __ldg(w4 + 2 * v); b = __ldg(w4 + 2 * v + 1); }
    float mn = fminf(fminf(fminf(a.x, a.y), fminf(a.z, a.w)), fminf(fminf(b.x, b.y), fminf(b.z, b.w)));
    float mx = fmaxf(fmaxf(fmaxf(a.x, a.y), fmaxf(a.z, a.w)), fmaxf(fmaxf(b.x, b.y), fmaxf(b.z, b.w)));
#pragma unroll
    for (int o = 2; o > 0; o >>= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    if (in && (lane & 3) == 0) { cmin[v >> 2] = mn; cmax[v >> 2] = mx; }
  }
  __syncthreads();

  auto finish_group = [&](int gi, float mn, float mx) {
    float s = __fdiv_rn(__fsub_rn(mx, mn), qmax);
    if (mx == mn) s = 1.0f;
    float z = rintf(__fdiv_rn(-mn, s));
    z = fminf(fmaxf(z, 0.0f), qmax);
    gscale[gi] = s;
    gzero[gi] = z;
    scales[(size_t)row * G + gi] = s;
    zeros[(size_t)row * G + gi] = (uint8_t)z;
  };
  if (cpg <= 32) {
    // narrow groups: one thread per group
    for (int gi = threadIdx.x; gi < G; gi += kQuantThreads) {
      float mn = INFINITY, mx = -INFINITY;
      for (int c = 0; c < cpg; ++c) {
        mn = fminf(mn, cmin[gi * cpg + c]);
        mx = fmaxf(mx, cmax[gi * cpg + c]);
      }
      finish_group(gi, mn, mx);
    }
  } else {
    // wide groups (per-channel above all): one warp per group
    for (int gi = warp; gi < G; gi += kQuantWarps) {
      float mn = INFINITY, mx = -INFINITY;
      for (int c = lane; c < cpg; c += 32) {
        mn = fminf(mn, cmin[gi * cpg + c]);
        mx = fmaxf(mx, cmax[gi * cpg + c]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      }
      if (lane == 0) finish_group(gi, mn, mx);
    }
  }
  __syncthreads();

  uint32_t* qrow = qweight + (size_t)row * chunks * BITS;
  for (int vb = 0; vb < nv8; vb += kQuantThreads) {
    const int v = vb + threadIdx.x;
    const bool in = v < nv8;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    if (in) { a = __ldg(w4 + 2 * v); b = __ldg(w4 + 2 * v + 1); }
    const int chunk = in ? (v >> 2) : 0;
    const int gi = cpg_shift >= 0 ? (chunk >> cpg_shift) : (chunk / cpg);
    const float s = gscale[gi], z = gzero[gi];
    const float rs = __frcp_rn(s);
    const float xs[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint32_t piece = 0u;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      float q = __fadd_rn(rint_of_quotient(xs[e], s, rs), z);
      q = fminf(fmaxf(q, 0.0f), qmax);
      piece |= (uint32_t)q << (BITS * e);
    }
    if constexpr (BITS == 4) {
      if (in) qrow[v] = piece;
    } else {
      // chunk = 96 bits = pieces p0..p3 of 24 bits: word j = (p_j >> 8j) | (p_{j+1} << (24 - 8j))
      const uint32_t nextp = __shfl_down_sync(0xffffffffu, piece, 1);
      const int j = lane & 3;
      const uint32_t word = (piece >> (8 * j)) | (nextp << (24 - 8 * j));
      if (in && j < 3) qrow[chunk * 3 + j] = word;
    }
  }
}

template <int BITS>
__global__ void pack_kernel(const uint8_t* __restrict__ codes, long long total_chunks,
                            uint32_t* __restrict__ qweight) {
  const int lane = threadIdx.x & 31;
  long long c = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long stride = ((long long)gridDim.x * blockDim.x) >> 5;
  for (; c < total_chunks; c += stride) {
    uint32_t code = codes[c * 32 + lane] & ((1u << BITS) - 1u);
    warp_pack_store<BITS>(code, lane, qweight + c * BITS);
  }
}

template <int BITS>
__global__ void unpack_kernel(const uint32_t* __restrict__ qweight, long long total_chunks,
                              uint8_t* __restrict__ codes) {
  const int lane = threadIdx.x & 31;
  long long c = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long stride = ((long long)gridDim.x * blockDim.x) >> 5;
  for (; c < total_chunks; c += stride)
    codes[c * 32 + lane] = (uint8_t)warp_unpack<BITS>(qweight + c * BITS, lane);
}

// Elementwise AdamW in binary32.  The bias corrections 1-b^t are formed on the
// host in double and passed in as reciprocals, as are 1-b1 and 1-b2 (the
// arguments are the binary32 values of lr, b1, b2, eps the caller passed).
__global__ void adamw_kernel(float* __restrict__ s, const float* __restrict__ grad,
                             float* __restrict__ m, float* __restrict__ v, long long n,
                             float lr, float b1, float b2, float omb1, float omb2, float eps,
                             float decay, float inv_c1, float inv_c2) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (; i < n; i += stride) {
    const float gr = grad[i];
    const float mn = b1 * m[i] + omb1 * gr;
    const float vn = b2 * v[i] + omb2 * gr * gr;
    const float denom = sqrtf(vn * inv_c2) + eps;
    s[i] = s[i] * decay - lr * (mn * inv_c1) / denom;
    m[i] = mn;
    v[i] = vn;
  }
}

int grid_for(long long work_items, int threads, int max_blocks = 148 * 16) {
  long long b = (work_items + threads - 1) / threads;
  if (b < 1) b = 1;
  if (b > max_blocks) b = max_blocks;
  return (int)b;
}

}  // namespace

}  // namespace peqa

using namespace peqa;

extern "C" int peqa_quantize_rtn(const float* W, int N, int K, int bits, int group_size,
                                 uint32_t* qweight, uint8_t* zeros, float* scales, void* stream) {
  if (!W || !qweight || !zeros || !scales) return PEQA_ERR_NULL;
  PEQA_TRY(check_bits_shape(N, K, bits, group_size));
  if ((K >> 5) > kMaxChunks) return PEQA_ERR_TOO_LARGE;
  if (!aligned16(W) || !aligned16(qweight) || !aligned16(scales)) return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  const int g = effective_group(K, group_size);
  cudaStream_t st = as_stream(stream);
  int cpg_shift = -1;
  for (int b = 0; b < 26; ++b)
    if ((32 << b) == g) cpg_shift = b;
  if (bits == 4)
    quantize_rtn_kernel<4><<<N, kQuantThreads, 0, st>>>(W, K, g, cpg_shift, qweight, zeros, scales);
  else
    quantize_rtn_kernel<3><<<N, kQuantThreads, 0, st>>>(W, K, g, cpg_shift, qweight, zeros, scales);
  PEQA_CUDA(cudaGetLastError());
  return PEQA_OK;
}

extern "C" int peqa_pack(const uint8_t* codes, int N, int K, int bits, uint32_t* qweight,
                         void* stream) {
  if (!codes || !qweight) return PEQA_ERR_NULL;
  PEQA_TRY(check_bits_shape(N, K, bits, 0));
  if (!aligned16(qweight)) return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  const long long chunks = (long long)N * (K >> 5);
  const int grid = grid_for(chunks * 32, 256);
  cudaStream_t st = as_stream(stream);
  if (bits == 4) pack_kernel<4><<<grid, 256, 0, st>>>(codes, chunks, qweight);
  else pack_kernel<3><<<grid, 256, 0, st>>>(codes, chunks, qweight);
  PEQA_CUDA(cudaGetLastError());
  return PEQA_OK;
}

extern "C" int peqa_unpack(const uint32_t* qweight, int N, int K, int bits, uint8_t* codes,
                           void* stream) {
  if (!codes || !qweight) return PEQA_ERR_NULL;
  PEQA_TRY(check_bits_shape(N, K, bits, 0));
  if (!aligned16(qweight)) return PEQA_ERR_ALIGNMENT;
  PEQA_TRY(check_arch());
  const long long chunks = (long long)N * (K >> 5);
  const int grid = grid_for(chunks * 32, 256);
  cudaStream_t st = as_stream(stream);
  if (bits == 4) unpack_kernel<4><<<grid, 256, 0, st>>>(qweight, chunks, codes);
  else unpack_kernel<3><<<grid, 256, 0, st>>>(qweight, chunks, codes);
  PEQA_CUDA(cudaGetLastError());
  return PEQA_OK;
}

extern "C" int peqa_scale_adamw(float* scales, const float* dS, float* m, float* v, int64_t numel,
                                float lr, float beta1, float beta2, float eps, float weight_decay,
                                int64_t step, void* stream) {
  if (!scales || !dS || !m || !v) return PEQA_ERR_NULL;
  if (numel <= 0 || step < 1) return PEQA_ERR_BAD_SHAPE;
  PEQA_TRY(check_arch());
  const double c1 = 1.0 - pow((double)beta1, (double)step);
  const double c2 = 1.0 - pow((double)beta2, (double)step);
  const float decay = (float)(1.0 - (double)lr * (double)weight_decay);
  const int grid = grid_for(numel, 256);
  adamw_kernel<<<grid, 256, 0, as_stream(stream)>>>(scales, dS, m, v, (long long)numel, lr, beta1,
                                                   beta2, (float)(1.0 - (double)beta1),
                                                   (float)(1.0 - (double)beta2), eps, decay,
                                                   (float)(1.0 / c1), (float)(1.0 / c2));
  PEQA_CUDA(cudaGetLastError());
  return PEQA_OK;
}
