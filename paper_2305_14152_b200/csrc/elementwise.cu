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

// Codes of eight consecutive columns of one group, as BITS-wide fields of a word
// (column e at bits [BITS*e, BITS*e + BITS)).
//
// Reference arithmetic (Eq. 1 in binary32): q = clamp(rint(fl(w / s)) + z, 0, qmax).
// Fast path, same result without a division or a float->int conversion per element:
//   t  = fl(w * fl(1/s))           within 3 ulp of fl(w / s)
//   tc = clamp(t, -z - 1/4, qmax - z + 1/4)   rint(tc) + z lands in [0, qmax] and equals
//                                  the clamped reference whenever rint(t) == rint(fl(w/s))
//   k  = (tc + 1.5*2^23) - 1.5*2^23           = rint(tc), ties to even, since |tc| < 2^22
//   word_f += k * 2^(BITS*e)       exact: the fields fill at most 24 bits of an fp32
// rint(t) can differ from rint(fl(w/s)) only if a half-integer lies within 3 ulp of t
// (|t| <= 16.25 inside the clamp, so 3 ulp < 6e-6).  The run keeps the smallest distance
// to a half-integer it has seen; if that is below 1e-5, or 1/s is not a normal number of
// moderate size, the eight codes are recomputed with the IEEE division.
template <int BITS>
__device__ __forceinline__ uint32_t quantize_run8(const float (&x)[8], float s, float z) {
  constexpr float kMagic = 12582912.0f;   // 1.5 * 2^23
  const float qmax = (float)((1 << BITS) - 1);
  const float rs = __frcp_rn(s);
  const float lo = __fsub_rn(-0.25f, z);
  const float hi = __fadd_rn(__fsub_rn(qmax, z), 0.25f);
  float near = 1.0f;
  uint32_t word;
  if constexpr (BITS == 3) {
    float acc = __fmul_rn(z, 2396745.0f);                 // z * sum_e 8^e
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float tc = fminf(fmaxf(__fmul_rn(x[e], rs), lo), hi);
      const float k = __fsub_rn(__fadd_rn(tc, kMagic), kMagic);
      near = fminf(near, fabsf(__fsub_rn(fabsf(__fsub_rn(tc, k)), 0.5f)));
      acc = __fmaf_rn(k, (float)(1 << (3 * e)), acc);
    }
    word = (uint32_t)acc;
  } else {
    float acc0 = __fmul_rn(z, 4369.0f), acc1 = acc0;      // z * sum_{e<4} 16^e
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float tc = fminf(fmaxf(__fmul_rn(x[e], rs), lo), hi);
      const float k = __fsub_rn(__fadd_rn(tc, kMagic), kMagic);
      near = fminf(near, fabsf(__fsub_rn(fabsf(__fsub_rn(tc, k)), 0.5f)));
      if (e < 4) acc0 = __fmaf_rn(k, (float)(1 << (4 * e)), acc0);
      else acc1 = __fmaf_rn(k, (float)(1 << (4 * (e - 4))), acc1);
    }
    word = (uint32_t)acc0 | ((uint32_t)acc1 << 16);
  }
  if (!(near > 1.0e-5f) || !(rs <= 1.0e30f)) {
    word = 0u;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      float q = __fadd_rn(rintf(__fdiv_rn(x[e], s)), z);
      q = fminf(fmaxf(q, 0.0f), qmax);
      word |= (uint32_t)q << (BITS * e);
    }
  }
  return word;
}

// One CTA per output row; a thread works on runs of 8 consecutive columns, so
// a 32-column chunk is 4 adjacent lanes.  Pass 1: read the row (kept in
// registers when RUNS > 0: run r of a thread is columns 8*(threadIdx.x +
// r*256)..+7, which covers K <= 2048*RUNS), min/max per chunk.  Pass 2: per
// group (s, z) in strict binary32 (division and rounding as single IEEE
// operations, no FMA).  Pass 3: codes and packing: eight 4-bit codes are exactly
// one word; eight 3-bit codes are 24 bits, and lanes 0..2 of a 4-lane chunk
// assemble the three words from their own and their right neighbour's piece.
// RUNS == 0 reads the row a second time in pass 3 instead (any K).
template <int BITS, int RUNS>
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
  constexpr int NR = RUNS > 0 ? RUNS : 1;
  float4 ra[NR], rb[NR];

  // Every thread runs the same number of iterations (the shuffles name the whole
  // warp); runs past the end of the row are predicated off.  nv8 is a multiple of 4,
  // so the 4 lanes of a chunk are all in or all out.
  auto minmax_run = [&](int v, bool in, const float4& a, const float4& b) {
    float mn = fminf(fminf(fminf(a.x, a.y), fminf(a.z, a.w)), fminf(fminf(b.x, b.y), fminf(b.z, b.w)));
    float mx = fmaxf(fmaxf(fmaxf(a.x, a.y), fmaxf(a.z, a.w)), fmaxf(fmaxf(b.x, b.y), fmaxf(b.z, b.w)));
#pragma unroll
    for (int o = 2; o > 0; o >>= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    if (in && (lane & 3) == 0) { cmin[v >> 2] = mn; cmax[v >> 2] = mx; }
  };
  if constexpr (RUNS > 0) {
#pragma unroll
    for (int r = 0; r < RUNS; ++r) {
      const int v = r * kQuantThreads + threadIdx.x;
      ra[r] = make_float4(0.f, 0.f, 0.f, 0.f);
      rb[r] = ra[r];
      if (v < nv8) { ra[r] = __ldg(w4 + 2 * v); rb[r] = __ldg(w4 + 2 * v + 1); }
    }
#pragma unroll
    for (int r = 0; r < RUNS; ++r) {
      const int v = r * kQuantThreads + threadIdx.x;
      minmax_run(v, v < nv8, ra[r], rb[r]);
    }
  } else {
    for (int vb = 0; vb < nv8; vb += kQuantThreads) {
      const int v = vb + threadIdx.x;
      const bool in = v < nv8;
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
      if (in) { a = __ldg(w4 + 2 * v); b = __ldg(w4 + 2 * v + 1); }
      minmax_run(v, in, a, b);
    }
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
  auto emit_run = [&](int v, bool in, const float4& a, const float4& b) {
    const int chunk = in ? (v >> 2) : 0;
    const int gi = cpg_shift >= 0 ? (chunk >> cpg_shift) : (chunk / cpg);
    const float xs[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    const uint32_t piece = quantize_run8<BITS>(xs, gscale[gi], gzero[gi]);
    if constexpr (BITS == 4) {
      if (in) qrow[v] = piece;
    } else {
      // chunk = 96 bits = pieces p0..p3 of 24 bits: word j = (p_j >> 8j) | (p_{j+1} << (24 - 8j))
      const uint32_t nextp = __shfl_down_sync(0xffffffffu, piece, 1);
      const int j = lane & 3;
      const uint32_t word = (piece >> (8 * j)) | (nextp << (24 - 8 * j));
      if (in && j < 3) qrow[chunk * 3 + j] = word;
    }
  };
  if constexpr (RUNS > 0) {
#pragma unroll
    for (int r = 0; r < RUNS; ++r) {
      const int v = r * kQuantThreads + threadIdx.x;
      emit_run(v, v < nv8, ra[r], rb[r]);
    }
  } else {
    for (int vb = 0; vb < nv8; vb += kQuantThreads) {
      const int v = vb + threadIdx.x;
      const bool in = v < nv8;
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
      if (in) { a = __ldg(w4 + 2 * v); b = __ldg(w4 + 2 * v + 1); }
      emit_run(v, in, a, b);
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
  // rows up to 2048 * RUNS columns stay in registers between the passes
  const int runs = K <= 4096 ? 2 : K <= 8192 ? 4 : K <= 12288 ? 6 : K <= 24576 ? 12 : 0;
#define PEQA_QUANT_LAUNCH(B, R) \
  quantize_rtn_kernel<B, R><<<N, kQuantThreads, 0, st>>>(W, K, g, cpg_shift, qweight, zeros, scales)
  if (bits == 4) {
    switch (runs) {
      case 2: PEQA_QUANT_LAUNCH(4, 2); break;
      case 4: PEQA_QUANT_LAUNCH(4, 4); break;
      case 6: PEQA_QUANT_LAUNCH(4, 6); break;
      case 12: PEQA_QUANT_LAUNCH(4, 12); break;
      default: PEQA_QUANT_LAUNCH(4, 0); break;
    }
  } else {
    switch (runs) {
      case 2: PEQA_QUANT_LAUNCH(3, 2); break;
      case 4: PEQA_QUANT_LAUNCH(3, 4); break;
      case 6: PEQA_QUANT_LAUNCH(3, 6); break;
      case 12: PEQA_QUANT_LAUNCH(3, 12); break;
      default: PEQA_QUANT_LAUNCH(3, 0); break;
    }
  }
#undef PEQA_QUANT_LAUNCH
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
