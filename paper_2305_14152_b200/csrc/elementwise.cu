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

__device__ __forceinline__ float min3(float a, float b, float c) {
  float r;
  asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// Per-group constants of the fast quantization path, written once per group.
struct GroupConst {
  float rs;   // fl(1/s), or NaN when the group must take the division path
  float zc;   // z * sum of the field weights (the accumulator's start value)
};

// Reference arithmetic (Eq. 1 in binary32): q = clamp(rint(fl(w / s)) + z, 0, qmax).
// The fast path computes t = fl(w * fl(1/s)), which is within 3 ulp of fl(w / s), and
// rounds it without a clamp.  That is only right for a group in which no code needs
// the clamp: t is monotone in w, so it is enough that the group's extremes satisfy
// -z - 1/2 < t(min) and t(max) < qmax - z + 1/2 (with a margin of 1e-5).  Groups that
// fail (all weights of one sign, so that z itself was clamped; an extreme next to a
// tie), and groups whose 1/s is not a normal number of moderate size, get rs = NaN.
template <int BITS>
__device__ __forceinline__ GroupConst group_const(float mn, float mx, float s, float z) {
  const float qmax = (float)((1 << BITS) - 1);
  GroupConst c;
  c.rs = __frcp_rn(s);
  const float t_lo = __fmul_rn(mn, c.rs), t_hi = __fmul_rn(mx, c.rs);
  const bool ok = c.rs <= 1.0e30f && t_lo > __fsub_rn(-0.49999f, z) &&
                  t_hi < __fadd_rn(__fsub_rn(qmax, z), 0.49999f);
  if (!ok) c.rs = __int_as_float(0x7fc00000);
  c.zc = __fmul_rn(z, BITS == 3 ? 2396745.0f : 4369.0f);   // sum_{e<8} 8^e, sum_{e<4} 16^e
  return c;
}

// Codes of eight consecutive columns of one group, as BITS-wide fields of a word
// (column e at bits [BITS*e, BITS*e + BITS)).  Fast path, per element:
//   t  = fl(w * rs)
//   k  = (t + 1.5*2^23) - 1.5*2^23   = rint(t), ties to even, since |t| < 2^22
//   word_f += k * 2^(BITS*e)         exact: the fields fill at most 24 bits of an fp32,
//                                    and word_f starts at z in every field
// rint(t) can differ from rint(fl(w/s)) only if a half-integer lies within 3 ulp of t
// (|t| <= 16.5 in a group that passed group_const, so 3 ulp < 6e-6).  The run keeps the
// largest |t - k| it has seen; if that is not below 1/2 - 1e-5, or the group's rs is
// NaN, the eight codes are recomputed with the IEEE division and the clamp.
template <int BITS>
__device__ __forceinline__ uint32_t quantize_run8(const float (&x)[8], float s, float z,
                                                  const GroupConst& c) {
  constexpr float kMagic = 12582912.0f;   // 1.5 * 2^23
  float k[8], r[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const float t = __fmul_rn(x[e], c.rs);
    k[e] = __fsub_rn(__fadd_rn(t, kMagic), kMagic);
    r[e] = fabsf(__fsub_rn(t, k[e]));
  }
  const float far = max3(max3(r[0], r[1], r[2]), max3(r[3], r[4], r[5]), fmaxf(r[6], r[7]));
  uint32_t word;
  if constexpr (BITS == 3) {
    float acc = c.zc;
#pragma unroll
    for (int e = 0; e < 8; ++e) acc = __fmaf_rn(k[e], (float)(1 << (3 * e)), acc);
    word = (uint32_t)acc;
  } else {
    float acc0 = c.zc, acc1 = c.zc;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      acc0 = __fmaf_rn(k[e], (float)(1 << (4 * e)), acc0);
      acc1 = __fmaf_rn(k[4 + e], (float)(1 << (4 * e)), acc1);
    }
    word = (uint32_t)acc0 | ((uint32_t)acc1 << 16);
  }
  // max drops a NaN operand, so a NaN rs has to be tested on its own
  if (!(far < 0.49999f) || c.rs != c.rs) {
    const float qmax = (float)((1 << BITS) - 1);
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

// A CTA takes rows blockIdx.x, blockIdx.x + gridDim.x, ...; a thread works on
// runs of 8 consecutive columns, so a 32-column chunk is 4 adjacent lanes.
// Pass 1: min/max per chunk of the row (kept in registers when RUNS > 0: run r
// of a thread is columns 8*(threadIdx.x + r*256)..+7, which covers K <=
// 2048*RUNS).  Pass 2: per group (s, z) in strict binary32 (division and
// rounding as single IEEE operations, no FMA).  Pass 3: codes and packing:
// eight 4-bit codes are exactly one word; eight 3-bit codes are 24 bits, and
// lanes 0..2 of a 4-lane chunk assemble the three words from their own and
// their right neighbour's piece.  With PREFETCH the loads of the CTA's next
// row are issued before pass 1 of the current one, so that the memory system
// stays busy while the row is being reduced and encoded.  RUNS == 0 reads the
// row a second time in pass 3 instead (any K).
template <int BITS, int RUNS, bool PREFETCH, int THREADS = kQuantThreads>
__global__ void __launch_bounds__(THREADS)
quantize_rtn_kernel(const float* __restrict__ W, int N, int K, int g, int cpg_shift,
                    uint32_t* __restrict__ qweight, uint8_t* __restrict__ zeros,
                    float* __restrict__ scales) {
  extern __shared__ __align__(16) uint8_t quant_smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunks = K >> 5;
  const int nv8 = K >> 3;
  const int G = K / g;
  GroupConst* gconst = reinterpret_cast<GroupConst*>(quant_smem);          // [G]
  float* gscale = reinterpret_cast<float*>(gconst + G);                    // [G]
  float* gzero = gscale + G;                                               // [G]
  float* cmin = gzero + G;                                                 // [chunks]
  float* cmax = cmin + chunks;                                             // [chunks]
  const int cpg = g >> 5;  // chunks per group
  const float qmax = (float)((1 << BITS) - 1);
  constexpr int NR = RUNS > 0 ? RUNS : 1;

  auto row_ptr = [&](int row) { return reinterpret_cast<const float4*>(W + (size_t)row * K); };
  auto load_row = [&](int row, float4 (&a)[NR], float4 (&b)[NR]) {
    const float4* w4 = row_ptr(row);
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      const int v = r * THREADS + threadIdx.x;
      a[r] = make_float4(0.f, 0.f, 0.f, 0.f);
      b[r] = a[r];
      if (row < N && v < nv8) { a[r] = __ldg(w4 + 2 * v); b[r] = __ldg(w4 + 2 * v + 1); }
    }
  };
  // Every thread runs the same number of iterations (the shuffles name the whole
  // warp); runs past the end of the row are predicated off.  nv8 is a multiple of 4,
  // so the 4 lanes of a chunk are all in or all out.
  auto minmax_run = [&](int v, bool in, const float4& a, const float4& b) {
    float mn = min3(min3(a.x, a.y, a.z), min3(a.w, b.x, b.y), fminf(b.z, b.w));
    float mx = max3(max3(a.x, a.y, a.z), max3(a.w, b.x, b.y), fmaxf(b.z, b.w));
#pragma unroll
    for (int o = 2; o > 0; o >>= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    if (in && (lane & 3) == 0) { cmin[v >> 2] = mn; cmax[v >> 2] = mx; }
  };

  // One row, from the registers ra, rb (RUNS > 0) or from memory (RUNS == 0).
  auto process_row = [&](int row, const float4 (&ra)[NR], const float4 (&rb)[NR]) {
    const float4* w4 = row_ptr(row);
    if constexpr (RUNS > 0) {
#pragma unroll
      for (int r = 0; r < RUNS; ++r) {
        const int v = r * THREADS + threadIdx.x;
        minmax_run(v, v < nv8, ra[r], rb[r]);
      }
    } else {
      for (int vb = 0; vb < nv8; vb += THREADS) {
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
      gconst[gi] = group_const<BITS>(mn, mx, s, z);
      scales[(size_t)row * G + gi] = s;
      zeros[(size_t)row * G + gi] = (uint8_t)z;
    };
    if (cpg <= 32) {
      // narrow groups: one thread per group
      for (int gi = threadIdx.x; gi < G; gi += THREADS) {
        float mn = INFINITY, mx = -INFINITY;
        for (int c = 0; c < cpg; ++c) {
          mn = fminf(mn, cmin[gi * cpg + c]);
          mx = fmaxf(mx, cmax[gi * cpg + c]);
        }
        finish_group(gi, mn, mx);
      }
    } else {
      // wide groups (per-channel above all): one warp per group
      for (int gi = warp; gi < G; gi += (THREADS / 32)) {
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
      const uint32_t piece = quantize_run8<BITS>(xs, gscale[gi], gzero[gi], gconst[gi]);
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
        const int v = r * THREADS + threadIdx.x;
        emit_run(v, v < nv8, ra[r], rb[r]);
      }
    } else {
      for (int vb = 0; vb < nv8; vb += THREADS) {
        const int v = vb + threadIdx.x;
        const bool in = v < nv8;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
        if (in) { a = __ldg(w4 + 2 * v); b = __ldg(w4 + 2 * v + 1); }
        emit_run(v, in, a, b);
      }
    }
    // The next row's pass 1 rewrites cmin/cmax, which pass 2 of this row has finished
    // with (second barrier above); its pass 2 rewrites the group arrays only after its
    // own first barrier, which every thread reaches after it has left this pass 3.
  };

  float4 a0[NR], b0[NR];
  if constexpr (RUNS > 0 && PREFETCH) {
    float4 a1[NR], b1[NR];
    int row = blockIdx.x;
    load_row(row, a0, b0);
    while (row < N) {
      load_row(row + gridDim.x, a1, b1);
      process_row(row, a0, b0);
      row += gridDim.x;
      if (row >= N) break;
      load_row(row + gridDim.x, a0, b0);
      process_row(row, a1, b1);
      row += gridDim.x;
    }
  } else {
    for (int row = blockIdx.x; row < N; row += gridDim.x) {
      if constexpr (RUNS > 0) load_row(row, a0, b0);
      process_row(row, a0, b0);
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

// Elementwise AdamW in binary32 (adamw_update in common.cuh).
__global__ void adamw_kernel(float* __restrict__ s, const float* __restrict__ grad,
                             float* __restrict__ m, float* __restrict__ v, long long n,
                             const AdamWConsts c) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (; i < n; i += stride) {
    float sv = s[i], mv = m[i], vv = v[i];
    adamw_update(sv, grad[i], mv, vv, c);
    s[i] = sv;
    m[i] = mv;
    v[i] = vv;
  }
}

int grid_for(long long work_items, int threads, int max_blocks = 0) {
  if (max_blocks <= 0) max_blocks = sm_count_or(148) * 16;
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
  // rows up to 8 * RUNS * threads columns stay in registers between the passes; rows of up to
  // 8192 columns (256 threads) and of 12289 to 24576 columns (512 threads) also prefetch the
  // CTA's next row
  const int runs = K <= 4096 ? 2 : K <= 8192 ? 4 : K <= 12288 ? 6 : K <= 24576 ? 12 : 0;
  const size_t smem = (size_t)(K / g) * (sizeof(GroupConst) + 8) + (size_t)(K >> 5) * 8;
  int sms = 0, dev = 0;
  PEQA_CUDA(cudaGetDevice(&dev));
  PEQA_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
#define PEQA_QUANT_LAUNCH(B, R, P, TH)                                                                 \
  do {                                                                                                 \
    auto kern = quantize_rtn_kernel<B, R, P, TH>;                                                      \
    if (smem > 48 * 1024)                                                                              \
      PEQA_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));   \
    int per_sm = 0;                                                                                    \
    PEQA_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, TH, smem));                 \
    if (per_sm < 1) per_sm = 1;                                                                        \
    const long long resident = (long long)sms * per_sm;                                                \
    const int grid = (int)(N < resident ? N : resident);                                               \
    kern<<<grid, TH, smem, st>>>(W, N, K, g, cpg_shift, qweight, zeros, scales);                       \
  } while (0)
  if (bits == 4) {
    switch (runs) {
      case 2: PEQA_QUANT_LAUNCH(4, 2, true, 256); break;
      case 4: PEQA_QUANT_LAUNCH(4, 4, true, 256); break;
      case 6: PEQA_QUANT_LAUNCH(4, 6, false, 256); break;
      case 12: PEQA_QUANT_LAUNCH(4, 6, true, 512); break;   // 512 threads: the next row is prefetched
      default: PEQA_QUANT_LAUNCH(4, 0, false, 256); break;
    }
  } else {
    switch (runs) {
      case 2: PEQA_QUANT_LAUNCH(3, 2, true, 256); break;
      case 4: PEQA_QUANT_LAUNCH(3, 4, true, 256); break;
      case 6: PEQA_QUANT_LAUNCH(3, 6, false, 256); break;
      case 12: PEQA_QUANT_LAUNCH(3, 6, true, 512); break;   // 512 threads: the next row is prefetched
      default: PEQA_QUANT_LAUNCH(3, 0, false, 256); break;
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
  const int grid = grid_for(numel, 256);
  adamw_kernel<<<grid, 256, 0, as_stream(stream)>>>(scales, dS, m, v, (long long)numel,
                                                   adamw_consts(lr, beta1, beta2, eps, weight_decay, step));
  PEQA_CUDA(cudaGetLastError());
  return PEQA_OK;
}

// App. K's "zero-points only" and "both" modes: the same AdamW step on the real-valued
// zero-points, driven by dZ.
extern "C" int peqa_zero_adamw(float* zeros_f, const float* dZ, float* m, float* v, int64_t numel,
                               float lr, float beta1, float beta2, float eps, float weight_decay,
                               int64_t step, void* stream) {
  return peqa_scale_adamw(zeros_f, dZ, m, v, numel, lr, beta1, beta2, eps, weight_decay, step, stream);
}
