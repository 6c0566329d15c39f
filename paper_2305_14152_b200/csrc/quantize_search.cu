// Quantization with a searched clipping range (Sec. 3.2: s0 and z0 "are
// initialized to minimize" the reconstruction error of Eq. 1; the paper gives no
// procedure, the search is this library's reading).  Per (row, group), candidate
// k = 0 .. n-1 shrinks the group's extremes by p_k = 1 - k/64 and then follows
// Eq. 1 in binary32:
//     lo = p*mn, hi = p*mx;  s = (hi - lo)/(2^b-1)  (s := 1 when hi == lo)
//     z = clamp(rint(-lo/s), 0, 2^b-1);  q_j = clamp(rint(w_j/s) + z, 0, 2^b-1)
//     e_j = w_j - s*(q_j - z);  err = sum_j e_j^2 in binary64, columns ascending.
// The first candidate with the smallest error wins; k = 0 is plain round-to-nearest.
//
// One warp owns a (row, group).  Lane k evaluates candidates k and k + 32, each a
// sequential pass over the group's columns (every lane reads the same weight, one
// broadcast load), which keeps the summation order the definition fixes; then the
// warp picks the winner and all lanes requantize and pack the group with its
// (s, z), one 32-column chunk at a time.  It is an initialisation step, run once per
// model: about a thousand operations per weight, a few milliseconds per layer.
#include <math.h>

#include "common.cuh"

namespace peqa {

namespace {

constexpr int kSearchWarps = 8;

template <int BITS>
__device__ __forceinline__ void candidate_consts(float mn, float mx, int k, float& s, float& z) {
  const float qmax = (float)((1 << BITS) - 1);
  const float p = __fsub_rn(1.0f, __fdiv_rn((float)k, 64.0f));
  const float lo = __fmul_rn(p, mn), hi = __fmul_rn(p, mx);
  s = __fdiv_rn(__fsub_rn(hi, lo), qmax);
  if (hi == lo) s = 1.0f;
  z = rintf(__fdiv_rn(-lo, s));
  z = fminf(fmaxf(z, 0.0f), qmax);
}

template <int BITS>
__device__ __forceinline__ float code_of(float w, float s, float z) {
  const float qmax = (float)((1 << BITS) - 1);
  const float q = __fadd_rn(rintf(__fdiv_rn(w, s)), z);
  return fminf(fmaxf(q, 0.0f), qmax);
}

template <int BITS>
__global__ void __launch_bounds__(kSearchWarps * 32)
quantize_search_kernel(const float* __restrict__ W, int N, int K, int g, int n_cand,
                       uint32_t* __restrict__ qweight, uint8_t* __restrict__ zeros,
                       float* __restrict__ scales, uint8_t* __restrict__ chosen) {
  const int G = K / g;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long item = (long long)blockIdx.x * kSearchWarps + warp;
  if (item >= (long long)N * G) return;
  const int row = (int)(item / G), gi = (int)(item - (long long)row * G);
  const float* w = W + (size_t)row * K + (size_t)gi * g;

  float mn = w[lane], mx = mn;
  for (int j = lane + 32; j < g; j += 32) {
    mn = fminf(mn, w[j]);
    mx = fmaxf(mx, w[j]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }

  // ---- this lane's candidates: k = lane and k = lane + 32
  double best_err = 0.0;
  int best_k = 1 << 20;
  float best_s = 1.0f, best_z = 0.0f;
#pragma unroll 1
  for (int k = lane; k < n_cand; k += 32) {
    float s, z;
    candidate_consts<BITS>(mn, mx, k, s, z);
    double err = 0.0;
    for (int j = 0; j < g; ++j) {
      const float x = __ldg(w + j);
      const float q = code_of<BITS>(x, s, z);
      const float e = __fsub_rn(x, __fmul_rn(s, __fsub_rn(q, z)));
      err = __dadd_rn(err, __dmul_rn((double)e, (double)e));
    }
    if (best_k == (1 << 20) || err < best_err) {
      best_err = err;
      best_k = k;
      best_s = s;
      best_z = z;
    }
  }
  // ---- the warp's winner: smallest error, then smallest k
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const double oe = __shfl_xor_sync(0xffffffffu, best_err, o);
    const int ok = __shfl_xor_sync(0xffffffffu, best_k, o);
    const float os = __shfl_xor_sync(0xffffffffu, best_s, o);
    const float oz = __shfl_xor_sync(0xffffffffu, best_z, o);
    const bool mine_valid = best_k != (1 << 20), other_valid = ok != (1 << 20);
    const bool take = other_valid && (!mine_valid || oe < best_err || (oe == best_err && ok < best_k));
    if (take) {
      best_err = oe;
      best_k = ok;
      best_s = os;
      best_z = oz;
    }
  }
  if (lane == 0) {
    scales[(size_t)row * G + gi] = best_s;
    zeros[(size_t)row * G + gi] = (uint8_t)best_z;
    if (chosen) chosen[(size_t)row * G + gi] = (uint8_t)best_k;
  }
  // ---- codes of the group with the winning (s, z): lane = column of a 32-column chunk
  uint32_t* qrow = qweight + (size_t)row * (K * BITS / 32) + (size_t)gi * (g * BITS / 32);
  for (int c = 0; c < g / 32; ++c) {
    const uint32_t code = (uint32_t)code_of<BITS>(w[c * 32 + lane], best_s, best_z);
    const int pos = BITS * lane;
    const int word = pos >> 5, sh = pos & 31;
    const uint32_t lo = code << sh;
    const uint32_t hi = (sh + BITS > 32) ? (code >> (32 - sh)) : 0u;
#pragma unroll
    for (int wi = 0; wi < BITS; ++wi) {
      const uint32_t contrib = (word == wi ? lo : 0u) | (word + 1 == wi ? hi : 0u);
      const uint32_t v = __reduce_or_sync(0xffffffffu, contrib);
      if (lane == wi) qrow[c * BITS + wi] = v;
    }
  }
}

}  // namespace

}  // namespace peqa

using namespace peqa;

extern "C" int peqa_quantize_search(const float* W, int N, int K, int bits, int group_size,
                                    int n_candidates, uint32_t* qweight, uint8_t* zeros,
                                    float* scales, uint8_t* chosen, void* stream) {
  if (!W || !qweight || !zeros || !scales) return PEQA_ERR_NULL;
  PEQA_TRY(check_bits_shape(N, K, bits, group_size));
  if (n_candidates < 1 || n_candidates > 64) return PEQA_ERR_BAD_SHAPE;
  if (!aligned16(W) || !aligned16(qweight)) return PEQA_ERR_ALIGNMENT;
  const int g = effective_group(K, group_size);
  const long long items = (long long)N * (K / g);
  const long long blocks = (items + kSearchWarps - 1) / kSearchWarps;
  if (blocks > 0x7fffffffLL) return PEQA_ERR_TOO_LARGE;
  cudaStream_t st = as_stream(stream);
  if (bits == 3)
    quantize_search_kernel<3><<<(unsigned)blocks, kSearchWarps * 32, 0, st>>>(W, N, K, g, n_candidates, qweight,
                                                                           zeros, scales, chosen);
  else
    quantize_search_kernel<4><<<(unsigned)blocks, kSearchWarps * 32, 0, st>>>(W, N, K, g, n_candidates, qweight,
                                                                           zeros, scales, chosen);
  PEQA_CUDA(cudaGetLastError());
  return PEQA_OK;
}
