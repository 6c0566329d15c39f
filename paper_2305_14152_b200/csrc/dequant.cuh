// Register-level dequantization of packed 3-/4-bit codes to bf16.
//
// The packed row is a little-endian bit string with column j at bits
// [b*j, b*j+b).  A "unit" is 32 consecutive columns: 4 words for b=4, 3 words
// for b=3.  Codes are turned into bf16 two at a time without any
// integer-to-float conversion: a code placed in the low mantissa bits of a
// bf16 whose exponent makes one code step equal 1.0 reads as (bias + q), and
// subtracting the bf16 constant (bias + z) gives (q - z) exactly (|q - z| <= 15).
//   code at mantissa bit 0 : bias 128 (bf16 0x4300)
//   code at mantissa bit 4 : bias 8   (bf16 0x4100)
// One 32-bit window of the bit string therefore yields the pair
// (column k, column k+4): b=4 has them 16 bits apart already, b=3 has them 12
// bits apart, so the window starts 4 bits early and the low code lands on
// mantissa bit 4.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace peqa {
namespace dq {

__device__ __forceinline__ uint32_t lop3_and_or(uint32_t x, uint32_t mask, uint32_t orv) {
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(x), "r"(mask), "r"(orv));  // (x & mask) | orv
  return r;
}

__device__ __forceinline__ uint32_t bf162_sub(uint32_t a, uint32_t b) {
  __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162*>(&a);
  __nv_bfloat162 y = *reinterpret_cast<__nv_bfloat162*>(&b);
  __nv_bfloat162 r = __hsub2(x, y);
  return *reinterpret_cast<uint32_t*>(&r);
}

__device__ __forceinline__ uint32_t bf162_mul(uint32_t a, uint32_t b) {
  __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162*>(&a);
  __nv_bfloat162 y = *reinterpret_cast<__nv_bfloat162*>(&b);
  __nv_bfloat162 r = __hmul2(x, y);
  return *reinterpret_cast<uint32_t*>(&r);
}

__device__ __forceinline__ uint32_t bf162_fma(uint32_t a, uint32_t b, uint32_t c) {
  __nv_bfloat162 x = *reinterpret_cast<__nv_bfloat162*>(&a);
  __nv_bfloat162 y = *reinterpret_cast<__nv_bfloat162*>(&b);
  __nv_bfloat162 z = *reinterpret_cast<__nv_bfloat162*>(&c);
  __nv_bfloat162 r = __hfma2(x, y, z);
  return *reinterpret_cast<uint32_t*>(&r);
}

__device__ __forceinline__ uint32_t bf162_broadcast(float s) {
  __nv_bfloat162 r = __float2bfloat162_rn(s);
  return *reinterpret_cast<uint32_t*>(&r);
}

// bf16x2 constant (bias_lo + z, bias_hi + z) matching pair_raw<BITS>().
template <int BITS>
__device__ __forceinline__ uint32_t zero_const(uint32_t z) {
  if (BITS == 4) return (0x4300u | z) * 0x00010001u;
  return ((0x4300u | z) << 16) | (0x4100u | (z << 4));
}

// 32-bit window of the 96-bit string (w0 lowest) starting at bit START
// (START may be negative: the string is shifted left).  Only bits 4..6 and
// 16..18 of the result are used by the caller.
template <int START>
__device__ __forceinline__ uint32_t window3(const uint32_t (&w)[3]) {
  if constexpr (START < 0) {
    return w[0] << (-START);
  } else {
    constexpr int a = START / 32;
    constexpr int sh = START % 32;
    if constexpr (sh == 0) {
      return w[a];
    } else if constexpr (sh + 19 <= 32 || a == 2) {
      return w[a] >> sh;
    } else {
      return __funnelshift_r(w[a], w[a + 1], sh);
    }
  }
}

// Biased bf16x2 of columns (K0, K0+4) of a unit, K0 = 8*blk + e, e in 0..3.
template <int BITS, int K0>
__device__ __forceinline__ uint32_t pair_raw(const uint32_t (&w)[BITS]) {
  if constexpr (BITS == 4) {
    constexpr int word = K0 / 8;
    constexpr int e = K0 % 8;
    return lop3_and_or(w[word] >> (4 * e), 0x000F000Fu, 0x43004300u);
  } else {
    return lop3_and_or(window3<3 * K0 - 4>(w), 0x00070070u, 0x43004100u);
  }
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}

// One block of 8 columns -> 4 bf16x2 registers in natural column order
// (out[0] = columns 0,1 ... out[3] = columns 6,7 of the block).
template <int BITS, int BLK, bool FOLD>
__device__ __forceinline__ void block8_natural(const uint32_t (&w)[BITS], uint32_t zc, uint32_t s2,
                                               uint32_t* out) {
  uint32_t d0 = bf162_sub(pair_raw<BITS, 8 * BLK + 0>(w), zc);  // (c0, c4)
  uint32_t d1 = bf162_sub(pair_raw<BITS, 8 * BLK + 1>(w), zc);  // (c1, c5)
  uint32_t d2 = bf162_sub(pair_raw<BITS, 8 * BLK + 2>(w), zc);  // (c2, c6)
  uint32_t d3 = bf162_sub(pair_raw<BITS, 8 * BLK + 3>(w), zc);  // (c3, c7)
  if (FOLD) {
    d0 = bf162_mul(d0, s2);
    d1 = bf162_mul(d1, s2);
    d2 = bf162_mul(d2, s2);
    d3 = bf162_mul(d3, s2);
  }
  out[0] = prmt(d0, d1, 0x5410u);
  out[1] = prmt(d2, d3, 0x5410u);
  out[2] = prmt(d0, d1, 0x7632u);
  out[3] = prmt(d2, d3, 0x7632u);
}

// A unit of 32 columns -> 16 bf16x2 registers holding (q - z) [* bf16(s) when
// FOLD] in natural column order.
template <int BITS, bool FOLD>
__device__ __forceinline__ void unit32_natural(const uint32_t (&w)[BITS], uint32_t z, float s,
                                               uint32_t (&out)[16]) {
  const uint32_t zc = zero_const<BITS>(z);
  const uint32_t s2 = FOLD ? bf162_broadcast(s) : 0u;
  block8_natural<BITS, 0, FOLD>(w, zc, s2, out + 0);
  block8_natural<BITS, 1, FOLD>(w, zc, s2, out + 4);
  block8_natural<BITS, 2, FOLD>(w, zc, s2, out + 8);
  block8_natural<BITS, 3, FOLD>(w, zc, s2, out + 12);
}

// A unit of 32 columns with a real-valued zero-point z = zi + delta (App. K trains z):
//   s*(q - z) = (q - zi)*s + c,  c = -delta*s,
// formed as one fused multiply-add per pair on the exact integers q - zi, so the operand is
// the product rounded once (with s and c rounded to bf16 first, as for grouped scales).
// zi must be an integer in [0, 2^BITS - 1].
template <int BITS>
__device__ __forceinline__ void unit32_affine(const uint32_t (&w)[BITS], uint32_t zi, float s, float c,
                                              uint32_t (&out)[16]) {
  const uint32_t zc = zero_const<BITS>(zi);
  const uint32_t s2 = bf162_broadcast(s), c2 = bf162_broadcast(c);
#pragma unroll
  for (int blk = 0; blk < 4; ++blk) {
    uint32_t d[4];
    if (blk == 0) {
      d[0] = pair_raw<BITS, 0>(w); d[1] = pair_raw<BITS, 1>(w); d[2] = pair_raw<BITS, 2>(w); d[3] = pair_raw<BITS, 3>(w);
    } else if (blk == 1) {
      d[0] = pair_raw<BITS, 8>(w); d[1] = pair_raw<BITS, 9>(w); d[2] = pair_raw<BITS, 10>(w); d[3] = pair_raw<BITS, 11>(w);
    } else if (blk == 2) {
      d[0] = pair_raw<BITS, 16>(w); d[1] = pair_raw<BITS, 17>(w); d[2] = pair_raw<BITS, 18>(w); d[3] = pair_raw<BITS, 19>(w);
    } else {
      d[0] = pair_raw<BITS, 24>(w); d[1] = pair_raw<BITS, 25>(w); d[2] = pair_raw<BITS, 26>(w); d[3] = pair_raw<BITS, 27>(w);
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) d[e] = bf162_fma(bf162_sub(d[e], zc), s2, c2);
    out[4 * blk + 0] = prmt(d[0], d[1], 0x5410u);
    out[4 * blk + 1] = prmt(d[2], d[3], 0x5410u);
    out[4 * blk + 2] = prmt(d[0], d[1], 0x7632u);
    out[4 * blk + 3] = prmt(d[2], d[3], 0x7632u);
  }
}

// Splits a real-valued zero-point into the integer the exact dequantization can use and
// the remainder the affine form carries: zi = clamp(rint(z), 0, 2^BITS - 1), delta = z - zi.
template <int BITS>
__device__ __forceinline__ void split_zero_point(float z, uint32_t& zi, float& delta) {
  const float r = fminf(fmaxf(rintf(z), 0.0f), (float)((1 << BITS) - 1));
  zi = (uint32_t)r;
  delta = z - r;
}

// ---------------------------------------------------------------------------
// Pairing for kernels whose contraction order is free (the streaming decode
// kernel: the activations are staged in whatever order the weights come out).
//
// A 3-bit code fits the 7 mantissa bits of a bf16 at any start bit p in 0..4,
// and with the exponent chosen so that one code step is 1.0 it reads as
// 2^(7-p) + q.  So one shifted window of the packed string can yield TWO pairs
// with two logic operations: with column A at bit 4 it holds
//   (A    at bit 4,  bias 8)   with  (A + 4 at bit 16, bias 128)   "std"
//   (A - 1 at bit 1, bias 64)  with  (A + 5 at bit 19, bias 16)    "alt"
// and a lone pair six columns apart can be taken as (bit 1, bit 19).  The 32
// columns of a unit split into six such double windows and four single ones
// (ten shifts, one of them by zero, and sixteen logic operations instead of
// sixteen of each).  Pair k of the unit, k = 0..15, is (stream_lo(k), stream_hi(k)); MMA
// m of the unit takes pairs 2m and 2m + 1.  4-bit codes have no second start
// position in a bf16 mantissa: their pairs stay (8b + e, 8b + e + 4).
// ---------------------------------------------------------------------------
// windows: A = 1, A = 3, (4,10), (9,13), A = 12, A = 15, (18,22), (21,27), A = 24, A = 26
__host__ __device__ constexpr int stream_lo(int bits, int k) {
  constexpr int lo3[16] = {1, 0, 3, 2, 4, 9, 12, 11, 15, 14, 18, 21, 24, 23, 26, 25};
  return bits == 3 ? lo3[k] : 8 * (k / 4) + k % 4;
}
__host__ __device__ constexpr int stream_hi(int bits, int k) {
  constexpr int hi3[16] = {5, 6, 7, 8, 10, 13, 16, 17, 19, 20, 22, 27, 28, 29, 30, 31};
  return bits == 3 ? hi3[k] : 8 * (k / 4) + k % 4 + 4;
}
// "alt" pairs sit at bits (1, 19) of their window and carry the biases (64, 16); the others
// sit at bits (4, 16) and carry (8, 128).  4-bit pairs carry (128, 128).
__host__ __device__ constexpr bool stream_alt(int bits, int k) {
  constexpr bool alt3[16] = {false, true, false, true, true, false, false, true,
                             false, true, false, true, false, true, false, true};
  return bits == 3 ? alt3[k] : false;
}
__host__ __device__ constexpr uint32_t stream_alt_mask3() {
  uint32_t m = 0;
  for (int k = 0; k < 16; ++k) m |= (stream_alt(3, k) ? 1u : 0u) << k;
  return m;
}

// 32-bit window of the 96-bit string starting at bit START (may be -1), of which bits
// 0..21 are used.
template <int START>
__device__ __forceinline__ uint32_t window3_wide(const uint32_t (&w)[3]) {
  if constexpr (START < 0) {
    return w[0] << (-START);
  } else {
    constexpr int a = START / 32;
    constexpr int sh = START % 32;
    if constexpr (sh == 0) {
      return w[a];
    } else if constexpr (sh + 22 <= 32 || a == 2) {
      return w[a] >> sh;
    } else {
      return __funnelshift_r(w[a], w[a + 1], sh);
    }
  }
}

// The two biased bf16x2 registers of MMA M (pairs 2M and 2M + 1) of a unit.
template <int BITS, int M>
__device__ __forceinline__ void mma_pairs_stream(const uint32_t (&w)[BITS], uint32_t& p0,
                                                 uint32_t& p1) {
  if constexpr (BITS == 4) {
    // pairs (8b + e, +4) and (8b + e + 1, +4) with b = M / 2, e = 2 * (M % 2)
    p0 = pair_raw<4, 8 * (M / 2) + 2 * (M % 2)>(w);
    p1 = pair_raw<4, 8 * (M / 2) + 2 * (M % 2) + 1>(w);
  } else {
    constexpr uint32_t kStdMask = 0x00070070u, kStdMagic = 0x43004100u;   // bits 4-6 | 16-18
    constexpr uint32_t kAltMask = 0x0038000Eu, kAltMagic = 0x41804280u;   // bits 1-3 | 19-21
    constexpr int k0 = 2 * M, k1 = 2 * M + 1;
    if constexpr (!stream_alt(3, k0) && stream_alt(3, k1) &&
                  stream_lo(3, k1) == stream_lo(3, k0) - 1) {
      // a double window: column lo[k0] at bit 4
      const uint32_t x = window3_wide<3 * stream_lo(3, k0) - 4>(w);
      p0 = lop3_and_or(x, kStdMask, kStdMagic);
      p1 = lop3_and_or(x, kAltMask, kAltMagic);
    } else {
      // two single windows
      if constexpr (stream_alt(3, k0))
        p0 = lop3_and_or(window3_wide<3 * stream_lo(3, k0) - 1>(w), kAltMask, kAltMagic);
      else
        p0 = lop3_and_or(window3_wide<3 * stream_lo(3, k0) - 4>(w), kStdMask, kStdMagic);
      if constexpr (stream_alt(3, k1))
        p1 = lop3_and_or(window3_wide<3 * stream_lo(3, k1) - 1>(w), kAltMask, kAltMagic);
      else
        p1 = lop3_and_or(window3_wide<3 * stream_lo(3, k1) - 4>(w), kStdMask, kStdMagic);
    }
  }
}

}  // namespace dq
}  // namespace peqa
