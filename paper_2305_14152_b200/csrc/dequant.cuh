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

}  // namespace dq
}  // namespace peqa
