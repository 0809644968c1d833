// The quantizer of Section 3.2 as a device function shared by the kernels that write the cache: affine 4-bit
// codes over groups of 64, 16-bit scale and bias (binary16, or bfloat16: the section names both).  Every arithmetic
// step is a single rounded binary32 operation in a fixed order, so that codes, scales and biases are reproducible
// bit for bit:
//   bias = RD_16(min) (-0 -> +0), scale = RU_16((max - bias) / 15), code = clamp(rne((x - bias) / scale), 0, 15),
//   all codes 0 when scale = 0; RD_16 / RU_16 round toward -inf / +inf into the 16-bit type.
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

namespace q4kv {

struct QuantOut { uint32_t word; uint32_t sb; };         // sb: scale in the low 16 bits, bias in the high 16 bits

// bfloat16 is the upper half of binary32: dropping the lower half rounds toward zero, and a value that lost bits on
// the far side of zero from the rounding direction moves one step away from zero.
__device__ inline uint32_t bf16_bits_rd(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u >> 16) + (((u & 0xFFFFu) != 0u && (u >> 31) != 0u) ? 1u : 0u);
}
__device__ inline uint32_t bf16_bits_ru(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u >> 16) + (((u & 0xFFFFu) != 0u && (u >> 31) == 0u) ? 1u : 0u);
}

// Scale and bias of one group from its minimum and maximum (the fixed binary32 sequence of the header comment):
// their 16-bit patterns and their values.
struct GroupScale { uint32_t hs, hb; float sf, bf; };
__device__ inline GroupScale group_scale(float mn, float mx, bool bf16) {
  GroupScale gs;
  if (bf16) {
    gs.hb = bf16_bits_rd(mn);
    if ((gs.hb & 0x7FFFu) == 0u) gs.hb = 0u;                                      // -0 -> +0
    gs.bf = __uint_as_float(gs.hb << 16);
    gs.hs = bf16_bits_ru(__fdiv_rn(__fsub_rn(mx, gs.bf), 15.0f));
    gs.sf = __uint_as_float(gs.hs << 16);
  } else {
    __half hb = __float2half_rd(mn);
    if (__half2float(hb) == 0.0f) hb = __ushort_as_half((unsigned short)0);       // -0 -> +0
    gs.hb = __half_as_ushort(hb);
    gs.bf = __half2float(hb);
    const __half hs = __float2half_ru(__fdiv_rn(__fsub_rn(mx, gs.bf), 15.0f));
    gs.hs = __half_as_ushort(hs);
    gs.sf = __half2float(hs);
  }
  return gs;
}

// A (scale, bias) pair of the cache as two binary32 numbers.
template <bool kBf16>
__device__ __forceinline__ float2 sb_to_f2(uint32_t u) {
  if (kBf16) return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
  return __half22float2(*reinterpret_cast<const __half2*>(&u));
}

// x[8]: eight consecutive elements owned by this lane; the 8 lanes of a group cooperate.
__device__ inline QuantOut quantize_eight(const float x[8], bool bf16) {
  float mn = x[0], mx = x[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) { mn = fminf(mn, x[i]); mx = fmaxf(mx, x[i]); }
#pragma unroll
  for (int o = 1; o < 8; o <<= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  const GroupScale gs = group_scale(mn, mx, bf16);
  const float bf = gs.bf, sf = gs.sf;
  uint32_t w = 0;
  if (sf != 0.0f) {
    // code = clamp(rne(fl((x - b) / s))).  The eight IEEE divisions dominate this function, so the quotient is
    // taken as t * (1/s) with one fused residual correction (within an ulp of the correctly rounded quotient,
    // 1/s being correctly rounded), which rounds to the same integer unless the quotient sits within a few ulps
    // of k + 1/2; only there is the division itself evaluated.
    const float inv = __frcp_rn(sf);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float t = __fsub_rn(x[i], bf);
      float q = __fmul_rn(t, inv);
      q = __fmaf_rn(__fmaf_rn(-sf, q, t), inv, q);
      if (fabsf(q - (floorf(q) + 0.5f)) < 1e-5f) q = __fdiv_rn(t, sf);
      int c = __float2int_rn(q);
      c = min(max(c, 0), 15);
      w |= (uint32_t)c << (4 * i);
    }
  }
  QuantOut o;
  o.word = w;
  o.sb = gs.hs | (gs.hb << 16);
  return o;
}

__device__ inline void load_eight_bf16(const void* base, size_t elem_index, float x[8]) {
  const uint4 v = *reinterpret_cast<const uint4*>((const uint16_t*)base + elem_index);
  const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    x[2 * i] = __uint_as_float(u[i] << 16);
    x[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
  }
}

}  // namespace q4kv
