// Device helpers shared by the kernels that turn target rows into picks (step a4): NaN-propagating maxima, the
// marker keys that report non-finite rows, the Philox4x32-10 draw and the integer weight of a logit.
#pragma once

#include "ubt_common.cuh"

namespace ubt {

// A NaN among the logits must not go unnoticed, so the maxima below let NaN win: a fragment that holds one has
// the maximum NaN, fails every "<=" and ">" test, and is reported through a marker key instead of a pick.
__device__ __forceinline__ float max_nan(float a, float b) {
  float d;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
  return d;
}
// Keys above the key of +inf never stand for a value: the first marks a row segment that holds a NaN, the
// second a segment whose CTA gave up a bounded wait.  The walk kernel turns them into status bits; the token
// they decode to is in range, so whatever follows stays memory-safe.
constexpr unsigned long long kKeyPlusInf = 0xff800000ull << 32;
constexpr unsigned long long kKeyNaNSeen = (0xffc00000ull << 32) | 0xffffffffull;
constexpr unsigned long long kKeyGaveUp = ~0ull;


// Fragment maximum without widening: packed bf16 max of the four words, then the two halves.
__device__ __forceinline__ float frag_max(const uint4& v, const __nv_bfloat16*) {
  const __nv_bfloat162 a = __hmax2_nan(*reinterpret_cast<const __nv_bfloat162*>(&v.x),
                                       *reinterpret_cast<const __nv_bfloat162*>(&v.y));
  const __nv_bfloat162 b = __hmax2_nan(*reinterpret_cast<const __nv_bfloat162*>(&v.z),
                                       *reinterpret_cast<const __nv_bfloat162*>(&v.w));
  const __nv_bfloat162 c = __hmax2_nan(a, b);
  const uint32_t w = *reinterpret_cast<const uint32_t*>(&c);
  return max_nan(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
__device__ __forceinline__ float frag_max(const uint4& v, const float*) {
  return max_nan(max_nan(__uint_as_float(v.x), __uint_as_float(v.y)), max_nan(__uint_as_float(v.z), __uint_as_float(v.w)));
}

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t (&out)[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
    const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = h1 ^ c1 ^ k0, n2 = h0 ^ c3 ^ k1;
    c0 = n0; c1 = l1; c2 = n2; c3 = l0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Integer weight of one logit: trunc(2^(40 + y)), y = max(fma(z, a, c), -42), with 2^y evaluated as
// 2^n * p(f), n = rint(y), f = y - n, p a fixed degree-5 polynomial in fma Horner form.  Every step
// is one IEEE-754 operation, so any machine reproduces the same integer.
__device__ __forceinline__ unsigned long long weight_of(float z, float a, float c) {
  float y = __fmaf_rn(z, a, c);
  y = fmaxf(y, -42.0f);
  const float big = 12582912.0f;
  const float tmp = __fadd_rn(y, big);
  const float nf = __fsub_rn(tmp, big);
  const float f = __fsub_rn(y, nf);
  float p = 0x1.5c7746p-10f;
  p = __fmaf_rn(p, f, 0x1.3cea8p-7f);
  p = __fmaf_rn(p, f, 0x1.c6b54ap-5f);
  p = __fmaf_rn(p, f, 0x1.ebf9bcp-3f);
  p = __fmaf_rn(p, f, 0x1.62e42cp-1f);
  p = __fmaf_rn(p, f, 1.0f);
  // p * 2^(n+40): add (n+40) to the exponent field; tmp's low mantissa bits hold n in two's complement
  const uint32_t e = __float_as_uint(p) + ((__float_as_uint(tmp) + 40u) << 23);
  return __float2ull_rz(__uint_as_float(e));
}

}  // namespace ubt
