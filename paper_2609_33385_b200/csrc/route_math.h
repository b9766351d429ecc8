// Device arithmetic of the gate that every kernel computing a routing decision shares: bf16
// unpacking, the gate-score exponential from individually rounded operations, and the
// order-preserving integer key of a logit.  One definition, so that the kernels cannot drift apart.
#pragma once
#include <cstdint>

namespace oled {

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// acc += x.lo * w.lo, then acc += x.hi * w.hi (ascending h) for two packed bf16 pairs, each step
// an fp32 fused multiply-add: fma.rn.f32.bf16 forms the exact product of its bf16 operands and
// rounds once - bit for bit __fmaf_rn of the widened operands - and saves the widening
// instructions, which outnumber the multiply-adds in the gate kernels' small register tiles.
__device__ __forceinline__ void fma_bf16_pair(float& acc, uint32_t x, uint32_t w) {
  asm("{\n .reg .b16 xl, xh, wl, wh;\n mov.b32 {xl, xh}, %1;\n mov.b32 {wl, wh}, %2;\n"
      " fma.rn.f32.bf16 %0, xl, wl, %0;\n fma.rn.f32.bf16 %0, xh, wh, %0;\n}"
      : "+f"(acc)
      : "r"(x), "r"(w));
}

// exp(x) for x <= 0 from individually rounded fp32 operations (no contraction, no fast math).
__device__ __forceinline__ float exp_spec(float x) {
  if (x < -80.0f) return 0.0f;
  const float kLog2e = __uint_as_float(0x3fb8aa3bu);  // fl32(1/ln 2)
  const float kLn2Hi = __uint_as_float(0x3f317000u);  // fl32(ln 2), low 12 significand bits cleared
  const float kLn2Lo = __uint_as_float(0x3805fdf4u);  // fl32(ln 2 - kLn2Hi)
  const float n = rintf(__fmul_rn(x, kLog2e));
  const float r = __fsub_rn(__fsub_rn(x, __fmul_rn(n, kLn2Hi)), __fmul_rn(n, kLn2Lo));
  float p = __uint_as_float(0x39500d01u);                        // 1/5040
  p = __fadd_rn(__fmul_rn(p, r), __uint_as_float(0x3ab60b61u));  // 1/720
  p = __fadd_rn(__fmul_rn(p, r), __uint_as_float(0x3c088889u));  // 1/120
  p = __fadd_rn(__fmul_rn(p, r), __uint_as_float(0x3d2aaaabu));  // 1/24
  p = __fadd_rn(__fmul_rn(p, r), __uint_as_float(0x3e2aaaabu));  // 1/6
  p = __fadd_rn(__fmul_rn(p, r), 0.5f);
  p = __fadd_rn(__fmul_rn(p, r), 1.0f);
  p = __fadd_rn(__fmul_rn(p, r), 1.0f);
  const float scale = __int_as_float(((int)n + 127) << 23);  // 2^n, n >= -116
  return __fmul_rn(p, scale);
}

__device__ __forceinline__ uint32_t order_key(float v) {  // v is not NaN and not -0
  const uint32_t bits = __float_as_uint(v);
  return (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
}

// A logit as the top-k sees it: NaN is read as -inf (the order stays total), -0 as +0 (they
// compare equal, the index decides).
__device__ __forceinline__ float topk_value(float x) {
  return (x == x) ? __fadd_rn(x, 0.0f) : __int_as_float(0xff800000);
}

// Integer numerator contribution of one assignment to the expert reuse score (Sec. 4.3 priority
// equation with psi(c) = c clamped to [0,1], NaN -> 0): floor(fl32(g * psi(c)) * 2^32).  A NaN
// product (non-finite activations) adds nothing; the 64-bit conversion of a NaN would return 2^63.
__device__ __forceinline__ unsigned long long score_quantum(float g, float c) {
  c = (c != c) ? 0.0f : fminf(fmaxf(c, 0.0f), 1.0f);
  const float pv = __fmul_rn(g, c);
  return (pv == pv) ? __float2ull_rz(__fmul_rn(pv, 4294967296.0f)) : 0ull;
}

}  // namespace oled
