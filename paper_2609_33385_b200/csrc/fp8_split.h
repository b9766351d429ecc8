// Token operands of the fp8 tensor-core form: a bf16 token row, scaled by a power of two, as the
// sum of two e4m3 terms, so that the MMA can read the experts' e4m3 codes as they are (an MMA
// takes both operands in the same 8-bit kind).  Shared by the kernels that produce the terms (the
// gathering permutation kernel, the split kernel between the two projections) and the FFN
// kernel's epilogue, which undoes the scale.
#pragma once
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include <cstdint>

namespace oled {

// The power of two that brings a token row's largest magnitude (bits of a
// non-negative fp32, see TokenAmax) into [128, 256), and its inverse.  The exponent is clamped so
// that both are normal numbers; an all-zero row takes the largest scale, which is as good as any.
__device__ __forceinline__ uint32_t token_exponent(uint32_t amax_bits) {
  return min(max((amax_bits >> 23) & 0xffu, 8u), 254u);
}
__device__ __forceinline__ float token_scale(uint32_t amax_bits) {
  return __uint_as_float((261u - token_exponent(amax_bits)) << 23);  // 2^(134 - biased exponent)
}
__device__ __forceinline__ float token_scale_inverse(uint32_t amax_bits) {
  return __uint_as_float((token_exponent(amax_bits) - 7u) << 23);
}
// Four bf16 (two words, ascending k) times `scale` -> their first e4m3 terms (one word, ascending
// k) and the e4m3 of sixteen times what the first terms leave.
__device__ __forceinline__ void split_bf16x4(uint32_t w0, uint32_t w1, float scale, uint32_t& t1, uint32_t& t2) {
  uint32_t q1[2], q2[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const uint32_t w = i == 0 ? w0 : w1;
    const float v0 = __uint_as_float(w << 16) * scale, v1 = __uint_as_float(w & 0xffff0000u) * scale;
    const __nv_fp8x2_storage_t a = __nv_cvt_float2_to_fp8x2(make_float2(v0, v1), __NV_SATFINITE, __NV_E4M3);
    const __half2_raw back_raw = __nv_cvt_fp8x2_to_halfraw2(a, __NV_E4M3);
    const float2 back = __half22float2(*reinterpret_cast<const __half2*>(&back_raw));
    const __nv_fp8x2_storage_t b = __nv_cvt_float2_to_fp8x2(
        make_float2((v0 - back.x) * 16.0f, (v1 - back.y) * 16.0f), __NV_SATFINITE, __NV_E4M3);
    q1[i] = a;
    q2[i] = b;
  }
  t1 = q1[0] | (q1[1] << 16);
  t2 = q2[0] | (q2[1] << 16);
}

}  // namespace oled
