// Bring-up path of the grouped SwiGLU expert FFN (plain FMA, one warp per output element).
// Same data flow as the tensor-core path: sorted token rows xp -> bf16 intermediate hbuf ->
// fp32 per-assignment outputs y; weights addressed through the expert->slot table.  Used to
// validate the rest of the step independently of the tcgen05 kernels; never the default.
#include <cuda_bf16.h>

#include "kernels.h"

namespace oled {
namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
  return v;
}

__device__ __forceinline__ float dot8(const uint4& a, const uint4& b) {
  const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    s = fmaf(__uint_as_float(aw[i] << 16), __uint_as_float(bw[i] << 16), s);
    s = fmaf(__uint_as_float(aw[i] & 0xffff0000u), __uint_as_float(bw[i] & 0xffff0000u), s);
  }
  return s;
}

// grid: (I/8, group experts); block 256 = 8 warps, warp w owns intermediate row i = blockIdx.x*8+w
__global__ void __launch_bounds__(256)
ffn1_simple_kernel(const __grid_constant__ FfnGroup grp, const uint8_t* __restrict__ pool,
                   size_t slot_bytes, const int32_t* __restrict__ offsets,
                   const uint16_t* __restrict__ xp, uint16_t* __restrict__ hbuf, int H, int I) {
  griddep_wait();
  const int e = grp.expert[blockIdx.y];
  const uint16_t* w = reinterpret_cast<const uint16_t*>(pool + (size_t)grp.slot[blockIdx.y] * slot_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = blockIdx.x * 8 + warp;
  const uint16_t* wg = w + (size_t)i * H;
  const uint16_t* wu = w + (size_t)(I + i) * H;
  for (int r = offsets[e]; r < offsets[e + 1]; ++r) {
    const uint16_t* xr = xp + (size_t)r * H;
    float a = 0.f, u = 0.f;
    for (int h = lane * 8; h < H; h += 256) {
      const uint4 xv = *reinterpret_cast<const uint4*>(xr + h);
      a += dot8(xv, *reinterpret_cast<const uint4*>(wg + h));
      u += dot8(xv, *reinterpret_cast<const uint4*>(wu + h));
    }
    a = warp_sum(a);
    u = warp_sum(u);
    if (lane == 0) {
      const float hm = a / (1.0f + __expf(-a)) * u;
      const __nv_bfloat16 b = __float2bfloat16_rn(hm);
      hbuf[(size_t)r * I + i] = *reinterpret_cast<const uint16_t*>(&b);
    }
  }
}

// grid: (H/8, group experts)
__global__ void __launch_bounds__(256)
ffn2_simple_kernel(const __grid_constant__ FfnGroup grp, const uint8_t* __restrict__ pool,
                   size_t slot_bytes, const int32_t* __restrict__ offsets,
                   const uint16_t* __restrict__ hbuf, float* __restrict__ y, int H, int I) {
  griddep_wait();
  const int e = grp.expert[blockIdx.y];
  const uint16_t* w = reinterpret_cast<const uint16_t*>(pool + (size_t)grp.slot[blockIdx.y] * slot_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int hh = blockIdx.x * 8 + warp;
  const uint16_t* wd = w + (size_t)2 * I * H + (size_t)hh * I;
  for (int r = offsets[e]; r < offsets[e + 1]; ++r) {
    const uint16_t* hr = hbuf + (size_t)r * I;
    float s = 0.f;
    for (int i = lane * 8; i < I; i += 256)
      s += dot8(*reinterpret_cast<const uint4*>(hr + i), *reinterpret_cast<const uint4*>(wd + i));
    s = warp_sum(s);
    if (lane == 0) y[(size_t)r * H + hh] = s;
  }
}

}  // namespace

void launch_ffn_simple(cudaStream_t st, const FfnGroup& grp, const uint8_t* pool, size_t slot_bytes,
                       const int32_t* offsets, const uint16_t* xp, uint16_t* hbuf, float* y, int H,
                       int I) {
  if (grp.n <= 0) return;
  ffn1_simple_kernel<<<dim3(I / 8, grp.n), 256, 0, st>>>(grp, pool, slot_bytes, offsets, xp, hbuf, H, I);
  ffn2_simple_kernel<<<dim3(H / 8, grp.n), 256, 0, st>>>(grp, pool, slot_bytes, offsets, hbuf, y, H, I);
}

}  // namespace oled
