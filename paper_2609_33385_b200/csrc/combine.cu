// Weighted un-permute / combine: the gate-weighted sum of the expert outputs of each token
// (paper Sec. 2.1: the MoE layer output is the gate-score-weighted sum over the top-k experts).
// Deterministic: ranks are added in ascending order in fp32, then rounded to bf16.
#include <cuda_bf16.h>

#include <algorithm>

#include "kernels.h"

namespace oled {
namespace {

// BATCH: the number of assignment rows whose loads are issued together.  Small steps (latency-
// bound) take 8 and split a token's row over gridDim.y CTAs, so that a 32-token step still puts
// a CTA on most SMs; large steps keep 1, where the extra registers cost occupancy.
template <bool Y_BF16, int BATCH>
__global__ void __launch_bounds__(256)
combine_kernel(const float* __restrict__ y, const float* __restrict__ gate,
               const int32_t* __restrict__ pos, int H, int K, uint16_t* __restrict__ out,
               const uint16_t* __restrict__ x, uint16_t* __restrict__ x_next,
               uint32_t* __restrict__ zero_words, int n_zero_words, StepTimeline* timeline) {
  const int t = blockIdx.x;
  const int slice = H / gridDim.y, h_begin = blockIdx.y * slice, h_end = h_begin + slice;
  griddep_launch_dependents();
  if (threadIdx.x == 0) timeline_entry(timeline, kTimelineSlots - 1);
  griddep_wait();
  if (threadIdx.x == 0) timeline_start(timeline, kTimelineSlots - 1);
  if (t == 0 && blockIdx.y == 0 && zero_words != nullptr)
    for (int i = threadIdx.x; i < n_zero_words; i += blockDim.x) zero_words[i] = 0u;
  __shared__ float s_g[OLED_MAX_TOPK];
  __shared__ int s_r[OLED_MAX_TOPK];
  if (threadIdx.x < K) {
    s_g[threadIdx.x] = gate[(size_t)t * K + threadIdx.x];
    s_r[threadIdx.x] = pos[(size_t)t * K + threadIdx.x];
  }
  __syncthreads();
  for (int h = h_begin + threadIdx.x * 4; h < h_end; h += blockDim.x * 4) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    // the rows of BATCH assignments are loaded together (independent requests in flight), then
    // accumulated in rank order
    for (int j0 = 0; j0 < K; j0 += BATCH) {
      float4 v[BATCH];
#pragma unroll
      for (int jj = 0; jj < BATCH; ++jj) {
        const int j = j0 + jj;
        if (j < K) {
          if (Y_BF16) {
            const uint2 p = *reinterpret_cast<const uint2*>(reinterpret_cast<const uint16_t*>(y) +
                                                            (size_t)s_r[j] * H + h);
            v[jj] = make_float4(__uint_as_float(p.x << 16), __uint_as_float(p.x & 0xffff0000u),
                                __uint_as_float(p.y << 16), __uint_as_float(p.y & 0xffff0000u));
          } else {
            v[jj] = *reinterpret_cast<const float4*>(y + (size_t)s_r[j] * H + h);
          }
        }
      }
#pragma unroll
      for (int jj = 0; jj < BATCH; ++jj) {
        const int j = j0 + jj;
        if (j < K) {
          const float g = s_g[j];
          acc.x = fmaf(g, v[jj].x, acc.x);
          acc.y = fmaf(g, v[jj].y, acc.y);
          acc.z = fmaf(g, v[jj].z, acc.z);
          acc.w = fmaf(g, v[jj].w, acc.w);
        }
      }
    }
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y);
    __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z, acc.w);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo);
    pk.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(out + (size_t)t * H + h) = pk;
    if (x_next != nullptr) {  // residual on the rounded output: bf16(x + bf16(out))
      const uint2 xv = *reinterpret_cast<const uint2*>(x + (size_t)t * H + h);
      const float2 o0 = __bfloat1622float2(lo), o1 = __bfloat1622float2(hi);
      __nv_bfloat162 r0 = __floats2bfloat162_rn(__uint_as_float(xv.x << 16) + o0.x,
                                                __uint_as_float(xv.x & 0xffff0000u) + o0.y);
      __nv_bfloat162 r1 = __floats2bfloat162_rn(__uint_as_float(xv.y << 16) + o1.x,
                                                __uint_as_float(xv.y & 0xffff0000u) + o1.y);
      uint2 rk;
      rk.x = *reinterpret_cast<uint32_t*>(&r0);
      rk.y = *reinterpret_cast<uint32_t*>(&r1);
      *reinterpret_cast<uint2*>(x_next + (size_t)t * H + h) = rk;
    }
  }
  if (threadIdx.x == 0) timeline_end(timeline, kTimelineSlots - 1);
}

// Large steps with bf16 assignment outputs: eight elements per thread, so that every access is
// a 16-byte vector (the four-element form above reads 8 bytes per lane and row).
__global__ void __launch_bounds__(256)
combine_bf16_wide_kernel(const uint16_t* __restrict__ y, const float* __restrict__ gate,
                         const int32_t* __restrict__ pos, int H, int K, uint16_t* __restrict__ out,
                         const uint16_t* __restrict__ x, uint16_t* __restrict__ x_next,
                         uint32_t* __restrict__ zero_words, int n_zero_words) {
  const int t = blockIdx.x;
  griddep_launch_dependents();
  griddep_wait();
  if (t == 0 && zero_words != nullptr)
    for (int i = threadIdx.x; i < n_zero_words; i += blockDim.x) zero_words[i] = 0u;
  __shared__ float s_g[OLED_MAX_TOPK];
  __shared__ int s_r[OLED_MAX_TOPK];
  if (threadIdx.x < K) {
    s_g[threadIdx.x] = gate[(size_t)t * K + threadIdx.x];
    s_r[threadIdx.x] = pos[(size_t)t * K + threadIdx.x];
  }
  __syncthreads();
  for (int h = threadIdx.x * 8; h < H; h += blockDim.x * 8) {
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    // four assignments' pieces are requested together, then accumulated in rank order
    for (int j0 = 0; j0 < K; j0 += 4) {
      uint4 p[4];
#pragma unroll
      for (int jj = 0; jj < 4; ++jj)
        if (j0 + jj < K) p[jj] = *reinterpret_cast<const uint4*>(y + (size_t)s_r[j0 + jj] * H + h);
#pragma unroll
      for (int jj = 0; jj < 4; ++jj)
        if (j0 + jj < K) {
          const float g = s_g[j0 + jj];
          const uint32_t w[4] = {p[jj].x, p[jj].y, p[jj].z, p[jj].w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            acc[2 * i] = fmaf(g, __uint_as_float(w[i] << 16), acc[2 * i]);
            acc[2 * i + 1] = fmaf(g, __uint_as_float(w[i] & 0xffff0000u), acc[2 * i + 1]);
          }
        }
    }
    uint32_t o[4];
    __nv_bfloat162 ob[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      ob[i] = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
      o[i] = *reinterpret_cast<uint32_t*>(&ob[i]);
    }
    *reinterpret_cast<uint4*>(out + (size_t)t * H + h) = make_uint4(o[0], o[1], o[2], o[3]);
    if (x_next != nullptr) {  // residual on the rounded output: bf16(x + bf16(out))
      const uint4 xv = *reinterpret_cast<const uint4*>(x + (size_t)t * H + h);
      const uint32_t xw[4] = {xv.x, xv.y, xv.z, xv.w};
      uint32_t r[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 of = __bfloat1622float2(ob[i]);
        __nv_bfloat162 rb = __floats2bfloat162_rn(__uint_as_float(xw[i] << 16) + of.x,
                                                  __uint_as_float(xw[i] & 0xffff0000u) + of.y);
        r[i] = *reinterpret_cast<uint32_t*>(&rb);
      }
      *reinterpret_cast<uint4*>(x_next + (size_t)t * H + h) = make_uint4(r[0], r[1], r[2], r[3]);
    }
  }
}

__global__ void __launch_bounds__(256)
residual_add_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ r,
                    uint16_t* __restrict__ y, size_t n) {
  griddep_launch_dependents();
  griddep_wait();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (size_t)gridDim.x * blockDim.x) {
    const float a = __uint_as_float((uint32_t)x[i] << 16);
    const float b = __uint_as_float((uint32_t)r[i] << 16);
    const __nv_bfloat16 s = __float2bfloat16_rn(a + b);
    y[i] = *reinterpret_cast<const uint16_t*>(&s);
  }
}

}  // namespace

void launch_combine(cudaStream_t st, const float* y, int y_bf16, const float* gate, const int32_t* pos, int T,
                    int H, int K, uint16_t* out, const uint16_t* x, uint16_t* x_next,
                    uint32_t* zero_words, int n_zero_words, StepTimeline* timeline) {
  static bool carveout_done = false;
  if (!carveout_done) {  // keep the FFN kernels' shared-memory carve-out: see gate_cluster.cu
    cudaFuncSetAttribute(combine_kernel<true, 8>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    cudaFuncSetAttribute(combine_kernel<false, 8>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    cudaGetLastError();
    carveout_done = true;
  }
  const bool small = (size_t)T * K <= 4096;
  // small steps: slices of 512 columns (128 threads x 4) while that leaves at most ~4 CTAs per SM
  int slices = 1;
  if (small)
    while (slices < 8 && H % (slices * 2 * 512) == 0 && (size_t)T * slices * 2 <= 592) slices *= 2;
  const dim3 sgrid(T, slices), sblock(slices > 1 ? 128 : 256);
  if (y_bf16 && small)
    launch_pdl(combine_kernel<true, 8>, sgrid, sblock, 0, st, y, gate, pos, H, K, out, x, x_next, zero_words,
               n_zero_words, timeline);
  else if (y_bf16 && H % 8 == 0)
    launch_pdl(combine_bf16_wide_kernel, dim3(T), dim3(256), 0, st, reinterpret_cast<const uint16_t*>(y), gate, pos, H,
               K, out, x, x_next, zero_words, n_zero_words);
  else if (y_bf16)
    launch_pdl(combine_kernel<true, 1>, dim3(T), dim3(256), 0, st, y, gate, pos, H, K, out, x, x_next, zero_words,
               n_zero_words, timeline);
  else if (small)
    launch_pdl(combine_kernel<false, 8>, sgrid, sblock, 0, st, y, gate, pos, H, K, out, x, x_next, zero_words,
               n_zero_words, timeline);
  else
    launch_pdl(combine_kernel<false, 1>, dim3(T), dim3(256), 0, st, y, gate, pos, H, K, out, x, x_next, zero_words,
               n_zero_words, timeline);
}

namespace {
constexpr uint32_t kPrefetchChunk = 16384;
// one thread per 16 KB chunk of a listed slot. (Pacing the requests - 1024 threads, a pause between a
// thread's chunks - was measured and made every workload slower.)
__global__ void __launch_bounds__(128)
l2_prefetch_kernel(const uint8_t* __restrict__ pool, unsigned long long slot_bytes, const __grid_constant__ SlotList slots,
                   unsigned long long bytes_per_slot) {
  const unsigned long long chunks_per_slot = (bytes_per_slot + kPrefetchChunk - 1) / kPrefetchChunk;
  const unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= chunks_per_slot * (unsigned long long)slots.n) return;
  const unsigned long long s = i / chunks_per_slot, c = i - s * chunks_per_slot;
  const unsigned long long off = c * kPrefetchChunk;
  const uint32_t bytes = (uint32_t)min((unsigned long long)kPrefetchChunk, bytes_per_slot - off) & ~15u;
  if (bytes == 0) return;
  const uint8_t* src = pool + (unsigned long long)slots.slot[s] * slot_bytes + off;
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
}  // namespace

void launch_l2_prefetch(cudaStream_t st, const uint8_t* pool, size_t slot_bytes, const SlotList& slots,
                        size_t bytes_per_slot) {
  if (slots.n <= 0 || bytes_per_slot == 0) return;
  const unsigned long long chunks = ((bytes_per_slot + kPrefetchChunk - 1) / kPrefetchChunk) * (unsigned long long)slots.n;
  l2_prefetch_kernel<<<(unsigned)((chunks + 127) / 128), 128, 0, st>>>(pool, (unsigned long long)slot_bytes, slots,
                                                                       (unsigned long long)bytes_per_slot);
}

void launch_residual_add(cudaStream_t st, const uint16_t* x, const uint16_t* r, uint16_t* y, size_t n) {
  const int blocks = (int)std::min<size_t>((n + 255) / 256, 148 * 8);
  launch_pdl(residual_add_kernel, dim3(blocks), dim3(256), 0, st, x, r, y, n);
}

}  // namespace oled
