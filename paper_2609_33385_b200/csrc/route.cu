// Gate of the MoE layer (paper Sec. 2.1 / Sec. 4.1: the gate yields each token's routed expert
// ids and gate scores), token->expert permutation, and the integer numerators of the expert
// reuse priority (Sec. 4.3 priority equation).
//
// Everything a keep/evict or routing decision depends on is computed in a fixed operation
// order so that it can be reproduced bit for bit elsewhere:
//   * logit(t,e): 32 chains, lane q owns h with (h/8) mod 32 == q, ascending h, one fused
//     multiply-add per term (bf16*bf16 is exact in fp32, so the fma rounds once, like a plain
//     add of the exact product); butterfly over xor distances 16,8,4,2,1; bias one rounded add.
//   * top-k: logit descending, ties to the lower expert index (a NaN logit counts as -inf).
//   * gate scores: z_j = exp_spec(L_j - L_0); S = ((z_0+z_1)+z_2)...; g_j = z_j / S.
//   * score numerators: v = g * psi(c) rounded once; floor(v * 2^32) summed as integers.
// The router stays off the tensor cores on purpose: their accumulation order is unspecified.
#include <cuda_bf16.h>

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <mutex>

#include "kernels.h"
#include "fp8_split.h"
#include "route_math.h"

namespace oled {
namespace {

// Top-k (ties to the lower index), gate scores over the selected logits, counts and integer
// reuse-score numerators of one token; executed by one warp.  row: the token's E logits.
template <int kMaxEPerLane>  // E <= 32 * kMaxEPerLane: bounds the per-lane candidate scan
__device__ __forceinline__ void route_token_tail_n(const float* row, int t, int lane, int E, int K,
                                                 const float* __restrict__ conf, int32_t* __restrict__ ids,
                                                 float* __restrict__ gate, int32_t* __restrict__ counts,
                                                 unsigned long long* __restrict__ scores,
                                                 int32_t* __restrict__ seg_counts, int seg_tokens) {
    float v[kMaxEPerLane];
#pragma unroll
    for (int i = 0; i < kMaxEPerLane; ++i) {
      const int e = lane + 32 * i;
      const float x = e < E ? row[e] : 0.0f;
      // a NaN logit is read as -inf: the order stays total; -0 becomes +0 (they compare equal)
      v[i] = (x == x) ? __fadd_rn(x, 0.0f) : __int_as_float(0xff800000);
    }
    uint32_t used = 0;
    int my_id = 0;
    float my_logit = 0.0f;
    for (int r = 0; r < K; ++r) {
      float bv = 0.0f;
      int be = 0x7fffffff;
#pragma unroll
      for (int i = 0; i < kMaxEPerLane; ++i) {
        const int e = lane + 32 * i;
        if (e < E && !((used >> i) & 1u)) {
          if (be == 0x7fffffff || v[i] > bv) {  // ascending e: strict > keeps the lower index
            bv = v[i];
            be = e;
          }
        }
      }
      // the warp's best: largest logit, then lowest index - two integer warp reductions (the logit
      // as an order-preserving unsigned key; a lane without a candidate holds key 0, below every
      // logit's key) and one broadcast of the winning logit
      const uint32_t bits = __float_as_uint(bv);
      const uint32_t key = be == 0x7fffffff ? 0u : ((bits & 0x80000000u) ? ~bits : (bits | 0x80000000u));
      const uint32_t kmax = __reduce_max_sync(0xffffffffu, key);
      be = (int)__reduce_min_sync(0xffffffffu, key == kmax ? (uint32_t)be : 0x7fffffffu);
      bv = __shfl_sync(0xffffffffu, bv, be & 31);
      if ((be & 31) == lane) used |= 1u << (be >> 5);
      if (lane == r) {
        my_id = be;
        my_logit = bv;
      }
    }
    const float top = __shfl_sync(0xffffffffu, my_logit, 0);
    const float z = lane < K ? exp_spec(__fsub_rn(my_logit, top)) : 0.0f;
    float s = __shfl_sync(0xffffffffu, z, 0);
    for (int j = 1; j < K; ++j) s = __fadd_rn(s, __shfl_sync(0xffffffffu, z, j));
    if (lane < K) {
      const float g = __fdiv_rn(z, s);
      ids[(size_t)t * K + lane] = my_id;
      gate[(size_t)t * K + lane] = g;
      float c = conf[t];
      c = (c != c) ? 0.0f : fminf(fmaxf(c, 0.0f), 1.0f);  // psi(c) = c, clamped; NaN -> 0
      const float pv = __fmul_rn(g, c);
      // a NaN product (non-finite activations) adds nothing; the 64-bit conversion of a NaN
      // would return 2^63
      const unsigned long long q = (pv == pv) ? __float2ull_rz(__fmul_rn(pv, 4294967296.0f)) : 0ull;
      atomicAdd(&counts[my_id], 1);
      atomicAdd(&scores[my_id], q);
      if (seg_counts != nullptr) atomicAdd(&seg_counts[(t / seg_tokens) * E + my_id], 1);
    }
  }

// The same selection whatever the bound: a tighter bound only drops candidates that do not exist.
__device__ __forceinline__ void route_token_tail(const float* row, int t, int lane, int E, int K,
                                                 const float* __restrict__ conf, int32_t* __restrict__ ids,
                                                 float* __restrict__ gate, int32_t* __restrict__ counts,
                                                 unsigned long long* __restrict__ scores,
                                                 int32_t* __restrict__ seg_counts = nullptr, int seg_tokens = 1) {
  if (E <= 64) route_token_tail_n<2>(row, t, lane, E, K, conf, ids, gate, counts, scores, seg_counts, seg_tokens);
  else if (E <= 128) route_token_tail_n<4>(row, t, lane, E, K, conf, ids, gate, counts, scores, seg_counts, seg_tokens);
  else route_token_tail_n<OLED_MAX_EXPERTS / 32>(row, t, lane, E, K, conf, ids, gate, counts, scores, seg_counts, seg_tokens);
}

// The previous layer's gate-weighted combine and residual, done by the gate kernel of the next
// layer for its own token (paper Sec. 2.1: the MoE output is the gate-score-weighted sum over the
// top-k experts; the stack adds it to the layer's input).  Arithmetic and order are those of
// combine_kernel: fp32 fused multiply-adds in rank order, out = bf16(sum), x = bf16(x_prev + out).
// n_rows tokens t0 .. t0 + n_rows - 1; their rows end up in s_x[row][H] as well.
__device__ __forceinline__ void combine_rows(const CombinePrev& p, int t0, int n_rows, int H, uint16_t* s_x_all,
                                             float* s_g_all, int* s_r_all) {
  const int K = p.K;
  // the small operands of all rows first (one round trip), then row after row
  for (int i = threadIdx.x; i < n_rows * K; i += blockDim.x) {
    s_g_all[i] = p.gate[(size_t)t0 * K + i];
    s_r_all[i] = p.pos[(size_t)t0 * K + i];
  }
  __syncthreads();
  for (int row = 0; row < n_rows; ++row) {
  const int t = t0 + row;
  const float* s_g = s_g_all + row * K;
  const int* s_r = s_r_all + row * K;
  uint16_t* s_x = s_x_all + (size_t)row * H;
  for (int h = threadIdx.x * 4; h < H; h += blockDim.x * 4) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const uint2 xv = *reinterpret_cast<const uint2*>(p.x + (size_t)t * H + h);
    for (int j0 = 0; j0 < K; j0 += 8) {  // the rows of eight assignments are loaded together
      float4 v[8];
#pragma unroll
      for (int jj = 0; jj < 8; ++jj)
        if (j0 + jj < K) v[jj] = *reinterpret_cast<const float4*>(p.y + (size_t)s_r[j0 + jj] * H + h);
#pragma unroll
      for (int jj = 0; jj < 8; ++jj)
        if (j0 + jj < K) {
          const float g = s_g[j0 + jj];
          acc.x = fmaf(g, v[jj].x, acc.x);
          acc.y = fmaf(g, v[jj].y, acc.y);
          acc.z = fmaf(g, v[jj].z, acc.z);
          acc.w = fmaf(g, v[jj].w, acc.w);
        }
    }
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y);
    __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z, acc.w);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo);
    pk.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p.out + (size_t)t * H + h) = pk;
    const float2 o0 = __bfloat1622float2(lo), o1 = __bfloat1622float2(hi);
    __nv_bfloat162 r0 = __floats2bfloat162_rn(__uint_as_float(xv.x << 16) + o0.x,
                                              __uint_as_float(xv.x & 0xffff0000u) + o0.y);
    __nv_bfloat162 r1 = __floats2bfloat162_rn(__uint_as_float(xv.y << 16) + o1.x,
                                              __uint_as_float(xv.y & 0xffff0000u) + o1.y);
    uint2 rk;
    rk.x = *reinterpret_cast<uint32_t*>(&r0);
    rk.y = *reinterpret_cast<uint32_t*>(&r1);
    *reinterpret_cast<uint2*>(p.x_next + (size_t)t * H + h) = rk;
    *reinterpret_cast<uint2*>(s_x + h) = rk;
  }
  }
}

// TT tokens per CTA, WARPS warps; each warp owns kEPerWarp experts per pass and all TT tokens.  Small
// blocks use TT = 1 with 16 warps (one pass covers 64 experts) and keep several 256-wide
// chunks of loads in flight; the chain order of every logit is the same in all variants.
// TT <= 4 (few-token steps): the tokens' rows are staged in shared memory - copied from x, or
// produced by the previous layer's combine (prev.y != nullptr), which this kernel then carries
// out for its tokens - and the top-k is a rank computation spread over all warps: expert e is
// selected iff fewer than K experts precede it in the order (logit descending, index ascending),
// and its rank is the number that do - the same total order a round-by-round selection walks.
// One token per CTA while that gives at most one wave of CTAs; two or four beyond (every CTA
// streams the whole router matrix, so a second wave costs as much as the first).
// The kernel reports nothing to the host: the permutation kernel, which follows it in every step,
// publishes the finished counts and scores without any ticket or fence.
template <int TT, int WARPS, int UNROLL, int kEPerWarp>
__global__ void __launch_bounds__(WARPS * 32)
route_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ wr,
             const float* __restrict__ bias, const float* __restrict__ conf, int T, int H, int E,
             int K, float* __restrict__ logits_out, int32_t* __restrict__ ids,
             float* __restrict__ gate, int32_t* __restrict__ counts,
             unsigned long long* __restrict__ scores, CombinePrev prev, StepTimeline* timeline) {
  extern __shared__ __align__(16) uint8_t s_dyn[];
  float* s_logits = reinterpret_cast<float*>(s_dyn);                       // [TT][E]
  constexpr bool staged = TT <= 4;
  constexpr int kST = staged ? TT : 1;
  // [TT][H] (staged forms only), on a 16-byte boundary: rows are moved with 16-byte vector accesses
  uint16_t* s_x = reinterpret_cast<uint16_t*>(s_dyn + (((size_t)TT * E * 4 + 15) & ~(size_t)15));
  __shared__ int s_sel_id[kST][OLED_MAX_TOPK];
  __shared__ float s_sel_logit[kST][OLED_MAX_TOPK];
  __shared__ float s_g[kST * OLED_MAX_TOPK];
  __shared__ int s_r[kST * OLED_MAX_TOPK];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t0 = blockIdx.x * TT;
  griddep_launch_dependents();
  if (threadIdx.x == 0) timeline_entry(timeline, 0);
  constexpr int kRouteWarps = WARPS;
  const int my_tokens = min(TT, T - t0);
  if (staged && gridDim.x <= 148) {
    // Small steps: the router weights do not depend on the predecessor (the previous layer's
    // expert FFN), but the expert weights streamed since their last use have pushed them out of
    // L2 - so they are called back in while this kernel still waits for its input.
    for (int eb = warp * kEPerWarp; eb < E; eb += kRouteWarps * kEPerWarp)
#pragma unroll
      for (int b = 0; b < kEPerWarp; ++b) {
        const int e = min(eb + b, E - 1);
        for (int off = lane * 64; off < H; off += 32 * 64)  // 128-byte lines of the row
          asm volatile("prefetch.global.L2 [%0];" ::"l"(wr + (size_t)e * H + off));
      }
  }
  griddep_wait();
  if (threadIdx.x == 0) timeline_start(timeline, 0);
  if (staged) {
    if (prev.y != nullptr) {
      // CTA 0 also clears the control block the previous step used (its kernels have completed)
      if (blockIdx.x == 0 && prev.zero_words != nullptr)
        for (int i = threadIdx.x; i < prev.n_zero_words; i += blockDim.x) prev.zero_words[i] = 0u;
      combine_rows(prev, t0, my_tokens, H, s_x, s_g, s_r);
    } else {
      for (int c = threadIdx.x; c < my_tokens * (H / 8); c += blockDim.x)
        reinterpret_cast<uint4*>(s_x)[c] = reinterpret_cast<const uint4*>(x + (size_t)t0 * H)[c];
    }
    __syncthreads();
  }

  for (int eb = warp * kEPerWarp; eb < E; eb += kRouteWarps * kEPerWarp) {
    float acc[TT][kEPerWarp];
#pragma unroll
    for (int a = 0; a < TT; ++a)
#pragma unroll
      for (int b = 0; b < kEPerWarp; ++b) acc[a][b] = 0.0f;

#pragma unroll UNROLL
    for (int hc = 0; hc < H; hc += 256) {
      const int h = hc + lane * 8;
      uint32_t xw[TT][4], ww[kEPerWarp][4];
#pragma unroll
      for (int a = 0; a < TT; ++a) {
        const int t = min(t0 + a, T - 1);
        // (staged rows beyond the step's last token hold stale shared memory: their logits are never used)
        const uint4 v = staged ? *reinterpret_cast<const uint4*>(s_x + (size_t)a * H + h)
                               : *reinterpret_cast<const uint4*>(x + (size_t)t * H + h);
        xw[a][0] = v.x; xw[a][1] = v.y; xw[a][2] = v.z; xw[a][3] = v.w;
      }
#pragma unroll
      for (int b = 0; b < kEPerWarp; ++b) {
        const int e = min(eb + b, E - 1);
        const uint4 v = *reinterpret_cast<const uint4*>(wr + (size_t)e * H + h);
        ww[b][0] = v.x; ww[b][1] = v.y; ww[b][2] = v.z; ww[b][3] = v.w;
      }
      // elements in ascending h: word 0 low half, word 0 high half, word 1 low half, ...
#pragma unroll
      for (int wi = 0; wi < 4; ++wi)
#pragma unroll
        for (int a = 0; a < TT; ++a)
#pragma unroll
          for (int b = 0; b < kEPerWarp; ++b) fma_bf16_pair(acc[a][b], xw[a][wi], ww[b][wi]);
    }
#pragma unroll
    for (int a = 0; a < TT; ++a)
#pragma unroll
      for (int b = 0; b < kEPerWarp; ++b) {
        float v = acc[a][b];
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) v = __fadd_rn(v, __shfl_xor_sync(0xffffffffu, v, d));
        const int e = eb + b;
        if (lane == 0 && e < E && t0 + a < T) {
          if (bias != nullptr) v = __fadd_rn(v, bias[e]);
          s_logits[a * E + e] = v;
          if (logits_out != nullptr) logits_out[(size_t)(t0 + a) * E + e] = v;
        }
      }
  }
  __syncthreads();

  if (staged) {
    // top-k by rank, work items (token, expert) over all warps; then one warp per token: gate
    // scores, counts and reuse-score numerators
    for (int w = warp; w < my_tokens * E; w += kRouteWarps) {
      const int a = w / E, e = w - a * E;
      const float* row = s_logits + a * E;
      const float ve = topk_value(row[e]);
      const uint32_t ke = order_key(ve);
      int before = 0;
      for (int o = lane; o < E; o += 32) {
        const uint32_t ko = order_key(topk_value(row[o]));
        before += (ko > ke || (ko == ke && o < e)) ? 1 : 0;
      }
      before = __reduce_add_sync(0xffffffffu, before);
      if (lane == 0 && before < K) {
        s_sel_id[a][before] = e;
        s_sel_logit[a][before] = ve;
      }
    }
    __syncthreads();
    for (int a = warp; a < my_tokens; a += kRouteWarps) {
      const int t = t0 + a;
      const int my_id = lane < K ? s_sel_id[a][lane] : 0;
      const float my_logit = lane < K ? s_sel_logit[a][lane] : 0.0f;
      const float top = __shfl_sync(0xffffffffu, my_logit, 0);
      const float z = lane < K ? exp_spec(__fsub_rn(my_logit, top)) : 0.0f;
      float sum = __shfl_sync(0xffffffffu, z, 0);
      for (int j = 1; j < K; ++j) sum = __fadd_rn(sum, __shfl_sync(0xffffffffu, z, j));
      if (lane < K) {
        const float g = __fdiv_rn(z, sum);
        ids[(size_t)t * K + lane] = my_id;
        gate[(size_t)t * K + lane] = g;
        atomicAdd(&counts[my_id], 1);
        atomicAdd(&scores[my_id], score_quantum(g, conf[t]));
      }
    }
  } else {
    // one warp per token
    for (int a = warp; a < TT; a += kRouteWarps) {
      const int t = t0 + a;
      if (t >= T) continue;
      route_token_tail(s_logits + a * E, t, lane, E, K, conf, ids, gate, counts, scores);
    }
  }
  if (threadIdx.x == 0) timeline_end(timeline, 0);
}

// Many-token steps: TT tokens per CTA, eight warps, every warp a register tile of TT tokens x 8
// experts.  The plain kernel above re-reads the router matrix once per eight tokens through the L1
// path and spends an ALU instruction on every bf16 -> fp32 conversion; it reaches a third of the
// FP32 pipe.  Here
//  - the operands are staged in shared memory by cp.async, a ring of k-chunks of 256 elements (the
//    TT token rows and 64 router rows of a chunk), so that the warps read only shared memory
//    (conflict-free 16-byte reads) and the global loads of later chunks are always in flight;
//  - the multiply-adds take their bf16 operands directly (fma.rn.f32.bf16: exact product, one
//    rounding - bit for bit the fp32 fused multiply-add of the converted operands), which removes
//    the conversions;
//  - TT is chosen by the launcher so that the CTAs fill whole waves of SMs (4096 tokens: 14 per
//    CTA, 293 CTAs, two waves on 148 SMs), and a larger TT re-reads the router matrix less often.
// Same chains, same order: lane q still owns the elements h with (h/8) mod 32 == q and walks them
// in ascending order.  Experts beyond 64 take further passes over the rows.
constexpr int kManyWarps = 8, kManyExperts = 64, kManyStages = 4;
__host__ __device__ constexpr int many_stage_bytes(int tt) { return (tt + kManyExperts) * 512; }  // one k-chunk of 256 bf16 per row

template <int TT>
__global__ void __launch_bounds__(kManyWarps * 32, 1)
route_many_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ wr,
                  const float* __restrict__ bias, const float* __restrict__ conf, int T, int H, int E,
                  int K, float* __restrict__ logits_out, int32_t* __restrict__ ids,
                  float* __restrict__ gate, int32_t* __restrict__ counts,
                  unsigned long long* __restrict__ scores, StepTimeline* timeline,
                  int32_t* __restrict__ seg_counts, int seg_tokens) {
  constexpr int kStageBytes = many_stage_bytes(TT);
  constexpr int kRows = TT + kManyExperts;
  extern __shared__ __align__(16) uint8_t s_dyn[];
  uint8_t* s_ring = s_dyn;                                                        // [stages][TT + 64 rows][512 B]
  float* s_logits = reinterpret_cast<float*>(s_dyn + kManyStages * kStageBytes);  // [TT][E]
  __shared__ const uint16_t* s_rowptr[kRows];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t0 = blockIdx.x * TT;
  griddep_launch_dependents();
  if (threadIdx.x == 0) timeline_entry(timeline, 0);
  griddep_wait();
  if (threadIdx.x == 0) timeline_start(timeline, 0);
  const int n_chunks = H / 256;
  const uint32_t ring_base = (uint32_t)__cvta_generic_to_shared(s_ring);

  for (int e0 = 0; e0 < E; e0 += kManyExperts) {
    // one stage: rows 0..TT-1 = tokens t0.., rows TT.. = experts e0..; each row 32 pieces of 16 bytes.
    // The rows' addresses are looked up in a table (one 8-byte read instead of a clamp and a 64-bit
    // multiply per copy: the copies' own instructions are a tenth of the loop otherwise).
    __syncthreads();  // the previous pass has finished with the ring and the table
    for (int row = threadIdx.x; row < kRows; row += kManyWarps * 32)
      s_rowptr[row] = row < TT ? x + (size_t)min(t0 + row, T - 1) * H
                               : wr + (size_t)min(e0 + row - TT, E - 1) * H;
    auto issue = [&](int chunk) {
      const uint32_t dst0 = ring_base + (uint32_t)(chunk % kManyStages) * kStageBytes + (uint32_t)lane * 16u;
#pragma unroll
      for (int j = 0; j < (kRows + kManyWarps - 1) / kManyWarps; ++j) {
        const int row = warp + j * kManyWarps;
        if (row < kRows)
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst0 + (uint32_t)row * 512u),
                       "l"(s_rowptr[row] + (size_t)chunk * 256 + lane * 8)
                       : "memory");
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    float acc[TT][8];
#pragma unroll
    for (int a = 0; a < TT; ++a)
#pragma unroll
      for (int b = 0; b < 8; ++b) acc[a][b] = 0.0f;
    __syncthreads();  // the table is complete
    for (int c = 0; c < kManyStages - 1; ++c) {
      if (c < n_chunks) issue(c);
      else asm volatile("cp.async.commit_group;" ::: "memory");
    }
    for (int c = 0; c < n_chunks; ++c) {
      asm volatile("cp.async.wait_group %0;" ::"n"(kManyStages - 2) : "memory");  // chunk c has landed (this thread's part)
      __syncthreads();                                                            // ... everyone's; and chunk c-1 is consumed
      if (c + kManyStages - 1 < n_chunks) issue(c + kManyStages - 1);
      else asm volatile("cp.async.commit_group;" ::: "memory");
      const uint8_t* st = s_ring + (size_t)(c % kManyStages) * kStageBytes;
      uint4 xw[TT], ww[8];
#pragma unroll
      for (int a = 0; a < TT; ++a) xw[a] = *reinterpret_cast<const uint4*>(st + a * 512 + lane * 16);
#pragma unroll
      for (int b = 0; b < 8; ++b) ww[b] = *reinterpret_cast<const uint4*>(st + (TT + warp * 8 + b) * 512 + lane * 16);
      // elements in ascending h: word 0 low half, word 0 high half, word 1 low half, ...
#pragma unroll
      for (int a = 0; a < TT; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) fma_bf16_pair(acc[a][b], xw[a].x, ww[b].x);
#pragma unroll
      for (int a = 0; a < TT; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) fma_bf16_pair(acc[a][b], xw[a].y, ww[b].y);
#pragma unroll
      for (int a = 0; a < TT; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) fma_bf16_pair(acc[a][b], xw[a].z, ww[b].z);
#pragma unroll
      for (int a = 0; a < TT; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) fma_bf16_pair(acc[a][b], xw[a].w, ww[b].w);
    }
    // The 32 partial sums of every (token, expert) pair are added in the order of the xor butterfly
    // (offsets 16, 8, 4, 2, 1; at every step a lane adds its partner's value to its own).  Addition
    // is commutative bit for bit, so every lane of the butterfly ends with the same value, and the
    // 32 pairs of a group can share the steps: at offset d a lane keeps the half of its pairs
    // whose index has bit d equal to its own lane's bit and hands the other half to its partner -
    // 31 shuffles per 32 pairs instead of 160, and lane l ends with the sum of pair l.
#pragma unroll
    for (int g = 0; g < (TT * 8 + 31) / 32; ++g) {
      float v[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const int p = g * 32 + i;  // pair p: token p / 8, expert column p % 8
        v[i] = p < TT * 8 ? acc[p / 8][p % 8] : 0.0f;
      }
#pragma unroll
      for (int d = 16; d >= 1; d >>= 1) {
        const bool upper = (lane & d) != 0;
#pragma unroll
        for (int i = 0; i < d; ++i) {
          const float keep = upper ? v[i + d] : v[i];
          const float send = upper ? v[i] : v[i + d];
          v[i] = __fadd_rn(keep, __shfl_xor_sync(0xffffffffu, send, d));
        }
      }
      const int p = g * 32 + lane, a = p / 8, e = e0 + warp * 8 + p % 8;
      if (p < TT * 8 && e < E && t0 + a < T) {
        float r = v[0];
        if (bias != nullptr) r = __fadd_rn(r, bias[e]);
        s_logits[a * E + e] = r;
        if (logits_out != nullptr) logits_out[(size_t)(t0 + a) * E + e] = r;
      }
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();
  // one warp per token
  for (int a = warp; a < TT; a += kManyWarps) {
    const int t = t0 + a;
    if (t >= T) continue;
    route_token_tail(s_logits + a * E, t, lane, E, K, conf, ids, gate, counts, scores, seg_counts, seg_tokens);
  }
  if (threadIdx.x == 0) timeline_end(timeline, 0);
}

// One CTA per expert (blockIdx.x): offset = sum of the counts before it; then a stable scan of the
// flat assignment list (ascending t*K+j) hands out consecutive sorted rows.
// If xp != nullptr the expert's CTAs (gridDim.y of them) also copy its token rows into sorted
// order (xp[r,:] = x[perm[r]/K,:]); used for small steps, larger ones run gather_kernel instead.
// Each of those CTAs repeats the scan for itself - a few hundred ids - keeps the token of every
// sorted row in shared memory (reading the rows' numbers back from global memory would cost a
// round trip before the first load), and takes every gridDim.y-th batch of RB rows, so that an
// expert that received many tokens does not make the step wait for one CTA's chain of batches.
// Only the CTAs with blockIdx.y == 0 write offsets, perm and pos.
constexpr int kGatherTokMax = 4096;  // rows of one expert in a step that gathers here (T * K <= 4096)
// RB: rows a CTA copies at a time.  Two, with eight CTAs per expert, in gathering launches: an
// expert's handful of rows is then spread over several SMs (with one CTA taking eight rows the
// step waited 3 us longer whenever an expert had more than eight, and the e4m3 terms of fp8
// steps, whose conversions are the long pole, came to 7 us).  (Eight: launches that do not gather.)
template <int RB>
__global__ void __launch_bounds__(256)
permute_kernel(const int32_t* __restrict__ ids, const int32_t* __restrict__ counts, int n, int E,
               int32_t* __restrict__ offsets, int32_t* __restrict__ perm, int32_t* __restrict__ pos,
               const uint16_t* __restrict__ x, uint16_t* __restrict__ xp, int H, int K, StepTimeline* timeline,
               TokenSplit split, const int32_t* __restrict__ seg_counts, int seg_tokens) {
  uint32_t* const amax_in = split.amax_in;
  uint32_t* const amax_mid = split.amax_mid;
  __shared__ int s_red[8];
  __shared__ int s_base;
  __shared__ int s_tok[kGatherTokMax];
  __shared__ uint32_t s_amax[3][RB];  // per batch of RB rows, three batches in rotation (see the gather loop)
  const int e = blockIdx.x;
  // segmented launches (no gathering): CTA (e, s) scans segment s of the assignment list only and
  // starts behind the expert's rows of the earlier segments, whose number the gate kernel counted
  const bool segmented = seg_counts != nullptr;
  const bool writer = blockIdx.y == 0 || segmented;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  griddep_launch_dependents();
  if (threadIdx.x == 0) timeline_entry(timeline, 1);
  griddep_wait();
  if (threadIdx.x == 0) timeline_start(timeline, 1);
  int part = 0;
  for (int i = threadIdx.x; i < e; i += blockDim.x) part += counts[i];
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) part += __shfl_xor_sync(0xffffffffu, part, d);
  if (lane == 0) s_red[warp] = part;
  __syncthreads();
  if (threadIdx.x == 0) {
    int off = 0;
    for (int w = 0; w < 8; ++w) off += s_red[w];
    s_base = off;
    if (blockIdx.y == 0) {
      offsets[e] = off;
      if (e == E - 1) offsets[E] = off + counts[e];
    }
    if (segmented) {
      for (int s = 0; s < (int)blockIdx.y; ++s) off += seg_counts[s * E + e];
      s_base = off;
    }
  }
  __syncthreads();
  // (a CTA beyond the first of an expert has work only if the expert has a batch of rows for it)
  if (segmented ? seg_counts[blockIdx.y * E + e] == 0 : (counts[e] == 0 || (int)blockIdx.y * RB >= counts[e])) {
    if (threadIdx.x == 0) timeline_end(timeline, 1);
    return;
  }
  int base = s_base;
  const int a_first = segmented ? (int)blockIdx.y * seg_tokens * K : 0;
  const int a_end = segmented ? min(n, a_first + seg_tokens * K) : n;
  // stable scan, 8 consecutive assignments per thread and 2048 per round
  for (int a0 = a_first; a0 < a_end; a0 += 8 * blockDim.x) {
    const int first = a0 + threadIdx.x * 8;
    int v[8];
    if (first + 8 <= a_end) {
      const int4 lo = *reinterpret_cast<const int4*>(ids + first);
      const int4 hi = *reinterpret_cast<const int4*>(ids + first + 4);
      v[0] = lo.x; v[1] = lo.y; v[2] = lo.z; v[3] = lo.w;
      v[4] = hi.x; v[5] = hi.y; v[6] = hi.z; v[7] = hi.w;
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = first + i < a_end ? ids[first + i] : -1;
    }
    uint32_t m = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) m |= (v[i] == e ? 1u : 0u) << i;
    const int c = __popc(m);
    int incl = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int o = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += o;
    }
    __syncthreads();  // previous round's s_red fully consumed
    if (lane == 31) s_red[warp] = incl;
    __syncthreads();
    int before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      const int cw = s_red[w];
      if (w < warp) before += cw;
      total += cw;
    }
    int r = base + before + incl - c;
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if ((m >> i) & 1u) {
        if (writer) {
          perm[r] = first + i;
          pos[first + i] = r;
        }
        if (xp != nullptr) s_tok[r - s_base] = (first + i) / K;
        ++r;
      }
    base += total;
  }
  if (xp == nullptr) {
    if (threadIdx.x == 0) timeline_end(timeline, 1);
    return;
  }
  if (threadIdx.x < 3 * RB) s_amax[threadIdx.x / RB][threadIdx.x % RB] = 0u;
  __syncthreads();  // the tokens of this expert's rows are in shared memory
  // eight rows at a time: their token numbers, then their loads, are independent memory
  // operations in flight together (a row-by-row loop is a chain of dependent round trips)
  const int vec_per_row = H / 8, first = s_base, rows = counts[e];
  const uint4* src = reinterpret_cast<const uint4*>(x);
  uint4* dst = reinterpret_cast<uint4*>(xp);
  int batch = 0;
  for (int r0 = (int)blockIdx.y * RB; r0 < rows; r0 += RB * (int)gridDim.y, ++batch) {
    int tok[RB];
#pragma unroll
    for (int j = 0; j < RB; ++j) tok[j] = r0 + j < rows ? s_tok[r0 + j] : -1;
    uint32_t big[RB];  // per row: max of |bf16| bit patterns, two per word
#pragma unroll
    for (int j = 0; j < RB; ++j) big[j] = 0u;
    uint4 v[RB];  // (the last vectors stay in registers for the e4m3 terms below)
    int c_last = -1;
    for (int c = threadIdx.x; c < vec_per_row; c += blockDim.x) {
      c_last = c;
#pragma unroll
      for (int j = 0; j < RB; ++j)
        if (tok[j] >= 0) v[j] = src[(size_t)tok[j] * vec_per_row + c];
#pragma unroll
      for (int j = 0; j < RB; ++j)
        if (tok[j] >= 0) {
          dst[(size_t)(first + r0 + j) * vec_per_row + c] = v[j];
          if (amax_in != nullptr)
            big[j] = __vmaxu2(__vmaxu2(big[j], __vmaxu2(v[j].x & 0x7fff7fffu, v[j].y & 0x7fff7fffu)),
                              __vmaxu2(v[j].z & 0x7fff7fffu, v[j].w & 0x7fff7fffu));
        }
    }
    if (amax_in != nullptr) {
      // the rows' largest magnitudes (a bf16 magnitude's bits order like the value) and a cleared
      // word per row for the intermediate rows' maxima.  One barrier per batch: a batch's words
      // were cleared two batches (two barriers) ago, and it clears the words of the batch after next.
      uint32_t* amax_now = s_amax[batch % 3];
#pragma unroll
      for (int j = 0; j < RB; ++j) {
        const uint32_t m = __reduce_max_sync(0xffffffffu, max(big[j] & 0xffffu, big[j] >> 16));
        if (lane == 0 && m != 0u) atomicMax(&amax_now[j], m);
      }
      __syncthreads();
      if (threadIdx.x < RB) {
        s_amax[(batch + 2) % 3][threadIdx.x] = 0u;
        if (r0 + (int)threadIdx.x < rows) {
          amax_in[first + r0 + threadIdx.x] = amax_now[threadIdx.x] << 16;
          amax_mid[first + r0 + threadIdx.x] = 0u;
        }
      }
      // the rows' two e4m3 terms (vectors of earlier rounds of the loop above are read back)
      for (int c = threadIdx.x; c < vec_per_row; c += blockDim.x) {
#pragma unroll
        for (int j = 0; j < RB; ++j)
          if (tok[j] >= 0) {
            const size_t r = (size_t)(first + r0 + j);
            const uint4 vv = c == c_last ? v[j] : dst[r * vec_per_row + c];
            const float scale = token_scale(amax_now[j] << 16);
            uint2 t1, t2;
            split_bf16x4(vv.x, vv.y, scale, t1.x, t2.x);
            split_bf16x4(vv.z, vv.w, scale, t1.y, t2.y);
            uint2* out1 = reinterpret_cast<uint2*>(split.terms_in + r * H);
            uint2* out2 = reinterpret_cast<uint2*>(split.terms_in + ((size_t)split.rows + r) * H);
            out1[c] = t1;
            out2[c] = t2;
          }
      }
    }
  }
  if (threadIdx.x == 0) timeline_end(timeline, 1);
}

// One warp per sorted row: the row's token number once, then the row's 16-byte vectors, four
// loads in flight per lane.
__global__ void __launch_bounds__(256)
gather_kernel(const uint16_t* __restrict__ x, const int32_t* __restrict__ perm, int n_rows, int H,
              int K, uint16_t* __restrict__ xp) {
  const int vec_per_row = H / 8;
  const int lane = threadIdx.x & 31;
  const int warps = gridDim.x * (blockDim.x >> 5);
  griddep_launch_dependents();
  griddep_wait();
  for (int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); r < n_rows; r += warps) {
    const int t = perm[r] / K;
    const uint4* src = reinterpret_cast<const uint4*>(x) + (size_t)t * vec_per_row;
    uint4* dst = reinterpret_cast<uint4*>(xp) + (size_t)r * vec_per_row;
    for (int c0 = lane; c0 < vec_per_row; c0 += 128) {
      uint4 v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (c0 + 32 * j < vec_per_row) v[j] = src[c0 + 32 * j];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (c0 + 32 * j < vec_per_row) dst[c0 + 32 * j] = v[j];
    }
  }
}

}  // namespace

constexpr int kRouteSmallMax = 1024;  // largest step that takes the one-token-per-CTA gate kernel

static thread_local bool g_pdl_step = true;
static std::atomic<bool> g_pdl_allowed{true};
void pdl_set_step(bool on) { g_pdl_step = on; }
void pdl_set_allowed(bool on) { g_pdl_allowed.store(on); }
bool pdl_enabled() { return g_pdl_allowed.load() && g_pdl_step; }

bool route_can_take_combine(int T) { return T <= kRouteSmallMax; }

void launch_route(cudaStream_t st, const uint16_t* x, const uint16_t* w_router, const float* bias,
                  const float* conf, int T, int H, int E, int K, float* logits, int32_t* ids,
                  float* gate, int32_t* counts, unsigned long long* scores, const CombinePrev& prev,
                  StepTimeline* timeline, int32_t* seg_counts, int seg_tokens) {
  if (T <= kRouteSmallMax) {
    constexpr int W = 16;
    static bool attr_done = false;
    if (!attr_done) {  // the staged rows: up to 4 x 16 K elements
      cudaFuncSetAttribute(route_kernel<1, W, 4, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
      cudaFuncSetAttribute(route_kernel<2, W, 4, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
      cudaFuncSetAttribute(route_kernel<4, W, 2, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
      cudaGetLastError();
      attr_done = true;
    }
    auto smem = [&](int tt) { return ((((size_t)tt * E * sizeof(float)) + 15) & ~(size_t)15) + (size_t)tt * H * 2; };
    if (T <= 148)
      launch_pdl(route_kernel<1, W, 4, 4>, dim3(T), dim3(W * 32), smem(1), st, x, w_router, bias, conf, T, H, E, K,
                 logits, ids, gate, counts, scores, prev, timeline);
    else if (T <= 296)  // (four tokens per CTA measured slower at 256 tokens x 128 experts: 33 against 20 us)
      launch_pdl(route_kernel<2, W, 4, 4>, dim3((T + 1) / 2), dim3(W * 32), smem(2), st, x, w_router, bias, conf, T, H,
                 E, K, logits, ids, gate, counts, scores, prev, timeline);
    else
      launch_pdl(route_kernel<4, W, 2, 4>, dim3((T + 3) / 4), dim3(W * 32), smem(4), st, x, w_router, bias, conf, T, H,
                 E, K, logits, ids, gate, counts, scores, prev, timeline);
  } else {
    // (re-tilings of the plain kernel - more tokens or experts per warp, more warps per CTA, deeper
    // unrolling - were all slower at 4096 tokens x 64 experts x 4096)
    // tokens per CTA: the time is (waves of CTAs) x (tokens per CTA); ties go to the larger tile,
    // which reads the router matrix less often
    static int n_sms = 0;
    if (n_sms == 0) {
      int dev = 0;
      cudaGetDevice(&dev);
      cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev);
      if (n_sms <= 0) n_sms = 148;
    }
    int best_tt = 8;
    long best_cost = -1;
    for (int tt : {8, 10, 12, 14}) {
      const int ctas = (T + tt - 1) / tt;
      const long cost = (long)((ctas + n_sms - 1) / n_sms) * tt;
      if (best_cost < 0 || cost <= best_cost) {
        best_cost = cost;
        best_tt = tt;
      }
    }
    auto go = [&](auto kernel, int tt) {
      const size_t smem = (size_t)kManyStages * many_stage_bytes(tt) + (size_t)tt * E * sizeof(float);
      cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
      launch_pdl(kernel, dim3((T + tt - 1) / tt), dim3(kManyWarps * 32), smem, st, x, w_router, bias, conf, T, H, E,
                 K, logits, ids, gate, counts, scores, timeline, seg_counts, seg_tokens);
    };
    switch (best_tt) {
      case 8: go(route_many_kernel<8>, 8); break;
      case 10: go(route_many_kernel<10>, 10); break;
      case 12: go(route_many_kernel<12>, 12); break;
      default: go(route_many_kernel<14>, 14); break;
    }
  }
}

void launch_permute(cudaStream_t st, const int32_t* ids, const int32_t* counts, int T, int E, int K,
                    int32_t* offsets, int32_t* perm, int32_t* pos, const uint16_t* x, uint16_t* xp, int H,
                    StepTimeline* timeline, const TokenSplit* split, const int32_t* seg_counts, int seg_tokens) {
  const TokenSplit sp = xp != nullptr && split != nullptr && split->complete() ? *split : TokenSplit{};
  if (xp != nullptr) {
    // gathering steps: two rows per CTA and batch, eight CTAs per expert (see the kernel) - fewer where
    // eight per expert would not be resident at once (four CTAs fit an SM; 128 experts take four each:
    // 7.2 instead of 8.9 us at 256 tokens, two each 9.5 us)
    int per_expert = 8;
    while (per_expert > 1 && E * per_expert > 4 * 148) per_expert >>= 1;
    launch_pdl(permute_kernel<2>, dim3(E, per_expert), dim3(256), 0, st, ids, counts, T * K, E, offsets, perm, pos, x, xp,
               H, K, timeline, sp, (const int32_t*)nullptr, 0);
  }
  else
    launch_pdl(permute_kernel<8>, dim3(E, seg_counts != nullptr ? kPermuteSegments : 1), dim3(256), 0, st, ids, counts,
               T * K, E, offsets, perm, pos, x, xp, H, K, timeline, sp, seg_counts, seg_tokens);
}

namespace {
__global__ void __launch_bounds__(128) report_kernel(RouteReport rep) {
  griddep_launch_dependents();
  griddep_wait();
  publish_report(rep, (int)threadIdx.x, (int)blockDim.x);
}
}  // namespace
void launch_report(cudaStream_t st, const RouteReport& rep) {
  launch_pdl(report_kernel, dim3(1), dim3(128), 0, st, rep);
}

void launch_gather(cudaStream_t st, const uint16_t* x, const int32_t* perm, int T, int H, int K,
                   uint16_t* xp) {
  const size_t total = (size_t)T * K * (H / 8);
  const int blocks = (int)std::min<size_t>((total + 255) / 256, 148 * 16);
  launch_pdl(gather_kernel, dim3(blocks), dim3(256), 0, st, x, perm, T * K, H, K, xp);
}

}  // namespace oled

// ---------------------------------------------------------------------------------------
// Allocation-free routing entry point (no counterpart in the paper).
//
// Some hosts cannot let a library allocate: an inference server that hands every byte of
// device memory to its own arena at start-up, or a latency-critical decode loop in which the
// implicit device-wide synchronisation of cudaMalloc / cudaFree is not acceptable.  For them
// this entry point runs the gate, top-k, gate scores and the token->expert permutation of one
// step with its scratch (gate logits, inverse permutation, reuse-score accumulators) in a
// fixed array that is part of the loaded module, so nothing is allocated or freed.
namespace oled {
namespace {

constexpr size_t kNaScoreBytes = (size_t)OLED_MAX_EXPERTS * sizeof(unsigned long long);
constexpr size_t kNaPosBytes = (size_t)OLED_NOALLOC_MAX_TOKENS * OLED_MAX_TOPK * sizeof(int32_t);
constexpr size_t kNaLogitBytes = (size_t)OLED_NOALLOC_MAX_TOKENS * OLED_MAX_EXPERTS * sizeof(float);
constexpr size_t kNaScratchBytes = kNaScoreBytes + kNaPosBytes + kNaLogitBytes;

// Lives in every GPU that loads the library until the process exits (about 0.55 MB).
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNaScratchBytes];

constexpr int kNaMaxDevices = 64;
std::mutex g_na_mutex;
void* g_na_ptr[kNaMaxDevices] = {};

// In host code g_noalloc_scratch is only a handle for the symbol, not an address a kernel can
// use: the device address is looked up once per device, with that device current.
int noalloc_scratch_ptr(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNaMaxDevices) return OLED_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_na_mutex);
  if (g_na_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return OLED_ERR_CUDA;
    }
    g_na_ptr[dev] = p;
  }
  *out = static_cast<unsigned char*>(g_na_ptr[dev]);
  return OLED_OK;
}

}  // namespace
}  // namespace oled

extern "C" int oled_route_noalloc(const void* hidden, const void* w_router, const float* bias,
                                  const float* confidences, int32_t n_tokens, int32_t hidden_dim,
                                  int32_t n_experts, int32_t top_k, void* cuda_stream, int32_t* ids,
                                  float* gate, int32_t* counts, int32_t* offsets, int32_t* perm) {
  using namespace oled;
  if (n_tokens < 0 || hidden_dim <= 0 || hidden_dim % 256 != 0 || n_experts <= 0 ||
      n_experts > OLED_MAX_EXPERTS || top_k <= 0 || top_k > OLED_MAX_TOPK || top_k > n_experts ||
      !counts || !offsets)
    return OLED_ERR_INVALID_ARG;
  if (n_tokens > OLED_NOALLOC_MAX_TOKENS) return OLED_ERR_TOO_MANY_TOKENS;
  if (n_tokens > 0 && (!hidden || !w_router || !confidences || !ids || !gate || !perm))
    return OLED_ERR_INVALID_ARG;
  {  // rows and ids are accessed with 16-byte vectors, everything else as 32-bit words
    auto off = [](const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; };
    if (off(hidden, 16) || off(w_router, 16) || off(ids, 16) || off(bias, 4) || off(confidences, 4) ||
        off(gate, 4) || off(counts, 4) || off(offsets, 4) || off(perm, 4))
      return OLED_ERR_INVALID_ARG;
  }
  unsigned char* scratch = nullptr;
  const int rc = noalloc_scratch_ptr(&scratch);
  if (rc != OLED_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned long long* scores = reinterpret_cast<unsigned long long*>(scratch);
  int32_t* pos = reinterpret_cast<int32_t*>(scratch + kNaScoreBytes);
  float* logits = reinterpret_cast<float*>(scratch + kNaScoreBytes + kNaPosBytes);
  // the array keeps the previous call's contents: the accumulators must start at zero
  if (cudaMemsetAsync(scores, 0, (size_t)n_experts * sizeof(unsigned long long), st) != cudaSuccess ||
      cudaMemsetAsync(counts, 0, (size_t)n_experts * sizeof(int32_t), st) != cudaSuccess ||
      cudaMemsetAsync(offsets, 0, (size_t)(n_experts + 1) * sizeof(int32_t), st) != cudaSuccess) {
    cudaGetLastError();
    return OLED_ERR_CUDA;
  }
  if (n_tokens == 0) return OLED_OK;
  launch_route(st, static_cast<const uint16_t*>(hidden), static_cast<const uint16_t*>(w_router), bias,
               confidences, n_tokens, hidden_dim, n_experts, top_k, logits, ids, gate, counts, scores,
               CombinePrev{}, nullptr);
  launch_permute(st, ids, counts, n_tokens, n_experts, top_k, offsets, perm, pos, nullptr, nullptr, hidden_dim,
                 nullptr);
  return cudaGetLastError() == cudaSuccess ? OLED_OK : OLED_ERR_CUDA;
}
