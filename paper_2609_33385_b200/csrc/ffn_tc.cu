// Grouped SwiGLU expert FFN on the 5th-generation tensor cores (paper Sec. 4.1: experts that hit
// the cache run on the GPU at once; misses follow once their weights have landed).
//
// Two persistent kernels per expert group, both "weights on M, tokens on N":
//   KIND 1:  D_g[i,n] = sum_h Wg[i,h] x[n,h],  D_u likewise with Wu  (two TMEM accumulators),
//            epilogue  hbuf[n,i] = bf16( silu(D_g) * D_u )
//   KIND 2:  D[c,n]   = sum_i Wd[c,i] hbuf[n,i],  epilogue  y[n,c] = D   (fp32)
// The 128 rows of a weight tile fill the MMA's M dimension whatever the number of tokens an
// expert received, so that the few-tokens-per-expert regime of a denoising block streams each
// resident expert's weights exactly once at HBM speed, and the many-token regime uses N up to
// 256.  Weights are addressed through the expert->slot table: one 3-D tensor map covers the
// whole slot pool and the slot number is a TMA coordinate.
//
// KIND 1 has a second form for small token tiles (N <= 32), "stacked": 64 gate rows and the 64 up
// rows of the same intermediate features share ONE 128-row MMA tile (lanes 0-63 gate, 64-127 up),
// so an item is half as large and twice as many items exist - with ~4 tokens per expert the
// kernel is a weight stream, and finer items are what keeps all 148 SMs streaming to the end of
// the launch.  The up values cross to the gate rows' warps through shared memory.
//
// In the many-token regime (N tile 256) both kernels work on two 128-row weight tiles that share
// one token tile (gate+up, or two row blocks of Wd): 64 KB of operands per 128x2x256x64 MACs.
// (By default those steps run on CTA pairs instead, ffn_pair.cu; this form is what remains where
// the pair form does not apply - shapes, fp8 stores - or is switched off.)
//
// Work items (expert, token tile, weight tile) are drawn from a global counter by each CTA's
// producer and handed to its other roles through a ring in shared memory (see take_item); a
// pipeline stage holds one k-block of 64, or two for small token tiles; KIND 2 starts its weight
// stream before its predecessor KIND 1 has finished (see the set-up in the kernel).
//
// Warp roles (704 threads): warps 0-15 epilogue (TMEM lane quarter = warp id mod 4, the warps of
// a quarter interleave 16-column chunks; only as many as the token tile has chunks are active),
// warp 16 lane 0 TMA producer, warp 17 lane 0 MMA issuer (warp 17 also owns the TMEM allocation),
// warps 18-21 widen fp8 weight tiles (fp8 expert stores only, idle otherwise).
//
// fp8 expert stores (e4m3 codes + one fp32 scale per weight row), token tiles of 64 and 128 rows
// (FP8 = 1, "widening"): a pipeline stage is a load
// slot in shared memory - the code tile of a k-block (64 bytes per weight row, half the bytes in
// flight of the bf16 form) next to its token tile - plus 32 (64) columns of TENSOR memory.
// Groups of four converter warps, one per TMEM lane quarter, read the codes, widen them to bf16
// (exact) and write them with tcgen05.st as the MMA's A operand: lane = weight row, two
// consecutive k per 32-bit column.  The MMA takes the weights from tensor memory and the tokens
// from the slot, runs in bf16 as before, and its completion frees the stage; the widened weights
// never touch shared memory.  The accumulators keep their place in front of the weight stages,
// which is why the fp8 form stops at token tiles of 128.  The epilogue multiplies each output
// row by its scale - the rows of a weight tile are the accumulator's lanes.
//
// fp8 expert stores, token tiles of at most 32 rows (FP8 = 2, "direct"): the widening form above
// is bound by the thread that issues the MMAs - an M = 128 instruction consumes 128 weight rows x
// 16 k whatever the element size, so half the bytes are not half the instructions.  Here the
// MMAs are kind::f8f6f4 (K = 32 per instruction) and read the e4m3 code tile as the TMA laid it
// down: a k-block is 128 rows x 128 k, the same 16 KB and the same four instructions as a bf16
// k-block of 64.  An MMA takes both operands in the same 8-bit kind, so the token rows enter as
// e4m3 too: every row, scaled by a power of two that brings its largest magnitude into
// [128, 256), is the sum of two e4m3 terms (fp8_split.h; exact for every element within 2^-14 of
// the row's maximum, which is as exact as bf16 tokens get next to an fp32 accumulator).  The
// terms are made once per step and operand - by the gathering permutation kernel for the input
// rows, by split_rows_kernel between the two projections for the intermediate rows, whose
// largest magnitudes the gate/up epilogue collects with atomicMax - and loaded as the B tile
// [term 1 rows | term 2 rows], N = 2 n_box; the epilogue adds the two accumulators (D1 + D2/16)
// and undoes the row's scale.  No converter warps and no proxy fences in the streaming loop:
// a form that split the tokens inside the kernel was bound by the fence between the converters'
// shared-memory writes and the MMA's reads (one per stage, each waiting for the copies in flight).
// The TMA thread issues one copy for the code tile (a 4-D map whose box takes the 64 gate and
// the 64 up rows at once) and one for both term tiles per k-block.
//
// Every mbarrier wait is bounded: on a timeout the CTA raises a flag in the status word, gives
// in-flight copies time to land, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include <algorithm>
#include <cstddef>
#include <cstdlib>

#include "fp8_split.h"
#include "kernels.h"
#include "sm100_ptx.h"

namespace oled {
namespace {

#ifndef OLED_EPI_WARPS
#define OLED_EPI_WARPS 16
#endif
#ifndef OLED_NAP_EPI  // nanoseconds between polls, fp8 form: epilogue, TMA producers, converters
#define OLED_NAP_EPI 128
#endif
#ifndef OLED_NAP_LOAD
#define OLED_NAP_LOAD 64
#endif
#ifndef OLED_NAP_CONV
#define OLED_NAP_CONV 32
#endif
constexpr int kEpiWarps = OLED_EPI_WARPS;  // up to four warps per TMEM lane quarter, interleaving 16-column chunks
constexpr int kProducerWarp = kEpiWarps;
constexpr int kMmaWarp = kEpiWarps + 1;
constexpr int kConvWarp0 = kEpiWarps + 2;     // four warps that widen fp8 weight tiles to bf16 (fp8 stores only)
constexpr int kThreads = (kEpiWarps + 6) * 32;
constexpr int kBlockM = 128;
constexpr int kBlockK = 64;   // one 128-byte swizzle atom of bf16
constexpr uint32_t kATile = kBlockM * kBlockK * 2;
constexpr int kMaxStages = 12;
constexpr int kItemRing = 8;  // items the producer may publish ahead of the slowest consumer
constexpr uint32_t kSmemMax = 232448;  // 227 KB

struct __align__(16) SharedCtl {
  unsigned long long full[kMaxStages];
  unsigned long long empty[kMaxStages];
  unsigned long long slot_full[kMaxStages];  // fp8 stores: the stage's code tile and token tile have landed
  unsigned long long item_full[kItemRing];   // the producer published the CTA's next item
  unsigned long long item_empty[kItemRing];  // every consumer role has read it
  unsigned long long tmem_full[2];
  unsigned long long tmem_empty[2];
  unsigned long long x_full[2][2];   // stacked gate/up mode: [buffer][chunk group], up rows -> gate rows
  unsigned long long x_empty[2][2];
  uint32_t tmem_base;
  int abort;
  int n_tiles_total;
  int pad;
  int item_ring[kItemRing];  // item numbers handed out by the producer; -1 = no more work
  int tile_prefix[OLED_MAX_EXPERTS + 1];
  int row_start[OLED_MAX_EXPERTS];
  int count[OLED_MAX_EXPERTS];
  // [buffer][chunk group][row][column]: up values of one 16-column chunk; read and written with
  // 16-byte vector accesses, hence the alignment
  __align__(16) float xchg[2][2][64][16];
};
static_assert(offsetof(SharedCtl, xchg) % 16 == 0, "xchg must be 16-byte aligned");
constexpr uint32_t kCtlBytes = (sizeof(SharedCtl) + 1023u) & ~1023u;

struct Item {
  int slot, m0, row0, valid;
  int kind;  // 1: gate/up (+SwiGLU), 2: down projection
  int g;     // index of the expert in the launch's group
};
// The second half of a FUSED launch's work list (KIND 3): items [n1, n1 + n2) are the down-
// projection items of the same experts and token tiles as the gate/up items [0, n1).
struct SecondPhase {
  int n1;            // number of first-phase items (INT_MAX: no second phase)
  int m_tiles, m_rows;
};
// A role's position in the expert list: items arrive in ascending order within a phase, so the
// search for an item's expert only moves forward; it restarts with the second phase.
struct ItemCursor {
  int g = 0;
  int phase2 = 0;
};
// Items (expert, token tile, weight tile) are handed out DYNAMICALLY: after its first item (its own
// CTA number) the producer thread of a CTA draws item numbers from a counter in global memory
// (one atomic per item, fetched one item ahead) and publishes them to the other roles of its CTA through a small ring in shared
// memory.  SMs that stream faster take more items, so the launch ends when the work does, not
// when the slowest SM has finished a fixed share.  Which CTA computes an item does not change
// its arithmetic.
// Consumer side: the seq-th item of this CTA, -1 when there is no more work, -2 on an abort.
__device__ __forceinline__ int take_item(SharedCtl* ctl, int seq, volatile int* abort_flag, uint32_t* status,
                                         uint32_t nap) {
  const int slot = seq % kItemRing;
  const uint32_t ph = (uint32_t)(seq / kItemRing) & 1u;
  if (!mbar_wait(smem_u32(&ctl->item_full[slot]), ph, abort_flag, status, nap)) return -2;
  const int item = *reinterpret_cast<volatile int*>(&ctl->item_ring[slot]);
  mbar_arrive(smem_u32(&ctl->item_empty[slot]));
  return item;
}
__device__ __forceinline__ void decode_item(const SharedCtl* ctl, const FfnGroup& grp, int item, int kind1, int m_tiles,
                                            int m_rows, int n_box, const SecondPhase& second, ItemCursor& cur,
                                            Item& it) {
  it.kind = kind1;
  if (item >= second.n1) {
    item -= second.n1;
    m_tiles = second.m_tiles;
    m_rows = second.m_rows;
    it.kind = 2;
    if (!cur.phase2) {
      cur.phase2 = 1;
      cur.g = 0;
    }
  }
  const int q = item / m_tiles;
  const int m = item - q * m_tiles;
  int g = cur.g;
  while (ctl->tile_prefix[g + 1] <= q) ++g;
  cur.g = g;
  const int nt = q - ctl->tile_prefix[g];
  it.g = g;
  it.slot = grp.slot[g];
  it.m0 = m * m_rows;
  it.row0 = ctl->row_start[g] + nt * n_box;
  it.valid = min(n_box, ctl->count[g] - nt * n_box);
}

// What a FUSED launch (KIND 3) needs on top: the down projection's tensor maps, its output and
// the completion counters.
struct FusedSecond {
  CUtensorMap tm_w2;    // down-projection weights
  CUtensorMap tm_act2;  // intermediate rows (hbuf)
  void* out2;           // y
  uint32_t* done;       // per expert of the group: epilogue warps that have stored gate/up rows; ZERO at start
};

// DUAL: two accumulators per item - gate and up (KIND 1, always), or two row blocks of Wd
// (KIND 2 with the 256-token tile).
// FP8: the slot pool holds fp8 expert blobs (tm_w is a byte map over the e4m3 codes).
// KIND 3 (bf16 stores, token tiles of at most 32 rows): the gate/up items in their stacked form,
// then the down-projection items of the same experts, in ONE launch.  A down item reads the
// intermediate rows that the gate/up items of its expert wrote, so its producer waits (bounded)
// until the expert's counter in `done` shows that all of them have been stored; items are handed
// out in order, gate/up first, so that wait is over long before it is reached except in launches
// with few items per SM - which is where this form pays: the two-kernel form leaves every SM that
// runs out of gate/up items idle until the last gate/up item of the whole launch is done, this
// one lets it go on with the down projection of experts that are already complete.
template <int KIND, bool DUAL, int FP8>
__global__ void __launch_bounds__(kThreads, 1)
ffn_tc_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_act,
              const __grid_constant__ FfnGroup grp, const int32_t* __restrict__ offsets,
              void* __restrict__ out_ptr, int H, int I, int n_stages, int k_atoms, int early_start, int out_bf16,
              const uint8_t* __restrict__ pool, unsigned long long slot_bytes,
              uint32_t* __restrict__ status, uint32_t* __restrict__ work_counter, StepTimeline* timeline,
              int timeline_slot, const __grid_constant__ RouteReport report,
              const __grid_constant__ FusedSecond fs, const uint32_t* __restrict__ amax_in,
              uint32_t* __restrict__ amax_out) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem_raw);
  const uint32_t tiles_base = (smem_u32(smem_raw) + kCtlBytes + 1023u) & ~1023u;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_box = grp.n_box;
  constexpr bool fused = KIND == 3;
  static_assert(!(fused && (DUAL || FP8)), "the fused form exists for bf16 stores and single tiles only");
  constexpr bool WIDEN = FP8 == 1;   // fp8 stores, codes widened to bf16 by converter warps
  constexpr bool DIRECT = FP8 == 2;  // fp8 stores, codes read by the MMA as they are (see the header comment)
  static_assert(!(DIRECT && DUAL), "the direct fp8 form exists for single 128-row tiles only");
  constexpr int kK = DIRECT ? 128 : kBlockK;  // k-values of a k-block (one 128-byte swizzle atom of weights)
  constexpr int kind1 = fused ? 1 : KIND;  // kind of the launch's first-phase (or only) items
  constexpr bool dual = DUAL;
  constexpr bool stacked = (KIND == 1 && !DUAL) || fused;  // gate/up items: 64 gate + 64 up rows in one 128-row tile
  constexpr uint32_t a_bytes = (dual ? 2u : 1u) * kATile;
  const uint32_t b_bytes = (uint32_t)n_box * 128u;
  // bf16 stores: a stage (shared memory) holds the weight tile(s) and the token tile of a k-block.
  // fp8 stores: a stage is a load slot in shared memory - the code tile (one byte per element)
  // followed by the token tile - plus a_cols columns of TENSOR memory, behind the accumulators,
  // for the widened weights.
  // A stage spans k_atoms (1 or 2) k-blocks of 64, laid out one after the other, each as
  // described above: small token tiles take two, which halves the waits and commits per byte on
  // the serial path of the MMA thread.
  // direct fp8 form: a stage is the code tile of a k-block of 128 (16 KB) and the two e4m3 term
  // tiles of the tokens (2 n_box rows of 128 bytes, term 2 behind term 1) - the MMA's B operand.
  constexpr uint32_t raw_bytes = WIDEN ? a_bytes / 2 : 0u;
  const uint32_t atom_bytes = DIRECT ? kATile + 2u * b_bytes
                              : WIDEN ? raw_bytes + b_bytes : a_bytes + b_bytes;  // one k-block in shared memory
  const uint32_t stage_bytes = (uint32_t)k_atoms * atom_bytes;
  constexpr uint32_t atom_cols = dual ? 64u : 32u;  // 64 k-values of one (two) 128-row tile(s), two per column
  const uint32_t a_cols = (uint32_t)k_atoms * atom_cols;
  const int k_blocks1 = (kind1 == 1 ? H : I) / (kK * k_atoms);  // stages per (first-phase) item
  const int k_blocks2 = I / (kK * k_atoms);                    // stages per down item of a fused launch
  constexpr int m_rows = (KIND == 2 && dual) ? 2 * kBlockM : stacked ? kBlockM / 2 : kBlockM;  // output features per item
  const int m_tiles = (kind1 == 1 ? I : H) / m_rows;
  const int acc_cols = (dual || DIRECT ? 2 : 1) * n_box;  // (direct fp8 form: one accumulator per token term)
  const int a_total = WIDEN ? n_stages * (int)a_cols : 0;
  const int acc_stages = (2 * acc_cols + a_total <= 512) ? 2 : 1;
  const uint32_t a_col0 = (uint32_t)(acc_stages * acc_cols);  // first column of the weight stages
  // warps that can own a 16-column chunk; the SwiGLU epilogue (KIND 1) profits from all 16, the
  // plain store epilogue of KIND 2 runs best with 8
  const int epi_warps = min((KIND != 2 || out_bf16) ? kEpiWarps : 8, 4 * (n_box / 16));
  // fp8 stores: the four dedicated converter warps plus epilogue warps this token tile leaves
  // idle form conv_groups (at most two: more of them take issue slots from the MMA thread and
  // measured slower) groups of four warps, one warp per TMEM lane quarter.
  // Group g owns the k-blocks i with i mod conv_groups == g; conv_groups divides both ring
  // depths, so every load slot and every weight stage belongs to ONE group, which visits the
  // rounds of its barriers in order - a parity wait can then never take an older phase for the
  // one it wants.
  int conv_groups = WIDEN ? 1 + (kEpiWarps - epi_warps) / 4 : 0;
  if (conv_groups > 2) conv_groups = 2;
  if (conv_groups > 1 && n_stages % conv_groups != 0) conv_groups = 1;
  const int conv_group = !WIDEN ? -1
                         : (warp >= kConvWarp0 && warp < kConvWarp0 + 4) ? 0
                         : (warp >= epi_warps && warp < kEpiWarps) ? 1 + (warp - epi_warps) / 4 : -1;
  const bool is_conv = WIDEN && conv_group >= 0 && conv_group < conv_groups;
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < acc_stages * acc_cols + a_total) tmem_cols <<= 1;

  // ---- set-up that depends on no earlier kernel: barriers, TMEM (overlaps the predecessor's tail)
  griddep_launch_dependents();
  if (threadIdx.x == 0) {
    timeline_entry(timeline, timeline_slot);
    for (int s = 0; s < kMaxStages; ++s) {
      // the stage's TMA transaction, or every lane of the four converting warps
      mbar_init(smem_u32(&ctl->full[s]), WIDEN ? 128u : 1u);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int s = 0; s < kMaxStages; ++s) mbar_init(smem_u32(&ctl->slot_full[s]), 1);
    for (int s = 0; s < kItemRing; ++s) {
      mbar_init(smem_u32(&ctl->item_full[s]), 1);
      // consumers: the MMA thread, one lane of every epilogue warp and of every converter warp
      mbar_init(smem_u32(&ctl->item_empty[s]), 1u + (uint32_t)epi_warps + (WIDEN ? 4u * (uint32_t)conv_groups : 0u));
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&ctl->tmem_full[a]), 1);
      mbar_init(smem_u32(&ctl->tmem_empty[a]), (uint32_t)epi_warps * 32u);
      for (int hgrp = 0; hgrp < 2; ++hgrp) {
        mbar_init(smem_u32(&ctl->x_full[a][hgrp]), 64);
        mbar_init(smem_u32(&ctl->x_empty[a][hgrp]), 64);
      }
    }
    ctl->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == kProducerWarp && lane == 0) {  // the two tensor maps, ahead of the first copy
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_act)) : "memory");
    if (fused) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&fs.tm_w2)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&fs.tm_act2)) : "memory");
    }
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&ctl->tmem_base)),
                 "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // ---- from here on the step's earlier kernels must have completed: work table from offsets.
  // KIND 1 follows the permutation, whose products it reads from the first instruction on.  KIND 2
  // follows KIND 1 of the same expert group: the offsets and the expert weights are older than
  // that kernel, only the token tiles (hbuf) are its product - so a KIND 2 CTA, which gets its SM
  // when a KIND 1 CTA leaves it, sets up and streams its first weight tiles while the slower SMs
  // still finish KIND 1; its producer waits for the predecessor before the first token-tile load.
  // (early_start is set by the host only where that is safe: see launch_ffn_tc and launch_variant)
  const bool early = KIND == 2 && early_start != 0;
  if (!early) griddep_wait();
  if (threadIdx.x == 0) timeline_start(timeline, timeline_slot);
  for (int g = threadIdx.x; g < grp.n; g += kThreads) {
    const int e = grp.expert[g];
    const int s = offsets[e];
    ctl->row_start[g] = s;
    ctl->count[g] = offsets[e + 1] - s;
  }
  __syncthreads();
  if (warp == 0) {  // exclusive scan of the experts' token-tile counts, 32 experts at a time
    int carry = 0;
    for (int g0 = 0; g0 < grp.n; g0 += 32) {
      const int g = g0 + lane;
      const int tiles = g < grp.n ? (ctl->count[g] + n_box - 1) / n_box : 0;
      int incl = tiles;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += o;
      }
      if (g < grp.n) ctl->tile_prefix[g] = carry + incl - tiles;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) {
      ctl->tile_prefix[grp.n] = carry;
      ctl->n_tiles_total = carry;
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  // polling back-off of the fp8 form, by role (the MMA thread never sleeps)
  constexpr uint32_t nap_epi = WIDEN ? OLED_NAP_EPI : 0u, nap_load = WIDEN ? OLED_NAP_LOAD : 0u,
                     nap_conv = WIDEN ? OLED_NAP_CONV : 0u;
  const uint32_t tmem_base = ctl->tmem_base;
  SecondPhase second;
  second.n1 = fused ? ctl->n_tiles_total * m_tiles : 0x7fffffff;
  second.m_rows = kBlockM;
  second.m_tiles = H / kBlockM;
  const int total_items = ctl->n_tiles_total * m_tiles + (fused ? ctl->n_tiles_total * second.m_tiles : 0);
  // KIND 3: epilogue warps that store intermediate rows per gate/up item, times the items of one token tile
  const uint32_t done_per_tile = (uint32_t)(m_tiles * (epi_warps / 2));
  volatile int* abort_flag = &ctl->abort;

  if (KIND != 2 && blockIdx.x == 0 && warp == kProducerWarp && lane != 0) {
    // the step's report to the host (see RouteReport): sent by lanes that have nothing else to do;
    // its trip across the host link ends long before this kernel does
    publish_report(report, lane - 1, 31);
  }
  if (warp == kProducerWarp && lane == 0) {
    // ------------------------------------------------------------ TMA producer
    // bf16 stores: weight rows and token tile of a k-block go to one operand stage; fp8 stores:
    // code rows and token tile go to one load slot
    int stage = 0, ready_g = -1;
    ItemCursor cur;
    uint32_t phase = 0;
    bool ok = true;
    const int ring = n_stages;
    // (with loads withheld - the test of the bounded waits - nothing is published either)
    // the CTA's first item is its own number (no round trip to the counter before the first
    // load); every later one is drawn from the counter, which hands out numbers from gridDim.x on
    int item = (int)blockIdx.x;
    for (int seq = 0; ok && !grp.withhold_loads; ++seq) {
      const bool none = item >= total_items;
      // the next item's number is fetched now: the atomic's latency lies under this item's loads
      const int next = none ? item : (int)(atomicAdd(work_counter, 1u) + gridDim.x);
      const int ring_slot = seq % kItemRing;
      if (!mbar_wait(smem_u32(&ctl->item_empty[ring_slot]), ((uint32_t)(seq / kItemRing) & 1u) ^ 1u, abort_flag, status,
                     nap_load)) {
        ok = false;
        break;
      }
      *reinterpret_cast<volatile int*>(&ctl->item_ring[ring_slot]) = none ? -1 : item;
      mbar_arrive(smem_u32(&ctl->item_full[ring_slot]));
      if (none) break;
      Item it;
      decode_item(ctl, grp, item, kind1, m_tiles, m_rows, n_box, second, cur, it);
      item = next;
      const bool down_of_fused = fused && it.kind == 2;
      const CUtensorMap* map_w = down_of_fused ? &fs.tm_w2 : &tm_w;
      const CUtensorMap* map_act = down_of_fused ? &fs.tm_act2 : &tm_act;
      const int k_blocks = down_of_fused ? k_blocks2 : k_blocks1;
      constexpr uint32_t w_tile = WIDEN ? kATile / 2 : kATile;  // bytes of 128 weight rows of a k-block
      auto load_weights = [&](int st, int kb) {
        const uint32_t bar = smem_u32(WIDEN ? &ctl->slot_full[st] : &ctl->full[st]);
        mbar_expect_tx(bar, stage_bytes);
        for (int atom = 0; atom < k_atoms; ++atom) {
          const uint32_t w_addr = tiles_base + (uint32_t)st * stage_bytes + (uint32_t)atom * atom_bytes;
          const int k0 = (kb * k_atoms + atom) * kK;
          if (DIRECT && stacked && it.kind == 1) {
            // one copy: the map is over [slot][gate | up][row][k], the box takes 64 rows of either
            // half (the copy instructions are the serial cost of this thread, see rings_for)
            tma_load_4d(map_w, w_addr, bar, k0, it.m0, 0, it.slot);
          } else if (stacked && it.kind == 1) {  // the map has 64-row boxes here
            tma_load_3d(map_w, w_addr, bar, k0, it.m0, it.slot);                  // 64 gate rows
            tma_load_3d(map_w, w_addr + w_tile / 2, bar, k0, I + it.m0, it.slot);  // 64 up rows
          } else if (it.kind == 1) {
            tma_load_3d(map_w, w_addr, bar, k0, it.m0, it.slot);               // gate rows
            tma_load_3d(map_w, w_addr + w_tile, bar, k0, I + it.m0, it.slot);  // up rows
          } else {
            tma_load_3d(map_w, w_addr, bar, k0, it.m0, it.slot);               // down rows
            if (dual) tma_load_3d(map_w, w_addr + w_tile, bar, k0, it.m0 + kBlockM, it.slot);
          }
        }
      };
      auto load_tokens = [&](int st, int kb) {
        const uint32_t bar = smem_u32(WIDEN ? &ctl->slot_full[st] : &ctl->full[st]);
        for (int atom = 0; atom < k_atoms; ++atom) {
          const uint32_t t_addr =
              tiles_base + (uint32_t)st * stage_bytes + (uint32_t)atom * atom_bytes + (WIDEN ? raw_bytes : a_bytes);
          const int k0 = (kb * k_atoms + atom) * kK;
          if (DIRECT) {  // (the map is over [term][row][k], the box takes both terms)
            tma_load_3d(map_act, t_addr, bar, k0, it.row0, 0);
          } else {
            tma_load_2d(map_act, t_addr, bar, k0, it.row0);
          }
        }
      };
      int kb = 0;
      if (early && seq == 0) {
        // the CTA's first stages (all free): weights now, token tiles once the predecessor is done
        const int pre = min(n_stages, k_blocks);
        for (int i = 0; i < pre; ++i) load_weights(i, i);
        griddep_wait();
        for (int i = 0; i < pre; ++i) load_tokens(i, i);
        kb = pre;
        if (pre == n_stages) phase ^= 1u;
        else stage = pre;
      }
      if (down_of_fused) {
        // The intermediate rows of every token tile of this expert must be in memory.  If they are
        // not yet (launches with few items per SM), the weights of as many stages as the ring
        // holds go first, then the wait, then those stages' token tiles.
        const uint32_t* flag = fs.done + it.g;
        const uint32_t target = done_per_tile * (uint32_t)(ctl->tile_prefix[it.g + 1] - ctl->tile_prefix[it.g]);
        uint32_t seen = target;  // (an expert seen complete stays complete: no second look)
        if (it.g != ready_g) asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(flag) : "memory");
        int pre = 0;
        const int stage0 = stage;
        if (seen < target) {
          pre = min(n_stages, k_blocks);
          for (int i = 0; i < pre && ok; ++i) {
            if (!mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag, status, nap_load)) {
              ok = false;
              break;
            }
            load_weights(stage, i);
            if (++stage == ring) {
              stage = 0;
              phase ^= 1u;
            }
          }
          unsigned long long t0 = 0;
          for (uint32_t spin = 0; ok; ++spin) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(flag) : "memory");
            if (seen >= target) break;
            if ((spin & 255u) == 255u) {
              if (*abort_flag) ok = false;
              const unsigned long long now = globaltimer();
              if (t0 == 0) t0 = now;
              if (now - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                atomicExch(status, (uint32_t)kStatusWaitTimeout);
                ok = false;
              }
            }
          }
          if (!ok) break;
        }
        ready_g = it.g;
        // the rows were written through the generic proxy; the loads below read through the async proxy
        asm volatile("fence.proxy.async;" ::: "memory");
        if (pre > 0) {
          int st = stage0;
          for (int i = 0; i < pre; ++i) {
            load_tokens(st, i);
            if (++st == ring) st = 0;
          }
          kb = pre;
        }
      }
      for (; kb < k_blocks; ++kb) {
        if (!mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag, status, nap_load)) {
          ok = false;
          break;
        }
        load_weights(stage, kb);
        load_tokens(stage, kb);
        if (++stage == ring) {
          stage = 0;
          phase ^= 1u;
        }
      }
    }
    if (!ok) {  // let copies already issued land before the CTA's shared memory is released
      const unsigned long long t0 = globaltimer();
      while (globaltimer() - t0 < 2000000ull) {
      }
    }
  } else if (warp == kMmaWarp && lane == 0) {
    // ------------------------------------------------------------ MMA issuer
    int stage = 0, local = 0;
    ItemCursor cur;
    uint32_t phase = 0;
    bool ok = true;
    // Descriptor words of stage 0 (K-major, 128-byte swizzle, 8-row groups 1024 bytes apart); the
    // low word holds the address in 16-byte units, the high word is the same for every operand.
    const uint32_t desc_hi = (uint32_t)(make_smem_desc(0) >> 32);
    const uint32_t ring_step = atom_bytes >> 4;  // one k-block further in shared memory
    const uint32_t a_lo0 = (uint32_t)make_smem_desc(tiles_base);
    const uint32_t b_lo0 = (uint32_t)make_smem_desc(tiles_base + (WIDEN ? raw_bytes : a_bytes));
    const uint32_t a_tmem0 = tmem_base + a_col0;  // fp8 stores: weights come from tensor memory
    const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
    uint32_t a_lo = a_lo0, b_lo = b_lo0, a_tmem = a_tmem0;
    for (; ok; ++local) {
      const int item = take_item(ctl, local, abort_flag, status, 0u);
      if (item < 0) break;
      Item it;
      decode_item(ctl, grp, item, kind1, m_tiles, m_rows, n_box, second, cur, it);
      const int k_blocks = (fused && it.kind == 2) ? k_blocks2 : k_blocks1;
      const int acc = local % acc_stages;
      const uint32_t acc_phase = (uint32_t)(local / acc_stages) & 1u;
      if (!mbar_wait(smem_u32(&ctl->tmem_empty[acc]), acc_phase ^ 1u, abort_flag, status)) break;
      tc_fence_after();
      const int n_mma = max(16, (it.valid + 15) & ~15);
      const uint32_t idesc = DIRECT ? make_idesc_e4m3(2 * n_box) : make_idesc(n_mma);
      const uint32_t d0 = tmem_base + (uint32_t)(acc * acc_cols);
      for (int kb = 0; kb < k_blocks; ++kb) {
        // (fp8 stores: the converters arrive on full[] only after the stage's slot has landed)
        if (!mbar_wait(full0 + (uint32_t)stage * 8u, phase, abort_flag, status)) {
          ok = false;
          break;
        }
        tc_fence_after();
        for (int atom = 0; atom < k_atoms; ++atom) {
          const uint32_t first = (kb | atom) != 0 ? 1u : 0u;
#pragma unroll
          for (int k = 0; k < kBlockK / 16; ++k) {  // 32 bytes along K = 2 address units
            const uint32_t accum = k != 0 ? 1u : first;
            if (DIRECT) {
              tc_mma_e4m3_lo(d0, a_lo + k * 2, b_lo + k * 2, desc_hi, idesc, accum);
            } else if (WIDEN) {
              tc_mma_ts_lo(d0, a_tmem + k * 8, b_lo + k * 2, desc_hi, idesc, accum);
              if (dual) tc_mma_ts_lo(d0 + (uint32_t)n_box, a_tmem + 32 + k * 8, b_lo + k * 2, desc_hi, idesc, accum);
            } else {
              tc_mma_lo(d0, a_lo + k * 2, b_lo + k * 2, desc_hi, idesc, accum);
              if (dual)
                tc_mma_lo(d0 + (uint32_t)n_box, a_lo + (kATile >> 4) + k * 2, b_lo + k * 2, desc_hi, idesc, accum);
            }
          }
          a_lo += ring_step;
          b_lo += ring_step;
          a_tmem += atom_cols;
        }
        tc_commit(empty0 + (uint32_t)stage * 8u);
        if (++stage == n_stages) {
          stage = 0;
          phase ^= 1u;
          a_lo = a_lo0;
          b_lo = b_lo0;
          a_tmem = a_tmem0;
        }
      }
      if (ok) tc_commit(smem_u32(&ctl->tmem_full[acc]));
    }
  } else if (is_conv) {
    // ------------------------------------------------------------ fp8 -> bf16 converters
    // The four warps of a group widen the code tile of one load slot into the weight stage (tensor
    // memory) of the same k-block, several groups (k-blocks) at a time.  A warp can write only
    // the TMEM lanes of its quarter (warp id mod 4): lane l of the warp owns weight row
    // 32 * quarter + l, reads its 64 codes (the TMA laid the 64-byte rows out with the 64-byte
    // swizzle, so that the 32 rows of a quarter spread over all banks), widens them and stores
    // 32 columns of packed bf16 pairs with one tcgen05.st.
    const int group = conv_group, quarter = warp & 3;
    const uint32_t row = (uint32_t)(quarter * 32 + lane);
    const uint32_t sw = (row >> 1) & 3u;  // SWIZZLE_64B: 16-byte chunk index xor address bits 7-8
    const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16) + a_col0;
    // The CTA's k-blocks form one sequence across its items; this group takes every
    // conv_groups-th of them (conv_groups divides the ring depth, so the group always meets the
    // same stages).  `mine`: the group's next k-block, counted from the current item's first.
    int stage = group, mine = group;
    uint32_t phase = 0;
    bool live = true;
    const int k_blocks = k_blocks1;
    for (int seq = 0; live; ++seq) {
      int item = 0;
      if (lane == 0) item = take_item(ctl, seq, abort_flag, status, nap_conv);
      item = __shfl_sync(0xffffffffu, item, 0);
      if (item < 0) break;  // (the converters need the item's length only: every item has k_blocks k-blocks)
      for (; mine < k_blocks; mine += conv_groups) {
        int ok = 0;
        if (lane == 0)
          ok = (mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag, status, nap_conv) &&
                mbar_wait(smem_u32(&ctl->slot_full[stage]), phase, abort_flag, status, nap_conv))
                   ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) {
          live = false;
          break;
        }
        __syncwarp();
        tc_fence_after();  // the stage was released by the completion of the MMAs that read it
        for (int atom = 0; atom < k_atoms; ++atom) {
          const uint32_t src = tiles_base + (uint32_t)stage * stage_bytes + (uint32_t)atom * atom_bytes + row * 64u;
#pragma unroll
          for (int tile = 0; tile < (dual ? 2 : 1); ++tile) {
            uint4 c[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
              c[j] = lds128(src + (uint32_t)tile * (kATile / 2) + (((uint32_t)j ^ sw) << 4));
            uint32_t r[32];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              e4m3x4_to_bf16x4(c[j].x, r[8 * j], r[8 * j + 1]);
              e4m3x4_to_bf16x4(c[j].y, r[8 * j + 2], r[8 * j + 3]);
              e4m3x4_to_bf16x4(c[j].z, r[8 * j + 4], r[8 * j + 5]);
              e4m3x4_to_bf16x4(c[j].w, r[8 * j + 6], r[8 * j + 7]);
            }
            tmem_st32(t_lane + (uint32_t)stage * a_cols + (uint32_t)atom * atom_cols + (uint32_t)tile * 32u, r);
          }
        }
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(smem_u32(&ctl->full[stage]));  // (the slot itself is released by the MMAs' completion)
        if ((stage += conv_groups) >= n_stages) {
          stage -= n_stages;
          phase ^= 1u;
        }
      }
      mine -= k_blocks;
    }
  } else if (warp < epi_warps) {
    // ------------------------------------------------------------ epilogue
    // (only as many warps per quarter as the token tile has 16-column chunks)
    int local = 0;
    ItemCursor cur;
    uint32_t xn = 0;  // stacked mode: 16-column chunks this warp's chunk group has exchanged so far
    bool alive = true;
    for (; alive; ++local) {
      int item = 0;
      if (lane == 0) item = take_item(ctl, local, abort_flag, status, nap_epi);
      item = __shfl_sync(0xffffffffu, item, 0);
      if (item < 0) break;
      Item it;
      decode_item(ctl, grp, item, kind1, m_tiles, m_rows, n_box, second, cur, it);
      const bool gate_up_item = it.kind == 1;  // (always true for KIND 1, never for KIND 2)
      const int acc = local % acc_stages;
      const uint32_t acc_phase = (uint32_t)(local / acc_stages) & 1u;
      // one lane polls (keeps issue slots free for the producer and MMA threads); the outcome is
      // warp-uniform because tcgen05.ld below is warp-collective
      int ready = 0;
      if (lane == 0) ready = mbar_wait(smem_u32(&ctl->tmem_full[acc]), acc_phase, abort_flag, status, nap_epi) ? 1 : 0;
      ready = __shfl_sync(0xffffffffu, ready, 0);
      if (!ready) break;
      tc_fence_after();
      const int quarter = warp & 3, half = warp >> 2;  // `half`: which 16-column chunks this warp takes
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * acc_cols);
      const int n_mma = max(16, (it.valid + 15) & ~15);
      const int col = it.m0 + quarter * 32 + lane;  // output feature owned by this thread
      // fp8 stores: one fp32 scale per weight row behind the codes: s_gate[I] | s_up[I] | s_down[H]
      const float* sc = FP8 ? reinterpret_cast<const float*>(pool + (size_t)it.slot * slot_bytes + (size_t)3 * H * I)
                            : nullptr;
      float s0 = 1.0f, s1 = 1.0f;
      if (FP8) {
        if (stacked) {
          const int f = it.m0 + (quarter & 1) * 32 + lane;
          s0 = quarter >= 2 ? sc[I + f] : sc[f];  // this thread's row: an up row or a gate row
        } else if (KIND == 1) {
          s0 = sc[col];
          s1 = sc[I + col];
        } else {
          s0 = sc[2 * I + col];
          if (dual) s1 = sc[2 * I + col + kBlockM];
        }
      }
      for (int c = half * 16; c < n_mma; c += 16 * (epi_warps / 4 > 0 ? epi_warps / 4 : 1)) {
        uint32_t ra[16];
        tmem_ld16(t_row + (uint32_t)c, ra);
        if (DIRECT) {
          // the two terms' accumulators: D = (D1 + D2 / 16) / row scale of the token
          uint32_t rt[16];
          tmem_ld16(t_row + (uint32_t)(n_box + c), rt);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float inv = c + j < it.valid ? token_scale_inverse(amax_in[it.row0 + c + j]) : 0.0f;
            ra[j] = __float_as_uint(__fmaf_rn(__uint_as_float(rt[j]), 0.0625f, __uint_as_float(ra[j])) * inv);
          }
        }
        if (stacked && gate_up_item) {
          // lanes 0-63 hold silu's argument (gate rows), lanes 64-127 the up rows of the same
          // features: warps 2,3 hand their chunk to warps 0,1 through a double-buffered slot
          tmem_ld_wait();
          const uint32_t buf = xn & 1u, ph = (xn >> 1) & 1u;
          ++xn;
          const int xrow = (quarter & 1) * 32 + lane;
          float* slot = &ctl->xchg[buf][half][xrow][0];
          int ok = 0;
          if (quarter >= 2) {
            if (lane == 0) ok = mbar_wait(smem_u32(&ctl->x_empty[buf][half]), ph ^ 1u, abort_flag, status) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) {
              alive = false;
              break;
            }
#pragma unroll
            for (int j = 0; j < 16; j += 4)
              *reinterpret_cast<float4*>(slot + j) =
                  make_float4(__uint_as_float(ra[j]) * s0, __uint_as_float(ra[j + 1]) * s0,
                              __uint_as_float(ra[j + 2]) * s0, __uint_as_float(ra[j + 3]) * s0);
            mbar_arrive(smem_u32(&ctl->x_full[buf][half]));
          } else {
            if (lane == 0) ok = mbar_wait(smem_u32(&ctl->x_full[buf][half]), ph, abort_flag, status) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) {
              alive = false;
              break;
            }
            __syncwarp();  // lane 0's acquire orders the whole warp's reads of the slot
            float u[16];
#pragma unroll
            for (int j = 0; j < 16; j += 4) {
              const float4 v = *reinterpret_cast<const float4*>(slot + j);
              u[j] = v.x; u[j + 1] = v.y; u[j + 2] = v.z; u[j + 3] = v.w;
            }
            mbar_arrive(smem_u32(&ctl->x_empty[buf][half]));
            uint16_t* hb = reinterpret_cast<uint16_t*>(out_ptr);
            uint32_t mag[16];  // direct fp8 form: magnitudes of the stored values (bf16 bit patterns)
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              mag[j] = 0u;
              if (c + j < it.valid) {
                const float a = __uint_as_float(ra[j]) * s0;
                const float hm = __fdividef(a, 1.0f + __expf(-a)) * u[j];
                const __nv_bfloat16 b = __float2bfloat16_rn(hm);
                hb[(size_t)(it.row0 + c + j) * I + it.m0 + xrow] = *reinterpret_cast<const uint16_t*>(&b);
                mag[j] = (uint32_t)(*reinterpret_cast<const uint16_t*>(&b) & 0x7fffu);
              }
            }
            if (DIRECT) {
              // the rows' largest magnitudes, for the down projection's token scaling: the warp's
              // 32 features of token c + j are reduced, lane j raises the row's word
              uint32_t top = 0u;
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                const uint32_t m = __reduce_max_sync(0xffffffffu, mag[j]);
                if (lane == j) top = m;
              }
              if (lane < 16 && c + lane < it.valid && top != 0u) atomicMax(amax_out + it.row0 + c + lane, top << 16);
            }
          }
        } else if (KIND == 1) {
          uint32_t rb[16];
          tmem_ld16(t_row + (uint32_t)(n_box + c), rb);
          tmem_ld_wait();
          uint16_t* hb = reinterpret_cast<uint16_t*>(out_ptr);
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            if (c + j < it.valid) {
              const float a = __uint_as_float(ra[j]) * s0;
              const float u = __uint_as_float(rb[j]) * s1;
              const float hm = __fdividef(a, 1.0f + __expf(-a)) * u;
              const __nv_bfloat16 b = __float2bfloat16_rn(hm);
              hb[(size_t)(it.row0 + c + j) * I + col] = *reinterpret_cast<const uint16_t*>(&b);
            }
          }
        } else {
          void* const out_y = fused ? fs.out2 : out_ptr;
          float* y = reinterpret_cast<float*>(out_y);
          uint16_t* yb = reinterpret_cast<uint16_t*>(out_y);  // many-token steps keep y in bf16
          uint32_t rb[16];
          if (dual) tmem_ld16(t_row + (uint32_t)(n_box + c), rb);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (c + j < it.valid) {
              const size_t o = (size_t)(it.row0 + c + j) * H + col;
              if (out_bf16) {
                const __nv_bfloat16 b0 = __float2bfloat16_rn(__uint_as_float(ra[j]) * s0);
                yb[o] = *reinterpret_cast<const uint16_t*>(&b0);
                if (dual) {
                  const __nv_bfloat16 b1 = __float2bfloat16_rn(__uint_as_float(rb[j]) * s1);
                  yb[o + kBlockM] = *reinterpret_cast<const uint16_t*>(&b1);
                }
              } else {
                y[o] = __uint_as_float(ra[j]) * s0;
                if (dual) y[o + kBlockM] = __uint_as_float(rb[j]) * s1;
              }
            }
        }
      }
      if (!alive) break;
      if (fused && gate_up_item && quarter < 2) {
        // this warp's intermediate rows of the item are stored: make them visible device-wide,
        // then count the warp in (the down items of this expert wait for the full count)
        __threadfence();
        asm volatile("fence.proxy.async;" ::: "memory");
        __syncwarp();
        if (lane == 0) atomicAdd(fs.done + it.g, 1u);
      }
      tc_fence_before();
      mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
    }
  }

  // ---- teardown
  // An early-start CTA reaches its dependency wait only on the path of its first item; every
  // other way out (no item drawn, loads withheld, an abort) passes it here, so that NO kernel of
  // a step completes before its predecessors have - the ordering of the kernels behind this one
  // rests on that.
  if (early) griddep_wait();
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols)
                 : "memory");
  }
  if (threadIdx.x == 0) timeline_end(timeline, timeline_slot);
}

// fp8 direct form, between the two projections: the intermediate rows of the group's experts
// (bf16, written by the gate/up epilogue together with every row's largest magnitude) as two e4m3
// terms per element.  Four CTAs per expert of the group (a quarter of the columns each); a warp
// takes a row at a time.
__global__ void __launch_bounds__(256)
split_rows_kernel(const __grid_constant__ FfnGroup grp, const int32_t* __restrict__ offsets,
                  const uint16_t* __restrict__ hbuf, const uint32_t* __restrict__ amax_mid,
                  uint8_t* __restrict__ terms_mid, int I, int rows_total) {
  griddep_launch_dependents();
  griddep_wait();
  const int e = grp.expert[blockIdx.x];
  const int first = offsets[e], last = offsets[e + 1];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int r = first + warp; r < last; r += 8) {
    const float scale = token_scale(amax_mid[r]);
    const uint4* src = reinterpret_cast<const uint4*>(hbuf + (size_t)r * I);
    uint2* out1 = reinterpret_cast<uint2*>(terms_mid + (size_t)r * I);
    uint2* out2 = reinterpret_cast<uint2*>(terms_mid + ((size_t)rows_total + r) * I);
    for (int c = lane + 32 * (int)blockIdx.y; c < I / 8; c += 32 * (int)gridDim.y) {
      const uint4 v = src[c];
      uint2 t1, t2;
      split_bf16x4(v.x, v.y, scale, t1.x, t2.x);
      split_bf16x4(v.z, v.w, scale, t1.y, t2.y);
      out1[c] = t1;
      out2[c] = t2;
    }
  }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

bool encode(CUtensorMap* m, int rank, const void* base, const cuuint64_t* dims, const cuuint64_t* strides,
            const cuuint32_t* box, bool bytes = false, bool bytes_swizzle_128 = false) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  const CUtensorMapL2promotion promo = CU_TENSOR_MAP_L2_PROMOTION_L2_256B;
  // bf16 operand tiles land in the 128-byte-swizzled layout the MMA reads; e4m3 rows for the
  // widening form (64 bytes per k-block) land with the 64-byte swizzle, which lets 32 lanes read
  // 32 rows free of bank conflicts; e4m3 rows the MMA reads itself (128 bytes per k-block) land
  // in the 128-byte-swizzled layout again
  return fn(m, bytes ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank,
            const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            bytes && !bytes_swizzle_128 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, promo,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct Rings {
  int stages;     // pipeline stages
  int k_atoms;    // k-blocks of 64 per stage
  uint32_t smem;  // dynamic shared memory of the launch
};
// Epilogue warps the kernel activates for a token tile (the others widen fp8 weights).
int epi_warps_for(int kind, int out_bf16, int n_box) {
  return std::min((kind != 2 || out_bf16) ? kEpiWarps : 8, 4 * (n_box / 16));
}
// Stage shape and count.  A stage holds two k-blocks where at least four such stages fit (small
// token tiles, one weight tile) and the contraction has an even number of k-blocks.  bf16 stores:
// as many stages (weight tile(s) + token tile) as fit in shared memory, ten k-blocks at most
// (eleven measured slower).  fp8 stores: a stage is a load slot in shared memory plus columns of
// tensor memory behind the accumulators (two accumulator stages if at least two weight stages
// still fit); the depth is a multiple of the number of converter groups (see the kernel).
// k_dim2: the second contraction length of a fused launch (0 otherwise).
// fp8: 0 = bf16 stores, 1 = fp8 stores widened by converter warps, 2 = fp8 stores read directly.
Rings rings_for(int kind, bool dual, int n_box, int out_bf16, int fp8, int k_dim, int k_dim2 = 0) {
  const uint32_t a = (dual ? 2u : 1u) * kATile, b = (uint32_t)n_box * 128u;
  const uint32_t avail = kSmemMax - kCtlBytes - 1024u;
  const uint32_t atom = fp8 == 2 ? kATile + 2u * b : fp8 ? a / 2 + b : a + b;  // one k-block in shared memory
  int kblocks = (int)std::min<uint32_t>((uint32_t)(fp8 == 2 ? kMaxStages : fp8 ? 2 * kMaxStages : 10), avail / atom);
  if (fp8 == 1) {
    const int acc_cols = (dual ? 2 : 1) * n_box, a_cols = dual ? 64 : 32;
    const int free_cols = 512 - 2 * acc_cols >= 2 * a_cols ? 512 - 2 * acc_cols : 512 - acc_cols;
    kblocks = std::min(kblocks, free_cols / a_cols);
  }
  Rings r;
  const int kk = fp8 == 2 ? 128 : kBlockK;  // k-values of a k-block
  r.k_atoms = (!dual && kblocks >= 8 && (k_dim / kk) % 2 == 0 && (k_dim2 / kk) % 2 == 0) ? 2 : 1;
  r.stages = std::min(kblocks / r.k_atoms, kMaxStages);
  if (fp8 == 1) {
    const int groups = std::min(2, 1 + (kEpiWarps - epi_warps_for(kind, out_bf16, n_box)) / 4);
    if (r.stages >= groups) r.stages -= r.stages % groups;
  }
  r.smem = kCtlBytes + 1024u + (uint32_t)(r.stages * r.k_atoms) * atom;
  return r;
}

template <int KIND, bool DUAL, int FP8>
bool set_smem_attr() {
  return cudaFuncSetAttribute(ffn_tc_kernel<KIND, DUAL, FP8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)kSmemMax) == cudaSuccess;
}

template <int KIND, bool DUAL>
void launch_variant(int fp8, int grid, cudaStream_t st, const CUtensorMap& tw, const CUtensorMap& ta,
                    const FfnGroup& grp, const int32_t* offsets, void* out, int H, int I, int out_bf16,
                    const uint8_t* pool, size_t slot_bytes, uint32_t* status, uint32_t* work_counter,
                    uint32_t smem_of_predecessor, bool early_allowed, StepTimeline* timeline, int timeline_slot,
                    const RouteReport& report, const FusedSecond& fs = FusedSecond{}, const uint32_t* amax_in = nullptr,
                    uint32_t* amax_out = nullptr) {
  const Rings r = rings_for(KIND, DUAL, grp.n_box, out_bf16, fp8, KIND == 2 ? I : H, KIND == 3 ? I : 0);
  // KIND 2 may start ahead of its dependency wait only where the caller vouches for the ordering
  // (early_allowed, see launch_ffn_tc) AND one of its CTAs and one of the KIND 1 kernel before it
  // cannot share an SM, so that it gets an SM only when a KIND 1 CTA has left it
  const int early = (KIND == 2 && early_allowed && smem_of_predecessor + r.smem > 228u * 1024u) ? 1 : 0;
  if constexpr (KIND == 3) {
    launch_pdl(ffn_tc_kernel<3, false, 0>, dim3(grid), dim3(kThreads), r.smem, st, tw, ta, grp, offsets, out, H, I,
               r.stages, r.k_atoms, 0, out_bf16, pool, (unsigned long long)slot_bytes, status, work_counter, timeline,
               timeline_slot, report, fs, amax_in, amax_out);
  } else if (fp8 == 2) {
    if constexpr (!DUAL)
      launch_pdl(ffn_tc_kernel<KIND, false, 2>, dim3(grid), dim3(kThreads), r.smem, st, tw, ta, grp, offsets, out, H,
                 I, r.stages, r.k_atoms, early, out_bf16, pool, (unsigned long long)slot_bytes, status, work_counter,
                 timeline, timeline_slot, report, fs, amax_in, amax_out);
  } else if (fp8) {
    launch_pdl(ffn_tc_kernel<KIND, DUAL, 1>, dim3(grid), dim3(kThreads), r.smem, st, tw, ta, grp, offsets, out, H,
               I, r.stages, r.k_atoms, early, out_bf16, pool, (unsigned long long)slot_bytes, status, work_counter, timeline,
               timeline_slot, report, fs, amax_in, amax_out);
  } else {
    launch_pdl(ffn_tc_kernel<KIND, DUAL, 0>, dim3(grid), dim3(kThreads), r.smem, st, tw, ta, grp, offsets, out, H,
               I, r.stages, r.k_atoms, early, out_bf16, pool, (unsigned long long)slot_bytes, status, work_counter, timeline,
               timeline_slot, report, fs, amax_in, amax_out);
  }
}

}  // namespace

static bool g_pairs_refused = false;  // a cluster launch of the pair kernel failed on this device once

int ffn_tc_setup(FfnTcMaps* maps, const uint8_t* pool, size_t slot_bytes, int n_slots, int H, int I, bool fp8,
                 const uint16_t* xp, const uint16_t* hbuf, int rows, const TokenSplit* split) {
  maps->fp8 = fp8;
  maps->pool = pool;
  maps->slot_bytes = slot_bytes;
  const cuuint64_t esz = fp8 ? 1 : 2;  // bytes per weight element in the slot pool
  {
    const cuuint64_t dims[3] = {(cuuint64_t)H, (cuuint64_t)(2 * I), (cuuint64_t)n_slots};
    const cuuint64_t strides[2] = {(cuuint64_t)H * esz, (cuuint64_t)slot_bytes};
    const cuuint32_t box[3] = {kBlockK, kBlockM, 1};
    const cuuint32_t box_half[3] = {kBlockK, kBlockM / 2, 1};  // stacked gate/up tiles
    if (!encode(&maps->w13, 3, pool, dims, strides, box, fp8)) return OLED_ERR_CUDA;
    if (!encode(&maps->w13_half, 3, pool, dims, strides, box_half, fp8)) return OLED_ERR_CUDA;
  }
  {
    const cuuint64_t dims[3] = {(cuuint64_t)I, (cuuint64_t)H, (cuuint64_t)n_slots};
    const cuuint64_t strides[2] = {(cuuint64_t)I * esz, (cuuint64_t)slot_bytes};
    const cuuint32_t box[3] = {kBlockK, kBlockM, 1};
    if (!encode(&maps->w2, 3, pool + (size_t)2 * I * H * esz, dims, strides, box, fp8)) return OLED_ERR_CUDA;
  }
  // fp8 stores: maps for the form whose MMAs read the codes themselves - k-blocks of 128 bytes
  maps->e4m3_direct = fp8 && H % 128 == 0 && I % 128 == 0 && split != nullptr && split->complete() && split->rows == rows;
  if (maps->e4m3_direct) {
    for (int i = 0; i < 2; ++i) {
      const cuuint32_t tbox[3] = {128, (cuuint32_t)(16 << i), 2};
      const cuuint64_t dims_in[3] = {(cuuint64_t)H, (cuuint64_t)rows, 2}, dims_mid[3] = {(cuuint64_t)I, (cuuint64_t)rows, 2};
      const cuuint64_t str_in[2] = {(cuuint64_t)H, (cuuint64_t)rows * H}, str_mid[2] = {(cuuint64_t)I, (cuuint64_t)rows * I};
      if (!encode(&maps->xp_terms[i], 3, split->terms_in, dims_in, str_in, tbox, true, true)) return OLED_ERR_CUDA;
      if (!encode(&maps->hbuf_terms[i], 3, split->terms_mid, dims_mid, str_mid, tbox, true, true)) return OLED_ERR_CUDA;
    }
    const cuuint32_t box_half[4] = {128, kBlockM / 2, 2, 1}, box[3] = {128, kBlockM, 1};
    const cuuint64_t dims13[4] = {(cuuint64_t)H, (cuuint64_t)I, 2, (cuuint64_t)n_slots};
    const cuuint64_t strides13[3] = {(cuuint64_t)H, (cuuint64_t)I * H, (cuuint64_t)slot_bytes};
    const cuuint64_t dims2[3] = {(cuuint64_t)I, (cuuint64_t)H, (cuuint64_t)n_slots};
    const cuuint64_t strides2[2] = {(cuuint64_t)I, (cuuint64_t)slot_bytes};
    if (!encode(&maps->w13_half_e4m3, 4, pool, dims13, strides13, box_half, true, true)) return OLED_ERR_CUDA;
    if (!encode(&maps->w2_e4m3, 3, pool + (size_t)2 * I * H, dims2, strides2, box, true, true)) return OLED_ERR_CUDA;
  }
  for (int i = 0; i < 5; ++i) {
    const cuuint32_t box[2] = {kBlockK, (cuuint32_t)(16 << i)};
    {
      const cuuint64_t dims[2] = {(cuuint64_t)H, (cuuint64_t)rows};
      const cuuint64_t strides[1] = {(cuuint64_t)H * 2};
      if (!encode(&maps->xp[i], 2, xp, dims, strides, box)) return OLED_ERR_CUDA;
    }
    {
      const cuuint64_t dims[2] = {(cuuint64_t)I, (cuuint64_t)rows};
      const cuuint64_t strides[1] = {(cuuint64_t)I * 2};
      if (!encode(&maps->hbuf[i], 2, hbuf, dims, strides, box)) return OLED_ERR_CUDA;
    }
  }
  static bool attr_done = false;
  if (!attr_done) {
    if (!set_smem_attr<1, true, 0>() || !set_smem_attr<1, false, 0>() || !set_smem_attr<2, true, 0>() ||
        !set_smem_attr<2, false, 0>() || !set_smem_attr<1, true, 1>() || !set_smem_attr<1, false, 1>() ||
        !set_smem_attr<2, true, 1>() || !set_smem_attr<2, false, 1>() || !set_smem_attr<3, false, 0>() ||
        !set_smem_attr<1, false, 2>() || !set_smem_attr<2, false, 2>())
      return OLED_ERR_CUDA;
    attr_done = true;
  }
  return OLED_OK;
}

static int box_index(int max_count, int cap) {
  int i = 0;
  while ((16 << i) < max_count && (16 << i) < cap) ++i;
  return i;
}

int launch_ffn_tc(cudaStream_t st, const FfnTcMaps& maps, const FfnGroup& grp_in, int max_count, int kind,
                  const int32_t* host_counts, const int32_t* offsets, uint16_t* hbuf, float* y, int y_bf16, int H, int I,
                  int n_sms, uint32_t* status, uint32_t* work_counter, bool behind_event_wait, StepTimeline* timeline,
                  int timeline_slot, const RouteReport& report_in, uint32_t* done, const TokenSplit* split) {
  const RouteReport report = kind != 2 ? report_in : RouteReport{};
  if (grp_in.n <= 0 || max_count <= 0) return OLED_OK;
  FfnGroup grp = grp_in;
  const bool fp8 = maps.fp8;
  grp.pad = 0;
  // N <= 128 keeps the accumulators double-buffered in TMEM; more tokens per expert than that
  // take N = 256 with two weight tiles per item (all 512 TMEM columns, one accumulator stage).
  // (fp8 stores stop at N = 128: the widened weights need tensor-memory columns of their own)
  const int ib = box_index(max_count, fp8 ? 128 : 256);
  grp.n_box = 16 << ib;
  // fp8 stores, token tiles of at most 32 rows, row magnitudes at hand: the MMAs read the codes
  // themselves (mode 2); otherwise converter warps widen them to bf16 (mode 1)
  const bool direct = fp8 && maps.e4m3_direct && grp.n_box <= 32 && split != nullptr && split->complete();
  const int mode = direct ? 2 : fp8 ? 1 : 0;
  // many-token tiles: the CTA-pair kernel, unless its cluster launch has failed before on this
  // device (the one-CTA form below computes the same)
  if (maps.use_pairs && !g_pairs_refused && ffn_pair_usable(maps, grp.n_box, H, I)) {
    if (launch_ffn_pair(st, maps, grp, kind, offsets, hbuf, y, y_bf16, H, I, n_sms, status, work_counter, timeline,
                        timeline_slot, report, done) == OLED_OK)
      return OLED_OK;
    cudaGetLastError();  // (a refused launch enqueues nothing)
    g_pairs_refused = true;
    if (maps.token_source.perm != nullptr) {  // the one-CTA form reads the gathered copy
      launch_gather(st, maps.token_source.x, maps.token_source.perm, maps.token_source.T, H, maps.token_source.K,
                    maps.token_source.xp);
      maps.token_source.perm = nullptr;
    }
  }
  if (kind == 3 && grp.n_box > 32) {
    // (only reached when the pair launch was refused: the two launches of the one-CTA form, the
    // work counter cleared in stream order between them)
    int rc = launch_ffn_tc(st, maps, grp_in, max_count, 1, host_counts, offsets, hbuf, y, y_bf16, H, I, n_sms, status,
                           work_counter, behind_event_wait, timeline, timeline_slot, report_in, done, split);
    if (rc != OLED_OK) return rc;
    if (cudaMemsetAsync(work_counter, 0, sizeof(uint32_t), st) != cudaSuccess) return OLED_ERR_CUDA;
    return launch_ffn_tc(st, maps, grp_in, max_count, 2, host_counts, offsets, hbuf, y, y_bf16, H, I, n_sms, status,
                         work_counter, false, timeline, timeline_slot, report_in, done, split);
  }
  // one CTA per SM, fewer if the group has fewer (weight tile, token tile) items than SMs
  auto grid_for = [&](int m_tiles) {
    if (host_counts == nullptr) return n_sms;  // counts not known on the host yet
    long long tiles = 0;
    for (int g = 0; g < grp.n; ++g) tiles += (host_counts[grp.expert[g]] + grp.n_box - 1) / grp.n_box;
    return (int)std::max<long long>(1, std::min<long long>(n_sms, tiles * m_tiles));
  };
  // shared memory of a CTA of this group's KIND 1 launch
  const bool stacked1 = grp.n_box <= 32;
  // A KIND 2 launch may start early only if nothing it reads besides the token tiles can still be
  // in the making: either every SM holds a CTA of the KIND 1 launch before it (full grid: a KIND 2
  // CTA then gets an SM only after a KIND 1 CTA, which waited for the permutation, has left it),
  // or the launch pair sits behind an event wait, which completes everything enqueued before it.
  const bool early_allowed = kind == 2 && (behind_event_wait || host_counts == nullptr);
  const uint32_t smem1 = kind == 2 ? rings_for(1, !stacked1, grp.n_box, 0, mode, H).smem : 0u;
  if (kind == 3) {
    if (fp8 || !stacked1 || done == nullptr) return OLED_ERR_INVALID_ARG;  // callers ask ffn_tc_can_fuse() first
    FusedSecond fs;
    fs.tm_w2 = maps.w2;
    fs.tm_act2 = maps.hbuf[ib];
    fs.out2 = y;
    fs.done = done;
    launch_variant<3, false>(0, grid_for(I / (kBlockM / 2) + H / kBlockM), st, maps.w13_half, maps.xp[ib], grp, offsets,
                             hbuf, H, I, 0, maps.pool, maps.slot_bytes, status, work_counter, 0u, false, timeline,
                             timeline_slot, report, fs);
  } else if (kind == 1 && stacked1) {
    launch_variant<1, false>(mode, grid_for(I / (kBlockM / 2)), st, direct ? maps.w13_half_e4m3 : maps.w13_half,
                             direct ? maps.xp_terms[ib] : maps.xp[ib], grp, offsets, hbuf, H, I, 0, maps.pool,
                             maps.slot_bytes, status, work_counter, smem1, early_allowed, timeline, timeline_slot, report,
                             FusedSecond{}, direct ? split->amax_in : nullptr, direct ? split->amax_mid : nullptr);
  } else if (kind == 1) {
    launch_variant<1, true>(mode, grid_for(I / kBlockM), st, maps.w13, maps.xp[ib], grp, offsets, hbuf, H, I, 0,
                            maps.pool, maps.slot_bytes, status, work_counter, smem1, early_allowed, timeline, timeline_slot, report);
  } else {
    const bool dual = grp.n_box == 256;
    if (dual)
      launch_variant<2, true>(mode, grid_for(H / (2 * kBlockM)), st, maps.w2, maps.hbuf[ib], grp, offsets, y, H, I,
                              y_bf16, maps.pool, maps.slot_bytes, status, work_counter, smem1, early_allowed, timeline, timeline_slot, report);
    else {
      if (direct)  // the intermediate rows as e4m3 terms, now that their magnitudes are complete
        launch_pdl(split_rows_kernel, dim3(grp.n, 4), dim3(256), 0, st, grp, offsets, (const uint16_t*)hbuf,
                   (const uint32_t*)split->amax_mid, split->terms_mid, I, split->rows);
      launch_variant<2, false>(mode, grid_for(H / kBlockM), st, direct ? maps.w2_e4m3 : maps.w2,
                               direct ? maps.hbuf_terms[ib] : maps.hbuf[ib], grp, offsets, y, H, I, y_bf16, maps.pool,
                               maps.slot_bytes, status, work_counter, smem1, early_allowed, timeline, timeline_slot,
                               report, FusedSecond{}, direct ? split->amax_mid : nullptr, nullptr);
    }
  }
  return cudaGetLastError() == cudaSuccess ? OLED_OK : OLED_ERR_CUDA;
}

bool ffn_tc_token_source_usable(const FfnTcMaps& maps, int H, int I) {
  return maps.use_pairs && !g_pairs_refused && ffn_pair_usable(maps, 256, H, I);
}
void ffn_tc_set_token_source(FfnTcMaps* maps, const uint16_t* x, int T, const int32_t* perm, int K, uint16_t* xp) {
  maps->token_source.perm = perm;
  maps->token_source.K = K;
  maps->token_source.T = T;
  maps->token_source.x = x;
  maps->token_source.xp = xp;
  maps->token_source.ready = nullptr;
}
void ffn_tc_clear_token_source(FfnTcMaps* maps) { maps->token_source.perm = nullptr; }

int ffn_tc_launches(const FfnTcMaps& maps, int max_count, int kind, const TokenSplit* split) {
  const bool direct = maps.fp8 && maps.e4m3_direct && (16 << box_index(max_count, 128)) <= 32 && split != nullptr &&
                      split->complete();
  return kind == 2 && direct ? 2 : 1;
}

bool ffn_tc_can_fuse(const FfnTcMaps& maps, int max_count) {
  return !maps.fp8 && (16 << box_index(max_count, 256)) <= 32;
}
bool ffn_pair_can_fuse(const FfnTcMaps& maps, int max_count, int H, int I) {
  return maps.use_pairs && !g_pairs_refused && ffn_pair_usable(maps, 16 << box_index(max_count, maps.fp8 ? 128 : 256), H, I);
}

}  // namespace oled
