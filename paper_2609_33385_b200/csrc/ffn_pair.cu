// Grouped SwiGLU expert FFN for many-token steps on CTA PAIRS (tcgen05 cta_group::2).
//
// In the many-token regime (token tiles of 256 rows) the expert FFN is a tensor-core GEMM, and
// TMEM fixes the tile one SM can accumulate: two 128-row weight tiles against 256 token rows use
// all 512 columns and take 64 KB of operands per k-block of 64.  Fewer operand bytes per
// multiply-add need two SMs to share a token tile: here a cluster of two CTAs computes 512
// output features x 256 tokens with M = 256 MMAs.  Each CTA holds its own two 128-row weight
// tiles, its own accumulators (its 128 lanes x 512 columns of TMEM) and HALF of the token tile;
// the MMA, issued by one thread of the pair's first CTA, reads both halves.  48 KB of operands per
// CTA and k-block instead of 64 (the tensor pipe's share of the active cycles went from 67 to
// 71 % on 4096 tokens x 4096 x 1536; the traffic alone was worth little - L2 runs at 39 % of its
// peak - the dynamic items across the pair, the pipelined epilogue and the single launch the rest).
//   KIND 1: features f0 + 128 r .. + 127 for CTA r: gate rows and up rows of those features,
//           epilogue hbuf[n, f] = bf16(silu(D_gate) * D_up)
//   KIND 2: output rows c0 + 256 r .. + 255 for CTA r (two row blocks of Wd), epilogue y[n, c] = D
// No TMA multicast: every CTA loads what lies in its own shared memory.
// 19 warps per CTA: 16 epilogue warps, the TMA thread's, the MMA thread's, and one whose first thread
// gathers token rows when the launch is asked to (PairTokens below); its lanes are idle otherwise.
//
// Protocol per pipeline stage (barriers at the same shared-memory offsets in both CTAs):
//   full[s]   lives in the FIRST CTA: its TMA thread announces the bytes of both CTAs' copies
//             (expect_tx), both CTAs' copies count their bytes there (cta_group::2 loads name a
//             cluster-wide barrier address);
//   empty[s]  lives in BOTH: the MMA thread's commit arrives on both (commit with a CTA mask)
//             when the MMAs that read the stage have completed.
// Accumulators: tmem_full in both CTAs (commit with the mask), tmem_empty in the first CTA (one
// arrival per epilogue warp of either CTA, the second CTA's across the cluster).
// Work items (expert, token tile, pair of weight-tile pairs) are numbered as in ffn_tc.cu and handed
// out dynamically: the first CTA's TMA thread takes the pair's number as its first item and draws
// every later one from a counter in global memory, and publishes each number to the item rings
// of BOTH CTAs (a remote store followed by a release arrival on the other CTA's barrier); all
// other roles take their items from their own CTA's ring.
// Every wait is bounded (a timeout raises the status word and the CTA winds down); a cluster
// barrier before the exit keeps a CTA's shared memory alive while its partner may still use it.
#include <cuda.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstddef>

#include "kernels.h"
#include "sm100_ptx.h"

namespace oled {
namespace {

constexpr int kPairEpiWarps = 16;
constexpr int kPairProducerWarp = kPairEpiWarps;
constexpr int kPairMmaWarp = kPairEpiWarps + 1;
constexpr int kPairGatherWarp = kPairEpiWarps + 2;
constexpr int kPairThreads = (kPairEpiWarps + 3) * 32;
constexpr int kPairK = 64;                              // k-values of a k-block (one 128-byte swizzle atom of bf16)
constexpr uint32_t kPairATile = 128 * kPairK * 2;       // 128 weight rows of a k-block
constexpr uint32_t kPairBHalf = 128 * kPairK * 2;       // this CTA's half of the token tile
constexpr uint32_t kPairStage = 2 * kPairATile + kPairBHalf;  // 48 KB
constexpr int kPairStages = 4;
constexpr int kPairRing = 8;      // item numbers in flight between the pair's roles (see take_pair_item)
constexpr int kPairN = 256;                             // token rows of a tile

struct __align__(16) PairCtl {
  unsigned long long full[kPairStages];
  unsigned long long empty[kPairStages];
  unsigned long long tmem_full;
  unsigned long long tmem_empty;
  unsigned long long item_full[kPairRing];
  unsigned long long row_full[4];  // (gathering thread) a row chunk has landed in its slot
  unsigned long long row_dst[4];   // where the slot's chunk goes
  uint32_t row_bytes[4];
  int row_tile[8];                 // the token tile (number within the launch) of the last chunks issued
  int item_ring[kPairRing];
  uint32_t tmem_base;
  int abort;
  int n_tiles_total;
  int pad;
  int tile_prefix[OLED_MAX_EXPERTS + 1];
  int row_start[OLED_MAX_EXPERTS];
  int count[OLED_MAX_EXPERTS];
};
constexpr uint32_t kPairCtlBytes = (sizeof(PairCtl) + 1023u) & ~1023u;
constexpr uint32_t kPairSmem = kPairCtlBytes + 1024u + kPairStages * kPairStage + 3u * 8192u;  // + the row ring

struct PairItem {
  int slot, m0, row0, valid;
  int kind;  // 1: gate/up (+SwiGLU), 2: down projection
  int g;     // index of the expert in the launch's group
};
// A role's position in the expert list: items arrive in ascending order within a phase, so the
// search for an item's expert only moves forward; it restarts with the second phase of a fused launch.
struct PairCursor {
  int g = 0;
  int phase2 = 0;
};
// How a launch's item numbers divide: [0, n1) items of kind1 with m_blocks1 feature blocks per
// token tile, then (a fused launch) the down items of the same token tiles with m_blocks2 blocks.
struct PairPlan {
  int kind1, n1, m_blocks1, m_blocks2;
};
// item -> (kind, expert, token tile, feature block of the pair)
__device__ __forceinline__ void pair_decode(const PairCtl* ctl, const FfnGroup& grp, int item, const PairPlan& plan,
                                            PairCursor& cur, PairItem& it) {
  int m_blocks = plan.m_blocks1;
  it.kind = plan.kind1;
  if (item >= plan.n1) {
    item -= plan.n1;
    m_blocks = plan.m_blocks2;
    it.kind = 2;
    if (!cur.phase2) {
      cur.phase2 = 1;
      cur.g = 0;
    }
  }
  const int m_rows = it.kind == 1 ? 256 : 512;  // features / output rows per pair item
  const int q = item / m_blocks;
  const int m = item - q * m_blocks;
  int g = cur.g;
  while (ctl->tile_prefix[g + 1] <= q) ++g;
  cur.g = g;
  const int nt = q - ctl->tile_prefix[g];
  it.g = g;
  it.slot = grp.slot[g];
  it.m0 = m * m_rows;
  it.row0 = ctl->row_start[g] + nt * kPairN;
  it.valid = min(kPairN, ctl->count[g] - nt * kPairN);
}

__device__ __forceinline__ bool mbar_try_cluster(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}
// The seq-th item of the pair, -1 when there is no more work, -2 on an abort or a timeout.
// No barrier guards the re-use of a ring slot; the pipeline does: the publisher hands out item
// n only after it has issued every copy of item n-1, so the MMA thread - at most a ring of stages
// behind the copies - is in item n-2 or later; it entered n-2 only after all epilogue warps of
// both CTAs had finished n-3 (one accumulator stage), and the other CTA's TMA thread is never
// behind the MMA thread.  Every reader is therefore past item n-4, and the ring holds 8.
__device__ __forceinline__ int take_pair_item(PairCtl* ctl, int seq, volatile int* abort_flag, uint32_t* status) {
  const int slot = seq % kPairRing;
  const uint32_t bar = smem_u32(&ctl->item_full[slot]), parity = (uint32_t)(seq / kPairRing) & 1u;
  unsigned long long t0 = 0;
  for (uint32_t spin = 0;; ++spin) {
    if (mbar_try_cluster(bar, parity)) break;
    if ((spin & 1023u) == 1023u) {
      if (*abort_flag) return -2;
      const unsigned long long now = globaltimer();
      if (t0 == 0) t0 = now;
      if (now - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(status, (uint32_t)kStatusWaitTimeout);
        return -2;
      }
    }
  }
  return *reinterpret_cast<volatile int*>(&ctl->item_ring[slot]);
}

// What a FUSED launch (KIND 3) needs on top: the down projection's tensor maps, its output and the
// completion counters (one ZERO word per expert of the group).
struct PairSecond {
  CUtensorMap tm_w2;    // down-projection weights
  CUtensorMap tm_act2;  // intermediate rows (hbuf)
  void* out2;           // y
  uint32_t* done;       // per expert: epilogue warps (of either CTA) that have stored gate/up rows
};

// The launch gathers its experts' token rows itself (kinds 1 and 3; perm == nullptr: the rows are in
// place already): sorted row r of the group's experts is row perm[r] / K of the step's input.  One
// thread per CTA moves the rows (CTA c takes every gridDim-th row of the group, in the order the items
// need them) through a small ring in shared memory with bulk copies, and counts each finished chunk
// on its token tile's word of `ready` (ZERO at the start); the TMA threads hold a gate/up item back
// until its tile's rows are complete.  The tensor pipe is the bound of these launches, so the
// copies ride along; a gather kernel in front would cost its full length.
struct PairTokens {
  const uint16_t* x;     // [T][H] the step's input
  uint16_t* xp;          // [rows][H] the sorted copy (read back through tm_act)
  const int32_t* perm;
  uint32_t* ready;       // per token tile of the launch (numbered expert by expert): chunks copied
  int K;
};
constexpr uint32_t kRowChunk = 8192;  // bytes per bulk copy of a row piece
constexpr int kRowSlots = 3;

// KIND 3: the gate/up items, then the down items of the same experts, in ONE launch (a launch
// boundary between cluster kernels is a full stop: a dependent cluster launch was never seen to
// start before its predecessor had finished, so the last gate/up items' uneven end and the next
// launch's set-up would leave SMs idle).  A down item reads the intermediate rows the gate/up
// items of its expert wrote; its TMA threads wait (bounded) until the expert's counter shows
// that all of them are stored - items are handed out in order, gate/up first, so that wait is
// over long before it is reached except at the switch of phases.
template <int KIND>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
ffn_pair_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_act,
                const __grid_constant__ FfnGroup grp, const int32_t* __restrict__ offsets, void* __restrict__ out_ptr,
                int H, int I, int out_bf16, uint32_t* __restrict__ status, uint32_t* __restrict__ work_counter,
                StepTimeline* timeline, int timeline_slot, const __grid_constant__ RouteReport report,
                const __grid_constant__ PairSecond sec, const __grid_constant__ PairTokens tok) {
  constexpr bool fused = KIND == 3;
  const bool gathers = KIND != 2 && tok.perm != nullptr;  // the launch gathers its token rows itself
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  PairCtl* ctl = reinterpret_cast<PairCtl*>(smem_raw);
  const uint32_t tiles_base = (smem_u32(smem_raw) + kPairCtlBytes + 1023u) & ~1023u;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_cta_rank();  // 0: the CTA whose thread issues the pair's MMAs
  const int pair = (int)blockIdx.x >> 1, n_pairs = (int)gridDim.x >> 1;

  griddep_launch_dependents();
  if (threadIdx.x == 0) {
    timeline_entry(timeline, timeline_slot);
    for (int s = 0; s < kPairStages; ++s) {
      mbar_init(smem_u32(&ctl->full[s]), 1);
      mbar_init(smem_u32(&ctl->empty[s]), 1);
    }
    for (int s = 0; s < kPairRing; ++s) mbar_init(smem_u32(&ctl->item_full[s]), 1);
    for (int s = 0; s < kRowSlots; ++s) mbar_init(smem_u32(&ctl->row_full[s]), 1);
    mbar_init(smem_u32(&ctl->tmem_full), 1);
    mbar_init(smem_u32(&ctl->tmem_empty), 2u * kPairEpiWarps);
    ctl->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == kPairProducerWarp && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tm_act)) : "memory");
    if (fused) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&sec.tm_w2)) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&sec.tm_act2)) : "memory");
    }
  }
  if (warp == kPairMmaWarp) {  // all 512 columns, allocated by the same warp of both CTAs
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  griddep_wait();
  if (threadIdx.x == 0) timeline_start(timeline, timeline_slot);
  for (int g = threadIdx.x; g < grp.n; g += kPairThreads) {
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
      const int tiles = g < grp.n ? (ctl->count[g] + kPairN - 1) / kPairN : 0;
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
  cluster_sync_all();  // both CTAs' barriers are initialised before either one signals across
  tc_fence_after();

  const uint32_t tmem_base = ctl->tmem_base;
  // per pair item: 256 features (kind 1: 128 per CTA, their gate and up rows) or 512 output rows
  // (kind 2: 256 per CTA, two row blocks of Wd)
  PairPlan plan;
  plan.kind1 = KIND == 2 ? 2 : 1;
  plan.m_blocks1 = KIND == 2 ? H / 512 : I / 256;
  plan.m_blocks2 = H / 512;
  plan.n1 = fused ? ctl->n_tiles_total * plan.m_blocks1 : 0x7fffffff;
  const int total_items = ctl->n_tiles_total * (plan.m_blocks1 + (fused ? plan.m_blocks2 : 0));
  // (a launch that gathers) the token tiles the pairs' first items read: copied by the epilogue warps
  const int first_tiles = min(ctl->n_tiles_total, (n_pairs + plan.m_blocks1 - 1) / plan.m_blocks1);
  // (fused) gate/up epilogue warps of both CTAs that store rows per item, times the gate/up items of a token tile
  const uint32_t done_per_tile = (uint32_t)(2 * kPairEpiWarps * (I / 256));
  volatile int* abort_flag = &ctl->abort;
  const uint32_t full_on_first = map_to_cta(smem_u32(&ctl->full[0]), 0);         // cluster-wide addresses
  const uint32_t tmem_empty_on_first = map_to_cta(smem_u32(&ctl->tmem_empty), 0);

  if (KIND != 2 && blockIdx.x == 0 && warp == kPairProducerWarp && lane != 0) publish_report(report, lane - 1, 31);

  if (warp == kPairProducerWarp && lane == 0) {
    // ------------------------------------------------------------ TMA producer (one per CTA)
    int stage = 0, ready_g = -1;
    PairCursor cur;
    uint32_t phase = 0;
    bool ok = true;
    int next_item = pair;  // (first CTA) the pair's first item is its own number
    // (with loads withheld - the test of the bounded waits - nothing is published either: every
    // other role of both CTAs runs into the limit of its wait for the first item)
    for (int seq = 0; ok && !(grp.withhold_loads && rank == 0); ++seq) {
      int item;
      if (rank == 0) {
        item = next_item < total_items ? next_item : -1;
        // the following item's number is fetched now: the atomic's latency lies under this item's copies
        if (item >= 0) next_item = (int)atomicAdd(work_counter, 1u) + n_pairs;
        const int slot = seq % kPairRing;
        *reinterpret_cast<volatile int*>(&ctl->item_ring[slot]) = item;
        asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(map_to_cta(smem_u32(&ctl->item_ring[slot]), 1)), "r"(item)
                     : "memory");
        mbar_arrive_cluster(map_to_cta(smem_u32(&ctl->item_full[slot]), 0));
        mbar_arrive_cluster(map_to_cta(smem_u32(&ctl->item_full[slot]), 1));
      } else {
        item = take_pair_item(ctl, seq, abort_flag, status);
      }
      if (item < 0) break;
      PairItem it;
      pair_decode(ctl, grp, item, plan, cur, it);
      const bool down_of_fused = fused && it.kind == 2;
      const CUtensorMap* map_w = down_of_fused ? &sec.tm_w2 : &tm_w;
      const CUtensorMap* map_act = down_of_fused ? &sec.tm_act2 : &tm_act;
      const int k_blocks = (it.kind == 1 ? H : I) / kPairK;
      // what the item's token operand waits for: (down items of a fused launch) all intermediate rows of
      // the expert stored by its gate/up items; (gate/up items of a launch that gathers) the tile's token
      // rows copied.  (What was seen complete stays complete.)
      const int tile = (it.row0 - ctl->row_start[it.g]) / kPairN + ctl->tile_prefix[it.g];
      const int wait_key = down_of_fused ? (1 << 30 | it.g) : tile;
      if ((down_of_fused || (gathers && it.kind == 1)) && wait_key != ready_g) {
        const uint32_t* counter = down_of_fused ? sec.done + it.g : tok.ready + tile;
        const uint32_t target =
            down_of_fused ? (uint32_t)(ctl->tile_prefix[it.g + 1] - ctl->tile_prefix[it.g]) * done_per_tile
                          : (uint32_t)it.valid * (((uint32_t)H * 2u + kRowChunk - 1) / kRowChunk);
        unsigned long long t0 = 0;
        for (uint32_t spin = 0; ok; ++spin) {
          uint32_t seen;
          asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
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
        ready_g = wait_key;
        // (the intermediate rows were written through the generic proxy; the copies below read through the async proxy)
        asm volatile("fence.proxy.async;" ::: "memory");
      }
      const int n_mma = max(32, (it.valid + 31) & ~31);
      const int my_row0 = it.row0 + (int)rank * (n_mma >> 1);  // this CTA's half of the tile's token rows
      const int my_m0 = it.m0 + (int)rank * (it.kind == 1 ? 128 : 256);
      for (int kb = 0; kb < k_blocks; ++kb) {
        if (!mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag, status)) {
          ok = false;
          break;
        }
        const uint32_t bar = full_on_first + (uint32_t)stage * 8u;
        if (rank == 0) mbar_expect_tx(smem_u32(&ctl->full[stage]), 2u * kPairStage);
        const uint32_t base = tiles_base + (uint32_t)stage * kPairStage;
        const int k0 = kb * kPairK;
        if (it.kind == 1) {
          tma_load_3d_pair(map_w, base, bar, k0, my_m0, it.slot);                   // gate rows
          tma_load_3d_pair(map_w, base + kPairATile, bar, k0, I + my_m0, it.slot);  // up rows
        } else {
          tma_load_3d_pair(map_w, base, bar, k0, my_m0, it.slot);
          tma_load_3d_pair(map_w, base + kPairATile, bar, k0, my_m0 + 128, it.slot);
        }
        tma_load_2d_pair(map_act, base + 2 * kPairATile, bar, k0, my_row0);
        if (++stage == kPairStages) {
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
  } else if (warp == kPairGatherWarp) {
    // ------------------------------------------------------------ token rows of the group's experts
    if (gathers && lane == 0 && !grp.withhold_loads) {
      const uint32_t ring0 = tiles_base + kPairStages * kPairStage;
      const uint32_t row_bytes = (uint32_t)H * 2u;
      const int chunks = (int)((row_bytes + kRowChunk - 1) / kRowChunk);
      // position in the group's rows: expert g, row r of it, chunk c; this CTA's next row is gridDim further
      // (the rows of the first tiles are the epilogue warps')
      int g = 0, r = (int)blockIdx.x, c = 0;
      auto settle = [&]() {
        for (;;) {
          while (g < grp.n && r >= ctl->count[g]) r -= ctl->count[g++];
          if (g >= grp.n || ctl->tile_prefix[g] + r / kPairN >= first_tiles) break;
          r += (int)gridDim.x;
        }
      };
      settle();
      int issued = 0;
      bool ok = true;
      auto issue = [&]() {
        const int slot = issued % kRowSlots;
        const int row = ctl->row_start[g] + r;
        const uint32_t off = (uint32_t)c * kRowChunk, bytes = min(kRowChunk, row_bytes - off);
        const uint8_t* src = reinterpret_cast<const uint8_t*>(tok.x) + (size_t)(__ldg(tok.perm + row) / tok.K) * row_bytes + off;
        ctl->row_dst[slot] = reinterpret_cast<unsigned long long>(tok.xp) + (unsigned long long)row * row_bytes + off;
        ctl->row_bytes[slot] = bytes;
        ctl->row_tile[issued & 7] = ctl->tile_prefix[g] + r / kPairN;
        const uint32_t bar = smem_u32(&ctl->row_full[slot]);
        mbar_expect_tx(bar, bytes);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                         ring0 + (uint32_t)slot * kRowChunk),
                     "l"(src), "r"(bytes), "r"(bar)
                     : "memory");
        ++issued;
        if (++c == chunks) {
          c = 0;
          r += (int)gridDim.x;
          settle();
        }
      };
      auto count_chunk = [&](int n) {  // chunk n is in global memory: visible device-wide, then counted
        asm volatile("fence.proxy.async;" ::: "memory");
        __threadfence();
        atomicAdd(tok.ready + ctl->row_tile[n & 7], 1u);
      };
      while (issued < kRowSlots - 1 && g < grp.n) issue();
      int n = 0;
      for (; ok && n < issued; ++n) {
        const int slot = n % kRowSlots;
        if (!mbar_wait(smem_u32(&ctl->row_full[slot]), (uint32_t)(n / kRowSlots) & 1u, abort_flag, status)) {
          ok = false;
          break;
        }
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(ctl->row_dst[slot]),
                     "r"(ring0 + (uint32_t)slot * kRowChunk), "r"(ctl->row_bytes[slot])
                     : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        if (g < grp.n) {
          // the slot the next copy lands in was read by the store before this one
          asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
          issue();
        }
        if (n >= 2) {
          asm volatile("cp.async.bulk.wait_group 2;" ::: "memory");
          count_chunk(n - 2);
        }
      }
      asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
      if (ok)
        for (int m = max(0, n - 2); m < n; ++m) count_chunk(m);
      if (!ok) {  // let copies already issued land before the CTA's shared memory is released
        const unsigned long long t0 = globaltimer();
        while (globaltimer() - t0 < 2000000ull) {
        }
      }
    }
  } else if (warp == kPairMmaWarp && lane == 0 && rank == 0) {
    // ------------------------------------------------------------ MMA issuer (first CTA only)
    int stage = 0, local = 0;
    PairCursor cur;
    uint32_t phase = 0;
    bool ok = true;
    const uint32_t desc_hi = (uint32_t)(make_smem_desc(0) >> 32);
    const uint32_t a_lo0 = (uint32_t)make_smem_desc(tiles_base);
    const uint32_t b_lo0 = (uint32_t)make_smem_desc(tiles_base + 2 * kPairATile);
    const uint32_t ring_step = kPairStage >> 4;
    uint32_t a_lo = a_lo0, b_lo = b_lo0;
    for (; ok; ++local) {
      const int item = take_pair_item(ctl, local, abort_flag, status);
      if (item < 0) break;
      PairItem it;
      pair_decode(ctl, grp, item, plan, cur, it);
      const int k_blocks = (it.kind == 1 ? H : I) / kPairK;
      // one accumulator stage: both CTAs' epilogues must have drained the previous item
      if (!mbar_wait(smem_u32(&ctl->tmem_empty), ((uint32_t)local & 1u) ^ 1u, abort_flag, status)) break;
      tc_fence_after();
      const int n_mma = max(32, (it.valid + 31) & ~31);
      const uint32_t idesc = make_idesc_pair(n_mma);
      for (int kb = 0; kb < k_blocks; ++kb) {
        if (!mbar_wait(smem_u32(&ctl->full[stage]), phase, abort_flag, status)) {
          ok = false;
          break;
        }
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < kPairK / 16; ++k) {  // 32 bytes along K = 2 address units
          const uint32_t accum = (kb | k) != 0 ? 1u : 0u;
          tc_mma_pair_lo(tmem_base, a_lo + k * 2, b_lo + k * 2, desc_hi, idesc, accum);
          tc_mma_pair_lo(tmem_base + (uint32_t)kPairN, a_lo + (kPairATile >> 4) + k * 2, b_lo + k * 2, desc_hi, idesc,
                         accum);
        }
        tc_commit_pair(smem_u32(&ctl->empty[stage]), 3u);
        a_lo += ring_step;
        b_lo += ring_step;
        if (++stage == kPairStages) {
          stage = 0;
          phase ^= 1u;
          a_lo = a_lo0;
          b_lo = b_lo0;
        }
      }
      if (ok) tc_commit_pair(smem_u32(&ctl->tmem_full), 3u);
    }
  } else if (warp < kPairEpiWarps) {
    // ------------------------------------------------------------ epilogue (both CTAs)
    // warp w: TMEM lane quarter w mod 4 (32 of the CTA's 128 rows), every fourth 16-column chunk
    if (gathers && !grp.withhold_loads) {
      // These warps have nothing to do until the first item's MMAs are through: they copy the token
      // rows of the tiles the first wave of items reads (one row per warp at a time, plain loads and
      // stores), so that wave waits a few microseconds instead of for the gathering threads' ring.
      const uint32_t row_bytes = (uint32_t)H * 2u;
      const uint32_t chunks = (row_bytes + kRowChunk - 1) / kRowChunk;
      const int W = (int)gridDim.x * kPairEpiWarps, w = (int)blockIdx.x * kPairEpiWarps + warp;
      int before = 0;  // rows of the experts before g
      for (int g = 0; g < grp.n && ctl->tile_prefix[g] < first_tiles; ++g) {
        const int rows = min(ctl->count[g], (first_tiles - ctl->tile_prefix[g]) * kPairN);
        for (int r = ((w - before) % W + W) % W; r < rows; r += W) {
          const int row = ctl->row_start[g] + r;
          const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(tok.x) +
                                                            (size_t)(__ldg(tok.perm + row) / tok.K) * row_bytes);
          uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(tok.xp) + (size_t)row * row_bytes);
          const int n16 = (int)(row_bytes >> 4);
          for (int i0 = lane; i0 < n16; i0 += 32 * 8) {
            uint4 v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (i0 + 32 * j < n16) v[j] = __ldg(src + i0 + 32 * j);
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (i0 + 32 * j < n16) dst[i0 + 32 * j] = v[j];
          }
          // visible device-wide and to the async proxy of the items' copies, then counted
          __threadfence();
          asm volatile("fence.proxy.async;" ::: "memory");
          __syncwarp();
          if (lane == 0) atomicAdd(tok.ready + ctl->tile_prefix[g] + r / kPairN, chunks);
        }
        before += ctl->count[g];
      }
    }
    int local = 0;
    PairCursor cur;
    const int quarter = warp & 3, part = warp >> 2;
    for (;; ++local) {
      int item = 0;
      if (lane == 0) item = take_pair_item(ctl, local, abort_flag, status);
      item = __shfl_sync(0xffffffffu, item, 0);
      if (item < 0) break;
      PairItem it;
      pair_decode(ctl, grp, item, plan, cur, it);
      int ready = 0;
      if (lane == 0) ready = mbar_wait(smem_u32(&ctl->tmem_full), (uint32_t)local & 1u, abort_flag, status) ? 1 : 0;
      ready = __shfl_sync(0xffffffffu, ready, 0);
      if (!ready) break;
      tc_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
      const int n_mma = max(32, (it.valid + 31) & ~31);
      const int col = it.m0 + (int)rank * (it.kind == 1 ? 128 : 256) + quarter * 32 + lane;  // feature / output row of this thread
      void* const out_y = fused ? sec.out2 : out_ptr;
      // The warp's chunks, one in registers while the next one's TMEM loads are in flight; the
      // accumulators are handed back as soon as the LAST chunk has been read - its arithmetic and
      // stores run while the MMAs of the next item already write the columns.
      constexpr int kStep = 16 * (kPairEpiWarps / 4);
      uint32_t na[16], nb[16];
      int c = part * 16;
      if (c < n_mma) {
        tmem_ld16(t_row + (uint32_t)c, na);
        tmem_ld16(t_row + (uint32_t)(kPairN + c), nb);
      }
      bool released = false;
      for (; c < n_mma; c += kStep) {
        uint32_t ra[16], rb[16];
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          ra[j] = na[j];
          rb[j] = nb[j];
        }
        if (c + kStep < n_mma) {
          tmem_ld16(t_row + (uint32_t)(c + kStep), na);
          tmem_ld16(t_row + (uint32_t)(kPairN + c + kStep), nb);
        } else {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(tmem_empty_on_first);
          released = true;
        }
        const bool whole = c + 16 <= it.valid;  // no ragged end inside this chunk
        if (it.kind == 1) {
          uint16_t* p = reinterpret_cast<uint16_t*>(out_ptr) + (size_t)(it.row0 + c) * I + col;
#pragma unroll
          for (int j = 0; j < 16; ++j, p += I)
            if (whole || c + j < it.valid) {
              const float a = __uint_as_float(ra[j]);
              const float hm = __fdividef(a, 1.0f + __expf(-a)) * __uint_as_float(rb[j]);
              const __nv_bfloat16 b = __float2bfloat16_rn(hm);
              *p = *reinterpret_cast<const uint16_t*>(&b);
            }
        } else if (out_bf16) {  // many-token steps keep y in bf16
          uint16_t* p = reinterpret_cast<uint16_t*>(out_y) + (size_t)(it.row0 + c) * H + col;
#pragma unroll
          for (int j = 0; j < 16; ++j, p += H)
            if (whole || c + j < it.valid) {
              const __nv_bfloat16 b0 = __float2bfloat16_rn(__uint_as_float(ra[j]));
              const __nv_bfloat16 b1 = __float2bfloat16_rn(__uint_as_float(rb[j]));
              p[0] = *reinterpret_cast<const uint16_t*>(&b0);
              p[128] = *reinterpret_cast<const uint16_t*>(&b1);
            }
        } else {
          float* p = reinterpret_cast<float*>(out_y) + (size_t)(it.row0 + c) * H + col;
#pragma unroll
          for (int j = 0; j < 16; ++j, p += H)
            if (whole || c + j < it.valid) {
              p[0] = __uint_as_float(ra[j]);
              p[128] = __uint_as_float(rb[j]);
            }
        }
      }
      if (!released) {  // (a warp without a chunk in this item)
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(tmem_empty_on_first);
      }
      if (fused && it.kind == 1) {
        // this warp's intermediate rows of the item are stored: visible device-wide (and to the
        // async proxy of the down items' copies), then counted
        __threadfence();
        asm volatile("fence.proxy.async;" ::: "memory");
        __syncwarp();
        if (lane == 0) atomicAdd(sec.done + it.g, 1u);
      }
    }
  }

  // ---- teardown: nobody leaves while the partner may still read this CTA's shared memory or
  // arrive on its barriers
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == kPairMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
  if (threadIdx.x == 0) timeline_end(timeline, timeline_slot);
}

}  // namespace

bool ffn_pair_usable(const FfnTcMaps& maps, int n_box, int H, int I) {
  return !maps.fp8 && n_box == kPairN && I % 256 == 0 && H % 512 == 0;
}

int launch_ffn_pair(cudaStream_t st, const FfnTcMaps& maps, const FfnGroup& grp, int kind, const int32_t* offsets,
                    uint16_t* hbuf, float* y, int y_bf16, int H, int I, int n_sms, uint32_t* status,
                    uint32_t* work_counter, StepTimeline* timeline, int timeline_slot, const RouteReport& report,
                    uint32_t* done) {
  static bool attr_done = false;
  if (!attr_done) {
    if (cudaFuncSetAttribute(ffn_pair_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmem) != cudaSuccess ||
        cudaFuncSetAttribute(ffn_pair_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmem) != cudaSuccess ||
        cudaFuncSetAttribute(ffn_pair_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmem) != cudaSuccess)
      return OLED_ERR_CUDA;
    attr_done = true;
  }
  const int grid = 2 * (n_sms / 2);  // one CTA per SM, in pairs
  cudaError_t err;
  PairSecond sec;
  sec.tm_w2 = maps.w2;
  sec.tm_act2 = maps.hbuf[3];
  sec.out2 = y;
  sec.done = done;
  PairTokens tok;
  const bool gathers = kind != 2 && maps.token_source.perm != nullptr;
  tok.x = maps.token_source.x;
  tok.xp = maps.token_source.xp;
  tok.perm = gathers ? maps.token_source.perm : nullptr;
  tok.ready = maps.token_source.ready;
  tok.K = maps.token_source.K;
  if (gathers && tok.ready == nullptr) return OLED_ERR_INVALID_ARG;
  if (kind == 3) {
    if (done == nullptr) return OLED_ERR_INVALID_ARG;
    err = launch_pdl(ffn_pair_kernel<3>, dim3(grid), dim3(kPairThreads), kPairSmem, st, maps.w13, maps.xp[3], grp, offsets,
                     (void*)hbuf, H, I, y_bf16, status, work_counter, timeline, timeline_slot, report, sec, tok);
  } else if (kind == 1)
    err = launch_pdl(ffn_pair_kernel<1>, dim3(grid), dim3(kPairThreads), kPairSmem, st, maps.w13, maps.xp[3], grp, offsets,
                     (void*)hbuf, H, I, 0, status, work_counter, timeline, timeline_slot, report, sec, tok);
  else
    err = launch_pdl(ffn_pair_kernel<2>, dim3(grid), dim3(kPairThreads), kPairSmem, st, maps.w2, maps.hbuf[3], grp,
                     offsets, (void*)y, H, I, y_bf16, status, work_counter, timeline, timeline_slot, RouteReport{}, sec, tok);
  return err == cudaSuccess ? OLED_OK : OLED_ERR_CUDA;
}

}  // namespace oled
