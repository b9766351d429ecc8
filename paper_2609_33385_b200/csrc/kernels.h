// Launch wrappers of the CUDA kernels of the denoise step (internal to the library).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstddef>
#include <cstdint>
#include <utility>

#include "../../include/oled.h"

namespace oled {

// ---- programmatic dependent launch ----------------------------------------------------------
// Every kernel of a step is launched with programmatic stream serialization: it may be scheduled
// while its predecessor drains, does its data-independent prologue, then blocks in
// griddep_wait() until the predecessor has completed and its writes are visible.  Every kernel
// executes griddep_wait() before touching global data, so dependencies hold transitively.
#ifdef __CUDACC__
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif
bool pdl_enabled();            // attribute on?
void pdl_set_step(bool on);    // per step and thread: used for small steps only (it costs ~2 % on many-token steps)
void pdl_set_allowed(bool on); // process-wide switch (OLED_OPT_PDL)

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---- device-side timeline (OLED_OPT_TIMELINE) ------------------------------------------------
// Per kernel slot of a step: the earliest time a CTA entered the kernel, the earliest time one got
// past its dependency wait, and the latest time one finished (GPU global timer, nanoseconds).
constexpr int kTimelineSlots = 12;   // 0 gate, 1 permutation, 2 gather, 3..10 FFN launches, 11 combine
struct StepTimeline {
  unsigned long long entry_min[kTimelineSlots];
  unsigned long long start_min[kTimelineSlots];
  unsigned long long end_max[kTimelineSlots];
};
#ifdef __CUDACC__
__device__ __forceinline__ unsigned long long timeline_now() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// called by one thread per CTA; tl == nullptr: tracing off
__device__ __forceinline__ void timeline_entry(StepTimeline* tl, int slot) {
  if (tl) atomicMin(&tl->entry_min[slot], timeline_now());
}
__device__ __forceinline__ void timeline_start(StepTimeline* tl, int slot) {
  if (tl) atomicMin(&tl->start_min[slot], timeline_now());
}
__device__ __forceinline__ void timeline_end(StepTimeline* tl, int slot) {
  if (tl) atomicMax(&tl->end_max[slot], timeline_now());
}
#endif

// The experts one FFN launch works on and the slot each one's weights sit in: the per-launch
// image of the expert->slot indirection table, passed by value in kernel-parameter space.
struct FfnGroup {
  int32_t n;
  int32_t n_box;  // token rows per TMA box / MMA N tile of this launch
  int32_t withhold_loads;  // test aid: the producer issues nothing, the consumers' waits run out
  int32_t pad;             // tuning aid: cap on the fp8 converter groups (0 = default)
  uint16_t expert[OLED_MAX_EXPERTS];
  uint16_t slot[OLED_MAX_EXPERTS];
};

// Device status word values (0 = ok).
enum : uint32_t { kStatusOk = 0, kStatusWaitTimeout = 1 };
// The context's status block (device words): a bounded wait that ran out; flags and smallest
// offending index of the self-check; one bit per scratch buffer whose guard words were overwritten.
enum : int { kStatusWait = 0, kStatusCheckFlags = 1, kStatusCheckIndex = 2, kStatusGuardMask = 3, kStatusWords = 4 };
constexpr uint32_t kStatusNoIndex = 0x7fffffffu;  // initial value of the index word

// Guard words behind the step's scratch buffers (checked when OLED_OPT_SELF_CHECK is on).
constexpr int kGuardWords = 16;
constexpr uint32_t kGuardPattern = 0xC0DEC0DEu;
struct GuardList {
  int n;
  uint32_t* words[12];
};

// Where a step's counts and scores are published for the host: mapped pinned host memory, one
// 8-byte word per value with the step's sequence number in the upper bits (scores: seq & 0xffff
// in bits 48..63; counts: seq in bits 32..63), so the host can tell word by word that the data is
// there: no ticket, no fence, no copy, no event.  The writer is a kernel that runs after the gate
// kernel has completed (counts and scores are final then) and that does NOT stand between the
// gate and the expert FFN: a kernel's completion waits for its writes to host memory to be
// acknowledged across the link (~4 us), so the report leaves from the first CTA of the step's
// first FFN launch - a kernel that runs for tens of microseconds anyway - or, in a step whose
// layer has no resident expert yet, from a one-CTA kernel of its own.  host_scores == nullptr:
// no report.
struct RouteReport {
  unsigned long long* host_scores = nullptr;    // mapped host [E]
  unsigned long long* host_counts = nullptr;    // mapped host [E]
  unsigned int seq = 0;
  const int32_t* counts = nullptr;              // device [E], final
  const unsigned long long* scores = nullptr;   // device [E], final
  int n_experts = 0;
  StepTimeline* timeline = nullptr;             // device, or null
};
#ifdef __CUDACC__
// Executed by `n_threads` threads with ranks 0..n_threads-1.
__device__ __forceinline__ void publish_report(const RouteReport& rep, int rank, int n_threads) {
  if (rep.host_scores == nullptr) return;
  const unsigned long long tag16 = (unsigned long long)(rep.seq & 0xffffu) << 48;
  const unsigned long long tag32 = (unsigned long long)rep.seq << 32;
  for (int e = rank; e < rep.n_experts; e += n_threads) {
    // score < 2^48 (at most 2^16 tokens of at most 2^32 each); masked so that no data can spoil the tag
    rep.host_scores[e] = tag16 | (rep.scores[e] & 0xffffffffffffull);
    rep.host_counts[e] = tag32 | (unsigned long long)(uint32_t)rep.counts[e];
  }
}
#endif
void launch_report(cudaStream_t st, const RouteReport& rep);  // the one-CTA kernel (route.cu)

// ---- route.cu -------------------------------------------------------------------------
// Gate logits in the contract order, top-k (ties to the lower index), softmax over the selected
// logits, per-expert counts and integer reuse-score numerators (atomics on zeroed arrays).
// A layer's combine handed to the next layer's gate kernel (few-token steps inside a stack
// iteration): out = bf16(sum_j gate[t,j] * y[pos[t*K+j],:]) in rank order, x_next = bf16(x + out),
// and x_next is the gate kernel's input.  y == nullptr: nothing to carry out.
struct CombinePrev {
  const float* y = nullptr;        // [T*K,H] fp32 per-assignment outputs of the previous layer
  const float* gate = nullptr;     // [T,K]   its gate scores
  const int32_t* pos = nullptr;    // [T*K]   its inverse permutation
  const uint16_t* x = nullptr;     // [T,H]   its input
  uint16_t* out = nullptr;         // [T,H]   its MoE output
  uint16_t* x_next = nullptr;      // [T,H]   its input plus its output
  int K = 0;
  uint32_t* zero_words = nullptr;  // the control block the previous step used, cleared by CTA 0
  int n_zero_words = 0;
};
// seg_counts (many-token steps; nullptr: none): ZERO words [kPermuteSegments][E]; the kernel also
// counts every expert's assignments per segment of seg_tokens consecutive tokens, so that the
// permutation kernel can work on the segments in parallel.
constexpr int kPermuteSegments = 16;
void launch_route(cudaStream_t st, const uint16_t* x, const uint16_t* w_router, const float* bias,
                  const float* conf, int T, int H, int E, int K, float* logits, int32_t* ids,
                  float* gate, int32_t* counts, unsigned long long* scores, const CombinePrev& prev,
                  StepTimeline* timeline, int32_t* seg_counts = nullptr, int seg_tokens = 0);
bool route_can_take_combine(int T);  // does the gate kernel of a T-token step carry out a CombinePrev?
// fp8 expert stores, direct form: the two token operands of a step's expert FFN - the gathered
// input rows and the intermediate rows - as sums of two e4m3 terms each, after scaling every row
// by a power of two taken from its largest magnitude (fp8_split.h).  The magnitudes are kept as the
// bit pattern of a non-negative fp32, so that an unsigned integer maximum orders them.
//   amax_in, terms_in:   written by the gathering permutation kernel, which also zeroes amax_mid
//   amax_mid:            raised with atomicMax by the gate/up epilogue
//   terms_mid:           written by the split kernel between the two projections
struct TokenSplit {
  uint32_t* amax_in = nullptr;   // [rows]
  uint32_t* amax_mid = nullptr;  // [rows]
  uint8_t* terms_in = nullptr;   // [2][rows][H] e4m3 codes: term 1 of every row, then term 2
  uint8_t* terms_mid = nullptr;  // [2][rows][I]
  int rows = 0;                  // rows of the buffers above (tokens x top-k of the context)
  bool complete() const { return amax_in && amax_mid && terms_in && terms_mid && rows > 0; }
};
// Offsets (exclusive scan), stable permutation by expert and its inverse.  With xp != nullptr the
// kernel also gathers the token rows (xp[r,:] = x[perm[r]/K,:]); meant for small steps.
// seg_counts (launches that do not gather; nullptr: none): the gate kernel's per-segment counts (see
// launch_route): kPermuteSegments CTAs per expert then scan one segment of the assignment list each.
// split (gathering launches only; nullptr: none): the kernel also writes, per sorted row, the
// largest magnitude of the row it copied and the row's two e4m3 terms, and zeroes amax_mid (see
// TokenSplit).
void launch_permute(cudaStream_t st, const int32_t* ids, const int32_t* counts, int T, int E, int K,
                    int32_t* offsets, int32_t* perm, int32_t* pos, const uint16_t* x, uint16_t* xp, int H,
                    StepTimeline* timeline, const TokenSplit* split = nullptr, const int32_t* seg_counts = nullptr,
                    int seg_tokens = 0);
// xp[r,:] = x[perm[r] / K, :] for the T*K sorted rows.
void launch_gather(cudaStream_t st, const uint16_t* x, const int32_t* perm, int T, int H, int K,
                   uint16_t* xp);

// Calls the first `bytes_per_slot` bytes of the listed slots of the pool into L2 (prefetch only:
// nothing is read into registers, nothing waits).  combine.cu.
struct SlotList {
  int32_t n;
  uint16_t slot[OLED_MAX_EXPERTS];
};
void launch_l2_prefetch(cudaStream_t st, const uint8_t* pool, size_t slot_bytes, const SlotList& slots,
                        size_t bytes_per_slot);

// ---- combine.cu -----------------------------------------------------------------------
// out[t,:] = bf16( sum_j gate[t,j] * y[pos[t*K+j],:] ), j ascending, fp32 accumulation.  With
// x_next != nullptr also x_next[t,:] = bf16(x[t,:] + out[t,:]) (the residual between layers).
// zero_words != nullptr: CTA 0 also clears n_zero_words 32-bit words there (the step's control
// block, ready for the next step's atomics).
// y_bf16 != 0: y holds bf16 rows (many-token steps) instead of fp32.
void launch_combine(cudaStream_t st, const float* y, int y_bf16, const float* gate, const int32_t* pos, int T,
                    int H, int K, uint16_t* out, const uint16_t* x, uint16_t* x_next,
                    uint32_t* zero_words, int n_zero_words, StepTimeline* timeline = nullptr);
void launch_residual_add(cudaStream_t st, const uint16_t* x, const uint16_t* r, uint16_t* y, size_t n);

// ---- ffn_simple.cu (bring-up path, plain FMA) ---------------------------------------------
void launch_ffn_simple(cudaStream_t st, const FfnGroup& grp, const uint8_t* pool, size_t slot_bytes,
                       const int32_t* offsets, const uint16_t* xp, uint16_t* hbuf, float* y, int H,
                       int I);

// ---- ffn_tc.cu (tcgen05 / TMEM / TMA) ------------------------------------------------------
struct FfnTcMaps {
  CUtensorMap w13_half_e4m3;  // fp8 stores: [slots][2][I][H] bytes, box {128,64,2,1}, 128-byte swizzle
  CUtensorMap w2_e4m3;        // fp8 stores: [slots][H][I] bytes, box {128,128,1}, 128-byte swizzle
  CUtensorMap xp_terms[2];    // [2][rows][H] bytes (TokenSplit::terms_in), box {128, 16<<i, 2}
  CUtensorMap hbuf_terms[2];  // [2][rows][I] bytes (TokenSplit::terms_mid), box {128, 16<<i, 2}
  bool e4m3_direct = false;   // the maps above exist (fp8 stores, H and I multiples of 128, term buffers given)
  CUtensorMap w13;       // [slots][2I][H] bf16, box {64,128,1}
  CUtensorMap w13_half;  // the same, box {64,64,1}
  CUtensorMap w2;        // [slots][H][I]  bf16, box {64,128,1}
  CUtensorMap xp[5];     // [rows][H] bf16, box {64, 16<<i}
  CUtensorMap hbuf[5];   // [rows][I] bf16, box {64, 16<<i}
  bool fp8 = false;      // slots hold fp8 blobs: the weight maps are byte maps over the e4m3 codes
  bool use_pairs = true; // token tiles of 256 rows go to the CTA-pair kernel where it applies (OLED_OPT_FFN_PAIRS)
  // The step made no gathered copy of the token rows (ffn_tc_set_token_source; perm == nullptr: it
  // did): every gate/up launch copies its own experts' rows into xp while it runs (sorted row r is
  // row perm[r] / K of x; CTA-pair kernel only).  Should a pair launch be refused, the gather kernel
  // fills xp after all and the source is dropped.
  struct TokenSource {
    const int32_t* perm = nullptr;
    int K = 0, T = 0;
    const uint16_t* x = nullptr;
    uint16_t* xp = nullptr;
    uint32_t* ready = nullptr;  // per launch: one ZERO word per token tile of 256 rows (at most rows / 256 + experts)
  };
  mutable TokenSource token_source;
  const uint8_t* pool = nullptr;
  size_t slot_bytes = 0;
};
// Builds the tensor maps; returns 0 or a negative oled_status.
int ffn_tc_setup(FfnTcMaps* maps, const uint8_t* pool, size_t slot_bytes, int n_slots, int H, int I, bool fp8,
                 const uint16_t* xp, const uint16_t* hbuf, int rows, const TokenSplit* split = nullptr);
// kind 1: gate/up + SwiGLU into hbuf; kind 2: down projection into y; kind 3: both in one launch
// (bf16 stores and token tiles of at most 32 rows only: ask ffn_tc_can_fuse; `done` then points at
// one ZERO word per expert of the group).  One launch each.
// work_counter: a device word that is ZERO when the kernel starts; its CTAs draw their work items
// from it (every launch that can be in flight at the same time needs a word of its own).
// report (kinds 1 and 3; host_scores == nullptr: none): the kernel's first CTA publishes the step's
// counts and scores to the host.
// behind_event_wait: the launch follows a cudaStreamWaitEvent (with, for kind 2, at most its own
// kind 1 launch in between), i.e. everything enqueued before that wait has completed.
// split (fp8 stores; nullptr: none): the token operands as e4m3 terms.  With them, token tiles of
// at most 32 rows take the form whose MMAs read the experts' e4m3 codes as they are; a kind 2
// launch is then preceded by the split kernel (ffn_tc_launches tells how many launches a call makes).
int launch_ffn_tc(cudaStream_t st, const FfnTcMaps& maps, const FfnGroup& grp, int max_count, int kind,
                  const int32_t* host_counts, const int32_t* offsets, uint16_t* hbuf, float* y, int y_bf16, int H,
                  int I, int n_sms, uint32_t* status, uint32_t* work_counter, bool behind_event_wait,
                  StepTimeline* timeline, int timeline_slot, const RouteReport& report, uint32_t* done = nullptr,
                  const TokenSplit* split = nullptr);
int ffn_tc_launches(const FfnTcMaps& maps, int max_count, int kind, const TokenSplit* split);
// No gathered copy of the step's token rows exists: every FFN launch until
// ffn_tc_clear_token_source must be one the CTA-pair kernel takes (token tile 256), and each gets
// maps->token_source.ready set to zeroed words of its own.
bool ffn_tc_token_source_usable(const FfnTcMaps& maps, int H, int I);
void ffn_tc_set_token_source(FfnTcMaps* maps, const uint16_t* x, int T, const int32_t* perm, int K, uint16_t* xp);
void ffn_tc_clear_token_source(FfnTcMaps* maps);
bool ffn_tc_can_fuse(const FfnTcMaps& maps, int max_count);
bool ffn_pair_can_fuse(const FfnTcMaps& maps, int max_count, int H, int I);  // kind 3 on CTA pairs
// ---- ffn_pair.cu: the many-token form on CTA pairs (bf16 stores, token tiles of 256 rows,
// intermediate a multiple of 256 and hidden a multiple of 512); kinds 1 and 2 as above, kind 3 both
// in one launch (`done`: one ZERO word per expert of the group).
bool ffn_pair_usable(const FfnTcMaps& maps, int n_box, int H, int I);
int launch_ffn_pair(cudaStream_t st, const FfnTcMaps& maps, const FfnGroup& grp, int kind, const int32_t* offsets,
                    uint16_t* hbuf, float* y, int y_bf16, int H, int I, int n_sms, uint32_t* status,
                    uint32_t* work_counter, StepTimeline* timeline, int timeline_slot, const RouteReport& report,
                    uint32_t* done = nullptr);
constexpr int kFfnWorkCounters = 8;  // FFN launches of one layer execution: 3 groups x 2 kinds, rounded up

// Self-check (check.cu): invariants of the routing and the permutation, guard words.
void launch_self_check(cudaStream_t st, const int32_t* ids, const int32_t* counts, const int32_t* offsets,
                       const int32_t* perm, const int32_t* pos, int T, int E, int K, uint32_t* status);
void launch_guard_check(cudaStream_t st, const GuardList& guards, uint32_t* status);
void launch_guard_fill(cudaStream_t st, const GuardList& guards);
void launch_corrupt_perm(cudaStream_t st, int32_t* perm, int n);  // test aid

}  // namespace oled
