// C ABI of the MoE denoise-step library: context, host expert store, the per-step
// orchestration (gate -> policy -> fills on a side stream -> grouped FFN -> combine) and the
// counters.  The flow follows the paper's per-layer order (Sec. 4.1) with the sets of Sec. 4.2
// and the retention rule of Sec. 4.2/4.3; every missed expert is fetched (no CPU execution).
#include <atomic>
#include <chrono>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <memory>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "kernels.h"
#include "policy.h"

using namespace oled;

namespace {

struct LayerData {
  LayerCacheState cache;
  int32_t last_active = -1;      // experts activated at the layer's previous execution (-1: none yet)
  int32_t last_max_count = -1;   // most token rows any expert received then
  int32_t last_misses = -1;      // its misses
  std::vector<int32_t> last_counts;  // its per-expert row counts
  const uint8_t* host_blob = nullptr;
  size_t host_stride = 0;
  uint16_t* w_router = nullptr;  // device [E,H]
  float* bias = nullptr;         // device [E] or null
  bool has_router = false;
  oled_stats_t stats{};
};

}  // namespace

struct oled_ctx {
  oled_model_shape shape{};
  cudaStream_t stream = nullptr;       // caller's
  cudaStream_t copy_stream = nullptr;  // expert fills
  std::vector<cudaEvent_t> fill_events;
  cudaEvent_t gate_event = nullptr;
  int n_sms = 148;
  size_t slot_bytes = 0;
  int n_slots = 0;
  uint8_t* pool = nullptr;
  SlotPool slots;
  std::vector<LayerData> layers;
  StepPlan plan;

  // scratch (device)
  // The step's control block (scores, counts, work-item counters of its FFN launches), all zero
  // when a step starts.  There are two, used by alternate steps: the kernel that clears a block -
  // the step's combine or, when that has been left to it, the next step's gate kernel - runs
  // after everything that used the block and never while the current step's atomics land in it.
  uint8_t* d_ctrl[2] = {nullptr, nullptr};
  int ctrl_sel = 0;
  unsigned long long* d_scores = nullptr;  // [E]   } the current step's block
  int32_t* d_counts = nullptr;             // [E]   }
  size_t ctrl_bytes = 0;
  float* d_logits = nullptr;   // [T,E]
  int32_t* d_ids = nullptr;    // [T,k]
  float* d_gate = nullptr;     // [T,k]  (the current step's of the two buffers below)
  float* d_gate_buf[2] = {nullptr, nullptr};
  int32_t* d_pos_buf[2] = {nullptr, nullptr};
  int buf_sel = 0;
  // a layer's combine that has been left to the next layer's gate kernel (few-token steps inside
  // oled_denoise_iteration): what that kernel, or a stand-alone combine, needs to carry it out
  struct PendingCombine {
    bool valid = false;
    int T = 0;
    const float* gate = nullptr;
    const int32_t* pos = nullptr;
    const uint16_t* x = nullptr;
    uint16_t* out = nullptr;
    uint16_t* x_next = nullptr;
    uint32_t* ctrl = nullptr;      // the control block that step used (to be cleared)
  } pending;
  int fuse_ffn = 1;            // OLED_OPT_FUSE_FFN: 0 never, 1 where few items per SM are expected, 2 wherever possible
  bool fuse_combine = true;    // stack iterations of few-token steps: a layer's combine runs inside the
                               // next layer's gate kernel (OLED_OPT_FUSE_COMBINE)
  int32_t* d_offsets = nullptr;// [E+1]
  int32_t* d_perm = nullptr;   // [T*k]
  int32_t* d_pos = nullptr;    // [T*k]
  uint16_t* d_xp = nullptr;    // [T*k,H]
  uint16_t* d_hbuf = nullptr;  // [T*k,I]
  TokenSplit split;            // fp8 stores: the FFN's token operands as e4m3 terms (see TokenSplit)
  const TokenSplit* step_split = nullptr;  // &split in steps whose permutation kernel fills it
  float* d_y = nullptr;        // [T*k,H]
  uint32_t* d_status = nullptr;
  uint32_t* d_work = nullptr;         // control block: work-item counters of the step's FFN launches
  uint32_t* d_done = nullptr;         // control block: [kFfnWorkCounters][E] completion counters of fused FFN launches
  uint32_t* d_ready = nullptr;        // control block: [kFfnWorkCounters][ready_words] row-copy counters of FFN launches that gather
  size_t ready_words = 0;             // token tiles of 256 rows a launch can have: max_tokens * K / 256 + E
  int32_t* d_seg = nullptr;           // control block, last: [kPermuteSegments][E] per-segment counts of many-token steps
  int work_next = 0;                  // next unused counter of the current layer execution
  bool ctrl_dirty = true;             // both control blocks must be cleared before the next gate launch
  unsigned int seq = 0;               // step sequence number echoed by the gate kernel
  volatile unsigned long long* h_report = nullptr;  // pinned, mapped: tagged scores [E] | tagged counts [E]
  std::vector<unsigned long long> host_scores;       // decoded copy of the last report
  std::vector<int32_t> host_counts;
  uint16_t* d_hidden_stage = nullptr;  // for the host-buffer entry point
  float* d_conf_stage = nullptr;
  uint16_t* d_out_stage = nullptr;
  uint16_t* d_iter[2] = {nullptr, nullptr};  // ping-pong hidden states of the stack iteration
  // pinned host mirror of the control block
  uint8_t* h_ctrl = nullptr;
  uint32_t* h_status = nullptr;

  FfnTcMaps maps;
  // optional per-kernel timing with CUDA events on the context's stream
  bool profile = false;
  struct ProfRec { int kernel; cudaEvent_t a, b; };
  std::vector<ProfRec> prof_pending;
  std::vector<cudaEvent_t> prof_free;
  oled_kernel_profile prof_acc[OLED_N_KERNELS] = {};
  int ffn_impl = 0;
  bool timeline_on = false;    // OLED_OPT_TIMELINE
  bool fp8_direct = true;      // OLED_OPT_FP8_DIRECT
  int l2_prefetch = 1;         // OLED_OPT_L2_PREFETCH (2: whatever the length of the expert stream)
  bool gather_in_ffn = true;   // OLED_OPT_GATHER_IN_FFN
  cudaEvent_t ev_layer_done = nullptr;  // recorded behind a layer's last kernel (L2 prefetch of the next layer)
  StepTimeline* d_timeline = nullptr;
  bool y_bf16 = false;         // this step keeps the per-assignment outputs in bf16 (many tokens)
  bool hit_fused = false;      // this step's resident-group FFN ran as one fused launch
  int miss_chunk = 4;
  bool split_last = true;      // the step's last blob is copied in two parts (gate|up first, down after)
  int withhold_loads = 0;      // test aid, see OLED_OPT_TEST_WITHHOLD_LOADS
  int self_check = 0;          // OLED_OPT_SELF_CHECK
  int corrupt_perm = 0;        // test aid, see OLED_OPT_TEST_CORRUPT_PERM
  GuardList guards{};          // guard words behind the step's scratch buffers
  uint64_t policy_ns = 0, policy_runs = 0;
  long long total_capacity = 0;
  int adapt_lo = 1;            // smallest capacity layer-adaptive sizing may hand out (see pool_plan)
  int adapt_period = 0;        // iterations between automatic capacity refreshes (0 = off)
  uint64_t iterations = 0;     // oled_denoise_iteration() calls so far
  uint64_t launches = 0;
  int last_cuda_error = 0;
  int last_layer = -1;
  int last_tokens = 0;
  std::vector<uint8_t> last_before, last_after;
};

namespace {

#define OLED_CUDA(ctx, call)                      \
  do {                                            \
    cudaError_t err__ = (call);                   \
    if (err__ != cudaSuccess) {                   \
      (ctx)->last_cuda_error = (int)err__;        \
      return OLED_ERR_CUDA;                       \
    }                                             \
  } while (0)

void select_ctrl(oled_ctx* ctx, int sel) {
  const size_t E = (size_t)ctx->shape.n_experts;
  uint8_t* b = ctx->d_ctrl[sel];
  ctx->ctrl_sel = sel;
  ctx->d_scores = reinterpret_cast<unsigned long long*>(b);
  ctx->d_counts = reinterpret_cast<int32_t*>(b + E * sizeof(unsigned long long));
  ctx->d_work = reinterpret_cast<uint32_t*>(b + E * (sizeof(unsigned long long) + sizeof(int32_t)));
  ctx->d_done = ctx->d_work + kFfnWorkCounters;
  ctx->d_ready = ctx->d_done + (size_t)kFfnWorkCounters * E;
  ctx->d_seg = reinterpret_cast<int32_t*>(ctx->d_ready + (size_t)kFfnWorkCounters * ctx->ready_words);
}

template <typename T>
int dev_alloc(oled_ctx* ctx, T** p, size_t n) {
  void* q = nullptr;
  cudaError_t err = cudaMalloc(&q, std::max<size_t>(n, 1) * sizeof(T));
  if (err != cudaSuccess) {
    ctx->last_cuda_error = (int)err;
    cudaGetLastError();
    return OLED_ERR_OOM;
  }
  *p = static_cast<T*>(q);
  return OLED_OK;
}

// A scratch buffer of n elements followed by guard words (16-byte aligned), which the self-check
// verifies after every step: a kernel that writes past its buffer shows up there.
template <typename T>
int dev_alloc_guarded(oled_ctx* ctx, T** p, size_t n) {
  const size_t bytes = (std::max<size_t>(n, 1) * sizeof(T) + 15) / 16 * 16;
  uint8_t* q = nullptr;
  const int rc = dev_alloc(ctx, &q, bytes + kGuardWords * sizeof(uint32_t));
  if (rc != OLED_OK) return rc;
  *p = reinterpret_cast<T*>(q);
  if (ctx->guards.n < (int)(sizeof(ctx->guards.words) / sizeof(ctx->guards.words[0])))
    ctx->guards.words[ctx->guards.n++] = reinterpret_cast<uint32_t*>(q + bytes);
  return OLED_OK;
}

inline bool misaligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }

int check_status(oled_ctx* ctx) {
  if (!ctx->h_status) return OLED_OK;
  if (ctx->h_status[kStatusWait] != kStatusOk) return OLED_ERR_TIMEOUT;
  if (ctx->h_status[kStatusCheckFlags] != 0 || ctx->h_status[kStatusGuardMask] != 0) return OLED_ERR_SELF_CHECK;
  return OLED_OK;
}

// Carries out a combine that was left to the next layer's gate kernel and never got one.
int flush_pending_combine(oled_ctx* ctx) {
  if (!ctx->pending.valid) return OLED_OK;
  const auto& p = ctx->pending;
  launch_combine(ctx->stream, ctx->d_y, 0, p.gate, p.pos, p.T, ctx->shape.hidden, ctx->shape.top_k, p.out, p.x, p.x_next,
                 p.ctrl, (int)(ctx->ctrl_bytes / 4));
  ctx->pending.valid = false;
  ctx->launches += 1;
  OLED_CUDA(ctx, cudaGetLastError());
  return OLED_OK;
}

int sync_all(oled_ctx* ctx) {
  {
    const int rcp = flush_pending_combine(ctx);
    if (rcp != OLED_OK) return rcp;
  }
  OLED_CUDA(ctx, cudaStreamSynchronize(ctx->copy_stream));
  OLED_CUDA(ctx, cudaMemcpyAsync(ctx->h_status, ctx->d_status, kStatusWords * sizeof(uint32_t), cudaMemcpyDeviceToHost,
                                 ctx->stream));
  OLED_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  return check_status(ctx);
}

void free_ctx(oled_ctx* ctx) {
  if (!ctx) return;
  if (ctx->stream || ctx->copy_stream) cudaDeviceSynchronize();
  for (auto& l : ctx->layers) {
    cudaFree(l.w_router);
    cudaFree(l.bias);
  }
  cudaFree(ctx->pool);
  cudaFree(ctx->d_ctrl[0]);
  cudaFree(ctx->d_logits);
  cudaFree(ctx->d_ids);
  cudaFree(ctx->d_gate_buf[0]);
  cudaFree(ctx->d_gate_buf[1]);
  cudaFree(ctx->d_offsets);
  cudaFree(ctx->d_perm);
  cudaFree(ctx->d_pos_buf[0]);
  cudaFree(ctx->d_pos_buf[1]);
  cudaFree(ctx->d_xp);
  cudaFree(ctx->d_hbuf);
  cudaFree(ctx->split.amax_in);
  cudaFree(ctx->split.amax_mid);
  cudaFree(ctx->split.terms_in);
  cudaFree(ctx->split.terms_mid);
  cudaFree(ctx->d_y);
  cudaFree(ctx->d_status);
  cudaFree(ctx->d_timeline);
  cudaFree(ctx->d_hidden_stage);
  cudaFree(ctx->d_conf_stage);
  cudaFree(ctx->d_out_stage);
  cudaFree(ctx->d_iter[0]);
  cudaFree(ctx->d_iter[1]);
  if (ctx->h_ctrl) cudaFreeHost(ctx->h_ctrl);
  if (ctx->h_status) cudaFreeHost(ctx->h_status);
  for (auto ev : ctx->fill_events) cudaEventDestroy(ev);
  for (auto& r : ctx->prof_pending) {
    cudaEventDestroy(r.a);
    cudaEventDestroy(r.b);
  }
  for (auto ev : ctx->prof_free) cudaEventDestroy(ev);
  if (ctx->gate_event) cudaEventDestroy(ctx->gate_event);
  if (ctx->ev_layer_done) cudaEventDestroy(ctx->ev_layer_done);
  if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
  cudaGetLastError();
  delete ctx;
}

cudaEvent_t prof_event(oled_ctx* ctx) {
  if (!ctx->prof_free.empty()) {
    cudaEvent_t e = ctx->prof_free.back();
    ctx->prof_free.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  if (cudaEventCreate(&e) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  return e;
}

// NVTX range around one of the five parts of a step (host side; shows up in a timeline profiler
// next to the kernels it enqueues).  Only with OLED_OPT_PROFILE on; the header-only NVTX API is a
// no-op unless a tool is attached.
struct NvtxRange {
  bool on;
  NvtxRange(const oled_ctx* ctx, const char* name);
  void end() {
    if (on) nvtxRangePop();
    on = false;
  }
  ~NvtxRange() { end(); }
};

// Brackets one kernel launch with events when profiling is on.
struct ProfScope {
  oled_ctx* ctx;
  cudaEvent_t a = nullptr, b = nullptr;
  int kernel;
  ProfScope(oled_ctx* c, int k, uint64_t bytes, uint64_t flops) : ctx(c), kernel(k) {
    if (!ctx->profile) return;
    a = prof_event(ctx);
    b = prof_event(ctx);
    if (a && b) {
      cudaEventRecord(a, ctx->stream);
      ctx->prof_acc[k].launches += 1;
      ctx->prof_acc[k].bytes += bytes;
      ctx->prof_acc[k].flops += flops;
    }
  }
  ~ProfScope() {
    if (a && b) {
      cudaEventRecord(b, ctx->stream);
      ctx->prof_pending.push_back({kernel, a, b});
    }
  }
};

NvtxRange::NvtxRange(const oled_ctx* ctx, const char* name) : on(ctx->profile) {
  if (on) nvtxRangePushA(name);
}

void prof_resolve(oled_ctx* ctx) {
  for (auto& r : ctx->prof_pending) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, r.a, r.b) == cudaSuccess) ctx->prof_acc[r.kernel].ms += ms;
    ctx->prof_free.push_back(r.a);
    ctx->prof_free.push_back(r.b);
  }
  ctx->prof_pending.clear();
  cudaGetLastError();
}

void prof_add(oled_ctx* ctx, int kernel, uint64_t bytes, uint64_t flops) {
  if (!ctx->profile) return;
  ctx->prof_acc[kernel].bytes += bytes;
  ctx->prof_acc[kernel].flops += flops;
}

// Algorithmic bytes / flops of the two FFN kernels for n experts with `rows` token rows in total:
// each expert's weights once, the token rows in, the result rows out.
void prof_add_ffn(oled_ctx* ctx, uint64_t n, uint64_t rows, bool fused) {
  const uint64_t H = ctx->shape.hidden, I = ctx->shape.intermediate, hi = H * I;
  const bool fp8 = ctx->shape.expert_format == OLED_EXPERTS_FP8;
  // weight bytes of one expert per kernel: bf16 elements, or e4m3 codes plus the fp32 row scales
  const uint64_t w13 = fp8 ? 2 * hi + 2 * I * 4 : 2 * hi * 2, w2 = fp8 ? hi + H * 4 : hi * 2;
  const uint64_t b1 = n * w13 + rows * H * 2 + rows * I * 2, b2 = n * w2 + rows * I * 2 + rows * H * (ctx->y_bf16 ? 2 : 4);
  if (fused) {
    prof_add(ctx, OLED_KERNEL_FFN_FUSED, b1 + b2, 6 * rows * hi);
  } else {
    prof_add(ctx, OLED_KERNEL_FFN_GATE_UP, b1, 4 * rows * hi);
    prof_add(ctx, OLED_KERNEL_FFN_DOWN, b2, 2 * rows * hi);
  }
}

// The FFN launches over one group: gate/up and down projection, or ONE fused launch where that
// form exists (bf16 stores, token tiles of at most 32 rows, no event to wait for between the two
// projections) and few items per SM are expected (expected_experts: how many of the group's
// experts are expected to have tokens).  host_counts == nullptr: the per-expert counts are not
// known on the host yet (the group is the resident set and experts without tokens cost nothing).
// before_down: an event the down projection (and nothing before it) has to wait for, or null.
// behind_event_wait: the caller has just enqueued a cudaStreamWaitEvent on the stream.
// report: the step's report to the host, sent by the first launch (the plain-FMA bring-up path
// and an empty group send it from a kernel of its own).
int run_ffn_launches(oled_ctx* ctx, const FfnGroup& grp, int max_count, const int32_t* host_counts,
                     cudaEvent_t before_down, bool behind_event_wait, int expected_experts, bool* fused_out,
                     const RouteReport& report = RouteReport{}) {
  if (fused_out) *fused_out = false;
  if ((grp.n <= 0 || max_count <= 0 || ctx->ffn_impl == 1) && report.host_scores != nullptr) {
    launch_report(ctx->stream, report);
    ctx->launches += 1;
  }
  if (grp.n <= 0) return OLED_OK;
  const int H = ctx->shape.hidden, I = ctx->shape.intermediate;
  // (no gathered copy of the token rows exists: every launch of the step takes the token tile of 256
  // rows, whatever its experts' counts, and gathers its own rows)
  if (ctx->maps.token_source.perm != nullptr) max_count = std::max(max_count, 129);
  if (ctx->ffn_impl == 1) {
    if (before_down) OLED_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, before_down, 0));
    launch_ffn_simple(ctx->stream, grp, ctx->pool, ctx->slot_bytes, ctx->d_offsets, ctx->d_xp, ctx->d_hbuf,
                      ctx->d_y, H, I);
    ctx->launches += 2;
  } else {
    // With many items per SM the two-kernel form is a little faster (the down projection's early
    // start hides the boundary; measured 125 against 129 us for 63 experts); with few, the SMs
    // that run out of gate/up items would idle until the whole gate/up launch has finished.
    const bool few_items = (long long)expected_experts * (I / 64) < 4ll * ctx->n_sms;
    // Many-token tiles on CTA pairs: always one launch (a boundary between cluster kernels is a full stop).
    const bool fuse_pairs = before_down == nullptr && ctx->fuse_ffn != 0 && ffn_pair_can_fuse(ctx->maps, max_count, H, I);
    const bool fuse = fuse_pairs ||
                      (before_down == nullptr && !ctx->y_bf16 && ffn_tc_can_fuse(ctx->maps, max_count) &&
                       (ctx->fuse_ffn == 2 || (ctx->fuse_ffn == 1 && few_items)));
    for (int kind = fuse ? 3 : 1; kind <= (fuse ? 3 : 2); ++kind) {
      if (kind == 2 && before_down) OLED_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, before_down, 0));
      ProfScope ps(ctx, kind == 3 ? OLED_KERNEL_FFN_FUSED : kind == 1 ? OLED_KERNEL_FFN_GATE_UP : OLED_KERNEL_FFN_DOWN, 0, 0);
      // a fresh (zero) work counter and, for a fused launch, a fresh row of completion counters
      // per launch; a layer execution has at most three launch pairs, should there ever be more,
      // used words are cleared in stream order and taken again
      const int li = ctx->work_next % kFfnWorkCounters;
      uint32_t* work = ctx->d_work + li;
      uint32_t* done = ctx->d_done + (size_t)li * ctx->shape.n_experts;
      uint32_t* ready = ctx->d_ready + (size_t)li * ctx->ready_words;
      if (ctx->work_next >= kFfnWorkCounters) {
        OLED_CUDA(ctx, cudaMemsetAsync(work, 0, sizeof(uint32_t), ctx->stream));
        OLED_CUDA(ctx, cudaMemsetAsync(done, 0, (size_t)ctx->shape.n_experts * sizeof(uint32_t), ctx->stream));
        OLED_CUDA(ctx, cudaMemsetAsync(ready, 0, ctx->ready_words * sizeof(uint32_t), ctx->stream));
      }
      ctx->maps.token_source.ready = ready;
      ctx->work_next += 1;
      const int rc = launch_ffn_tc(ctx->stream, ctx->maps, grp, max_count, kind, host_counts, ctx->d_offsets,
                                   ctx->d_hbuf, ctx->d_y, ctx->y_bf16 ? 1 : 0, H, I, ctx->n_sms, ctx->d_status, work,
                                   behind_event_wait || (kind == 2 && before_down != nullptr),
                                   ctx->timeline_on ? ctx->d_timeline + ctx->last_layer : nullptr, 3 + li, report, done,
                                   ctx->step_split);
      if (rc != OLED_OK) return rc;
      ctx->launches += ffn_tc_launches(ctx->maps, max_count, kind, ctx->step_split);
    }
    if (fused_out) *fused_out = fuse;
  }
  OLED_CUDA(ctx, cudaGetLastError());
  return OLED_OK;
}

// FFN over experts[begin, end) (ids) with known counts, weights through the layer's slot table.
int run_ffn_group(oled_ctx* ctx, LayerData& L, const std::vector<int32_t>& experts, size_t begin, size_t end,
                  const int32_t* counts, cudaEvent_t before_down, bool behind_event_wait) {
  if (begin >= end) return OLED_OK;
  FfnGroup grp;
  grp.n = (int32_t)(end - begin);
  grp.n_box = 16;
  grp.withhold_loads = ctx->withhold_loads;
  grp.pad = 0;
  int max_count = 0;
  uint64_t rows = 0;
  for (size_t i = begin; i < end; ++i) {
    const int32_t e = experts[i];
    grp.expert[i - begin] = (uint16_t)e;
    grp.slot[i - begin] = (uint16_t)L.cache.slot_of[e];
    max_count = std::max(max_count, counts[e]);
    rows += (uint64_t)counts[e];
  }
  bool fused = false;
  const int rc = run_ffn_launches(ctx, grp, max_count, counts, before_down, behind_event_wait, grp.n, &fused);
  prof_add_ffn(ctx, (uint64_t)grp.n, rows, fused);
  return rc;
}

// Blocks until the gate kernel of step `seq` has published counts and scores, and decodes them.
int wait_gate_report(oled_ctx* ctx) {
  const size_t E = (size_t)ctx->shape.n_experts;
  const unsigned long long tag16 = (unsigned long long)(ctx->seq & 0xffffu);
  const unsigned long long tag32 = (unsigned long long)ctx->seq;
  const auto t0 = std::chrono::steady_clock::now();
  bool synced = false;
  for (size_t i = 0; i < 2 * E; ++i) {
    for (uint64_t spin = 0;; ++spin) {
      const unsigned long long v = ctx->h_report[i];
      if (i < E ? (v >> 48) == tag16 : (v >> 32) == tag32) {
        if (i < E) ctx->host_scores[i] = v & 0xffffffffffffull;
        else ctx->host_counts[i - E] = (int32_t)(uint32_t)v;
        break;
      }
      if ((spin & 0xFFFF) == 0xFFFF) {
        const double s = std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count();
        if (s > 20.0) {  // the kernel did not report: find out why instead of spinning for ever
          if (synced) return OLED_ERR_TIMEOUT;
          OLED_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
          synced = true;
        }
      }
    }
  }
  std::atomic_thread_fence(std::memory_order_acquire);
  return OLED_OK;
}

}  // namespace

extern "C" {

size_t oled_expert_blob_bytes(int32_t hidden, int32_t intermediate, int32_t expert_format) {
  const size_t hi = (size_t)hidden * (size_t)intermediate;
  if (expert_format == OLED_EXPERTS_FP8)
    return (3 * hi + 4 * (2 * (size_t)intermediate + (size_t)hidden) + 255) / 256 * 256;
  return 3 * hi * 2;
}

const char* oled_strerror(int code) {
  switch (code) {
    case OLED_OK: return "ok";
    case OLED_ERR_INVALID_ARG: return "invalid argument";
    case OLED_ERR_NOT_PINNED: return "host expert store is not pinned host memory";
    case OLED_ERR_NOT_REGISTERED: return "layer has no router or no expert store registered";
    case OLED_ERR_TOO_MANY_TOKENS: return "n_tokens exceeds max_tokens";
    case OLED_ERR_OOM: return "out of memory";
    case OLED_ERR_CUDA: return "CUDA error (see oled_last_cuda_error)";
    case OLED_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case OLED_ERR_NO_SLOT: return "not enough staging slots for this step's misses";
    case OLED_ERR_STALE_DEBUG: return "the most recent step was on another layer";
    case OLED_ERR_SELF_CHECK: return "the self-check found a violation (see oled_self_check_report)";
    default: return "unknown error";
  }
}

int oled_create(const oled_model_shape* shape, const int32_t* cache_capacity, void* cuda_stream,
                oled_ctx** out_ctx) {
  if (!shape || !cache_capacity || !out_ctx) return OLED_ERR_INVALID_ARG;
  *out_ctx = nullptr;
  const oled_model_shape& s = *shape;
  if (s.n_layers <= 0 || s.hidden <= 0 || s.hidden % 256 != 0 || s.hidden > 16384 || s.intermediate <= 0 ||
      s.intermediate % 128 != 0 || s.n_experts <= 0 || s.n_experts > OLED_MAX_EXPERTS || s.top_k <= 0 ||
      s.top_k > OLED_MAX_TOPK || s.top_k > s.n_experts || s.max_tokens <= 0 || s.max_tokens > 65535 ||
      s.staging_slots < 0 || (s.expert_format != OLED_EXPERTS_BF16 && s.expert_format != OLED_EXPERTS_FP8))
    return OLED_ERR_INVALID_ARG;
  int min_cap = s.n_experts;
  long long total_cap = 0;
  for (int l = 0; l < s.n_layers; ++l) {
    if (cache_capacity[l] <= 0 || cache_capacity[l] > s.n_experts) return OLED_ERR_INVALID_ARG;
    min_cap = std::min(min_cap, cache_capacity[l]);
    total_cap += cache_capacity[l];
  }
  oled_ctx* ctx = new (std::nothrow) oled_ctx();
  if (!ctx) return OLED_ERR_OOM;
  ctx->shape = s;
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  int rc = OLED_OK;
  auto fail = [&](int code) {
    const int cu = ctx->last_cuda_error;
    (void)cu;
    free_ctx(ctx);
    return code;
  };

  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
    cudaGetLastError();
    return fail(OLED_ERR_CUDA);
  }
  ctx->n_sms = prop.multiProcessorCount;
  if (cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&ctx->gate_event, cudaEventDisableTiming) != cudaSuccess)
    return fail(OLED_ERR_CUDA);
  ctx->fill_events.resize(s.n_experts);
  for (auto& ev : ctx->fill_events) {
    ev = nullptr;
    if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) return fail(OLED_ERR_CUDA);
  }

  (void)min_cap;
  const PoolPlan pp = pool_plan(s.n_experts, total_cap, s.staging_slots);
  ctx->adapt_lo = pp.adapt_lo;
  ctx->slot_bytes = oled_expert_blob_bytes(s.hidden, s.intermediate, s.expert_format);
  if (pp.n_slots > 65535) return fail(OLED_ERR_INVALID_ARG);
  ctx->n_slots = (int)pp.n_slots;
  ctx->slots.init(ctx->n_slots);
  ctx->total_capacity = total_cap;
  ctx->layers.resize(s.n_layers);
  for (int l = 0; l < s.n_layers; ++l) ctx->layers[l].cache.init(s.n_experts, cache_capacity[l]);

  const size_t T = (size_t)s.max_tokens, E = (size_t)s.n_experts, K = (size_t)s.top_k;
  const size_t H = (size_t)s.hidden, I = (size_t)s.intermediate;
  ctx->ready_words = T * K / 256 + E;
  ctx->ctrl_bytes = E * (sizeof(unsigned long long) + sizeof(int32_t)) + kFfnWorkCounters * sizeof(uint32_t) +
                    (size_t)kFfnWorkCounters * (E + ctx->ready_words) * sizeof(uint32_t) +
                    (size_t)kPermuteSegments * E * sizeof(int32_t);
  ctx->ctrl_bytes = (ctx->ctrl_bytes + 15) / 16 * 16;
  if ((rc = dev_alloc(ctx, &ctx->pool, (size_t)ctx->n_slots * ctx->slot_bytes)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_ctrl[0], 2 * ctx->ctrl_bytes)) != OLED_OK) return fail(rc);
  ctx->d_ctrl[1] = ctx->d_ctrl[0] + ctx->ctrl_bytes;
  select_ctrl(ctx, 0);
  if ((rc = dev_alloc_guarded(ctx, &ctx->d_logits, T * E)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc_guarded(ctx, &ctx->d_ids, T * K)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc_guarded(ctx, &ctx->d_gate_buf[0], T * K)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc_guarded(ctx, &ctx->d_gate_buf[1], T * K)) != OLED_OK) return fail(rc);
  ctx->d_gate = ctx->d_gate_buf[0];
  if ((rc = dev_alloc_guarded(ctx, &ctx->d_offsets, E + 1)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc_guarded(ctx, &ctx->d_perm, T * K)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc_guarded(ctx, &ctx->d_pos_buf[0], T * K)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc_guarded(ctx, &ctx->d_pos_buf[1], T * K)) != OLED_OK) return fail(rc);
  ctx->d_pos = ctx->d_pos_buf[0];
  if ((rc = dev_alloc_guarded(ctx, &ctx->d_xp, T * K * H)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc_guarded(ctx, &ctx->d_hbuf, T * K * I)) != OLED_OK) return fail(rc);
  if (s.expert_format == OLED_EXPERTS_FP8 && H % 128 == 0 && I % 128 == 0) {
    if ((rc = dev_alloc(ctx, &ctx->split.amax_in, T * K)) != OLED_OK) return fail(rc);
    if ((rc = dev_alloc(ctx, &ctx->split.amax_mid, T * K)) != OLED_OK) return fail(rc);
    if ((rc = dev_alloc(ctx, &ctx->split.terms_in, 2 * T * K * H)) != OLED_OK) return fail(rc);
    if ((rc = dev_alloc(ctx, &ctx->split.terms_mid, 2 * T * K * I)) != OLED_OK) return fail(rc);
    ctx->split.rows = (int)(T * K);
  }
  if ((rc = dev_alloc_guarded(ctx, &ctx->d_y, T * K * H)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_status, kStatusWords)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_timeline, (size_t)s.n_layers)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_hidden_stage, T * H)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_conf_stage, T)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_out_stage, T * H)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_iter[0], T * H)) != OLED_OK) return fail(rc);
  if ((rc = dev_alloc(ctx, &ctx->d_iter[1], T * H)) != OLED_OK) return fail(rc);
  for (int l = 0; l < s.n_layers; ++l) {
    if ((rc = dev_alloc(ctx, &ctx->layers[l].w_router, E * H)) != OLED_OK) return fail(rc);
    if (s.has_router_bias && (rc = dev_alloc(ctx, &ctx->layers[l].bias, E)) != OLED_OK) return fail(rc);
  }
  if (cudaMallocHost(reinterpret_cast<void**>(&ctx->h_ctrl), 2 * E * sizeof(unsigned long long)) != cudaSuccess ||
      cudaMallocHost(reinterpret_cast<void**>(&ctx->h_status), kStatusWords * sizeof(uint32_t)) != cudaSuccess)
    return fail(OLED_ERR_OOM);
  memset(ctx->h_status, 0, kStatusWords * sizeof(uint32_t));
  ctx->h_status[kStatusCheckIndex] = kStatusNoIndex;
  memset(ctx->h_ctrl, 0, 2 * E * sizeof(unsigned long long));
  ctx->h_report = reinterpret_cast<volatile unsigned long long*>(ctx->h_ctrl);
  ctx->host_scores.assign(E, 0);
  ctx->host_counts.assign(E, 0);
  launch_guard_fill(ctx->stream, ctx->guards);
  if (cudaMemcpy(ctx->d_status, ctx->h_status, kStatusWords * sizeof(uint32_t), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemset(ctx->d_xp, 0, T * K * H * 2) != cudaSuccess ||
      cudaMemset(ctx->d_hbuf, 0, T * K * I * 2) != cudaSuccess ||
      cudaMemset(ctx->d_y, 0, T * K * H * 4) != cudaSuccess)
    return fail(OLED_ERR_CUDA);
  rc = ffn_tc_setup(&ctx->maps, ctx->pool, ctx->slot_bytes, ctx->n_slots, s.hidden, s.intermediate,
                    s.expert_format == OLED_EXPERTS_FP8, ctx->d_xp,
                    ctx->d_hbuf, (int)(T * K), ctx->split.complete() ? &ctx->split : nullptr);
  if (rc != OLED_OK) return fail(rc);
  if (cudaDeviceSynchronize() != cudaSuccess) return fail(OLED_ERR_CUDA);
  *out_ctx = ctx;
  return OLED_OK;
}

int oled_register_router(oled_ctx* ctx, int32_t layer, const void* w_router, const float* bias) {
  if (!ctx || !w_router || layer < 0 || layer >= ctx->shape.n_layers) return OLED_ERR_INVALID_ARG;
  if ((bias != nullptr) != (ctx->shape.has_router_bias != 0)) return OLED_ERR_INVALID_ARG;
  LayerData& L = ctx->layers[layer];
  const size_t bytes = (size_t)ctx->shape.n_experts * ctx->shape.hidden * 2;
  OLED_CUDA(ctx, cudaMemcpyAsync(L.w_router, w_router, bytes, cudaMemcpyDefault, ctx->stream));
  if (bias)
    OLED_CUDA(ctx, cudaMemcpyAsync(L.bias, bias, (size_t)ctx->shape.n_experts * sizeof(float),
                                   cudaMemcpyDefault, ctx->stream));
  OLED_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  L.has_router = true;
  return OLED_OK;
}

int oled_register_experts(oled_ctx* ctx, int32_t layer, const void* host_blob, size_t expert_stride_bytes) {
  if (!ctx || !host_blob || layer < 0 || layer >= ctx->shape.n_layers) return OLED_ERR_INVALID_ARG;
  if (expert_stride_bytes < ctx->slot_bytes || expert_stride_bytes % 16 != 0 ||
      reinterpret_cast<uintptr_t>(host_blob) % 16 != 0)
    return OLED_ERR_INVALID_ARG;
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, host_blob) != cudaSuccess) {
    cudaGetLastError();
    return OLED_ERR_NOT_PINNED;
  }
  if (a.type != cudaMemoryTypeHost) return OLED_ERR_NOT_PINNED;
  // the last byte must be pinned too
  const uint8_t* last = static_cast<const uint8_t*>(host_blob) +
                        (size_t)(ctx->shape.n_experts - 1) * expert_stride_bytes + ctx->slot_bytes - 1;
  if (cudaPointerGetAttributes(&a, last) != cudaSuccess || a.type != cudaMemoryTypeHost) {
    cudaGetLastError();
    return OLED_ERR_NOT_PINNED;
  }
  LayerData& L = ctx->layers[layer];
  // a new store invalidates whatever this layer has cached
  OLED_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  drop_all(L.cache, ctx->slots);
  L.host_blob = static_cast<const uint8_t*>(host_blob);
  L.host_stride = expert_stride_bytes;
  return OLED_OK;
}

// x_next != nullptr: also write x_next = bf16(hidden + out), the residual between layers.
// defer_combine: the caller promises that the next step on this context takes x_next as its
// input with the same n_tokens; the combine may then be left to that step's gate kernel.
static int step_impl(oled_ctx* ctx, int32_t layer, const void* hidden, const float* confidences,
                     int32_t n_tokens, void* out, void* x_next, bool defer_combine = false) {
  if (!ctx || layer < 0 || layer >= ctx->shape.n_layers || n_tokens < 0) return OLED_ERR_INVALID_ARG;
  if (n_tokens > ctx->shape.max_tokens) return OLED_ERR_TOO_MANY_TOKENS;
  LayerData& L = ctx->layers[layer];
  if (!L.has_router || !L.host_blob) return OLED_ERR_NOT_REGISTERED;
  const int T = n_tokens, H = ctx->shape.hidden, E = ctx->shape.n_experts, K = ctx->shape.top_k;
  if (T > 0) {
    if (!hidden || !confidences || !out) return OLED_ERR_INVALID_ARG;
    const uint8_t* a = static_cast<const uint8_t*>(hidden);
    const uint8_t* b = static_cast<const uint8_t*>(out);
    const size_t bytes = (size_t)T * H * 2;
    if (a < b + bytes && b < a + bytes) return OLED_ERR_INVALID_ARG;  // out aliases hidden
    // the kernels read and write rows with 16-byte vector accesses
    if (misaligned(hidden, 16) || misaligned(out, 16) || misaligned(x_next, 16) || misaligned(confidences, 4))
      return OLED_ERR_INVALID_ARG;
  }
  cudaStream_t st = ctx->stream;
  ctx->last_layer = layer;
  ctx->last_tokens = T;
  if (T == 0) {  // nothing is activated: R' = R, only the step counter moves
    ctx->last_before = L.cache.resident;
    ctx->last_after = L.cache.resident;
    L.stats.steps += 1;
    return OLED_OK;
  }

  pdl_set_step((size_t)T * K <= 4096);
  // per-assignment outputs y: fp32 for small steps; bf16 once y's traffic matters (the rounding
  // adds at most 2^-9 relative per term, far inside the output tolerance)
  ctx->y_bf16 = ctx->ffn_impl == 0 && (size_t)T * K > 4096;
  // 1. gate, counts and reuse-score numerators, permutation; the permutation kernel reports
  // counts and scores to the host.  This step takes the control block the last step did not use.
  if (ctx->ctrl_dirty) OLED_CUDA(ctx, cudaMemsetAsync(ctx->d_ctrl[0], 0, 2 * ctx->ctrl_bytes, st));
  ctx->ctrl_dirty = true;
  select_ctrl(ctx, ctx->ctrl_sel ^ 1);
  ctx->work_next = 0;
  ctx->seq += 1;
  RouteReport rep;
  rep.host_scores = reinterpret_cast<unsigned long long*>(ctx->h_ctrl);
  rep.host_counts = reinterpret_cast<unsigned long long*>(ctx->h_ctrl) + E;
  rep.seq = ctx->seq;
  rep.counts = ctx->d_counts;
  rep.scores = ctx->d_scores;
  rep.n_experts = E;
  StepTimeline* const tl = ctx->timeline_on ? ctx->d_timeline + layer : nullptr;
  rep.timeline = tl;
  if (tl) {  // earliest times start at the maximum, latest at zero
    OLED_CUDA(ctx, cudaMemsetAsync(tl, 0xff, 2 * kTimelineSlots * sizeof(unsigned long long), st));
    OLED_CUDA(ctx, cudaMemsetAsync(tl->end_max, 0, kTimelineSlots * sizeof(unsigned long long), st));
  }
  // many-token steps: the gate kernel counts every expert's assignments per segment of the token
  // range, and the permutation kernel then scans the segments in parallel
  int32_t* const seg_counts = (size_t)T * K > 4096 && !route_can_take_combine(T) ? ctx->d_seg : nullptr;
  const int seg_tokens = ((T + kPermuteSegments - 1) / kPermuteSegments + 3) / 4 * 4;
  // the current step's gate-score and inverse-permutation buffers (the previous step's stay
  // intact for a combine that has been left to this step's gate kernel)
  ctx->buf_sel ^= 1;
  ctx->d_gate = ctx->d_gate_buf[ctx->buf_sel];
  ctx->d_pos = ctx->d_pos_buf[ctx->buf_sel];
  const bool fuse_prev = ctx->pending.valid && ctx->pending.T == T && route_can_take_combine(T) &&
                         ctx->pending.x_next == static_cast<const uint16_t*>(hidden);
  if (ctx->pending.valid && !fuse_prev) {
    const int rcp = flush_pending_combine(ctx);
    if (rcp != OLED_OK) return rcp;
  }
  {
    NvtxRange nv(ctx, "oled.step.1_gate_topk_scores");
    ProfScope ps(ctx, OLED_KERNEL_ROUTE,
                 ((uint64_t)T * H + (uint64_t)E * H) * 2 + (uint64_t)T * K * 8 +
                     (fuse_prev ? (uint64_t)T * K * H * 4 + (uint64_t)T * H * 6 : 0),
                 2ull * T * H * E + (fuse_prev ? 2ull * T * K * H : 0));
    CombinePrev prev;
    if (fuse_prev) {
      prev.y = ctx->d_y;
      prev.gate = ctx->pending.gate;
      prev.pos = ctx->pending.pos;
      prev.x = ctx->pending.x;
      prev.out = ctx->pending.out;
      prev.x_next = ctx->pending.x_next;
      prev.K = K;
      prev.zero_words = ctx->pending.ctrl;
      prev.n_zero_words = (int)(ctx->ctrl_bytes / 4);
      ctx->pending.valid = false;
    }
    launch_route(st, static_cast<const uint16_t*>(hidden), L.w_router, L.bias, confidences, T, H, E, K,
                 ctx->d_logits, ctx->d_ids, ctx->d_gate, ctx->d_counts, ctx->d_scores, prev, tl, seg_counts, seg_tokens);
  }
  const bool fuse_gather = (size_t)T * K <= 4096;  // few rows per expert: one CTA per expert copies them
  // Many rows per expert (every FFN launch of the step on CTA pairs, token tiles of 256 rows): no
  // gather kernel, each gate/up launch copies its experts' token rows while its first items run.
  const bool gather_in_ffn = !fuse_gather && ctx->gather_in_ffn && ctx->ffn_impl == 0 &&
                             std::min<size_t>(T, 2 * (((size_t)T * K + E - 1) / E)) > 128 &&
                             (reinterpret_cast<uintptr_t>(hidden) & 15u) == 0 &&  // (bulk copies of whole rows)
                             ffn_tc_token_source_usable(ctx->maps, H, ctx->shape.intermediate);
  if (gather_in_ffn)
    ffn_tc_set_token_source(&ctx->maps, static_cast<const uint16_t*>(hidden), T, ctx->d_perm, K, ctx->d_xp);
  else
    ffn_tc_clear_token_source(&ctx->maps);
  NvtxRange nv_perm(ctx, "oled.step.2_permutation_counts");
  {
    ProfScope ps(ctx, OLED_KERNEL_PERMUTE, (uint64_t)T * K * 12 + (fuse_gather ? (uint64_t)T * K * H * 4 : 0), 0);
    // (fp8 stores: a gathering permutation kernel also leaves the rows' magnitudes for the FFN)
    ctx->step_split = fuse_gather && ctx->fp8_direct && ctx->split.complete() ? &ctx->split : nullptr;
    launch_permute(st, ctx->d_ids, ctx->d_counts, T, E, K, ctx->d_offsets, ctx->d_perm, ctx->d_pos,
                   static_cast<const uint16_t*>(hidden), fuse_gather ? ctx->d_xp : nullptr, H, tl, ctx->step_split,
                   seg_counts, seg_tokens);
  }
  if (!fuse_gather && !gather_in_ffn) {
    ProfScope ps(ctx, OLED_KERNEL_GATHER, (uint64_t)T * K * H * 4, 0);
    launch_gather(st, static_cast<const uint16_t*>(hidden), ctx->d_perm, T, H, K, ctx->d_xp);
  }
  ctx->launches += fuse_gather || gather_in_ffn ? 2 : 3;
  nv_perm.end();
  if (ctx->corrupt_perm) {
    launch_corrupt_perm(st, ctx->d_perm, T * K);
    ctx->launches += 1;
  }
  if (ctx->self_check) {
    launch_self_check(st, ctx->d_ids, ctx->d_counts, ctx->d_offsets, ctx->d_perm, ctx->d_pos, T, E, K, ctx->d_status);
    ctx->launches += 1;
  }
  OLED_CUDA(ctx, cudaGetLastError());

  NvtxRange nv_ffn_hits(ctx, "oled.step.3_expert_ffn_hits");
  // 1b. cache hits need no decision: the FFN over the experts resident BEFORE the step is
  // enqueued at once (experts that received no token contribute no tile), so the GPU does not
  // wait for the host's round trip below.
  {
    FfnGroup grp;
    grp.n = 0;
    grp.n_box = 16;
    grp.withhold_loads = ctx->withhold_loads;
    grp.pad = 0;
    for (int32_t e = 0; e < E; ++e)
      if (L.cache.resident[e] && L.cache.slot_of[e] >= 0) {
        grp.expert[grp.n] = (uint16_t)e;
        grp.slot[grp.n] = (uint16_t)L.cache.slot_of[e];
        ++grp.n;
      }
    // token tile of this launch (the counts are not known on the host yet): twice the mean load
    // per expert, but at least 32 rows - an expert that received more rows than the tile holds
    // has its weights streamed once per tile, and in a block of 32 tokens whose routing is
    // concentrated on few experts (the regime the paper reports) counts of 17..32 are common
    const int mean_load = (int)(((size_t)T * K + E - 1) / E);
    // (how many of the residents will have tokens is not known yet: the layer's previous
    // execution is the estimate - adjacent iterations activate mostly the same experts, Sec. 3.3)
    const int expected = std::min<int>(grp.n, L.last_active >= 0 ? L.last_active : E);
    // (direct fp8 form: its token operand is two rows per token and a third of a stage at 32, so
    // where the layer's previous execution gave no expert more than 16 rows the tile is 16)
    const int floor_rows = ctx->step_split != nullptr && L.last_max_count >= 0 && L.last_max_count <= 16 ? 16 : 32;
    const int rc0 = run_ffn_launches(ctx, grp, std::min(T, std::max(floor_rows, 2 * mean_load)), nullptr, nullptr, false,
                                     expected, &ctx->hit_fused, rep);
    if (rc0 != OLED_OK) return rc0;
  }

  nv_ffn_hits.end();
  NvtxRange nv_policy(ctx, "oled.step.5_reuse_score_retention_fills");
  // The report implies that everything enqueued before this step has completed, so slots
  // released earlier are free to be overwritten by the side stream.
  {
    const int rcw = wait_gate_report(ctx);
    if (rcw != OLED_OK) return rcw;
  }
  const unsigned long long* scores = ctx->host_scores.data();
  const int32_t* counts = ctx->host_counts.data();

  // 2. hits / misses against the pre-step resident set, Top-C retention, slot plan
  StepPlan& plan = ctx->plan;
  {
    const auto p0 = std::chrono::steady_clock::now();
    const bool ok = plan_step(L.cache, ctx->slots, counts, reinterpret_cast<const uint64_t*>(scores), plan);
    ctx->policy_ns += (uint64_t)std::chrono::duration_cast<std::chrono::nanoseconds>(
                          std::chrono::steady_clock::now() - p0).count();
    ctx->policy_runs += 1;
    if (!ok) return OLED_ERR_NO_SLOT;
  }
  ctx->last_before = plan.before;
  ctx->last_after = plan.after;

  // 3. fills: one pinned-host -> HBM copy per miss on the side stream.  The misses form two
  // groups: everything but the last `miss_chunk` experts, then those last few.  The first group's
  // FFN is one large launch that runs under the copies of the second; only the small second
  // group's FFN is exposed after the last byte has arrived - and of that only the down
  // projection: the step's LAST blob is copied in two parts, what the gate/up kernel reads (and
  // the row scales of an fp8 blob) first, the down-projection weights after it, so the last
  // group's gate/up kernel runs while the last down-projection weights are still on the link.
  const size_t n_miss = plan.misses.size();
  // byte range of the down-projection weights inside a blob (bf16 elements or e4m3 codes)
  const size_t esz = ctx->shape.expert_format == OLED_EXPERTS_FP8 ? 1 : 2;
  const size_t hi_elems = (size_t)ctx->shape.hidden * (size_t)ctx->shape.intermediate;
  const size_t down_off = 2 * hi_elems * esz, down_bytes = hi_elems * esz;
  const bool split_last = ctx->split_last && n_miss > 0 && E >= 3;
  const size_t tail = std::min(n_miss, (size_t)ctx->miss_chunk);
  const size_t bounds[3] = {0, n_miss - tail, n_miss};
  size_t n_groups = 0;
  size_t group_begin[2], group_end[2];
  for (int gi = 0; gi < 2; ++gi) {
    if (bounds[gi] == bounds[gi + 1]) continue;
    for (size_t i = bounds[gi]; i < bounds[gi + 1]; ++i) {
      const int32_t e = plan.misses[i];
      uint8_t* dst = ctx->pool + (size_t)L.cache.slot_of[e] * ctx->slot_bytes;
      const uint8_t* src = L.host_blob + (size_t)e * L.host_stride;
      if (i + 1 < n_miss || !split_last) {
        OLED_CUDA(ctx, cudaMemcpyAsync(dst, src, ctx->slot_bytes, cudaMemcpyHostToDevice, ctx->copy_stream));
      } else {  // the step's last blob: gate|up (and the scales behind the codes) now, down below
        OLED_CUDA(ctx, cudaMemcpyAsync(dst, src, down_off, cudaMemcpyHostToDevice, ctx->copy_stream));
        if (ctx->slot_bytes > down_off + down_bytes)
          OLED_CUDA(ctx, cudaMemcpyAsync(dst + down_off + down_bytes, src + down_off + down_bytes,
                                         ctx->slot_bytes - down_off - down_bytes, cudaMemcpyHostToDevice,
                                         ctx->copy_stream));
      }
    }
    OLED_CUDA(ctx, cudaEventRecord(ctx->fill_events[n_groups], ctx->copy_stream));
    if (split_last && bounds[gi + 1] == n_miss) {
      const int32_t e = plan.misses[n_miss - 1];
      OLED_CUDA(ctx, cudaMemcpyAsync(ctx->pool + (size_t)L.cache.slot_of[e] * ctx->slot_bytes + down_off,
                                     L.host_blob + (size_t)e * L.host_stride + down_off, down_bytes,
                                     cudaMemcpyHostToDevice, ctx->copy_stream));
      OLED_CUDA(ctx, cudaEventRecord(ctx->fill_events[2], ctx->copy_stream));
    }
    group_begin[n_groups] = bounds[gi];
    group_end[n_groups] = bounds[gi + 1];
    ++n_groups;
  }

  nv_policy.end();
  NvtxRange nv_ffn_miss(ctx, "oled.step.3_expert_ffn_misses");
  // 4. grouped FFN over the misses as their weights land (hits: step 1b)
  {
    uint64_t hit_rows = 0;
    for (int32_t e : plan.hits) hit_rows += (uint64_t)counts[e];
    prof_add_ffn(ctx, plan.hits.size(), hit_rows, ctx->hit_fused);
  }
  int rc = OLED_OK;
  for (size_t c = 0; c < n_groups; ++c) {
    OLED_CUDA(ctx, cudaStreamWaitEvent(st, ctx->fill_events[c], 0));
    rc = run_ffn_group(ctx, L, plan.misses, group_begin[c], group_end[c], counts,
                       split_last && group_end[c] == n_miss ? ctx->fill_events[2] : nullptr, true);
    if (rc != OLED_OK) return rc;
  }

  nv_ffn_miss.end();
  NvtxRange nv_comb(ctx, "oled.step.4_combine");
  // 5. combine - or, inside a stack iteration of few-token steps, left to the next layer's gate kernel
  const bool defer = defer_combine && ctx->fuse_combine && route_can_take_combine(T) && x_next != nullptr &&
                     !ctx->y_bf16 && !ctx->self_check && ctx->ffn_impl == 0;
  if (defer) {
    ctx->pending.valid = true;
    ctx->pending.T = T;
    ctx->pending.gate = ctx->d_gate;
    ctx->pending.pos = ctx->d_pos;
    ctx->pending.x = static_cast<const uint16_t*>(hidden);
    ctx->pending.out = static_cast<uint16_t*>(out);
    ctx->pending.x_next = static_cast<uint16_t*>(x_next);
    ctx->pending.ctrl = reinterpret_cast<uint32_t*>(ctx->d_ctrl[ctx->ctrl_sel]);
    ctx->ctrl_dirty = false;  // the gate kernel that carries the combine out clears this step's block
  } else {
    {
      ProfScope ps(ctx, OLED_KERNEL_COMBINE, (uint64_t)T * K * H * (ctx->y_bf16 ? 2 : 4) + (uint64_t)T * H * 2,
                   2ull * T * K * H);
      launch_combine(st, ctx->d_y, ctx->y_bf16 ? 1 : 0, ctx->d_gate, ctx->d_pos, T, H, K, static_cast<uint16_t*>(out),
                     static_cast<const uint16_t*>(hidden), static_cast<uint16_t*>(x_next),
                     reinterpret_cast<uint32_t*>(ctx->d_scores), (int)(ctx->ctrl_bytes / 4), tl);
    }
    ctx->launches += 1;
    if (ctx->self_check) {
      launch_guard_check(st, ctx->guards, ctx->d_status);
      ctx->launches += 1;
    }
    OLED_CUDA(ctx, cudaGetLastError());
    ctx->ctrl_dirty = false;  // combine's CTA 0 cleared this step's control block
  }

  finish_step(L.cache, ctx->slots, plan);
  L.stats.steps += 1;
  L.stats.hits += plan.hits.size();
  L.stats.misses += n_miss;
  L.stats.bytes_moved += (uint64_t)n_miss * ctx->slot_bytes;
  L.stats.evictions += (uint64_t)plan.n_evictions;
  L.stats.active_experts += (uint64_t)plan.n_active;
  L.last_active = plan.n_active;
  L.last_max_count = 0;
  for (int32_t e = 0; e < E; ++e) L.last_max_count = std::max(L.last_max_count, counts[e]);
  L.last_misses = n_miss;
  L.last_counts.assign(counts, counts + E);
  L.stats.assignments += (uint64_t)T * K;
  L.stats.fills_reused += (uint64_t)plan.n_fills_reused;
  L.stats.ideal_hits += (uint64_t)std::min<int64_t>(plan.n_active, plan.capacity_used);
  static const bool log_steps = getenv("OLED_LOG") != nullptr;  // one line per layer execution on stderr
  if (log_steps) {
    int resident = 0;
    for (uint8_t r : plan.after) resident += r;
    fprintf(stderr, "oled: layer %d tokens %d active %d hits %zu misses %zu evicted %d resident %d/%d\n", (int)layer, T,
            (int)plan.n_active, plan.hits.size(), n_miss, (int)plan.n_evictions, resident, (int)plan.capacity_used);
  }
  return OLED_OK;
}

int oled_denoise_step(oled_ctx* ctx, int32_t layer, const void* hidden, const float* confidences,
                      int32_t n_tokens, void* out) {
  return step_impl(ctx, layer, hidden, confidences, n_tokens, out, nullptr);
}

int oled_denoise_step_host(oled_ctx* ctx, int32_t layer, const void* host_hidden,
                           const float* host_confidences, int32_t n_tokens, void* host_out) {
  if (!ctx || n_tokens < 0) return OLED_ERR_INVALID_ARG;
  if (n_tokens > ctx->shape.max_tokens) return OLED_ERR_TOO_MANY_TOKENS;
  if (n_tokens > 0 && (!host_hidden || !host_confidences || !host_out)) return OLED_ERR_INVALID_ARG;
  const size_t bytes = (size_t)n_tokens * ctx->shape.hidden * 2;
  if (n_tokens > 0) {
    OLED_CUDA(ctx, cudaMemcpyAsync(ctx->d_hidden_stage, host_hidden, bytes, cudaMemcpyHostToDevice, ctx->stream));
    OLED_CUDA(ctx, cudaMemcpyAsync(ctx->d_conf_stage, host_confidences, (size_t)n_tokens * sizeof(float),
                                   cudaMemcpyHostToDevice, ctx->stream));
  }
  const int rc = oled_denoise_step(ctx, layer, ctx->d_hidden_stage, ctx->d_conf_stage, n_tokens, ctx->d_out_stage);
  if (rc != OLED_OK) return rc;
  if (n_tokens > 0) {
    OLED_CUDA(ctx, cudaMemcpyAsync(host_out, ctx->d_out_stage, bytes, cudaMemcpyDeviceToHost, ctx->stream));
    OLED_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  }
  return OLED_OK;
}

// While the next layer's gate and permutation kernels run the HBM is idle: if that layer's
// previous execution hit the cache with every activated expert, the weights its FFN will stream
// first - the residents activated then, in the order of the FFN's expert list - are called into
// L2 from the side stream (idle as well when nothing misses), behind the current layer's last
// kernel.  A prefetch only: what the gate then decides changes nothing but the hit rate in L2.
static int prefetch_next_layer(oled_ctx* ctx, int32_t next) {
  if (!ctx->l2_prefetch || ctx->ffn_impl != 0) return OLED_OK;
  const LayerData& N = ctx->layers[next];
  if (N.last_misses != 0 || (int32_t)N.last_counts.size() != ctx->shape.n_experts) return OLED_OK;
  constexpr size_t kPrefetchBytes = 64u << 20;  // about what the HBM delivers during gate + permutation (32-96 MB measured alike, more costs)
  // the gate/up matrices only (they lead a blob): the down matrices are read a whole gate/up launch later
  const size_t esz = ctx->shape.expert_format == OLED_EXPERTS_FP8 ? 1 : 2;
  const size_t lead_bytes = (size_t)2 * ctx->shape.hidden * ctx->shape.intermediate * esz;
  // Worth it only in front of a long expert stream: measured, streams of 0.4 and 0.8 GB per layer gained
  // 2-3 % and one of 0.27 GB lost 2 % (the prefetch delays the gate kernel's own loads by 2 us now and then).
  size_t stream_bytes = 0;
  for (int32_t e = 0; e < ctx->shape.n_experts; ++e)
    if (N.last_counts[e] > 0) stream_bytes += (size_t)3 * ctx->shape.hidden * ctx->shape.intermediate * esz;
  if (stream_bytes < 5 * kPrefetchBytes && ctx->l2_prefetch != 2) return OLED_OK;
  SlotList list;
  list.n = 0;
  const int cap = (int)std::max<size_t>(1, kPrefetchBytes / lead_bytes);
  for (int32_t e = 0; e < ctx->shape.n_experts && list.n < cap; ++e)
    if (N.cache.resident[e] && N.cache.slot_of[e] >= 0 && N.last_counts[e] > 0) list.slot[list.n++] = (uint16_t)N.cache.slot_of[e];
  if (list.n == 0) return OLED_OK;
  if (ctx->ev_layer_done == nullptr)
    OLED_CUDA(ctx, cudaEventCreateWithFlags(&ctx->ev_layer_done, cudaEventDisableTiming));
  OLED_CUDA(ctx, cudaEventRecord(ctx->ev_layer_done, ctx->stream));
  OLED_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_layer_done, 0));
  launch_l2_prefetch(ctx->copy_stream, ctx->pool, ctx->slot_bytes, list, lead_bytes);
  ctx->launches += 1;
  OLED_CUDA(ctx, cudaGetLastError());
  return OLED_OK;
}

int oled_denoise_iteration(oled_ctx* ctx, const void* hidden, const float* confidences, int32_t n_tokens,
                           void* hidden_out) {
  if (!ctx || n_tokens < 0) return OLED_ERR_INVALID_ARG;
  if (n_tokens > ctx->shape.max_tokens) return OLED_ERR_TOO_MANY_TOKENS;
  if (n_tokens > 0 && (!hidden || !confidences || !hidden_out)) return OLED_ERR_INVALID_ARG;
  const void* x = hidden;
  for (int l = 0; l < ctx->shape.n_layers; ++l) {
    void* nxt = (l + 1 == ctx->shape.n_layers) ? hidden_out : (void*)ctx->d_iter[l & 1];
    const int rc = step_impl(ctx, l, x, confidences, n_tokens, ctx->d_out_stage, nxt, l + 1 < ctx->shape.n_layers);
    if (rc != OLED_OK) return rc;
    x = nxt;
    {  // (behind the last layer: the first layer of the iteration that is likely to follow)
      const int rcp = prefetch_next_layer(ctx, l + 1 < ctx->shape.n_layers ? l + 1 : 0);
      if (rcp != OLED_OK) return rcp;
    }
  }
  ctx->iterations += 1;
  if (ctx->adapt_period > 0 && ctx->iterations % (uint64_t)ctx->adapt_period == 0)
    return oled_adapt_capacity(ctx, nullptr);
  return OLED_OK;
}

int oled_adapt_capacity(oled_ctx* ctx, int32_t* new_capacity) {
  if (!ctx) return OLED_ERR_INVALID_ARG;
  std::vector<LayerCacheState*> layers;
  for (auto& L : ctx->layers) layers.push_back(&L.cache);
  const std::vector<int32_t> caps = adaptive_capacities(layers, ctx->total_capacity, ctx->adapt_lo);
  // Slots of residents evicted here may still be read by kernels already enqueued; they are
  // reused only after the next step's gate report, which those kernels precede in stream order.
  for (size_t l = 0; l < layers.size(); ++l)
    ctx->layers[l].stats.evictions += (uint64_t)shrink_to(*layers[l], ctx->slots, caps[l]);
  if (new_capacity)
    for (size_t l = 0; l < caps.size(); ++l) new_capacity[l] = caps[l];
  return OLED_OK;
}

int oled_get_capacity(oled_ctx* ctx, int32_t* capacity) {
  if (!ctx || !capacity) return OLED_ERR_INVALID_ARG;
  for (size_t l = 0; l < ctx->layers.size(); ++l) capacity[l] = ctx->layers[l].cache.capacity;
  return OLED_OK;
}

int oled_denoise_iteration_host(oled_ctx* ctx, const void* host_hidden, const float* host_confidences,
                                int32_t n_tokens, void* host_hidden_out) {
  if (!ctx || n_tokens < 0) return OLED_ERR_INVALID_ARG;
  if (n_tokens > ctx->shape.max_tokens) return OLED_ERR_TOO_MANY_TOKENS;
  if (n_tokens == 0) return oled_denoise_iteration(ctx, nullptr, nullptr, 0, nullptr);
  if (!host_hidden || !host_confidences || !host_hidden_out) return OLED_ERR_INVALID_ARG;
  const size_t bytes = (size_t)n_tokens * ctx->shape.hidden * 2;
  OLED_CUDA(ctx, cudaMemcpyAsync(ctx->d_hidden_stage, host_hidden, bytes, cudaMemcpyHostToDevice, ctx->stream));
  OLED_CUDA(ctx, cudaMemcpyAsync(ctx->d_conf_stage, host_confidences, (size_t)n_tokens * sizeof(float),
                                 cudaMemcpyHostToDevice, ctx->stream));
  // the last layer's residual writes into the staging buffer the input came from: by then the
  // input has been consumed (layer 0 reads it; later layers read the ping-pong buffers)
  uint16_t* final_dev = ctx->shape.n_layers > 1 ? ctx->d_hidden_stage : ctx->d_iter[0];
  const int rc = oled_denoise_iteration(ctx, ctx->d_hidden_stage, ctx->d_conf_stage, n_tokens, final_dev);
  if (rc != OLED_OK) return rc;
  OLED_CUDA(ctx, cudaMemcpyAsync(host_hidden_out, final_dev, bytes, cudaMemcpyDeviceToHost, ctx->stream));
  OLED_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  return OLED_OK;
}

int oled_stats(oled_ctx* ctx, int32_t layer, oled_stats_t* out) {
  if (!ctx || !out || layer < -1 || layer >= ctx->shape.n_layers) return OLED_ERR_INVALID_ARG;
  const int rc = sync_all(ctx);
  oled_stats_t acc{};
  for (int l = 0; l < ctx->shape.n_layers; ++l) {
    if (layer >= 0 && l != layer) continue;
    const oled_stats_t& s = ctx->layers[l].stats;
    acc.steps += s.steps;
    acc.hits += s.hits;
    acc.misses += s.misses;
    acc.bytes_moved += s.bytes_moved;
    acc.evictions += s.evictions;
    acc.active_experts += s.active_experts;
    acc.assignments += s.assignments;
    acc.fills_reused += s.fills_reused;
    acc.ideal_hits += s.ideal_hits;
  }
  *out = acc;
  return rc;
}

int oled_debug_last(oled_ctx* ctx, int32_t layer, int32_t* ids, float* gate, int32_t* perm, int32_t* counts,
                    uint64_t* scores, uint8_t* resident_before, uint8_t* resident_after) {
  if (!ctx || layer < 0 || layer >= ctx->shape.n_layers) return OLED_ERR_INVALID_ARG;
  if (ctx->last_layer != layer) return OLED_ERR_STALE_DEBUG;
  const int rc = sync_all(ctx);
  if (rc != OLED_OK && rc != OLED_ERR_TIMEOUT) return rc;
  const size_t n = (size_t)ctx->last_tokens * ctx->shape.top_k, E = (size_t)ctx->shape.n_experts;
  if (n > 0) {
    if (ids) OLED_CUDA(ctx, cudaMemcpy(ids, ctx->d_ids, n * sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (gate) OLED_CUDA(ctx, cudaMemcpy(gate, ctx->d_gate, n * sizeof(float), cudaMemcpyDeviceToHost));
    if (perm) OLED_CUDA(ctx, cudaMemcpy(perm, ctx->d_perm, n * sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (counts) memcpy(counts, ctx->host_counts.data(), E * sizeof(int32_t));
    if (scores) memcpy(scores, ctx->host_scores.data(), E * sizeof(uint64_t));
  } else {
    if (counts) memset(counts, 0, E * sizeof(int32_t));
    if (scores) memset(scores, 0, E * sizeof(uint64_t));
  }
  if (resident_before) memcpy(resident_before, ctx->last_before.data(), E);
  if (resident_after) memcpy(resident_after, ctx->last_after.data(), E);
  return rc;
}

int oled_debug_perm(oled_ctx* ctx, int32_t layer, int32_t* offsets, int32_t* pos) {
  if (!ctx || layer < 0 || layer >= ctx->shape.n_layers) return OLED_ERR_INVALID_ARG;
  if (ctx->last_layer != layer) return OLED_ERR_STALE_DEBUG;
  const int rc = sync_all(ctx);
  if (rc != OLED_OK && rc != OLED_ERR_TIMEOUT) return rc;
  const size_t n = (size_t)ctx->last_tokens * ctx->shape.top_k, E = (size_t)ctx->shape.n_experts;
  if (n > 0) {
    if (offsets) OLED_CUDA(ctx, cudaMemcpy(offsets, ctx->d_offsets, (E + 1) * sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (pos) OLED_CUDA(ctx, cudaMemcpy(pos, ctx->d_pos, n * sizeof(int32_t), cudaMemcpyDeviceToHost));
  } else if (offsets) {
    memset(offsets, 0, (E + 1) * sizeof(int32_t));
  }
  return rc;
}

int oled_debug_timeline(oled_ctx* ctx, int32_t layer, uint64_t* times) {
  if (!ctx || !times || layer < 0 || layer >= ctx->shape.n_layers) return OLED_ERR_INVALID_ARG;
  const int rc = sync_all(ctx);
  if (rc != OLED_OK && rc != OLED_ERR_TIMEOUT) return rc;
  OLED_CUDA(ctx, cudaMemcpy(times, ctx->d_timeline + layer, sizeof(StepTimeline), cudaMemcpyDeviceToHost));
  return rc;
}

int oled_debug_logits(oled_ctx* ctx, int32_t layer, float* logits) {
  if (!ctx || !logits || layer < 0 || layer >= ctx->shape.n_layers) return OLED_ERR_INVALID_ARG;
  if (ctx->last_layer != layer) return OLED_ERR_STALE_DEBUG;
  const int rc = sync_all(ctx);
  if (rc != OLED_OK && rc != OLED_ERR_TIMEOUT) return rc;
  const size_t n = (size_t)ctx->last_tokens * ctx->shape.n_experts;
  if (n > 0) OLED_CUDA(ctx, cudaMemcpy(logits, ctx->d_logits, n * sizeof(float), cudaMemcpyDeviceToHost));
  return rc;
}

int oled_reset_cache(oled_ctx* ctx) {
  if (!ctx) return OLED_ERR_INVALID_ARG;
  const int rc = sync_all(ctx);
  for (auto& L : ctx->layers) {
    drop_all(L.cache, ctx->slots);
    L.stats = oled_stats_t{};
  }
  ctx->iterations = 0;
  ctx->last_layer = -1;
  return rc;
}

int oled_residual_add(oled_ctx* ctx, const void* x, const void* r, void* y, size_t n) {
  if (!ctx || !x || !r || !y) return OLED_ERR_INVALID_ARG;
  if (n == 0) return OLED_OK;
  launch_residual_add(ctx->stream, static_cast<const uint16_t*>(x), static_cast<const uint16_t*>(r),
                      static_cast<uint16_t*>(y), n);
  ctx->launches += 1;
  OLED_CUDA(ctx, cudaGetLastError());
  return OLED_OK;
}

int oled_set_option(oled_ctx* ctx, int32_t option, int64_t value) {
  if (!ctx) return OLED_ERR_INVALID_ARG;
  switch (option) {
    case OLED_OPT_FFN_IMPL:
      if (value != 0 && value != 1) return OLED_ERR_INVALID_ARG;
      if (value == 1 && ctx->shape.expert_format != OLED_EXPERTS_BF16) return OLED_ERR_INVALID_ARG;
      ctx->ffn_impl = (int)value;
      return OLED_OK;
    case OLED_OPT_PROFILE:
      ctx->profile = value != 0;
      return OLED_OK;
    case OLED_OPT_POLICY:
      if (value < OLED_POLICY_PRIORITY || value > OLED_POLICY_LFU) return OLED_ERR_INVALID_ARG;
      for (auto& L : ctx->layers) L.cache.policy = (int32_t)value;
      return OLED_OK;
    case OLED_OPT_ADAPT_PERIOD:
      if (value < 0) return OLED_ERR_INVALID_ARG;
      ctx->adapt_period = (int)value;
      return OLED_OK;
    case OLED_OPT_TEST_WITHHOLD_LOADS:
      ctx->withhold_loads = value != 0 ? 1 : 0;
      return OLED_OK;
    case OLED_OPT_SELF_CHECK:
      ctx->self_check = value != 0 ? 1 : 0;
      return OLED_OK;
    case OLED_OPT_TEST_CORRUPT_PERM:
      ctx->corrupt_perm = value != 0 ? 1 : 0;
      return OLED_OK;
    case OLED_OPT_MISS_CHUNK:
      if (value < 1) return OLED_ERR_INVALID_ARG;
      ctx->miss_chunk = (int)std::min<int64_t>(value, OLED_MAX_EXPERTS);
      return OLED_OK;
    case OLED_OPT_SPLIT_LAST_FILL:
      ctx->split_last = value != 0;
      return OLED_OK;
    case OLED_OPT_FUSE_FFN:
      if (value < 0 || value > 2) return OLED_ERR_INVALID_ARG;
      ctx->fuse_ffn = (int)value;
      return OLED_OK;
    case OLED_OPT_FUSE_COMBINE:
      ctx->fuse_combine = value != 0;
      return OLED_OK;
    case OLED_OPT_PDL:
      pdl_set_allowed(value != 0);
      return OLED_OK;
    case OLED_OPT_TIMELINE:
      ctx->timeline_on = value != 0;
      return OLED_OK;
    case OLED_OPT_FP8_DIRECT:
      ctx->fp8_direct = value != 0;
      return OLED_OK;
    case OLED_OPT_L2_PREFETCH:
      ctx->l2_prefetch = value;
      return OLED_OK;
    case OLED_OPT_FFN_PAIRS:
      ctx->maps.use_pairs = value != 0;
      return OLED_OK;
    case OLED_OPT_GATHER_IN_FFN:
      ctx->gather_in_ffn = value != 0;
      return OLED_OK;
    default:
      return OLED_ERR_INVALID_ARG;
  }
}

int oled_profile_read(oled_ctx* ctx, int32_t kernel, int32_t reset, oled_kernel_profile* out) {
  if (!ctx || !out || kernel < 0 || kernel >= OLED_N_KERNELS) return OLED_ERR_INVALID_ARG;
  const int rc = sync_all(ctx);
  prof_resolve(ctx);
  *out = ctx->prof_acc[kernel];
  if (reset) ctx->prof_acc[kernel] = oled_kernel_profile{};
  return rc;
}

int oled_clear_status(oled_ctx* ctx) {
  if (!ctx) return OLED_ERR_INVALID_ARG;
  OLED_CUDA(ctx, cudaStreamSynchronize(ctx->copy_stream));
  memset(ctx->h_status, 0, kStatusWords * sizeof(uint32_t));
  ctx->h_status[kStatusCheckIndex] = kStatusNoIndex;
  OLED_CUDA(ctx, cudaMemcpyAsync(ctx->d_status, ctx->h_status, kStatusWords * sizeof(uint32_t), cudaMemcpyHostToDevice,
                                 ctx->stream));
  OLED_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
  return OLED_OK;
}

int oled_self_check_report(oled_ctx* ctx, uint32_t* flags, int32_t* first_index, uint32_t* guard_mask) {
  if (!ctx) return OLED_ERR_INVALID_ARG;
  const int rc = sync_all(ctx);
  if (rc != OLED_OK && rc != OLED_ERR_SELF_CHECK && rc != OLED_ERR_TIMEOUT) return rc;
  const uint32_t f = ctx->h_status[kStatusCheckFlags];
  if (flags) *flags = f;
  if (first_index) *first_index = f != 0 ? (int32_t)ctx->h_status[kStatusCheckIndex] : -1;
  if (guard_mask) *guard_mask = ctx->h_status[kStatusGuardMask];
  return OLED_OK;
}

int oled_policy_time(oled_ctx* ctx, uint64_t* nanoseconds, uint64_t* runs) {
  if (!ctx || !nanoseconds || !runs) return OLED_ERR_INVALID_ARG;
  *nanoseconds = ctx->policy_ns;
  *runs = ctx->policy_runs;
  return OLED_OK;
}

int oled_launch_count(oled_ctx* ctx, uint64_t* out) {
  if (!ctx || !out) return OLED_ERR_INVALID_ARG;
  *out = ctx->launches;
  return OLED_OK;
}

int oled_synchronize(oled_ctx* ctx) {
  if (!ctx) return OLED_ERR_INVALID_ARG;
  return sync_all(ctx);
}

void oled_destroy(oled_ctx* ctx) { free_ctx(ctx); }

int oled_last_cuda_error(oled_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

// ---- host-only policy simulator -----------------------------------------------------------
struct oled_policy {
  LayerCacheState cache;
  std::shared_ptr<SlotPool> pool;  // one per simulated layer, or shared by the layers of a simulated stack
  StepPlan plan;
  uint64_t fills_reused = 0;
  int32_t adapt_lo = 1;
};

int oled_policy_create(int32_t n_experts, int32_t capacity, int32_t pool_slots, oled_policy** out) {
  if (!out || n_experts <= 0 || n_experts > OLED_MAX_EXPERTS || capacity <= 0 || capacity > n_experts ||
      pool_slots < capacity)
    return OLED_ERR_INVALID_ARG;
  oled_policy* p = new (std::nothrow) oled_policy();
  if (!p) return OLED_ERR_OOM;
  p->cache.init(n_experts, capacity);
  p->pool = std::make_shared<SlotPool>();
  p->pool->init(pool_slots);
  *out = p;
  return OLED_OK;
}

int oled_policy_create_stack(int32_t n_layers, int32_t n_experts, const int32_t* capacity, int32_t staging_slots,
                             oled_policy** out, int32_t* pool_slots) {
  if (!out || !capacity || n_layers <= 0 || n_experts <= 0 || n_experts > OLED_MAX_EXPERTS || staging_slots < 0)
    return OLED_ERR_INVALID_ARG;
  long long total = 0;
  for (int32_t l = 0; l < n_layers; ++l) {
    if (capacity[l] <= 0 || capacity[l] > n_experts) return OLED_ERR_INVALID_ARG;
    total += capacity[l];
  }
  const PoolPlan pp = pool_plan(n_experts, total, staging_slots);  // the sizing rule of oled_create()
  auto pool = std::make_shared<SlotPool>();
  pool->init((int32_t)pp.n_slots);
  for (int32_t l = 0; l < n_layers; ++l) {
    oled_policy* p = new (std::nothrow) oled_policy();
    if (!p) {
      for (int32_t j = 0; j < l; ++j) delete out[j];
      return OLED_ERR_OOM;
    }
    p->cache.init(n_experts, capacity[l]);
    p->pool = pool;
    p->adapt_lo = pp.adapt_lo;
    out[l] = p;
  }
  if (pool_slots) *pool_slots = (int32_t)pp.n_slots;
  return OLED_OK;
}

int oled_policy_step(oled_policy* p, const int32_t* counts, const uint64_t* scores, uint8_t* resident_before,
                     uint8_t* resident_after, int32_t* slot_of, int32_t* n_hits, int32_t* n_misses,
                     int32_t* n_evictions) {
  if (!p || !counts || !scores) return OLED_ERR_INVALID_ARG;
  if (!plan_step(p->cache, *p->pool, counts, scores, p->plan)) return OLED_ERR_NO_SLOT;
  const size_t E = (size_t)p->cache.n_experts;
  if (resident_before) memcpy(resident_before, p->plan.before.data(), E);
  if (resident_after) memcpy(resident_after, p->plan.after.data(), E);
  if (slot_of)
    for (size_t e = 0; e < E; ++e) slot_of[e] = counts[e] > 0 ? p->cache.slot_of[e] : -1;
  if (n_hits) *n_hits = (int32_t)p->plan.hits.size();
  if (n_misses) *n_misses = (int32_t)p->plan.misses.size();
  if (n_evictions) *n_evictions = p->plan.n_evictions;
  p->fills_reused += (uint64_t)p->plan.n_fills_reused;
  finish_step(p->cache, *p->pool, p->plan);
  return OLED_OK;
}

void oled_policy_destroy(oled_policy* p) { delete p; }

int oled_policy_set_policy(oled_policy* p, int32_t policy) {
  if (!p || policy < OLED_POLICY_PRIORITY || policy > OLED_POLICY_LFU) return OLED_ERR_INVALID_ARG;
  p->cache.policy = policy;
  return OLED_OK;
}

int oled_policy_fills_reused(oled_policy* p, uint64_t* out) {
  if (!p || !out) return OLED_ERR_INVALID_ARG;
  *out = p->fills_reused;
  return OLED_OK;
}

int oled_policy_adapt(oled_policy** layers, int32_t n_layers, int32_t total_capacity, int32_t* new_capacity) {
  if (!layers || n_layers <= 0 || !new_capacity) return OLED_ERR_INVALID_ARG;
  std::vector<LayerCacheState*> ls;
  for (int32_t l = 0; l < n_layers; ++l) {
    if (!layers[l]) return OLED_ERR_INVALID_ARG;
    ls.push_back(&layers[l]->cache);
  }
  if (total_capacity < n_layers || total_capacity > (int64_t)n_layers * ls[0]->n_experts)
    return OLED_ERR_INVALID_ARG;
  const std::vector<int32_t> caps = adaptive_capacities(ls, total_capacity, layers[0]->adapt_lo);
  for (int32_t l = 0; l < n_layers; ++l) {
    shrink_to(*ls[l], *layers[l]->pool, caps[l]);
    new_capacity[l] = caps[l];
  }
  return OLED_OK;
}

}  // extern "C"
