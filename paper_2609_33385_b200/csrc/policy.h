// Host-side cache policy of the denoise step: hit/miss resolution against the resident set
// before execution (paper Sec. 4.2: A, R, M = A \ R), the cache update
// R' = Top_C(R u G, p) (Sec. 4.2) with G = M, stale residents at priority zero (Sec. 4.3),
// and the slot bookkeeping behind the expert->slot indirection table.
//
// Integer-only: priorities arrive as the 64-bit integer numerators of the Sec. 4.3 priority
// equation, so every keep/evict decision is exact.  No CUDA in this file.
#pragma once
#include <algorithm>
#include <cstdint>
#include <vector>

namespace oled {

// Physical expert slots shared by all layers.  A layer at rest owns at most C_l of them; during
// a step it may borrow more for misses that will not be retained.
struct SlotPool {
  std::vector<int32_t> free_;
  void init(int32_t n_slots) {
    free_.clear();
    for (int32_t s = n_slots - 1; s >= 0; --s) free_.push_back(s);  // pop_back hands out 0,1,2,...
  }
  size_t n_free() const { return free_.size(); }
  int32_t alloc() {
    int32_t s = free_.back();
    free_.pop_back();
    return s;
  }
  void release(int32_t s) { free_.push_back(s); }
};

struct LayerCacheState {
  int32_t n_experts = 0;
  int32_t capacity = 0;
  std::vector<int32_t> slot_of;   // expert -> slot, -1 = weights not in HBM
  std::vector<uint8_t> resident;  // R: the policy's resident set
  void init(int32_t e, int32_t c) {
    n_experts = e;
    capacity = c;
    slot_of.assign(e, -1);
    resident.assign(e, 0);
  }
};

struct StepPlan {
  std::vector<int32_t> hits;           // A n R, ascending id
  std::vector<int32_t> misses;         // A \ R, ascending id
  std::vector<uint8_t> before, after;  // R and R'
  std::vector<int32_t> release_after;  // activated experts that are not retained
  int32_t n_evictions = 0;             // #(R \ R')
  int32_t n_active = 0;
};

// Decide the step.  Returns false (and changes nothing) if the pool cannot hold the misses.
// On success every activated expert has a slot in L.slot_of; the caller copies the misses
// into theirs, runs the FFN, then calls finish_step().
inline bool plan_step(LayerCacheState& L, SlotPool& pool, const int32_t* counts,
                      const uint64_t* scores, StepPlan& plan) {
  const int32_t E = L.n_experts;
  plan.hits.clear();
  plan.misses.clear();
  plan.release_after.clear();
  plan.before = L.resident;
  plan.after.assign(E, 0);

  std::vector<int32_t> cand;
  for (int32_t e = 0; e < E; ++e) {
    const bool act = counts[e] > 0;
    if (act && L.resident[e]) plan.hits.push_back(e);
    if (act && !L.resident[e]) plan.misses.push_back(e);
    if (act || L.resident[e]) cand.push_back(e);
  }
  plan.n_active = (int32_t)(plan.hits.size() + plan.misses.size());

  auto value = [&](int32_t e) -> uint64_t { return counts[e] > 0 ? scores[e] : 0ull; };
  std::stable_sort(cand.begin(), cand.end(), [&](int32_t a, int32_t b) {
    const uint64_t va = value(a), vb = value(b);
    if (va != vb) return va > vb;
    return a < b;
  });
  const size_t keep = std::min<size_t>(cand.size(), (size_t)L.capacity);
  for (size_t i = 0; i < keep; ++i) plan.after[cand[i]] = 1;

  // Slots of residents that are neither activated nor retained can be reused at once.
  size_t stale_evicted = 0;
  plan.n_evictions = 0;
  for (int32_t e = 0; e < E; ++e) {
    if (L.resident[e] && !plan.after[e]) {
      ++plan.n_evictions;
      if (counts[e] <= 0) ++stale_evicted;
    }
  }
  if (pool.n_free() + stale_evicted < plan.misses.size()) return false;

  for (int32_t e = 0; e < E; ++e) {
    if (L.resident[e] && !plan.after[e] && counts[e] <= 0) {
      pool.release(L.slot_of[e]);
      L.slot_of[e] = -1;
    }
  }
  for (int32_t e : plan.misses) L.slot_of[e] = pool.alloc();
  for (int32_t e = 0; e < E; ++e)
    if (counts[e] > 0 && !plan.after[e]) plan.release_after.push_back(e);
  L.resident = plan.after;
  return true;
}

// After the step's FFN work has been enqueued: give back the slots of activated experts that
// are not retained.  (They are reused only after a later host synchronisation that follows
// this step's kernels in stream order.)
inline void finish_step(LayerCacheState& L, SlotPool& pool, const StepPlan& plan) {
  for (int32_t e : plan.release_after) {
    pool.release(L.slot_of[e]);
    L.slot_of[e] = -1;
  }
}

inline void drop_all(LayerCacheState& L, SlotPool& pool) {
  for (int32_t e = 0; e < L.n_experts; ++e) {
    if (L.slot_of[e] >= 0) pool.release(L.slot_of[e]);
    L.slot_of[e] = -1;
    L.resident[e] = 0;
  }
}

}  // namespace oled
