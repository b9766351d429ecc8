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

// Retention value of a candidate: the paper's confidence- and gate-guided priority (Sec. 4.3),
// or the recency / frequency values of the LRU and LFU comparison policies (Sec. 5.1, 5.3).
enum Policy : int32_t { kPolicyPriority = 0, kPolicyLru = 1, kPolicyLfu = 2 };

struct LayerCacheState {
  int32_t n_experts = 0;
  int32_t capacity = 0;
  int32_t policy = kPolicyPriority;
  std::vector<int32_t> slot_of;   // expert -> slot, -1 = weights not in HBM
  std::vector<uint8_t> resident;  // R: the policy's resident set
  uint64_t executions = 0;        // layer executions so far
  std::vector<uint64_t> last_used;    // LRU: last execution that activated the expert
  std::vector<uint64_t> frequency;    // LFU: executions that activated the expert
  std::vector<uint64_t> last_value;   // value of every expert at the last update
  std::vector<uint8_t> pending_fill;  // fetched and retained at the last execution
  // statistics of the current sizing period and their smoothed Q16 values (Sec. 4.3)
  uint64_t period_steps = 0, period_active = 0, period_hits = 0, period_capacity = 0;
  int64_t a_q16 = -1, u_q16 = -1;     // -1: no period observed yet
  void init(int32_t e, int32_t c) {
    n_experts = e;
    capacity = c;
    slot_of.assign(e, -1);
    resident.assign(e, 0);
    clear_history();
  }
  void clear_history() {
    executions = 0;
    last_used.assign(n_experts, 0);
    frequency.assign(n_experts, 0);
    last_value.assign(n_experts, 0);
    pending_fill.assign(n_experts, 0);
    period_steps = period_active = period_hits = period_capacity = 0;
    a_q16 = u_q16 = -1;
  }
};

struct StepPlan {
  std::vector<int32_t> hits;           // A n R, ascending id
  std::vector<int32_t> misses;         // A \ R, ascending id
  std::vector<uint8_t> before, after;  // R and R'
  std::vector<int32_t> release_after;  // activated experts that are not retained
  int32_t n_evictions = 0;             // #(R \ R')
  int32_t n_active = 0;
  int32_t n_fills_reused = 0;          // fetched at the last execution, retained, activated again now
  int32_t capacity_used = 0;           // the layer's capacity at this execution
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
  plan.capacity_used = L.capacity;

  // values under the layer's policy (history is advanced on a copy: a failed plan changes nothing)
  const uint64_t now = L.executions + 1;
  std::vector<uint64_t> val(E);
  for (int32_t e = 0; e < E; ++e) {
    const bool act = counts[e] > 0;
    if (L.policy == kPolicyPriority) val[e] = act ? scores[e] : 0ull;   // stale residents: priority 0
    else if (L.policy == kPolicyLru) val[e] = act ? now : L.last_used[e];
    else val[e] = L.frequency[e] + (act ? 1 : 0);
  }
  auto value = [&](int32_t e) -> uint64_t { return val[e]; };
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
  // history, effective-transfer bookkeeping (Sec. 5.3) and sizing statistics (Sec. 4.3)
  plan.n_fills_reused = 0;
  for (int32_t e = 0; e < E; ++e) {
    const bool act = counts[e] > 0;
    if (act) {
      L.last_used[e] = now;
      L.frequency[e] += 1;
      if (L.pending_fill[e]) ++plan.n_fills_reused;
    }
    L.pending_fill[e] = (act && !plan.before[e] && plan.after[e]) ? 1 : 0;
  }
  L.last_value = val;
  L.executions = now;
  L.period_steps += 1;
  L.period_active += (uint64_t)plan.n_active;
  L.period_hits += plan.hits.size();
  L.period_capacity += (uint64_t)L.capacity;
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
  L.clear_history();
}

// New capacity for a layer.  If fewer slots than residents remain, the residents with the highest
// value at the last update stay (ties to the lower id); the others are evicted at once, which is a
// table update only.  Returns the number of evictions.
inline int32_t shrink_to(LayerCacheState& L, SlotPool& pool, int32_t capacity) {
  L.capacity = capacity;
  std::vector<int32_t> res;
  for (int32_t e = 0; e < L.n_experts; ++e)
    if (L.resident[e]) res.push_back(e);
  if ((int32_t)res.size() <= capacity) return 0;
  std::stable_sort(res.begin(), res.end(), [&](int32_t a, int32_t b) {
    if (L.last_value[a] != L.last_value[b]) return L.last_value[a] > L.last_value[b];
    return a < b;
  });
  for (size_t i = (size_t)capacity; i < res.size(); ++i) {
    const int32_t e = res[i];
    L.resident[e] = 0;
    L.pending_fill[e] = 0;
    if (L.slot_of[e] >= 0) pool.release(L.slot_of[e]);
    L.slot_of[e] = -1;
  }
  return (int32_t)res.size() - capacity;
}

// C_l = total * w_l / sum_j w_j in integers (Sec. 4.3 proportional allocation): floor of the quota
// clamped to [lo, hi]; spare units go one by one to the layer furthest below its quota (ties to the
// lower index), surplus units are taken from the layer furthest above it (ties to the higher index).
inline std::vector<int32_t> apportion(std::vector<uint64_t> w, int64_t total, int32_t lo, int32_t hi) {
  const size_t n = w.size();
  unsigned __int128 sw = 0;
  for (uint64_t x : w) sw += x;
  if (sw == 0) {
    w.assign(n, 1);
    sw = n;
  }
  std::vector<int32_t> c(n);
  int64_t sum = 0;
  for (size_t l = 0; l < n; ++l) {
    const int64_t q = (int64_t)(((unsigned __int128)total * w[l]) / sw);
    c[l] = (int32_t)std::min<int64_t>(hi, std::max<int64_t>(lo, q));
    sum += c[l];
  }
  auto deficit = [&](size_t l) -> __int128 {
    return (__int128)((unsigned __int128)total * w[l]) - (__int128)c[l] * (__int128)sw;
  };
  while (sum < total) {
    long best = -1;
    for (size_t l = 0; l < n; ++l)
      if (c[l] < hi && (best < 0 || deficit(l) > deficit((size_t)best))) best = (long)l;
    c[(size_t)best] += 1;
    ++sum;
  }
  while (sum > total) {
    long best = -1;
    for (size_t l = 0; l < n; ++l)
      if (c[l] > lo && (best < 0 || deficit(l) <= deficit((size_t)best))) best = (long)l;
    c[(size_t)best] -= 1;
    --sum;
  }
  return c;
}

// Layer-adaptive sizing (Sec. 4.3): w_l = a_l * u_l from the statistics of the period that just
// ended, smoothed over periods by s <- (s + new) / 2 in Q16; returns the new capacities.
// lo: smallest capacity a layer may be given (see pool_plan: a layer that shrinks further could
// need more transient slots during one of its steps than the pool has).
inline std::vector<int32_t> adaptive_capacities(std::vector<LayerCacheState*>& layers, int64_t total, int32_t lo = 1) {
  std::vector<uint64_t> w;
  for (LayerCacheState* L : layers) {
    if (L->period_steps > 0) {
      const int64_t a_new = (int64_t)(L->period_active * 65536ull / (L->period_steps * (uint64_t)L->n_experts));
      const int64_t u_new = (int64_t)(L->period_hits * 65536ull / std::max<uint64_t>(1, L->period_capacity));
      L->a_q16 = L->a_q16 < 0 ? a_new : (L->a_q16 + a_new) / 2;
      L->u_q16 = L->u_q16 < 0 ? u_new : (L->u_q16 + u_new) / 2;
      L->period_steps = L->period_active = L->period_hits = L->period_capacity = 0;
    }
    w.push_back((uint64_t)std::max<int64_t>(0, L->a_q16) * (uint64_t)std::max<int64_t>(0, L->u_q16));
  }
  return apportion(w, total, std::max<int32_t>(1, lo), layers.empty() ? 1 : layers[0]->n_experts);
}

// Size of the shared slot pool.  While layer l executes, the other layers hold at most
// C_total - C_l slots (the resident sets never exceed the capacities, also right after a
// resize) and layer l itself needs at most E (every expert activated), so the pool never runs
// out iff C_total + staging - (C_total - C_l) >= E, i.e. staging >= E - C_l for every capacity a
// layer can ever have.  Layer-adaptive sizing may shrink a layer down to `adapt_lo`; the default
// staging (E - 1) allows 1, a smaller caller-chosen staging raises the floor accordingly.
struct PoolPlan {
  int32_t staging;   // transient slots beyond the capacities
  int64_t n_slots;   // C_total + staging
  int32_t adapt_lo;  // smallest capacity layer-adaptive sizing may hand out
};
inline PoolPlan pool_plan(int32_t n_experts, int64_t total_capacity, int32_t staging_requested) {
  PoolPlan p;
  p.staging = staging_requested > 0 ? staging_requested : std::max<int32_t>(1, n_experts - 1);
  p.n_slots = total_capacity + p.staging;
  p.adapt_lo = std::max<int32_t>(1, n_experts - p.staging);
  return p;
}

}  // namespace oled
