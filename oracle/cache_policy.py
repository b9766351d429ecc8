"""CPU oracle for the expert-cache policy of a denoising step.  TEST INFRASTRUCTURE ONLY.

A scalar simulation, in the paper's notation, of:

* the sets of Sec. 4.2 (problem formulation): A (activated by the gate),
  R (resident in the layer's GPU cache *before* execution), M = A \\ R
  (misses);  G, the misses fetched to the GPU, is all of M here because the
  hot path has no CPU execution path;
* the expert reuse priority of Sec. 4.3,
      p_e = sum_{t in T_e} g_{t,e} * psi(c_t)  /  sum_{e'} sum_{t in T_e'} g_{t,e'} * psi(c_t),
  psi(c) = c, with resident-but-not-activated experts set to priority zero;
* the cache update of Sec. 4.2,  R' = Top_C( R u G, p ).

So that two implementations can agree on every keep/evict decision bit for
bit, the numerator is accumulated as an integer: each term g*psi(c) is one
rounded fp32 product v, quantised to floor(v * 2^32), summed in 64-bit
integers (order-free).  Ranking uses these integer scores s_e; p_e = s_e/sum s
is derived for reporting.  Ties in the ranking go to the lower expert index.

Also here, for the comparison points of the paper's evaluation:

* LRU and LFU retention (Sec. 5.1 "Naive-LRU ... inter-iteration expert cache with LRU
  replacement"; Sec. 5.3 compares Priority with LRU and LFU): the same cache update with the
  value of a candidate being the index of the last layer execution that activated it (LRU) or
  the number of executions that activated it so far (LFU);
* the ideal cache bound of Sec. 5.1 (clairvoyant: as many of the activated experts as fit are
  already resident): hits = min(C, #A);
* the effective transfer ratio of Sec. 5.3: fetched experts that are retained and activated
  again at the layer's next execution, over all fetched experts;
* layer-adaptive cache sizing (Sec. 4.3): w_l = a_l * u_l, C_l = C_total * w_l / sum_j w_j.

Pins (tests/test_oracle_policy.py, tests/test_oracle_adaptive.py): hand-worked priority cases,
sum p = 1, brute force over all C-subsets, subset/size invariants, stale-first eviction,
hit/miss accounting identities, full-capacity and repeated-input cases; LRU / LFU against
textbook list-based caches on single-access traces; apportionment against its defining
properties and a hand case.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Set

import numpy as np

F32 = np.float32
_TWO32 = F32(4294967296.0)


def psi(c: np.ndarray) -> np.ndarray:
    """psi(c) = c (Sec. 4.3 default), clamped to [0,1]; NaN counts as 0."""
    c = np.asarray(c, dtype=F32)
    c = np.where(np.isnan(c), F32(0.0), c)
    return np.minimum(np.maximum(c, F32(0.0)), F32(1.0)).astype(F32)


def reuse_scores(ids: np.ndarray, gate: np.ndarray, conf: np.ndarray, n_experts: int) -> List[int]:
    """Integer numerators s_e of the reuse priority (Sec. 4.3 priority equation)."""
    ids = np.asarray(ids)
    gate = np.asarray(gate, dtype=F32)
    w = psi(conf)
    s = [0] * n_experts
    t, k = ids.shape
    for tt in range(t):
        for j in range(k):
            v = F32(gate[tt, j] * w[tt])                 # one rounded fp32 product
            # exact scaling, then floor; a NaN product (non-finite activations) adds nothing
            q = 0 if v != v else int(np.floor(np.float64(v) * 4294967296.0))
            s[int(ids[tt, j])] += q
    return s


def priorities(scores: List[int]) -> np.ndarray:
    """p_e = s_e / sum_e' s_e' (all zero when the denominator is zero)."""
    tot = sum(scores)
    if tot == 0:
        return np.zeros(len(scores), dtype=np.float64)
    return np.array([sc / tot for sc in scores], dtype=np.float64)


def retain_top_c(resident: Set[int], fetched: Set[int], scores: List[int], activated: Set[int],
                 capacity: int) -> Set[int]:
    """R' = Top_C(R u G, p): keep the C candidates with the highest priority.

    Residents that were not activated have priority zero (Sec. 4.3); ties go
    to the lower expert index.
    """
    cand = sorted(resident | fetched)
    value = {e: (scores[e] if e in activated else 0) for e in cand}
    ranked = sorted(cand, key=lambda e: (-value[e], e))
    return set(ranked[:capacity])


def retain_by_value(resident: Set[int], fetched: Set[int], value: List[int], capacity: int) -> Set[int]:
    """Top_C(R u G, value) for the LRU / LFU comparison policies: the value of a candidate is
    taken as it stands (no stale rule); ties go to the lower expert index."""
    cand = sorted(resident | fetched)
    ranked = sorted(cand, key=lambda e: (-value[e], e))
    return set(ranked[:capacity])


def ideal_hits(n_activated: int, capacity: int) -> int:
    """Hits of the clairvoyant bound (Sec. 5.1): min(C, #A) per layer execution."""
    return min(capacity, n_activated)


@dataclass
class LayerStats:
    steps: int = 0
    hits: int = 0
    misses: int = 0
    bytes_moved: int = 0
    evictions: int = 0
    active_experts: int = 0
    assignments: int = 0
    fills_reused: int = 0      # fetched, retained and activated again at the next execution
    ideal_hits: int = 0        # hits of the clairvoyant bound under the same capacity

    def add(self, o: "LayerStats") -> None:
        for f in ("steps", "hits", "misses", "bytes_moved", "evictions", "active_experts",
                  "assignments", "fills_reused", "ideal_hits"):
            setattr(self, f, getattr(self, f) + getattr(o, f))


@dataclass
class LayerCache:
    """Resident set and counters of one layer's cache pool (Sec. 4.1: one pool per layer)."""
    n_experts: int
    capacity: int
    expert_bytes: int
    resident: Set[int] = field(default_factory=set)
    stats: LayerStats = field(default_factory=LayerStats)
    policy: str = "priority"            # "priority" (Sec. 4.3), "lru", "lfu"
    last_used: List[int] = field(default_factory=list)   # LRU: last execution that activated e
    frequency: List[int] = field(default_factory=list)   # LFU: executions that activated e
    last_value: List[int] = field(default_factory=list)  # value of each expert at the last update
    pending_fills: Set[int] = field(default_factory=set)  # fetched and retained at the last execution
    # accumulators of the current sizing period (Sec. 4.3 runtime statistics)
    period_steps: int = 0
    period_active: int = 0
    period_hits: int = 0
    period_capacity: int = 0

    def __post_init__(self):
        self.last_used = [0] * self.n_experts
        self.frequency = [0] * self.n_experts
        self.last_value = [0] * self.n_experts

    def step(self, ids: np.ndarray, gate: np.ndarray, conf: np.ndarray) -> dict:
        """One layer execution: hits/misses against the pre-step R, then retention."""
        ids = np.asarray(ids)
        activated = set(int(v) for v in ids.reshape(-1))
        before = set(self.resident)
        hits = activated & before
        misses = activated - before
        scores = reuse_scores(ids, gate, conf, self.n_experts)
        now = self.stats.steps + 1
        for e in activated:
            self.last_used[e] = now
            self.frequency[e] += 1
        if self.policy == "priority":
            after = retain_top_c(before, misses, scores, activated, self.capacity)
            value = [scores[e] if e in activated else 0 for e in range(self.n_experts)]
        else:
            value = list(self.last_used if self.policy == "lru" else self.frequency)
            after = retain_by_value(before, misses, value, self.capacity)
        self.last_value = value
        self.stats.fills_reused += len(self.pending_fills & activated)
        self.stats.ideal_hits += ideal_hits(len(activated), self.capacity)
        self.pending_fills = misses & after
        self.period_steps += 1
        self.period_active += len(activated)
        self.period_hits += len(hits)
        self.period_capacity += self.capacity
        self.resident = after
        st = self.stats
        st.steps += 1
        st.hits += len(hits)
        st.misses += len(misses)
        st.bytes_moved += len(misses) * self.expert_bytes
        st.evictions += len(before - after)
        st.active_experts += len(activated)
        st.assignments += int(ids.size)
        return dict(activated=activated, resident_before=before, resident_after=after,
                    hits=hits, misses=misses, scores=scores, priority=priorities(scores))

    def shrink_to(self, capacity: int) -> int:
        """Set a new capacity; if fewer slots than residents remain, keep the residents with the
        highest value at the last update (ties to the lower id).  Returns the evictions."""
        self.capacity = capacity
        if len(self.resident) <= capacity:
            return 0
        ranked = sorted(self.resident, key=lambda e: (-self.last_value[e], e))
        kept = set(ranked[:capacity])
        n = len(self.resident) - len(kept)
        self.resident = kept
        self.pending_fills &= kept
        self.stats.evictions += n
        return n

    def reset(self) -> None:
        self.resident = set()
        self.stats = LayerStats()
        self.__post_init__()
        self.pending_fills = set()
        self.period_steps = self.period_active = self.period_hits = self.period_capacity = 0


# --------------------------------------------------------------------------
# Layer-adaptive cache sizing (Sec. 4.3, "From expert priority to layer-adaptive cache sizing")
# --------------------------------------------------------------------------
Q16 = 1 << 16


def apportion(weights: List[int], total: int, lo: int, hi: int) -> List[int]:
    """C_l = total * w_l / sum_j w_j in integers: floor of the quota clamped to [lo, hi], then
    the remaining units go one by one to the layer furthest below its quota (ties to the lower
    index), or are taken from the layer furthest above it (ties to the higher index)."""
    n = len(weights)
    sw = sum(weights)
    assert n * lo <= total <= n * hi
    if sw == 0:
        weights, sw = [1] * n, n
    c = [min(hi, max(lo, total * w // sw)) for w in weights]
    # deficit of layer l relative to its quota, scaled by sw: total*w_l - c_l*sw
    while sum(c) < total:
        cand = [l for l in range(n) if c[l] < hi]
        l = max(cand, key=lambda j: (total * weights[j] - c[j] * sw, -j))
        c[l] += 1
    while sum(c) > total:
        cand = [l for l in range(n) if c[l] > lo]
        l = min(cand, key=lambda j: (total * weights[j] - c[j] * sw, -j))
        c[l] -= 1
    return c


class AdaptiveSizer:
    """Smoothed per-layer statistics and the proportional allocation of Sec. 4.3.

    a_l: activation ratio (#A / E), u_l: cache utilisation (hits / capacity), both averaged
    over the layer executions of the period that just ended, held as Q16 fixed point and
    smoothed over periods by s <- (s + new) / 2 (integer floor); w_l = a_l * u_l.
    """

    def __init__(self, n_layers: int, n_experts: int):
        self.n_experts = n_experts
        self.a = [None] * n_layers
        self.u = [None] * n_layers

    def refresh(self, caches: List[LayerCache], total: int) -> List[int]:
        weights = []
        for l, c in enumerate(caches):
            if c.period_steps > 0:
                a_new = c.period_active * Q16 // (c.period_steps * self.n_experts)
                u_new = c.period_hits * Q16 // max(1, c.period_capacity)
                self.a[l] = a_new if self.a[l] is None else (self.a[l] + a_new) // 2
                self.u[l] = u_new if self.u[l] is None else (self.u[l] + u_new) // 2
                c.period_steps = c.period_active = c.period_hits = c.period_capacity = 0
            weights.append((self.a[l] or 0) * (self.u[l] or 0))
        return apportion(weights, total, 1, self.n_experts)
