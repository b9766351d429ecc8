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

Pins (tests/test_oracle_policy.py): hand-worked priority cases, sum p = 1,
brute force over all C-subsets, subset/size invariants, stale-first eviction,
hit/miss accounting identities, full-capacity and repeated-input cases.
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
            q = int(np.floor(np.float64(v) * 4294967296.0))   # exact scaling, then floor
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


@dataclass
class LayerStats:
    steps: int = 0
    hits: int = 0
    misses: int = 0
    bytes_moved: int = 0
    evictions: int = 0
    active_experts: int = 0
    assignments: int = 0

    def add(self, o: "LayerStats") -> None:
        for f in ("steps", "hits", "misses", "bytes_moved", "evictions", "active_experts",
                  "assignments"):
            setattr(self, f, getattr(self, f) + getattr(o, f))


@dataclass
class LayerCache:
    """Resident set and counters of one layer's cache pool (Sec. 4.1: one pool per layer)."""
    n_experts: int
    capacity: int
    expert_bytes: int
    resident: Set[int] = field(default_factory=set)
    stats: LayerStats = field(default_factory=LayerStats)

    def step(self, ids: np.ndarray, gate: np.ndarray, conf: np.ndarray) -> dict:
        """One layer execution: hits/misses against the pre-step R, then retention."""
        ids = np.asarray(ids)
        activated = set(int(v) for v in ids.reshape(-1))
        before = set(self.resident)
        hits = activated & before
        misses = activated - before
        scores = reuse_scores(ids, gate, conf, self.n_experts)
        after = retain_top_c(before, misses, scores, activated, self.capacity)
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

    def reset(self) -> None:
        self.resident = set()
        self.stats = LayerStats()
