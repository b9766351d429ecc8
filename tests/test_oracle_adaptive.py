"""Pins for the comparison policies (LRU, LFU, ideal bound, effective transfer ratio) and the
layer-adaptive cache sizing of the policy oracle."""
import itertools
from collections import OrderedDict

import numpy as np

from oracle import cache_policy as cp
from oracle import OracleStack

F32 = np.float32


def _one(e):
    return np.array([[e]]), np.array([[1.0]], F32), np.array([0.5], F32)


def test_lru_matches_textbook_lru_on_single_accesses():
    rng = np.random.default_rng(0)
    for cap in (1, 2, 3, 5):
        cache = cp.LayerCache(8, cap, 10, policy="lru")
        book = OrderedDict()
        for x in rng.integers(0, 8, size=200):
            x = int(x)
            cache.step(*_one(x))
            if x in book:
                book.move_to_end(x)
            else:
                if len(book) == cap:
                    book.popitem(last=False)        # least recently used
                book[x] = True
            assert cache.resident == set(book)


def test_lfu_matches_textbook_lfu_on_single_accesses():
    rng = np.random.default_rng(1)
    for cap in (1, 2, 4):
        cache = cp.LayerCache(6, cap, 10, policy="lfu")
        freq = [0] * 6
        book = set()
        for x in rng.integers(0, 6, size=300):
            x = int(x)
            cache.step(*_one(x))
            freq[x] += 1
            book.add(x)
            if len(book) > cap:                     # drop the least frequent, ties: the higher id
                book.remove(min(book, key=lambda e: (freq[e], -e)))
            assert cache.resident == book


def test_priority_policy_is_the_default_and_differs_from_lru():
    # two experts activated, capacity 1: priority keeps the one with the confident token,
    # LRU (both equally recent) keeps the lower id
    ids = np.array([[0], [1]])
    gate = np.array([[1.0], [1.0]], F32)
    conf = np.array([0.1, 0.9], F32)
    a, b = cp.LayerCache(4, 1, 10), cp.LayerCache(4, 1, 10, policy="lru")
    assert a.step(ids, gate, conf)["resident_after"] == {1}
    assert b.step(ids, gate, conf)["resident_after"] == {0}


def test_ideal_bound_and_it_dominates_every_policy():
    assert [cp.ideal_hits(a, 4) for a in (0, 3, 4, 9)] == [0, 3, 4, 4]
    rng = np.random.default_rng(2)
    caches = {p: cp.LayerCache(16, 5, 10, policy=p) for p in ("priority", "lru", "lfu")}
    ideal = 0
    for _ in range(50):
        ids = np.stack([rng.permutation(16)[:2] for _ in range(4)])
        g = rng.dirichlet(np.ones(2), size=4).astype(F32)
        c = rng.uniform(0, 1, 4).astype(F32)
        for ch in caches.values():
            r = ch.step(ids, g, c)
        ideal += cp.ideal_hits(len(r["activated"]), 5)
    assert all(ch.stats.hits <= ideal for ch in caches.values())


def test_effective_transfer_counter_by_hand():
    cache = cp.LayerCache(6, 2, 10)
    two = lambda a, b: (np.array([[a], [b]]), np.array([[1.0], [1.0]], F32), np.array([0.9, 0.5], F32))
    cache.step(*two(0, 1))            # fetch 0, 1; both retained
    assert cache.stats.fills_reused == 0 and cache.pending_fills == {0, 1}
    cache.step(*two(1, 2))            # 1 reused; 2 fetched; candidates {0,1,2}: keep 1 (0.9), 2 (0.5)
    assert cache.stats.fills_reused == 1 and cache.resident == {1, 2} and cache.pending_fills == {2}
    cache.step(*two(3, 4))            # 2 not activated: not reused
    assert cache.stats.fills_reused == 1 and cache.stats.misses == 5


def test_apportion_properties():
    rng = np.random.default_rng(3)
    assert cp.apportion([1, 1, 2], 10, 1, 10) == [3, 2, 5]        # quotas 2.5, 2.5, 5: tie to lower index
    assert cp.apportion([0, 0, 0, 0], 8, 1, 8) == [2, 2, 2, 2]     # no information: uniform
    assert cp.apportion([5, 0], 6, 1, 4) == [4, 2]                 # cap binds, rest flows on
    assert cp.apportion([0, 9], 6, 1, 8) == [1, 5]                 # floor of one slot per layer
    for _ in range(300):
        n = int(rng.integers(1, 9))
        hi = int(rng.integers(2, 20))
        total = int(rng.integers(n, n * hi + 1))
        w = [int(v) for v in rng.integers(0, 1000, size=n)]
        c = cp.apportion(w, total, 1, hi)
        assert sum(c) == total and all(1 <= v <= hi for v in c)
        sw = sum(w)
        if sw and all(1 <= total * x // sw and -(-total * x // sw) <= hi for x in w):
            # nothing clamps: every share is the floor or the ceiling of its quota (Hamilton)
            assert all(total * x // sw <= v <= -(-total * x // sw) for x, v in zip(w, c))
        for i, j in itertools.combinations(range(n), 2):          # more weight, never fewer slots
            if w[i] > w[j]:
                assert c[i] >= c[j]


def test_adaptive_sizer_hand_case_and_uniform_case():
    # layer 0: 4 of 8 experts active, 2 hits in 4 slots -> a = .5, u = .5, w = .25
    # layer 1: 8 of 8 active, 4 hits in 4 slots       -> a = 1,  u = 1,  w = 1
    # quotas of 8 slots: 1.6 and 6.4 -> floors 1, 6 -> the spare slot goes to layer 0 (remainder .6)
    caches = [cp.LayerCache(8, 4, 10), cp.LayerCache(8, 4, 10)]
    for c, (act, hit) in zip(caches, ((4, 2), (8, 4))):
        c.period_steps, c.period_active, c.period_hits, c.period_capacity = 5, 5 * act, 5 * hit, 5 * 4
    sizer = cp.AdaptiveSizer(2, 8)
    assert sizer.refresh(caches, 8) == [2, 6]
    assert all(c.period_steps == 0 for c in caches)               # a new period starts
    # identical statistics on every layer: the uniform allocation is a fixed point
    caches = [cp.LayerCache(8, 3, 10) for _ in range(4)]
    for c in caches:
        c.period_steps, c.period_active, c.period_hits, c.period_capacity = 5, 20, 10, 15
    assert cp.AdaptiveSizer(4, 8).refresh(caches, 12) == [3, 3, 3, 3]


def test_smoothing_halves_the_distance_each_period():
    c = [cp.LayerCache(8, 4, 10)]
    s = cp.AdaptiveSizer(1, 8)
    c[0].period_steps, c[0].period_active, c[0].period_hits, c[0].period_capacity = 1, 8, 4, 4
    s.refresh(c, 4)
    assert s.a[0] == cp.Q16 and s.u[0] == cp.Q16
    c[0].period_steps, c[0].period_active, c[0].period_hits, c[0].period_capacity = 1, 0, 0, 4
    s.refresh(c, 4)
    assert s.a[0] == cp.Q16 // 2 and s.u[0] == cp.Q16 // 2
    s.refresh(c, 4)                                               # no execution in the period: unchanged
    assert s.a[0] == cp.Q16 // 2


def test_shrink_keeps_the_most_valuable_residents():
    cache = cp.LayerCache(6, 4, 10)
    ids = np.array([[0], [1], [2], [3]])
    cache.step(ids, np.ones((4, 1), F32), np.array([0.2, 0.9, 0.9, 0.4], F32))
    assert cache.resident == {0, 1, 2, 3}
    assert cache.shrink_to(2) == 2 and cache.resident == {1, 2} and cache.capacity == 2
    assert cache.shrink_to(3) == 0 and cache.resident == {1, 2}
    assert cache.stats.evictions == 2


def test_stack_adapt_capacity_conserves_the_budget_and_moves_slots_to_demand():
    st = OracleStack(2, 256, 8, 1, 128, [3, 3])
    rng = np.random.default_rng(5)
    for it in range(5):
        # layer 0 always uses the same expert; layer 1 cycles over many
        st.policy_step(0, np.array([[0]]), np.array([[1.0]], F32), np.array([0.9], F32))
        ids = np.stack([rng.permutation(8)[:1] for _ in range(6)])
        st.policy_step(1, ids, np.ones((6, 1), F32), rng.uniform(0.1, 1, 6).astype(F32))
    caps = st.adapt_capacity()
    assert sum(caps) == 6 and caps[1] > caps[0] >= 1
    assert [c.capacity for c in st.caches] == caps
    assert all(len(c.resident) <= c.capacity for c in st.caches)
