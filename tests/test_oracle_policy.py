"""Pins for the cache-policy oracle (priority, Top-C retention, hit/miss accounting)."""
import itertools
import os

import numpy as np
import pytest

from oracle import cache_policy as cp
from oracle import OracleStack
from paper_2609_33385_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
F32 = np.float32


# ------------------------------------------------------------------ fixtures from text files
def _priority_cases():
    cases, cur = [], None
    for line in open(os.path.join(GOLD, "priority_cases.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, _, rest = line.partition(" ")
        if key == "case":
            cur = {"name": rest}
            cases.append(cur)
        elif key == "experts":
            cur["e"] = int(rest)
        elif key in ("ids", "gate"):
            rows = [r.split() for r in rest.split(";")]
            cur[key] = np.array(rows, dtype=np.int32 if key == "ids" else F32)
        else:
            cur[key] = np.array(rest.split(), dtype=np.float64)
    return cases


def _retention_cases():
    out = []
    for line in open(os.path.join(GOLD, "retention_cases.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        parts = {p.split()[0]: [int(v) for v in p.split()[1:]] for p in line.split("|")}
        out.append(parts)
    return out


@pytest.mark.parametrize("case", _priority_cases(), ids=lambda c: c["name"])
def test_priority_hand_cases(case):
    s = cp.reuse_scores(case["ids"], case["gate"], case["conf"].astype(F32), case["e"])
    p = cp.priorities(s)
    assert np.allclose(p, case["p"], atol=2e-7)
    assert abs(p.sum() - 1.0) < 1e-12


@pytest.mark.parametrize("case", _retention_cases())
def test_retention_hand_cases(case):
    got = cp.retain_top_c(set(case["R"]), set(case["A"]) - set(case["R"]), case["s"],
                          set(case["A"]), case["C"][0])
    assert got == set(case["R'"])


# ------------------------------------------------------------------ scores
def test_score_quantisation_by_hand():
    # g = 1, c = fl32(0.8) = 13421773 * 2^-24  ->  floor(v * 2^32) = 13421773 * 256
    s = cp.reuse_scores(np.array([[1]]), np.array([[1.0]], F32), np.array([0.8], F32), 3)
    assert s == [0, 13421773 * 256, 0]
    # product rounded once in fp32: 0.3 * 0.7
    v = F32(F32(0.3) * F32(0.7))
    s = cp.reuse_scores(np.array([[0]]), np.array([[0.3]], F32), np.array([0.7], F32), 1)
    assert s == [int(np.float64(v) * 2.0 ** 32)]


def test_scores_zero_iff_not_activated_and_sum_to_one():
    rng = np.random.default_rng(3)
    t, k, e = 40, 4, 32
    ids = np.stack([rng.permutation(e)[:k] for _ in range(t)]).astype(np.int32)
    g = rng.dirichlet(np.ones(k), size=t).astype(F32)
    c = rng.uniform(0.05, 1.0, size=t).astype(F32)
    s = cp.reuse_scores(ids, g, c, e)
    act = set(ids.reshape(-1).tolist())
    assert all((s[i] > 0) == (i in act) for i in range(e))
    p = cp.priorities(s)
    assert abs(p.sum() - 1.0) < 1e-12
    # against the definition evaluated in fp64
    num = np.zeros(e)
    for tt in range(t):
        for j in range(k):
            num[ids[tt, j]] += float(g[tt, j]) * float(c[tt])
    assert np.allclose(p, num / num.sum(), rtol=1e-6, atol=1e-9)


def test_scores_order_independent_and_scale_invariant_ranking():
    rng = np.random.default_rng(4)
    t, k, e = 16, 2, 8
    ids = np.stack([rng.permutation(e)[:k] for _ in range(t)]).astype(np.int32)
    g = rng.dirichlet(np.ones(k), size=t).astype(F32)
    c = rng.uniform(0.1, 1.0, size=t).astype(F32)
    s = cp.reuse_scores(ids, g, c, e)
    perm = rng.permutation(t)
    assert cp.reuse_scores(ids[perm], g[perm], c[perm], e) == s
    half = cp.reuse_scores(ids, g, (c * F32(0.5)).astype(F32), e)      # exact halving
    rank = lambda v: sorted(range(e), key=lambda i: (-v[i], i))
    assert rank(half) == rank(s)


def test_psi_clamps_and_all_zero_priorities():
    assert cp.psi(np.array([-1.0, 0.25, 2.0, np.nan], F32)).tolist() == [0.0, 0.25, 1.0, 0.0]
    s = cp.reuse_scores(np.array([[0, 1]]), np.array([[0.5, 0.5]], F32), np.array([0.0], F32), 2)
    assert s == [0, 0] and cp.priorities(s).tolist() == [0.0, 0.0]


# ------------------------------------------------------------------ retention
def test_retention_brute_force():
    rng = np.random.default_rng(5)
    e = 7
    for trial in range(300):
        resident = set(np.flatnonzero(rng.random(e) < 0.4).tolist())
        activated = set(np.flatnonzero(rng.random(e) < 0.5).tolist())
        scores = [int(v) for v in rng.integers(0, 4, size=e)]       # many ties
        cap = int(rng.integers(1, e + 1))
        cand = sorted(resident | activated)
        val = {i: (scores[i] if i in activated else 0) for i in cand}
        n = min(cap, len(cand))
        # max total value; among those, the lexicographically smallest id tuple
        best = min(itertools.combinations(cand, n),
                   key=lambda sub: (-sum(val[i] for i in sub), sub))
        got = cp.retain_top_c(resident, activated - resident, scores, activated, cap)
        assert got == set(best)
        assert got <= (resident | activated) and len(got) == n
        if cap >= len(cand):
            assert got == set(cand)
        stale = resident - activated
        kept_stale = got & stale
        if kept_stale:                       # a stale expert survives only if every
            assert all(i in got for i in activated if val[i] > 0)   # valued expert did


# ------------------------------------------------------------------ cache simulation
def _route(rng, t, k, e):
    ids = np.stack([rng.permutation(e)[:k] for _ in range(t)]).astype(np.int32)
    g = rng.dirichlet(np.ones(k), size=t).astype(F32)
    c = rng.uniform(0.0, 1.0, size=t).astype(F32)
    return ids, g, c


def test_cache_accounting_identities():
    rng = np.random.default_rng(6)
    cache = cp.LayerCache(16, 5, 1000)
    prev = set()
    for step in range(30):
        ids, g, c = _route(rng, 6, 2, 16)
        r = cache.step(ids, g, c)
        assert r["resident_before"] == prev
        assert r["hits"] | r["misses"] == r["activated"] and not (r["hits"] & r["misses"])
        assert r["hits"] == r["activated"] & prev
        assert r["resident_after"] <= prev | r["activated"] and len(r["resident_after"]) <= 5
        prev = r["resident_after"]
    st = cache.stats
    assert st.steps == 30 and st.hits + st.misses == st.active_experts
    assert st.bytes_moved == st.misses * 1000 and st.assignments == 30 * 12


def test_full_capacity_misses_at_most_once():
    rng = np.random.default_rng(7)
    cache = cp.LayerCache(12, 12, 10)
    for step in range(40):
        cache.step(*_route(rng, 5, 2, 12))
    assert cache.stats.misses == len(cache.resident) <= 12 and cache.stats.evictions == 0


def test_repeated_input_hits_after_first_step():
    rng = np.random.default_rng(8)
    ids, g, c = _route(rng, 8, 2, 32)
    n_act = len(set(ids.reshape(-1).tolist()))
    cache = cp.LayerCache(32, n_act, 10)
    cache.step(ids, g, c)
    m1 = cache.stats.misses
    for _ in range(3):
        r = cache.step(ids, g, c)
        assert not r["misses"]
    assert m1 == n_act == cache.stats.misses


def test_hits_counted_against_pre_step_state():
    cache = cp.LayerCache(4, 1, 10)
    one = lambda e: (np.array([[e]]), np.array([[1.0]], F32), np.array([0.5], F32))
    assert cache.step(*one(2))["misses"] == {2}
    r = cache.step(*one(3))                 # 2 is resident but stale; 3 misses, then replaces it
    assert r["misses"] == {3} and r["resident_before"] == {2} and r["resident_after"] == {3}
    assert cache.stats.evictions == 1


# ------------------------------------------------------------------ whole step, capacity invariance
def _stack(w, caps):
    st = OracleStack(w.n_layers, w.hidden, w.n_experts, w.top_k, w.intermediate, caps)
    for l in range(w.n_layers):
        wr, b = synth.router_weights(w, l)
        st.register_router(l, wr, b)
        blobs = np.empty((w.n_experts, w.expert_elems), np.uint16)
        synth.fill_layer_blobs(w, l, blobs)
        st.register_experts(l, blobs)
    return st


def test_output_and_routing_identical_at_every_capacity():
    w = synth.tiny(n_layers=1, blocks=1, iters=3)
    runs = []
    for cap in (1, 3, w.n_experts):
        st = _stack(w, [cap])
        outs = [st.denoise_step(0, h, c) for _, _, h, c in synth.denoise_inputs(w)]
        runs.append((outs, st.stats()))
    for outs, _ in runs[1:]:
        for a, b in zip(runs[0][0], outs):
            assert np.array_equal(a["ids"], b["ids"]) and np.array_equal(a["out"], b["out"])
            assert a["scores"] == b["scores"]
    assert runs[0][1].misses >= runs[1][1].misses >= runs[2][1].misses
    assert runs[2][1].evictions == 0


def test_policy_replay_matches_full_step():
    w = synth.tiny(n_layers=1, blocks=1, iters=4)
    full, replay = _stack(w, [3]), _stack(w, [3])
    for _, _, h, c in synth.denoise_inputs(w):
        r = full.denoise_step(0, h, c)
        q = replay.policy_step(0, r["ids"], r["gate"], c)
        assert q["resident_after"] == r["resident_after"] and q["misses"] == r["misses"]
    assert full.stats() == replay.stats()


def test_synth_is_seeded_and_bf16():
    w = synth.config(0)
    a = list(synth.denoise_inputs(w))
    b = list(synth.denoise_inputs(w))
    assert len(a) == w.iters * w.blocks
    assert all(np.array_equal(x[2], y[2]) and np.array_equal(x[3], y[3]) for x, y in zip(a, b))
    assert a[0][2].dtype == np.uint16 and a[0][2].shape == (32, 512)
    wr, bias = synth.router_weights(w, 0)
    assert wr.shape == (16, 512) and bias is None
    assert synth.config(1).capacity == 26 and synth.config(2).capacity == 51
    assert [synth.capacity_for(f, 64) for f in (0.1, 0.2, 0.4, 0.6, 1.0)] == [6, 13, 26, 38, 64]
    x = np.array([1.0, 1.00390625, 1.01171875, -3.0e-5], np.float32)   # ties and odd cases
    r = synth.round_to_bf16(x)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.015625           # tie to even, tie to even up
