"""Host-side checks that need no GPU: the library loads, exports every symbol the header
declares, and its C++ cache policy agrees with the oracle's policy decision for decision."""
import os
import re

import numpy as np
import pytest

from oracle import cache_policy as cp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2609_33385_b200 import build
    build.build()
    from paper_2609_33385_b200 import binding as b
    b.load()
    return b


def test_library_exports_every_declared_symbol(binding):
    header = open(os.path.join(ROOT, "include", "oled.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(oled_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    lib = binding.load()
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in include/oled.h but not exported"
    assert declared == set(binding.EXPORTS)


def test_strerror_and_arg_checks_without_gpu(binding):
    assert binding.strerror(0) == "ok"
    assert "pinned" in binding.strerror(binding.ERR_NOT_PINNED)
    assert binding.strerror(-12345) == "unknown error"
    with pytest.raises(binding.OledError):
        binding.PolicySim(8, 0, 8)            # capacity 0
    with pytest.raises(binding.OledError):
        binding.PolicySim(8, 4, 3)            # pool smaller than capacity
    lib = binding.load()
    assert lib.oled_denoise_step(None, 0, None, None, 1, None) == binding.ERR_INVALID_ARG
    assert lib.oled_stats(None, 0, None) == binding.ERR_INVALID_ARG


@pytest.mark.parametrize("e,cap,seed", [(16, 8, 0), (64, 26, 1), (12, 1, 2), (9, 9, 3), (128, 51, 4)])
def test_host_policy_matches_oracle(binding, e, cap, seed):
    rng = np.random.default_rng(seed)
    sim = binding.PolicySim(e, cap, e)        # worst-case pool: E slots
    ref = cp.LayerCache(e, cap, 100)
    for step in range(60):
        t, k = int(rng.integers(1, 12)), int(rng.integers(1, min(4, e) + 1))
        ids = np.stack([rng.permutation(e)[:k] for _ in range(t)]).astype(np.int32)
        gate = rng.dirichlet(np.ones(k), size=t).astype(np.float32)
        conf = rng.choice([0.0, 0.25, 0.5, 1.0], size=t).astype(np.float32)   # many ties, zeros
        r = ref.step(ids, gate, conf)
        counts = np.bincount(ids.reshape(-1), minlength=e).astype(np.int32)
        got = sim.step(counts, np.array(r["scores"], dtype=np.uint64))
        assert set(np.flatnonzero(got["resident_before"])) == r["resident_before"]
        assert set(np.flatnonzero(got["resident_after"])) == r["resident_after"]
        assert got["hits"] == len(r["hits"]) and got["misses"] == len(r["misses"])
        assert got["evictions"] == len(r["resident_before"] - r["resident_after"])
        # slot table: every activated expert has a distinct slot during the step
        slots = got["slot_of"][counts > 0]
        assert np.all(slots >= 0) and len(set(slots.tolist())) == len(slots)
        assert np.all(got["slot_of"][counts == 0] == -1)


def test_host_policy_pool_exhaustion_is_an_error_not_a_crash(binding):
    sim = binding.PolicySim(8, 2, 3)          # capacity 2 plus one transient slot
    counts = np.zeros(8, np.int32)
    counts[[0, 1, 2]] = 1
    sim.step(counts, np.arange(8, dtype=np.uint64) + 1)    # 3 misses fit in 3 slots
    counts[:] = 0
    counts[[3, 4, 5, 6]] = 1                                # 4 misses: 2 stale slots + 1 free < 4
    with pytest.raises(binding.OledError) as ei:
        sim.step(counts, np.arange(8, dtype=np.uint64) + 1)
    assert ei.value.code == binding.ERR_NO_SLOT
    counts[:] = 0
    counts[[3, 4, 5]] = 1                                   # the failed step changed nothing
    got = sim.step(counts, np.arange(8, dtype=np.uint64) + 1)
    assert got["misses"] == 3


@pytest.mark.parametrize("policy", ["priority", "lru", "lfu"])
def test_host_policy_variants_match_oracle(binding, policy):
    rng = np.random.default_rng(11)
    e, cap = 24, 7
    sim = binding.PolicySim(e, cap, e, policy=policy)
    ref = cp.LayerCache(e, cap, 100, policy=policy)
    for step in range(80):
        t, k = int(rng.integers(1, 8)), 2
        ids = np.stack([rng.permutation(e)[:k] for _ in range(t)]).astype(np.int32)
        gate = rng.dirichlet(np.ones(k), size=t).astype(np.float32)
        conf = rng.choice([0.0, 0.3, 1.0], size=t).astype(np.float32)
        r = ref.step(ids, gate, conf)
        counts = np.bincount(ids.reshape(-1), minlength=e).astype(np.int32)
        got = sim.step(counts, np.array(r["scores"], dtype=np.uint64))
        assert set(np.flatnonzero(got["resident_after"])) == r["resident_after"]
        assert got["misses"] == len(r["misses"])
    assert sim.fills_reused() == ref.stats.fills_reused


def test_host_adaptive_sizing_matches_oracle(binding):
    from oracle import OracleStack
    rng = np.random.default_rng(12)
    n_layers, e, caps = 5, 16, [4, 4, 4, 4, 4]
    sims = [binding.PolicySim(e, c, e) for c in caps]
    ora = OracleStack(n_layers, 256, e, 2, 128, caps)
    width = [2, 4, 8, 12, 16]                       # layer l draws its experts from the first width[l]
    for it in range(23):
        for l in range(n_layers):
            t = 6
            ids = np.stack([rng.permutation(width[l])[:2] for _ in range(t)]).astype(np.int32)
            gate = rng.dirichlet(np.ones(2), size=t).astype(np.float32)
            conf = rng.uniform(0, 1, size=t).astype(np.float32)
            r = ora.policy_step(l, ids, gate, conf)
            counts = np.bincount(ids.reshape(-1), minlength=e).astype(np.int32)
            got = sims[l].step(counts, np.array(r["scores"], dtype=np.uint64))
            assert set(np.flatnonzero(got["resident_after"])) == r["resident_after"], (it, l)
        if it % 5 == 4:                              # the paper's refresh period
            want = ora.adapt_capacity()
            assert binding.PolicySim.adapt(sims, sum(caps)) == want
            assert sum(want) == sum(caps)
    assert want[0] < want[-1]                        # slots moved to the layers with the larger working sets


def test_shared_pool_never_runs_out_after_adaptive_shrinking(binding):
    """The slot pool of a stack, sized by the rule oled_create() uses with default staging: a layer
    that layer-adaptive sizing has shrunk to ONE slot, while the other layers fill their enlarged
    capacities, must still be able to activate every expert in one step (Sec. 4.3 sizing on top of
    the Sec. 4.2 cache update)."""
    e, n_layers = 16, 4
    caps = [4] * n_layers
    sims, pool_slots = binding.PolicySim.stack(e, caps)
    assert pool_slots == sum(caps) + e - 1
    ones = np.ones(e, np.uint64)
    # period 1: layer 0 activates one expert per step, the others all of them -> layer 0 starves
    for it in range(5):
        for l, sim in enumerate(sims):
            counts = np.zeros(e, np.int32)
            if l == 0:
                counts[0] = 1
            else:
                counts[:] = 1
            sim.step(counts, ones * (it + 1))
    new = binding.PolicySim.adapt(sims, sum(caps))
    assert sum(new) == sum(caps) and new[0] == 1 and max(new[1:]) > 4
    # the grown layers fill their capacities, then the shrunk layer activates everything
    for l in (1, 2, 3):
        got = sims[l].step(np.ones(e, np.int32), np.arange(e, dtype=np.uint64) + 1)
        assert int(got["resident_after"].sum()) == new[l]
    got = sims[0].step(np.ones(e, np.int32), np.arange(e, dtype=np.uint64) + 1)
    assert got["hits"] + got["misses"] == e and int(got["resident_after"].sum()) == 1
    slots = got["slot_of"]
    assert np.all(slots >= 0) and len(set(slots.tolist())) == e


def test_small_caller_chosen_staging_raises_the_adaptive_floor(binding):
    """With fewer staging slots than E - 1 a layer of capacity C could need E - C transient slots
    that do not exist; the sizing then never hands out less than E - staging."""
    e, caps, staging = 16, [6, 6, 6], 10
    sims, pool_slots = binding.PolicySim.stack(e, caps, staging_slots=staging)
    assert pool_slots == sum(caps) + staging
    for it in range(5):
        for l, sim in enumerate(sims):
            counts = np.zeros(e, np.int32)
            counts[: (1 if l == 0 else e)] = 1
            sim.step(counts, np.ones(e, np.uint64))
    new = binding.PolicySim.adapt(sims, sum(caps))
    assert sum(new) == sum(caps) and min(new) == e - staging
    for l in (1, 2, 0):                                   # worst case still fits
        got = sims[l].step(np.ones(e, np.int32), np.arange(e, dtype=np.uint64) + 1)
        assert got["hits"] + got["misses"] == e


def test_misaligned_pointers_are_rejected_before_anything_is_launched(binding):
    """oled_route_noalloc accesses rows and ids with 16-byte vectors: a pointer into the middle of
    such a vector is an argument error (nothing touches the GPU, so this runs without one)."""
    ok16, ok4 = 0x7000_0000_0100, 0x7000_0000_0204
    args = dict(hidden=ok16, w_router=ok16 + 0x1000, bias=None, conf=ok4, ids=ok16 + 0x2000, gate=ok4 + 0x3000,
                counts=ok4 + 0x4000, offsets=ok4 + 0x5000, perm=ok4 + 0x6000)

    def call(**kw):
        a = dict(args, **kw)
        return binding.route_noalloc(a["hidden"], a["w_router"], a["bias"], a["conf"], 4, 256, 8, 2, 0, a["ids"],
                                     a["gate"], a["counts"], a["offsets"], a["perm"])
    for name in ("hidden", "w_router", "ids"):
        assert call(**{name: args[name] + 8}) == binding.ERR_INVALID_ARG, name
    for name in ("conf", "gate", "counts", "offsets", "perm"):
        assert call(**{name: args[name] + 2}) == binding.ERR_INVALID_ARG, name
    assert call(bias=ok4 + 1) == binding.ERR_INVALID_ARG


def test_two_e4m3_terms_hold_a_scaled_bf16_row():
    """The arithmetic the direct fp8 tensor-core form rests on (csrc/fp8_split.h), restated in numpy
    with the oracle's decoder: a bf16 row scaled by the power of two that brings its largest
    magnitude into [128, 256) equals t1 + t2/16 with t1 = e4m3(v), t2 = e4m3(16 (v - t1)) -
    exactly for every element within 2^-14 of the row's maximum, and to 2^-22 of the maximum
    below that."""
    from oracle.moe_layer import fp8_e4m3_to_f32
    from paper_2609_33385_b200 import synth
    rng = np.random.default_rng(5)
    rows = []
    for spread in (0, 6, 14, 20, 30):                      # binades between a row's largest and smallest elements
        mant = rng.integers(128, 256, size=(64, 512)).astype(np.float64)          # 8 significant bits
        expo = rng.integers(-spread, 1, size=(64, 512)) + rng.integers(-40, 40, size=(64, 1))
        rows.append(np.ldexp(mant, expo - 7) * rng.choice([-1.0, 1.0], size=(64, 512)))
    x = np.concatenate(rows)
    x[3] = 0.0                                              # an all-zero row
    assert np.array_equal(synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(x.astype(np.float32))).astype(np.float64), x)
    amax = np.abs(x).max(axis=1, keepdims=True)
    _, ex = np.frexp(np.where(amax > 0, amax, 1.0))        # amax = m * 2^ex, m in [0.5, 1)
    scale = np.ldexp(1.0, 8 - ex)                          # amax * scale in [128, 256)
    v = x * scale
    assert np.all((np.abs(v).max(axis=1) >= 128) | (amax[:, 0] == 0)) and np.abs(v).max() < 256
    t1 = fp8_e4m3_to_f32(synth.f32_to_e4m3_codes(v)).astype(np.float64)
    t2 = fp8_e4m3_to_f32(synth.f32_to_e4m3_codes((v - t1) * 16.0)).astype(np.float64)
    err = np.abs(t1 + t2 / 16.0 - v)
    exact_zone = np.abs(v) >= 2.0 ** -6                    # within 2^-14 of a maximum of at least 128
    assert exact_zone.mean() > 0.5 and np.all(err[exact_zone] == 0.0)
    assert err.max() <= 2.0 ** -14 and (~exact_zone).any()  # 2^-22 of the smallest scaled maximum (128)
