"""Pins for the MoE-layer oracle: each test ties an oracle function to something
other than itself (fp64 arithmetic, hand-built cases, brute force, closed forms,
library routines), so that a dropped term, a wrong index or a transposed
operand fails at least one of them."""
import itertools
import math

import numpy as np
import pytest

from oracle import moe_layer as om
from paper_2609_33385_b200 import synth

F32 = np.float32


def _bf16_vals(rng, shape, scale=1.0):
    return synth.round_to_bf16(rng.standard_normal(shape).astype(F32) * F32(scale))


# ------------------------------------------------------------------ logits
def test_logits_close_to_fp64_dot():
    rng = np.random.default_rng(1)
    x = _bf16_vals(rng, (7, 512))
    w = _bf16_vals(rng, (5, 512), 0.05)
    b = rng.standard_normal(5).astype(F32)
    got = om.gate_logits(x, w, b)
    ref = x.astype(np.float64) @ w.astype(np.float64).T + b.astype(np.float64)
    bound = 1e-5 * np.linalg.norm(x, axis=1)[:, None] * np.linalg.norm(w, axis=1)[None, :] + 1e-6
    assert got.dtype == F32 and got.shape == (7, 5)
    assert np.all(np.abs(got - ref) <= bound)


def test_logits_one_hot_returns_weight_exactly():
    rng = np.random.default_rng(2)
    w = _bf16_vals(rng, (6, 256))
    for h0 in (0, 9, 255):
        x = np.zeros((1, 256), F32)
        x[0, h0] = 1.0
        assert np.array_equal(om.gate_logits(x, w)[0], w[:, h0])


def test_logits_not_transposed():
    # T != E and asymmetric data: element (t,e) must use row t of x and row e of w
    x = np.zeros((2, 256), F32)
    w = np.zeros((3, 256), F32)
    x[1, 4] = 2.0
    w[2, 4] = 3.0
    got = om.gate_logits(x, w)
    assert got.shape == (2, 3) and got[1, 2] == 6.0 and np.count_nonzero(got) == 1


def _single(vals):
    """logit of one token/expert where x holds vals at given h and w is all ones"""
    x = np.zeros((1, 512), F32)
    for h, v in vals.items():
        x[0, h] = v
    return float(om.gate_logits(x, np.ones((1, 512), F32))[0, 0])


def test_logits_chain_membership_and_order():
    big = float(2 ** 24)
    # h = 0,1,2 all belong to chain 0 and are visited in ascending h:
    # (2^24 + 1) rounds back to 2^24, minus 2^24 gives 0.
    assert _single({0: big, 1: 1.0, 2: -big}) == 0.0
    # h = 8 belongs to chain 1: the 1 survives in its own chain.
    assert _single({0: big, 8: 1.0, 1: -big}) == 1.0
    # h = 256 is chain 0 again (next 256-wide group), visited after h < 256.
    assert _single({0: big, 256: 1.0, 257: -big}) == 0.0
    # ascending order inside a chain: -2^24 at h=0 first, then +2^24, then 1 -> 1
    assert _single({0: -big, 1: big, 2: 1.0}) == 1.0


def test_logits_butterfly_order():
    big = float(2 ** 24)
    # chains 0 and 16 meet in the first butterfly step: 2^24 + 1 -> 2^24; chain 1 (-2^24)
    # joins in the last step: 0.  A left-to-right sum of the chains would give 1.
    assert _single({0: big, 16 * 8: 1.0, 8: -big}) == 0.0
    # chains 0 and 1 only meet in the last step; 0+16 first: (2^24 - 2^24) then + 1 -> 1
    assert _single({0: big, 16 * 8: -big, 8: 1.0}) == 1.0


def test_logits_bias_added_once():
    x = np.zeros((1, 256), F32)
    w = np.zeros((2, 256), F32)
    assert np.array_equal(om.gate_logits(x, w, np.array([0.25, -3.0], F32))[0], [0.25, -3.0])


# ------------------------------------------------------------------ exp
def test_exp_spec_vs_libm_within_2ulp():
    xs = np.linspace(-80.0, 0.0, 200001).astype(F32)
    got = om.exp_spec(xs)
    ref64 = np.exp(xs.astype(np.float64))
    ref = ref64.astype(F32)
    ulp = np.spacing(ref)
    assert np.all(np.abs(got.astype(np.float64) - ref64) <= 2.0 * ulp)
    assert om.exp_spec(np.array([0.0], F32))[0] == 1.0
    assert om.exp_spec(np.array([-80.5, -1000.0], F32)).tolist() == [0.0, 0.0]
    assert np.all(np.diff(got) >= 0)          # monotone on the grid


def test_exp_spec_known_values():
    got = om.exp_spec(np.array([-math.log(2.0), -1.0, -math.log(3.0)], F32))
    assert np.allclose(got, [0.5, math.exp(-1.0), 1.0 / 3.0], rtol=3e-7, atol=0)


# ------------------------------------------------------------------ top-k
@pytest.mark.parametrize("e,k", [(16, 2), (8, 3)])
def test_topk_brute_force(e, k):
    rng = np.random.default_rng(e * 10 + k)
    logits = rng.standard_normal((20, e)).astype(F32)
    ids, g = om.topk_route(logits, k)
    for t in range(20):
        best = max(itertools.combinations(range(e), k),
                   key=lambda s: sum(float(logits[t, i]) for i in s))
        assert set(ids[t]) == set(best)
        sel = logits[t, ids[t]]
        assert np.all(np.diff(sel) <= 0)      # rank 0 is the largest
        # softmax over the selected logits, against an fp64 evaluation
        z = np.exp(sel.astype(np.float64) - float(sel[0]))
        assert np.allclose(g[t], z / z.sum(), rtol=1e-6, atol=1e-9)


def test_topk_ties_go_to_lower_index():
    logits = np.array([[1.0, 3.0, 3.0, 0.0, 3.0],
                       [0.0, -0.0, 0.0, -1.0, -1.0]], F32)
    ids, g = om.topk_route(logits, 2)
    assert ids.tolist() == [[1, 2], [0, 1]]
    assert g.tolist() == [[0.5, 0.5], [0.5, 0.5]]
    ids3, g3 = om.topk_route(logits, 4)
    assert ids3[0].tolist() == [1, 2, 4, 0]
    assert ids3[1].tolist() == [0, 1, 2, 3]


def test_topk_ties_from_duplicate_router_rows():
    rng = np.random.default_rng(5)
    w = _bf16_vals(rng, (6, 256), 0.05)
    w[4] = w[1]                                # experts 1 and 4 always tie
    x = _bf16_vals(rng, (9, 256))
    logits = om.gate_logits(x, w)
    ids, _ = om.topk_route(logits, 6)
    for t in range(9):
        row = ids[t].tolist()
        assert row.index(1) + 1 == row.index(4)


def test_gate_closed_forms():
    for k in (1, 2, 4, 8):
        ids, g = om.topk_route(np.zeros((1, 8), F32), k)
        assert ids[0].tolist() == list(range(k))
        assert g[0].tolist() == [1.0 / k] * k          # exact for k a power of two
    ids, g = om.topk_route(np.array([[0.0, F32(math.log(3.0))]], F32), 2)
    assert ids[0].tolist() == [1, 0]
    assert np.allclose(g[0], [0.75, 0.25], atol=1e-6)


def test_gate_sums_to_one():
    rng = np.random.default_rng(7)
    logits = (rng.standard_normal((200, 64)) * 3).astype(F32)
    _, g = om.topk_route(logits, 8)
    s = g.astype(np.float64).sum(axis=1)
    assert np.all(np.abs(s - 1.0) <= 8 * 2.0 ** -24)
    assert np.all(g > 0) and np.all(np.diff(g, axis=1) <= 0)


# ------------------------------------------------------------------ permutation
def test_permutation_properties():
    rng = np.random.default_rng(8)
    t, k, e = 37, 3, 11
    ids = np.stack([rng.permutation(e)[:k] for _ in range(t)]).astype(np.int32)
    cnt, off, perm, pos = om.permutation(ids, e)
    n = t * k
    assert sorted(perm.tolist()) == list(range(n))              # bijection
    assert cnt.sum() == n and off[0] == 0 and off[-1] == n
    assert np.array_equal(np.diff(off), cnt)
    assert np.array_equal(pos[perm], np.arange(n))              # inverse
    flat = ids.reshape(-1)
    for ee in range(e):
        seg = perm[off[ee]:off[ee + 1]]
        assert np.all(flat[seg] == ee)                          # right expert
        assert np.all(np.diff(seg) > 0)                         # stable: ascending t*k+j
        assert cnt[ee] == np.count_nonzero(flat == ee)


def test_permutation_tiny_by_hand():
    ids = np.array([[2, 0], [0, 1], [2, 1]], np.int32)
    cnt, off, perm, pos = om.permutation(ids, 4)
    assert cnt.tolist() == [2, 2, 2, 0]
    assert off.tolist() == [0, 2, 4, 6, 6]
    assert perm.tolist() == [1, 2, 3, 5, 0, 4]
    assert pos.tolist() == [4, 0, 1, 2, 5, 3]


# ------------------------------------------------------------------ FFN / layer
def _layer(rng, t=6, h=256, e=4, k=2, i=64):
    x = synth.f32_to_bf16_bits(rng.standard_normal((t, h)).astype(F32))
    wr = synth.f32_to_bf16_bits((rng.standard_normal((e, h)) * 0.1).astype(F32))
    blobs = synth.f32_to_bf16_bits((rng.standard_normal((e, 3 * h * i)) * 0.1).astype(F32))

    def get(ee, blobs=blobs):
        b = blobs[ee]
        return b[:h * i].reshape(i, h), b[h * i:2 * h * i].reshape(i, h), b[2 * h * i:].reshape(h, i)
    return x, wr, blobs, get


def test_ffn_matches_dense_swiglu_mlp_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(9)
    x, wr, blobs, get = _layer(rng, t=5, e=1, k=1)
    res = om.moe_layer_forward(x, wr, None, get, 1)
    wg, wu, wd = (torch.from_numpy(om.bf16_to_f32(a).astype(np.float64)) for a in get(0))
    xt = torch.from_numpy(om.bf16_to_f32(x).astype(np.float64))
    ref = (torch.nn.functional.silu(xt @ wg.T) * (xt @ wu.T)) @ wd.T
    assert np.all(res["gate"] == 1.0)
    assert np.allclose(res["out"], ref.numpy(), rtol=1e-12, atol=1e-12)


def test_ffn_not_gate_up_swapped_and_silu_sign():
    # one hidden unit: silu acts on the gate projection only
    x = np.array([[2.0]])
    out = om.expert_ffn(x, np.array([[-1.0]]), np.array([[3.0]]), np.array([[1.0]]))
    a = -2.0
    assert np.allclose(out, [[a / (1 + math.exp(-a)) * 6.0]])
    out2 = om.expert_ffn(x, np.array([[3.0]]), np.array([[-1.0]]), np.array([[1.0]]))
    assert not np.allclose(out, out2)


def test_layer_zero_gate_weights_and_linearity():
    rng = np.random.default_rng(10)
    x, wr, blobs, get = _layer(rng)
    h, i = 256, 64
    base = om.moe_layer_forward(x, wr, None, get, 2)["out"]
    zero = blobs.copy()
    zero[:, :h * i] = 0                                   # Wg = 0  =>  silu(0) = 0
    res0 = om.moe_layer_forward(x, wr, None, lambda e: _views(zero, e, h, i), 2)
    assert np.all(res0["out"] == 0)
    dbl = blobs.copy()
    dbl[:, 2 * h * i:] = synth.f32_to_bf16_bits(om.bf16_to_f32(blobs[:, 2 * h * i:]) * F32(2))
    res2 = om.moe_layer_forward(x, wr, None, lambda e: _views(dbl, e, h, i), 2)
    assert np.allclose(res2["out"], 2.0 * base, rtol=1e-12, atol=0)


def _views(blobs, e, h, i):
    b = blobs[e]
    return b[:h * i].reshape(i, h), b[h * i:2 * h * i].reshape(i, h), b[2 * h * i:].reshape(h, i)


def test_layer_relabelling_invariance():
    rng = np.random.default_rng(11)
    x, wr, blobs, get = _layer(rng, e=5, k=2)
    base = om.moe_layer_forward(x, wr, None, get, 2)
    p = np.array([3, 0, 4, 1, 2])                         # new id n holds old expert p[n]
    res = om.moe_layer_forward(x, wr[p], None, lambda e: get(int(p[e])), 2)
    assert np.array_equal(p[res["ids"]], base["ids"])
    assert np.allclose(res["out"], base["out"], rtol=1e-12, atol=1e-15)


def test_layer_top1_output_is_expert_output():
    rng = np.random.default_rng(12)
    x, wr, blobs, get = _layer(rng, e=3, k=1)
    res = om.moe_layer_forward(x, wr, None, get, 1)
    xf = om.bf16_to_f32(x)
    for t in range(x.shape[0]):
        wg, wu, wd = (om.bf16_to_f32(a) for a in get(int(res["ids"][t, 0])))
        ref = om.expert_ffn(xf[t:t + 1], wg, wu, wd)[0]      # g = 1 exactly, so out is the expert's y
        assert res["gate"][t, 0] == 1.0 and np.allclose(res["out"][t], ref, rtol=1e-12, atol=1e-15)


def test_layer_weighted_sum_by_hand():
    # every expert e returns (e+1)*x-independent constant direction: check the g-weighted sum
    rng = np.random.default_rng(13)
    x, wr, blobs, get = _layer(rng, t=4, e=4, k=2)
    res = om.moe_layer_forward(x, wr, None, get, 2)
    xf = om.bf16_to_f32(x)
    for t in range(4):
        acc = np.zeros(256)
        for j in range(2):
            wg, wu, wd = (om.bf16_to_f32(a) for a in get(int(res["ids"][t, j])))
            acc += float(res["gate"][t, j]) * om.expert_ffn(xf[t:t + 1], wg, wu, wd)[0]
        assert np.allclose(res["out"][t], acc, rtol=1e-10, atol=1e-13)


def test_layer_empty_step():
    rng = np.random.default_rng(14)
    x, wr, blobs, get = _layer(rng)
    res = om.moe_layer_forward(x[:0], wr, None, get, 2)
    assert res["out"].shape == (0, 256) and res["counts"].sum() == 0


# ------------------------------------------------------------------ fp8 expert blobs
def test_fp8_decode_against_format_definition_and_torch():
    codes = np.arange(256, dtype=np.uint8)
    got = om.fp8_e4m3_to_f32(codes)
    assert got[0] == 0.0 and got[0x80] == 0.0 and np.signbit(got[0x80])
    assert got[0x01] == 2.0 ** -9 and got[0x07] == 7 * 2.0 ** -9          # subnormals
    assert got[0x08] == 2.0 ** -6 and got[0x38] == 1.0 and got[0x3C] == 1.5
    assert got[0x7E] == 448.0 and got[0xFE] == -448.0                       # largest finite
    assert np.isnan(got[0x7F]) and np.isnan(got[0xFF])
    finite = got[:0x7F]
    assert np.all(np.diff(finite) > 0)                                      # codes are monotone
    torch = pytest.importorskip("torch")
    if hasattr(torch, "float8_e4m3fn"):
        ref = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float32).numpy()
        ok = ~np.isnan(ref)
        assert np.array_equal(got[ok], ref[ok]) and np.array_equal(np.isnan(got), np.isnan(ref))


def test_fp8_encode_roundtrip_and_rounding():
    vals = om.fp8_e4m3_to_f32(np.arange(256, dtype=np.uint8))
    fin = ~np.isnan(vals)
    back = synth.f32_to_e4m3_codes(vals[fin])
    assert np.array_equal(om.fp8_e4m3_to_f32(back), vals[fin])              # every code survives
    # midpoints go to the even code; anything beyond 448 saturates
    assert synth.f32_to_e4m3_codes(np.array([1.0625, 1.1875, 1000.0, -1000.0])).tolist() == \
        [0x38, 0x3A, 0x7E, 0xFE]
    rng = np.random.default_rng(0)
    x = rng.standard_normal(20000) * 50
    q = om.fp8_e4m3_to_f32(synth.f32_to_e4m3_codes(x)).astype(np.float64)
    pos = np.sort(np.abs(vals[fin]).astype(np.float64))
    xa = np.minimum(np.abs(x), 448.0)
    nearest = pos[np.abs(pos[None, :] - xa[:, None]).argmin(axis=1)]
    assert np.allclose(np.abs(q), nearest)                                   # nearest representable


def test_fp8_blob_layout_and_dequantisation_error():
    w = synth.tiny(n_layers=1)
    blob = synth.expert_blob_bits(w, 0, 3)
    q = synth.quantize_expert_blob(w, blob)
    assert q.size == synth.fp8_blob_bytes(w) and q.size % 256 == 0
    g, u, d = om.fp8_expert_weights(q, w.hidden, w.intermediate)
    for deq, ref in zip((g, u, d), synth.split_blob(w, blob)):
        r = om.bf16_to_f32(ref).astype(np.float64)
        assert deq.shape == r.shape
        # per-row scaling: error at most half an e4m3 step of the row maximum (1/16 relative)
        bound = np.abs(r).max(axis=1, keepdims=True) / 16.0 + 1e-12
        assert np.all(np.abs(deq - r) <= bound)
        assert np.allclose(np.abs(deq).max(axis=1), np.abs(r).max(axis=1), rtol=1e-6)


def test_fp8_layer_matches_layer_on_dequantised_weights():
    rng = np.random.default_rng(21)
    w = synth.tiny(n_layers=1)
    x, conf = synth.flat_tokens(w, 6)
    wr, _ = synth.router_weights(w, 0)
    blobs = np.stack([synth.quantize_expert_blob(w, synth.expert_blob_bits(w, 0, e)) for e in range(w.n_experts)])
    res = om.moe_layer_forward(x, wr, None, lambda e: om.fp8_expert_weights(blobs[e], w.hidden, w.intermediate),
                               w.top_k)
    # the same layer evaluated token by token with explicit fp64 formulas
    xf = om.bf16_to_f32(x).astype(np.float64)
    for t in range(6):
        acc = np.zeros(w.hidden)
        for j in range(w.top_k):
            g, u, d = om.fp8_expert_weights(blobs[res["ids"][t, j]], w.hidden, w.intermediate)
            a = g @ xf[t]
            acc += float(res["gate"][t, j]) * (d @ (a / (1 + np.exp(-a)) * (u @ xf[t])))
        assert np.allclose(res["out"][t], acc, rtol=1e-10, atol=1e-13)


def test_nan_logit_ranks_below_every_number_and_ids_stay_distinct():
    """Non-finite activations: a NaN logit is read as -inf, so the order is total; the ids of a
    token are distinct, NaN entries come last and among themselves in index order."""
    logits = np.array([[np.nan, 1.0, np.nan, -3.0, 2.0],
                       [np.nan, np.nan, np.nan, np.nan, np.nan],
                       [np.inf, 0.0, -np.inf, np.nan, 5.0]], dtype=np.float32)
    with np.errstate(all="ignore"):
        ids, g = om.topk_route(logits, 4)
    assert ids.tolist() == [[4, 1, 3, 0], [0, 1, 2, 3], [0, 4, 1, 2]]
    assert g[0, 3] == 0.0 and np.isclose(g[0, :3].sum(), 1.0)       # exp_spec(-inf) is 0
    assert np.isnan(g[1]).all()                                       # -inf - -inf
    assert np.isnan(g[2]).all()                                       # inf - inf poisons the sum


def test_nan_reuse_score_adds_nothing():
    from oracle import cache_policy as P
    ids = np.array([[0, 1]], dtype=np.int32)
    gate = np.array([[np.nan, 0.5]], dtype=np.float32)
    assert P.reuse_scores(ids, gate, np.array([1.0], np.float32), 2) == [0, 2 ** 31]
