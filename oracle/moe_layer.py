"""CPU oracle for the MoE layer of one denoising step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct restatement of what the hot path computes:
gate -> top-k experts and gate scores -> expert FFNs -> gate-weighted sum
(paper Sec. 2.1 "MoE-based dLLMs" and Sec. 4.1, system overview: "the MoE gate
first produces the routed expert IDs, gate scores ...").  The paper never
writes the formulas of the gate or of the expert; the readings used here are
the softmax/top-k gate with ties to the lower expert index and the SwiGLU
expert  Wd( silu(Wg x) * (Wu x) )  without biases.

Only tests, the smoke check and the benchmark's cpu-baseline leg may import
this package.  It shares no code with the CUDA path.

Decision-bearing arithmetic (logits, top-k, gate scores) is evaluated in fp32
in a fixed, documented operation order so that a second implementation can
reproduce the routing bit for bit; everything that is only compared within a
tolerance (expert FFN, combine) is fp64.

Pins (tests/test_oracle_*.py): fp64 dot products, one-hot inputs, brute-force
top-k over all subsets, closed-form softmax cases, libm exp on a dense grid,
bijection/segment properties of the permutation, E=1/k=1 reduction to a dense
SwiGLU MLP, linearity in Wd, relabelling invariance.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp32 exactly."""
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def fp8_e4m3_to_f32(codes: np.ndarray) -> np.ndarray:
    """Decode fp8 e4m3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities,
    0x7F / 0xFF are NaN; exponent field 0 is subnormal: m * 2^-9)."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int32)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e, m = (c >> 3) & 0xF, c & 7
    mag = np.where(e == 0, m * 2.0 ** -9, (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64)))
    mag = np.where((e == 15) & (m == 7), np.nan, mag)
    return (sign * mag).astype(np.float32)


def fp8_expert_weights(blob: np.ndarray, hidden: int, intermediate: int):
    """Dequantised (gate[I,H], up[I,H], down[H,I]) in fp64 from an fp8 expert blob: e4m3 codes of
    the three matrices followed by fp32 scales s_gate[I] | s_up[I] | s_down[H], one per row."""
    h, i = hidden, intermediate
    n = 3 * h * i
    sc = np.asarray(blob[n:n + 4 * (2 * i + h)], dtype=np.uint8).view(np.float32).astype(np.float64)
    vals = fp8_e4m3_to_f32(blob[:n]).astype(np.float64)
    gate = vals[:h * i].reshape(i, h) * sc[:i, None]
    up = vals[h * i:2 * h * i].reshape(i, h) * sc[i:2 * i, None]
    down = vals[2 * h * i:].reshape(h, i) * sc[2 * i:, None]
    return gate, up, down


# --------------------------------------------------------------------------
# Gate logits, fixed reduction order
# --------------------------------------------------------------------------
def gate_logits(x: np.ndarray, w_router: np.ndarray, bias=None) -> np.ndarray:
    """L[t,e] = sum_h x[t,h]*w[e,h] (+ bias[e]) in fp32, in the contract order.

    x [T,H] and w_router [E,H] are fp32 arrays holding bf16-representable
    values, so every product is exact in fp32.  The sum runs over 32 chains:
    chain q owns the indices h with (h // 8) % 32 == q, visited in ascending
    h, each step one rounded fp32 addition starting from +0.  The 32 chain
    sums are then combined by a butterfly: for d in 16, 8, 4, 2, 1 every
    chain adds the chain whose number differs in bit d; chain 0 holds the
    result.  The bias, if any, is one more rounded addition.
    """
    x = np.asarray(x, dtype=F32)
    w = np.asarray(w_router, dtype=F32)
    t, h = x.shape
    e = w.shape[0]
    assert w.shape[1] == h and h % 256 == 0, "hidden must be a multiple of 256"
    xs = x.reshape(t, h // 256, 32, 8)
    ws = w.reshape(e, h // 256, 32, 8)
    acc = np.zeros((t, e, 32), dtype=F32)
    for i in range(h // 256):
        for j in range(8):
            prod = xs[:, None, i, :, j] * ws[None, :, i, :, j]   # exact products
            acc = (acc + prod).astype(F32)
    lanes = np.arange(32)
    for d in (16, 8, 4, 2, 1):
        acc = (acc + acc[:, :, lanes ^ d]).astype(F32)
    out = acc[:, :, 0]
    if bias is not None:
        out = (out + np.asarray(bias, dtype=F32)[None, :]).astype(F32)
    return np.ascontiguousarray(out)


# --------------------------------------------------------------------------
# exp for the gate softmax, built from individually rounded fp32 operations
# --------------------------------------------------------------------------
_LOG2E = F32(1.4426950408889634)          # fl32(1/ln 2)
_LN2_HI = F32(0.693115234375)             # fl32(ln 2) with the low 12 significand bits cleared
_LN2_LO = F32(0.6931471805599453 - 0.693115234375)
_EXP_COEF = [F32(1.0), F32(1.0), F32(1.0 / 2), F32(1.0 / 6), F32(1.0 / 24),
             F32(1.0 / 120), F32(1.0 / 720), F32(1.0 / 5040)]
EXP_CUTOFF = F32(-80.0)


def exp_spec(x: np.ndarray) -> np.ndarray:
    """exp(x) for x <= 0 in fp32 using only rounded multiplies, adds, subtracts.

    x < -80 gives 0.  Otherwise n = rint(x*log2(e)) (ties to even),
    r = (x - n*LN2_HI) - n*LN2_LO, P = degree-7 Taylor polynomial of e^r by
    Horner's rule (multiply, then add, each rounded), result = P * 2^n.
    exp_spec(0) is exactly 1.
    """
    x = np.asarray(x, dtype=F32)
    n = np.rint((x * _LOG2E).astype(F32)).astype(F32)
    r = ((x - (n * _LN2_HI).astype(F32)).astype(F32) - (n * _LN2_LO).astype(F32)).astype(F32)
    p = np.full(x.shape, _EXP_COEF[7], dtype=F32)
    for c in (6, 5, 4, 3, 2, 1, 0):
        p = ((p * r).astype(F32) + _EXP_COEF[c]).astype(F32)
    scale = np.ldexp(F32(1.0), np.maximum(n, F32(-126)).astype(np.int32)).astype(F32)
    res = (p * scale).astype(F32)
    return np.where(x < EXP_CUTOFF, F32(0.0), res).astype(F32)


# --------------------------------------------------------------------------
# Top-k and gate scores
# --------------------------------------------------------------------------
def topk_route(logits: np.ndarray, k: int):
    """Top-k experts per token and softmax gate scores over the selected k.

    Order: logit descending, ties to the lower expert index; rank 0 is the
    largest.  Scores: z_j = exp_spec(L_j - L_0), S = ((z_0+z_1)+z_2)+...,
    g_j = z_j / S, every operation a rounded fp32 operation.
    A NaN logit is read as -inf (the paper does not say what a router does
    with non-finite activations; this keeps the order total, so the k ids of
    a token stay distinct).
    Returns ids [T,k] int32 and g [T,k] fp32.
    """
    logits = np.asarray(logits, dtype=F32)
    logits = np.where(np.isnan(logits), F32(-np.inf), logits).astype(F32)
    t, e = logits.shape
    assert 1 <= k <= e
    ids = np.empty((t, k), dtype=np.int32)
    g = np.empty((t, k), dtype=F32)
    for tt in range(t):
        row = logits[tt]
        order = sorted(range(e), key=lambda ee: (-float(row[ee]), ee))[:k]
        ids[tt] = order
        sel = row[order]
        z = exp_spec((sel - sel[0]).astype(F32))
        s = z[0]
        for j in range(1, k):
            s = F32(s + z[j])
        g[tt] = (z / s).astype(F32)
    return ids, g


# --------------------------------------------------------------------------
# Token -> expert permutation
# --------------------------------------------------------------------------
def permutation(ids: np.ndarray, n_experts: int):
    """Counting sort of the T*k assignments by expert, stable in (token, rank).

    Returns counts [E], offsets [E+1] (exclusive scan), perm [T*k] with
    perm[r] = t*k+j (the assignment placed at sorted row r) and its inverse
    pos [T*k] with pos[t*k+j] = r.
    """
    ids = np.asarray(ids, dtype=np.int32)
    flat = ids.reshape(-1)
    n = flat.size
    counts = np.zeros(n_experts, dtype=np.int32)
    for a in range(n):
        counts[flat[a]] += 1
    offsets = np.zeros(n_experts + 1, dtype=np.int32)
    for e in range(n_experts):
        offsets[e + 1] = offsets[e] + counts[e]
    cursor = offsets[:-1].copy()
    perm = np.empty(n, dtype=np.int32)
    pos = np.empty(n, dtype=np.int32)
    for a in range(n):
        e = flat[a]
        perm[cursor[e]] = a
        pos[a] = cursor[e]
        cursor[e] += 1
    return counts, offsets, perm, pos


# --------------------------------------------------------------------------
# Expert FFN and combine (toleranced part, fp64)
# --------------------------------------------------------------------------
def expert_ffn(x: np.ndarray, w_gate: np.ndarray, w_up: np.ndarray, w_down: np.ndarray) -> np.ndarray:
    """SwiGLU expert: y = Wd ( silu(Wg x) * (Wu x) ), rows of x are tokens.

    x [n,H]; w_gate, w_up [I,H]; w_down [H,I]; returns [n,H] in fp64.
    """
    x = np.asarray(x, dtype=np.float64)
    a = x @ np.asarray(w_gate, dtype=np.float64).T
    u = x @ np.asarray(w_up, dtype=np.float64).T
    hmid = a / (1.0 + np.exp(-a)) * u
    return hmid @ np.asarray(w_down, dtype=np.float64).T


def moe_layer_forward(x_bits, w_router_bits, bias, expert_weights, k: int):
    """The whole layer for one step.

    x_bits [T,H] bf16 bits; w_router_bits [E,H] bf16 bits; bias fp32 [E] or
    None; expert_weights(e) -> (gate, up, down) as bf16 bit arrays.
    Returns a dict with logits, ids, gate, counts, offsets, perm, pos and
    out [T,H] fp64 where out[t] = sum_j g[t,j] * FFN_{ids[t,j]}(x[t]), j ascending.
    """
    x = bf16_to_f32(x_bits)
    wr = bf16_to_f32(w_router_bits)
    t, h = x.shape
    e = wr.shape[0]
    if t == 0:
        z = np.zeros
        return dict(logits=z((0, e), F32), ids=z((0, k), np.int32), gate=z((0, k), F32),
                    counts=z(e, np.int32), offsets=z(e + 1, np.int32), perm=z(0, np.int32),
                    pos=z(0, np.int32), out=z((0, h), np.float64))
    logits = gate_logits(x, wr, bias)
    ids, g = topk_route(logits, k)
    counts, offsets, perm, pos = permutation(ids, e)
    y = np.zeros((t * k, h), dtype=np.float64)           # per sorted assignment row
    for ee in range(e):
        if counts[ee] == 0:
            continue
        rows = perm[offsets[ee]:offsets[ee + 1]]
        toks = rows // k
        wg, wu, wd = expert_weights(ee)
        if wg.dtype == np.uint16:           # bf16 bit patterns; fp8 stores hand over decoded floats
            wg, wu, wd = bf16_to_f32(wg), bf16_to_f32(wu), bf16_to_f32(wd)
        y[offsets[ee]:offsets[ee + 1]] = expert_ffn(x[toks], wg, wu, wd)
    out = np.zeros((t, h), dtype=np.float64)
    for tt in range(t):
        for j in range(k):
            out[tt] += np.float64(g[tt, j]) * y[pos[tt * k + j]]
    return dict(logits=logits, ids=ids, gate=g, counts=counts, offsets=offsets, perm=perm,
                pos=pos, out=out)
