"""Seeded synthetic dLLM-shaped workloads (inputs only).

This module draws random numbers and lays them out; it contains none of the
method's arithmetic (no routing, no FFN, no cache policy).  It is the one
module that the CPU oracle's tests and the CUDA path's tests/bench may both
use, so that both sides see identical inputs.

Shapes follow the five workload configurations this library is measured on; value
distributions follow the regime the paper reports for semi-autoregressive
dLLM decoding (Sec. 2.1: a block of masked tokens is refined over several
denoising iterations; Sec. 3.3: adjacent iterations have highly similar
hidden states).

bf16 tensors are carried as ``uint16`` bit patterns (``*_bits``) or as
``float32`` arrays whose low 16 bits are zero.
"""
from __future__ import annotations

import dataclasses
import math
from concurrent.futures import ThreadPoolExecutor
from typing import Iterator, Optional, Tuple

import numpy as np


# --------------------------------------------------------------------------
# bf16 <-> fp32 bit helpers (input formatting only)
# --------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even) and return uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """fp32 array whose values are exactly representable in bf16."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


# --------------------------------------------------------------------------
# Workload description
# --------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    cfg_id: int
    n_layers: int
    hidden: int
    n_experts: int
    top_k: int
    intermediate: int
    batch: int
    block_len: int
    iters: int
    blocks: int
    rho: float                 # hidden-state correlation between iterations
    literal_mix: bool          # True: h' = rho*h + (1-rho)*eps ; False: h' = rho*h + sqrt(1-rho^2)*eps
    beta_a: float
    beta_b: float
    residency: float           # fraction of experts resident per layer
    router_std: float          # std of router weights
    weight_std: float = 0.02
    zipf_bias: float = 0.0     # >0: per-expert bias b_e = -zipf_bias*ln(1+pi(e))
    finalize_threshold: float = 0.9
    shared_beta: float = 0.0   # >0: "dLLM-shaped" variant, tokens share a block direction
    conf_coupling: float = 0.0 # >0: a confident token's hidden state changes less (Sec. 4.3)
    layer_zipf: float = 0.0    # >0: per-layer gate bias of growing strength (layers differ in footprint)
    seed: int = 0

    @property
    def has_bias(self) -> bool:
        return self.zipf_bias > 0.0 or self.layer_zipf > 0.0

    @property
    def tokens(self) -> int:
        return self.batch * self.block_len

    @property
    def capacity(self) -> int:
        return capacity_for(self.residency, self.n_experts)

    @property
    def expert_elems(self) -> int:
        return 3 * self.hidden * self.intermediate

    @property
    def expert_bytes(self) -> int:
        return 2 * self.expert_elems

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def capacity_for(residency: float, n_experts: int) -> int:
    """Slots for a residency fraction: round half up, at least 1, at most E."""
    c = int(math.floor(residency * n_experts + 0.5))
    return max(1, min(n_experts, c))


def config(idx: int, **overrides) -> Workload:
    """The five workload configurations (index 0..4)."""
    if idx == 0:
        w = Workload("cfg1-1L-h512-e16-top2-T32", 1, 1, 512, 16, 2, 1024, 1, 32, 4, 1,
                     0.9, True, 2.0, 2.0, 0.5, 0.02)
    elif idx == 1:
        w = Workload("cfg2-16L-h2048-e64-top8-T32", 2, 16, 2048, 64, 8, 1024, 1, 32, 8, 4,
                     0.9, False, 2.0, 2.0, 0.4, 0.02)
    elif idx == 2:
        w = Workload("cfg3-48L-h2048-e128-top8-T256", 3, 48, 2048, 128, 8, 768, 4, 64, 16, 1,
                     0.85, False, 1.5, 3.0, 0.4, 0.02)
    elif idx == 3:
        w = Workload("cfg4-sweep-16L-h2048-e64-top8-T32", 4, 16, 2048, 64, 8, 1024, 1, 32, 8, 1,
                     0.9, False, 2.0, 2.0, 0.4, 0.02)
    elif idx == 4:
        w = Workload("cfg5-1L-h4096-e64-top8-T4096", 5, 1, 4096, 64, 8, 1536, 64, 64, 1, 1,
                     0.9, False, 2.0, 2.0, 1.0, 1.0 / math.sqrt(4096.0), zipf_bias=1.1)
    else:
        raise ValueError("config index must be 0..4")
    return w.replace(**overrides) if overrides else w


def tiny(**kw) -> Workload:
    """A small ragged shape for unit tests (hidden must stay a multiple of 256)."""
    base = Workload("tiny", 99, 2, 256, 8, 2, 128, 1, 5, 3, 2, 0.9, False, 2.0, 2.0, 0.5, 0.05,
                    weight_std=0.05)
    return base.replace(**kw) if kw else base


# --------------------------------------------------------------------------
# Random streams
# --------------------------------------------------------------------------
_STREAM_ROUTER, _STREAM_EXPERT, _STREAM_HIDDEN, _STREAM_CONF, _STREAM_BIAS = 1, 2, 3, 4, 5


def _rng(w: Workload, stream: int, *ids: int) -> np.random.Generator:
    return np.random.default_rng([w.seed, w.cfg_id, stream, *ids])


def router_weights(w: Workload, layer: int) -> Tuple[np.ndarray, Optional[np.ndarray]]:
    """Router matrix [E,H] as bf16 bits and the optional fp32 bias [E]."""
    g = _rng(w, _STREAM_ROUTER, layer)
    wr = g.standard_normal((w.n_experts, w.hidden), dtype=np.float32) * np.float32(w.router_std)
    bias = None
    if w.has_bias:
        strength = w.zipf_bias + w.layer_zipf * (layer / max(1, w.n_layers - 1))
        perm = _rng(w, _STREAM_BIAS, layer).permutation(w.n_experts)
        bias = (-strength * np.log1p(perm.astype(np.float64))).astype(np.float32)
    return f32_to_bf16_bits(wr), bias


def expert_blob_bits(w: Workload, layer: int, expert: int, out: Optional[np.ndarray] = None) -> np.ndarray:
    """One expert's weights as bf16 bits, laid out gate[I,H] | up[I,H] | down[H,I]."""
    g = _rng(w, _STREAM_EXPERT, layer, expert)
    n = w.expert_elems
    if out is None:
        out = np.empty(n, dtype=np.uint16)
    chunk = 1 << 22
    std = np.float32(w.weight_std)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        out[s:e] = f32_to_bf16_bits(g.standard_normal(e - s, dtype=np.float32) * std)
    return out


def fill_layer_blobs(w: Workload, layer: int, out: np.ndarray, threads: int = 0,
                     alias_of: Optional[int] = None) -> None:
    """Fill ``out`` (uint16 [E, 3*H*I]) with every expert of ``layer``."""
    src_layer = layer if alias_of is None else alias_of
    assert out.shape == (w.n_experts, w.expert_elems) and out.dtype == np.uint16
    if threads <= 1:
        for e in range(w.n_experts):
            expert_blob_bits(w, src_layer, e, out[e])
        return
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(lambda e: expert_blob_bits(w, src_layer, e, out[e]), range(w.n_experts)))


def split_blob(w: Workload, blob_bits: np.ndarray):
    """Views (gate[I,H], up[I,H], down[H,I]) of one expert blob."""
    hi = w.hidden * w.intermediate
    gate = blob_bits[:hi].reshape(w.intermediate, w.hidden)
    up = blob_bits[hi:2 * hi].reshape(w.intermediate, w.hidden)
    down = blob_bits[2 * hi:3 * hi].reshape(w.hidden, w.intermediate)
    return gate, up, down


# --------------------------------------------------------------------------
# Hidden states and confidences of the denoising loop
# --------------------------------------------------------------------------
def _noise(w: Workload, g: np.random.Generator) -> np.ndarray:
    t, h = w.tokens, w.hidden
    z = g.standard_normal((t, h), dtype=np.float32)
    if w.shared_beta > 0.0:
        # one shared direction per sequence of the batch
        s = g.standard_normal((w.batch, 1, h), dtype=np.float32)
        s = np.broadcast_to(s, (w.batch, w.block_len, h)).reshape(t, h)
        z = np.float32(math.sqrt(w.shared_beta)) * s + np.float32(math.sqrt(1.0 - w.shared_beta)) * z
    return z


def denoise_inputs(w: Workload) -> Iterator[Tuple[int, int, np.ndarray, np.ndarray]]:
    """Yield (block, iteration, hidden_bits [T,H] uint16, confidences [T] fp32).

    The layer-0 input of iteration i+1 is a noisy copy of iteration i's;
    confidences are drawn per iteration from Beta(a,b); a token whose
    confidence exceeds the threshold is finalised: its confidence is pinned
    to 1 and its hidden state no longer changes within the block.
    """
    t = w.tokens
    for b in range(w.blocks):
        gh = _rng(w, _STREAM_HIDDEN, b)
        gc = _rng(w, _STREAM_CONF, b)
        h = _noise(w, gh)
        final = np.zeros(t, dtype=bool)
        c = None
        for i in range(w.iters):
            if i > 0:
                eps = _noise(w, gh)
                if w.literal_mix:
                    nh = np.float32(w.rho) * h + np.float32(1.0 - w.rho) * eps
                elif w.conf_coupling > 0.0:
                    # per-token correlation: the previous iteration's confidence decides how far a
                    # token moves (high confidence => stable hidden state => stable routing)
                    rt = np.clip(w.rho + w.conf_coupling * (c.astype(np.float64) - 0.5), 0.0, 0.999)
                    nh = (rt[:, None] * h + np.sqrt(1.0 - rt * rt)[:, None] * eps).astype(np.float32)
                else:
                    nh = np.float32(w.rho) * h + np.float32(math.sqrt(1.0 - w.rho * w.rho)) * eps
                h = np.where(final[:, None], h, nh).astype(np.float32)
            c = gc.beta(w.beta_a, w.beta_b, size=t).astype(np.float32)
            c = np.where(final, np.float32(1.0), c).astype(np.float32)
            yield b, i, f32_to_bf16_bits(h), c
            final = final | (c > np.float32(w.finalize_threshold))


def flat_tokens(w: Workload, n_tokens: int, stream_id: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """A single step's inputs with an arbitrary token count (edge-case tests)."""
    g = _rng(w, _STREAM_HIDDEN, 1000 + stream_id, n_tokens)
    h = g.standard_normal((n_tokens, w.hidden), dtype=np.float32)
    c = g.beta(w.beta_a, w.beta_b, size=n_tokens).astype(np.float32)
    return f32_to_bf16_bits(h), c


# --------------------------------------------------------------------------
# Narrow expert blobs: fp8 (e4m3) weights with one fp32 scale per output row
# --------------------------------------------------------------------------
def f32_to_e4m3_codes(x: np.ndarray) -> np.ndarray:
    """Round to the nearest e4m3 value (ties to the even code), saturating at +-448."""
    xf = np.asarray(x, dtype=np.float64)
    a = np.minimum(np.abs(xf), 448.0)
    _, ex = np.frexp(a)                                   # a = m * 2^ex, m in [0.5, 1)
    qe = np.maximum(ex - 1, -6) - 3                       # exponent of the rounding quantum
    v = np.rint(np.ldexp(a, -qe))                         # 0..16 quanta, ties to even
    val = np.ldexp(v, qe)                                 # the rounded magnitude (may reach the next binade)
    _, ex2 = np.frexp(val)
    e_field = np.where(val < 2.0 ** -6, 0, ex2 - 1 + 7)
    m_field = np.where(val < 2.0 ** -6, np.ldexp(val, 9), (np.ldexp(val, -(ex2 - 1)) - 1.0) * 8.0)
    code = (e_field.astype(np.int64) << 3 | m_field.astype(np.int64)).astype(np.uint8)
    return code | (np.signbit(xf).astype(np.uint8) << 7)


def fp8_blob_bytes(w: Workload) -> int:
    """Bytes of one fp8 expert blob: gate[I,H] | up[I,H] | down[H,I] codes, then fp32 scales
    s_gate[I] | s_up[I] | s_down[H]; padded to a multiple of 256."""
    n = 3 * w.hidden * w.intermediate + 4 * (2 * w.intermediate + w.hidden)
    return (n + 255) // 256 * 256


def quantize_expert_blob(w: Workload, blob_bits: np.ndarray, out: Optional[np.ndarray] = None) -> np.ndarray:
    """bf16 expert blob -> fp8 blob.  Every row of the three matrices gets the scale
    max|row| / 448 (1 for an all-zero row) and its elements are rounded to e4m3."""
    h, i = w.hidden, w.intermediate
    if out is None:
        out = np.zeros(fp8_blob_bytes(w), dtype=np.uint8)
    mats = split_blob(w, blob_bits)
    off, scales = 0, []
    for m in mats:
        f = bf16_bits_to_f32(m)
        amax = np.abs(f).max(axis=1)
        sc = np.where(amax > 0, amax / np.float32(448.0), np.float32(1.0)).astype(np.float32)
        q = f32_to_e4m3_codes(f.astype(np.float64) / sc[:, None].astype(np.float64))
        out[off:off + q.size] = q.reshape(-1)
        off += q.size
        scales.append(sc)
    sc_all = np.concatenate(scales).astype(np.float32)
    out[off:off + 4 * sc_all.size] = sc_all.view(np.uint8)
    return out
