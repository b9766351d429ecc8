"""CPU oracle of the denoise step over a stack of MoE layers.  TEST INFRASTRUCTURE ONLY.

Mirrors the per-layer flow of the paper's system overview (Sec. 4.1): the gate
produces expert ids and gate scores; cache hits and misses are decided against
the layer's resident set before execution; every activated expert is computed
(misses are fetched, never executed on the CPU); after execution the
retention rule of Sec. 4.2/4.3 yields the resident set the same layer sees in
the next denoising iteration.  Offloading is lossless (Sec. 5.1 measurement
protocol): the layer output does not depend on the cache capacity.
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence

import numpy as np

from .cache_policy import AdaptiveSizer, LayerCache, LayerStats
from .moe_layer import (bf16_to_f32, fp8_expert_weights, gate_logits, moe_layer_forward, permutation,
                        topk_route)


class OracleStack:
    """Weights, per-layer cache state and counters of an L-layer MoE stack."""

    def __init__(self, n_layers: int, hidden: int, n_experts: int, top_k: int, intermediate: int,
                 capacity: Sequence[int], policy: str = "priority"):
        assert len(capacity) == n_layers
        self.n_layers, self.hidden, self.n_experts = n_layers, hidden, n_experts
        self.top_k, self.intermediate = top_k, intermediate
        self.expert_bytes = 3 * hidden * intermediate * 2
        self.caches: List[LayerCache] = [LayerCache(n_experts, int(c), self.expert_bytes, policy=policy)
                                         for c in capacity]
        self.total_capacity = sum(int(c) for c in capacity)
        self.sizer = AdaptiveSizer(n_layers, n_experts)
        self.router: List[Optional[np.ndarray]] = [None] * n_layers
        self.bias: List[Optional[np.ndarray]] = [None] * n_layers
        self.experts: List[Optional[Callable[[int], tuple]]] = [None] * n_layers

    def register_router(self, layer: int, w_router_bits: np.ndarray, bias=None) -> None:
        assert w_router_bits.shape == (self.n_experts, self.hidden)
        self.router[layer] = w_router_bits
        self.bias[layer] = None if bias is None else np.asarray(bias, dtype=np.float32)

    def register_experts(self, layer: int, blobs_bits: np.ndarray) -> None:
        """blobs_bits: uint16 [E, 3*H*I], each row gate[I,H] | up[I,H] | down[H,I]."""
        h, i = self.hidden, self.intermediate
        assert blobs_bits.shape == (self.n_experts, 3 * h * i)

        def get(e: int):
            b = blobs_bits[e]
            return (b[:h * i].reshape(i, h), b[h * i:2 * h * i].reshape(i, h),
                    b[2 * h * i:].reshape(h, i))
        self.experts[layer] = get

    def register_experts_fp8(self, layer: int, blobs: np.ndarray) -> None:
        """blobs: uint8 [E, blob_bytes], each row an fp8 expert blob (codes, then row scales)."""
        h, i = self.hidden, self.intermediate
        assert blobs.shape[0] == self.n_experts and blobs.shape[1] >= 3 * h * i + 4 * (2 * i + h)
        self.experts[layer] = lambda e: fp8_expert_weights(blobs[e], h, i)
        self.expert_bytes = int(blobs.shape[1])
        for c in self.caches:
            c.expert_bytes = self.expert_bytes

    def denoise_step(self, layer: int, hidden_bits: np.ndarray, conf: np.ndarray) -> dict:
        """One layer execution of one denoising iteration; returns every intermediate."""
        res = moe_layer_forward(hidden_bits, self.router[layer], self.bias[layer], self.experts[layer],
                        self.top_k)
        res.update(self.caches[layer].step(res["ids"], res["gate"], conf))
        return res

    def route_step(self, layer: int, hidden_bits: np.ndarray, conf: np.ndarray) -> dict:
        """Gate, permutation and cache policy of one layer execution, without the expert FFNs
        (for large shapes, where outputs are checked on sampled tokens with ``token_outputs``)."""
        x = bf16_to_f32(hidden_bits)
        logits = gate_logits(x, bf16_to_f32(self.router[layer]), self.bias[layer])
        ids, g = topk_route(logits, self.top_k)
        counts, offsets, perm, pos = permutation(ids, self.n_experts)
        res = dict(logits=logits, ids=ids, gate=g, counts=counts, offsets=offsets, perm=perm, pos=pos)
        res.update(self.caches[layer].step(ids, g, conf))
        return res

    def token_outputs(self, layer: int, hidden_bits: np.ndarray, tokens) -> np.ndarray:
        """Layer output rows of the given tokens only (each token's output depends on no other)."""
        sel = np.asarray(hidden_bits)[list(tokens)]
        return moe_layer_forward(sel, self.router[layer], self.bias[layer], self.experts[layer],
                                 self.top_k)["out"]

    def policy_step(self, layer: int, ids: np.ndarray, gate: np.ndarray, conf: np.ndarray) -> dict:
        """Cache simulation alone, from recorded routing."""
        return self.caches[layer].step(ids, gate, conf)

    def adapt_capacity(self) -> List[int]:
        """Layer-adaptive sizing (Sec. 4.3): new C_l from the statistics of the period that just
        ended; a layer left with more residents than slots drops its lowest-valued ones at once."""
        caps = self.sizer.refresh(self.caches, self.total_capacity)
        for c, cap in zip(self.caches, caps):
            c.shrink_to(cap)
        return caps

    def stats(self, layer: int = -1) -> LayerStats:
        if layer >= 0:
            return self.caches[layer].stats
        tot = LayerStats()
        for c in self.caches:
            tot.add(c.stats)
        return tot

    def reset_cache(self) -> None:
        for c in self.caches:
            c.reset()
        self.sizer = AdaptiveSizer(self.n_layers, self.n_experts)
