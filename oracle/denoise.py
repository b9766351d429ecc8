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

from .cache_policy import LayerCache, LayerStats
from .moe_layer import moe_layer_forward


class OracleStack:
    """Weights, per-layer cache state and counters of an L-layer MoE stack."""

    def __init__(self, n_layers: int, hidden: int, n_experts: int, top_k: int, intermediate: int,
                 capacity: Sequence[int]):
        assert len(capacity) == n_layers
        self.n_layers, self.hidden, self.n_experts = n_layers, hidden, n_experts
        self.top_k, self.intermediate = top_k, intermediate
        self.expert_bytes = 3 * hidden * intermediate * 2
        self.caches: List[LayerCache] = [LayerCache(n_experts, int(c), self.expert_bytes)
                                         for c in capacity]
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

    def denoise_step(self, layer: int, hidden_bits: np.ndarray, conf: np.ndarray) -> dict:
        """One layer execution of one denoising iteration; returns every intermediate."""
        res = moe_layer_forward(hidden_bits, self.router[layer], self.bias[layer], self.experts[layer],
                        self.top_k)
        res.update(self.caches[layer].step(res["ids"], res["gate"], conf))
        return res

    def policy_step(self, layer: int, ids: np.ndarray, gate: np.ndarray, conf: np.ndarray) -> dict:
        """Cache simulation alone, from recorded routing."""
        return self.caches[layer].step(ids, gate, conf)

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
