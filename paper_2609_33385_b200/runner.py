"""Harness that feeds a synthetic workload to the library: memory, streams and the decode loop.

torch is used for device memory, pinned host memory and the CUDA stream only; every step of
the hot path runs inside liboled.so through the C ABI (``binding.OledContext``).

The loop mimics block-wise semi-autoregressive decoding (paper Sec. 2.1): for each block, for
each denoising iteration, every layer of the stack executes once; the residual between the
layers of this MoE-only stack is x_{l+1} = bf16(x_l + out_l).
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from typing import List, Optional, Sequence

import numpy as np
import torch

from . import synth
from .binding import (EXPERTS_BF16, EXPERTS_FP8, OPT_ADAPT_PERIOD, OPT_FFN_IMPL, OPT_MISS_CHUNK, OPT_POLICY, POLICY_IDS,
                      OledContext)


def bits_to_dev(bits: np.ndarray, device) -> torch.Tensor:
    """uint16 bf16 bit patterns -> bf16 tensor on ``device``."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


def dev_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)


class StackRunner:
    """An L-layer MoE stack registered with one library context."""

    def __init__(self, w: synth.Workload, capacity: Optional[Sequence[int]] = None,
                 device: str = "cuda:0", distinct_layers: Optional[int] = None,
                 gen_threads: Optional[int] = None, ffn_impl: Optional[int] = None,
                 miss_chunk: Optional[int] = None, max_tokens: Optional[int] = None,
                 staging_slots: int = 0, share_store_of: Optional["StackRunner"] = None,
                 policy: Optional[str] = None, adapt_period: Optional[int] = None, fp8: bool = False):
        self.w = w
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        caps = [w.capacity] * w.n_layers if capacity is None else [int(c) for c in capacity]
        self.capacity = caps
        self.max_tokens = max_tokens or w.tokens
        self.stream = torch.cuda.current_stream(self.device)
        self.ctx = OledContext(w.n_layers, w.hidden, w.n_experts, w.top_k, w.intermediate,
                               self.max_tokens, caps, self.stream.cuda_stream,
                               has_router_bias=w.has_bias, staging_slots=staging_slots,
                               expert_format=EXPERTS_FP8 if fp8 else EXPERTS_BF16)
        self.fp8 = fp8
        if ffn_impl is not None:
            self.ctx.set_option(OPT_FFN_IMPL, ffn_impl)
        if miss_chunk is not None:
            self.ctx.set_option(OPT_MISS_CHUNK, miss_chunk)
        if policy is not None:
            self.ctx.set_option(OPT_POLICY, POLICY_IDS[policy])
        if adapt_period is not None:
            self.ctx.set_option(OPT_ADAPT_PERIOD, adapt_period)
        threads = gen_threads or min(32, len(os.sched_getaffinity(0)))
        n_distinct = w.n_layers if distinct_layers is None else max(1, min(distinct_layers, w.n_layers))
        self.n_distinct = n_distinct
        # host expert store: pinned, one [E, 3*H*I] block of bf16 bits per distinct layer
        self._host_t: List[torch.Tensor] = []
        self.blobs: List[np.ndarray] = []
        if share_store_of is not None:         # same pinned host expert store, another context
            self.n_distinct = n_distinct = share_store_of.n_distinct
            self._host_t = share_store_of._host_t
            self.blobs = share_store_of.blobs
        for d in range(0 if share_store_of is not None else n_distinct):
            if fp8:   # bf16 weights are generated, then quantised row by row into the pinned fp8 store
                nb = synth.fp8_blob_bytes(w)
                t = torch.zeros((w.n_experts, nb), dtype=torch.uint8, pin_memory=True)
                a = t.numpy()
                def one(e, d=d, a=a):
                    synth.quantize_expert_blob(w, synth.expert_blob_bits(w, d, e), a[e])
                with ThreadPoolExecutor(max_workers=max(1, threads)) as ex:
                    list(ex.map(one, range(w.n_experts)))
            else:
                t = torch.empty((w.n_experts, w.expert_elems), dtype=torch.int16, pin_memory=True)
                a = t.numpy().view(np.uint16)
                synth.fill_layer_blobs(w, d, a, threads=threads)
            self._host_t.append(t)
            self.blobs.append(a)
        self.router_bits: List[np.ndarray] = []
        self.bias: List[Optional[np.ndarray]] = []
        self._router_dev = []
        for l in range(w.n_layers):
            wr, b = synth.router_weights(w, l)
            self.router_bits.append(wr)
            self.bias.append(b)
            wr_d = bits_to_dev(wr, self.device)
            b_d = None if b is None else torch.from_numpy(b).to(self.device)
            self._router_dev.append((wr_d, b_d))
            self.ctx.register_router(l, wr_d.data_ptr(), None if b_d is None else b_d.data_ptr())
            ht = self._host_t[l % n_distinct]
            self.ctx.register_experts(l, ht.data_ptr(), self.ctx.expert_bytes)

    def layer_blobs(self, layer: int) -> np.ndarray:
        return self.blobs[layer % self.n_distinct]

    # -- one layer execution with device tensors (bf16 [T,H], fp32 [T], bf16 [T,H])
    def step(self, layer: int, hidden: torch.Tensor, conf: torch.Tensor, out: torch.Tensor) -> None:
        n = hidden.shape[0]
        self.ctx.denoise_step(layer, hidden.data_ptr(), conf.data_ptr(), n, out.data_ptr())

    def step_host(self, layer: int, hidden: torch.Tensor, conf: torch.Tensor, out: torch.Tensor) -> None:
        n = hidden.shape[0]
        self.ctx.denoise_step_host(layer, hidden.data_ptr(), conf.data_ptr(), n, out.data_ptr())

    def iteration(self, x0: torch.Tensor, conf: torch.Tensor, bufs: List[torch.Tensor],
                  out: torch.Tensor) -> torch.Tensor:
        """All layers once: x_{l+1} = bf16(x_l + out_l).  ``bufs``: two [T,H] bf16 scratch tensors."""
        x = x0
        n = x0.numel()
        for l in range(self.w.n_layers):
            self.step(l, x, conf, out)
            nxt = bufs[l & 1]
            self.ctx.residual_add(x.data_ptr(), out.data_ptr(), nxt.data_ptr(), n)
            x = nxt
        return x

    def close(self) -> None:
        self.ctx.destroy()
