"""ctypes binding of the C ABI in include/oled.h — argument marshalling only.

Every step of the hot path runs inside liboled.so; nothing here computes.  The library must be
present (``python -m paper_2609_33385_b200.build``): there is no CPU fallback, and a missing or
unloadable library raises at load time.

Tensors are passed as raw device/host pointers (``tensor.data_ptr()``); torch is used by the
callers for device memory, pinned host memory and streams only.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liboled.so")

OLED_OK = 0
ERR_INVALID_ARG, ERR_NOT_PINNED, ERR_NOT_REGISTERED, ERR_TOO_MANY_TOKENS = -1, -2, -3, -4
ERR_OOM, ERR_CUDA, ERR_TIMEOUT, ERR_NO_SLOT, ERR_STALE_DEBUG = -5, -6, -7, -8, -9
OPT_FFN_IMPL, OPT_MISS_CHUNK, OPT_PROFILE, OPT_POLICY, OPT_ADAPT_PERIOD = 1, 2, 3, 4, 5
OPT_TEST_WITHHOLD_LOADS = 6
OPT_SELF_CHECK, OPT_TEST_CORRUPT_PERM = 7, 8
OPT_SPLIT_LAST_FILL, OPT_FUSE_COMBINE, OPT_FUSE_FFN, OPT_PDL, OPT_TIMELINE, OPT_FP8_DIRECT = 9, 10, 11, 12, 13, 14
OPT_FFN_PAIRS = 15
OPT_L2_PREFETCH = 16
OPT_GATHER_IN_FFN = 17
TIMELINE_SLOTS = 12
ERR_SELF_CHECK = -10
CHECK_FLAGS = {0x01: "id_range", 0x02: "id_duplicate", 0x04: "offsets", 0x08: "perm_range", 0x10: "inverse",
               0x20: "row_expert", 0x40: "order"}
POLICY_PRIORITY, POLICY_LRU, POLICY_LFU = 0, 1, 2
POLICY_IDS = {"priority": 0, "lru": 1, "lfu": 2}
KERNEL_NAMES = ["route", "permute", "gather", "ffn_gate_up", "ffn_down", "combine", "ffn_fused"]

EXPORTS = [
    "oled_create", "oled_register_router", "oled_register_experts", "oled_denoise_step",
    "oled_denoise_step_host", "oled_denoise_iteration", "oled_denoise_iteration_host", "oled_stats", "oled_debug_last", "oled_debug_logits",
    "oled_reset_cache", "oled_residual_add", "oled_set_option", "oled_profile_read", "oled_launch_count",
    "oled_synchronize", "oled_destroy", "oled_strerror", "oled_last_cuda_error",
    "oled_policy_create", "oled_policy_step", "oled_policy_destroy", "oled_route_noalloc",
    "oled_adapt_capacity", "oled_get_capacity", "oled_policy_set_policy", "oled_policy_fills_reused",
    "oled_policy_adapt", "oled_clear_status", "oled_policy_time", "oled_expert_blob_bytes",
    "oled_self_check_report", "oled_debug_perm", "oled_policy_create_stack", "oled_debug_timeline",
]
EXPERTS_BF16, EXPERTS_FP8 = 0, 1
NOALLOC_MAX_TOKENS = 256


class ModelShape(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("hidden", C.c_int32), ("n_experts", C.c_int32),
                ("top_k", C.c_int32), ("intermediate", C.c_int32), ("max_tokens", C.c_int32),
                ("has_router_bias", C.c_int32), ("staging_slots", C.c_int32),
                ("expert_format", C.c_int32)]


class KernelProfile(C.Structure):
    _fields_ = [("launches", C.c_uint64), ("ms", C.c_double), ("bytes", C.c_uint64),
                ("flops", C.c_uint64)]


class StatsStruct(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("steps", "hits", "misses", "bytes_moved", "evictions",
                                          "active_experts", "assignments", "fills_reused", "ideal_hits")]


@dataclass
class Stats:
    steps: int = 0
    hits: int = 0
    misses: int = 0
    bytes_moved: int = 0
    evictions: int = 0
    active_experts: int = 0
    assignments: int = 0
    fills_reused: int = 0
    ideal_hits: int = 0


class OledError(RuntimeError):
    def __init__(self, code: int, what: str, cuda_error: int = 0):
        self.code = code
        self.cuda_error = cuda_error
        msg = f"{what}: {strerror(code)} ({code})"
        if cuda_error:
            msg += f" [cudaError {cuda_error}]"
        super().__init__(msg)


_lib = None


def load() -> C.CDLL:
    """Load liboled.so; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                           "`python -m paper_2609_33385_b200.build` (nvcc, sm_100a); "
                           "there is no CPU fallback")
    lib = C.CDLL(LIB_PATH)
    vp, i32, u64p = C.c_void_p, C.c_int32, C.POINTER(C.c_uint64)
    lib.oled_create.argtypes = [C.POINTER(ModelShape), C.POINTER(C.c_int32), vp, C.POINTER(vp)]
    lib.oled_register_router.argtypes = [vp, i32, vp, vp]
    lib.oled_register_experts.argtypes = [vp, i32, vp, C.c_size_t]
    lib.oled_denoise_step.argtypes = [vp, i32, vp, vp, i32, vp]
    lib.oled_denoise_step_host.argtypes = [vp, i32, vp, vp, i32, vp]
    lib.oled_denoise_iteration.argtypes = [vp, vp, vp, i32, vp]
    lib.oled_denoise_iteration_host.argtypes = [vp, vp, vp, i32, vp]
    lib.oled_stats.argtypes = [vp, i32, C.POINTER(StatsStruct)]
    lib.oled_debug_last.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.oled_debug_logits.argtypes = [vp, i32, vp]
    lib.oled_debug_perm.argtypes = [vp, i32, vp, vp]
    lib.oled_debug_timeline.argtypes = [vp, i32, vp]
    lib.oled_policy_create_stack.argtypes = [i32, i32, C.POINTER(i32), i32, C.POINTER(vp), C.POINTER(i32)]
    lib.oled_reset_cache.argtypes = [vp]
    lib.oled_residual_add.argtypes = [vp, vp, vp, vp, C.c_size_t]
    lib.oled_set_option.argtypes = [vp, i32, C.c_int64]
    lib.oled_profile_read.argtypes = [vp, i32, i32, C.POINTER(KernelProfile)]
    lib.oled_launch_count.argtypes = [vp, u64p]
    lib.oled_synchronize.argtypes = [vp]
    lib.oled_destroy.argtypes = [vp]
    lib.oled_destroy.restype = None
    lib.oled_strerror.argtypes = [C.c_int]
    lib.oled_strerror.restype = C.c_char_p
    lib.oled_last_cuda_error.argtypes = [vp]
    lib.oled_policy_create.argtypes = [i32, i32, i32, C.POINTER(vp)]
    lib.oled_policy_step.argtypes = [vp, vp, vp, vp, vp, vp, C.POINTER(i32), C.POINTER(i32),
                                     C.POINTER(i32)]
    lib.oled_policy_destroy.argtypes = [vp]
    lib.oled_policy_destroy.restype = None
    lib.oled_expert_blob_bytes.argtypes = [i32, i32, i32]
    lib.oled_expert_blob_bytes.restype = C.c_size_t
    lib.oled_clear_status.argtypes = [vp]
    lib.oled_self_check_report.argtypes = [vp, vp, vp, vp]
    lib.oled_policy_time.argtypes = [vp, u64p, u64p]
    lib.oled_adapt_capacity.argtypes = [vp, vp]
    lib.oled_get_capacity.argtypes = [vp, vp]
    lib.oled_policy_set_policy.argtypes = [vp, i32]
    lib.oled_policy_fills_reused.argtypes = [vp, u64p]
    lib.oled_policy_adapt.argtypes = [C.POINTER(vp), i32, i32, vp]
    lib.oled_route_noalloc.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp]
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().oled_strerror(int(code)).decode()


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


class OledContext:
    """Thin handle over ``oled_ctx*``; method names follow the C entry points."""

    def __init__(self, n_layers: int, hidden: int, n_experts: int, top_k: int, intermediate: int,
                 max_tokens: int, cache_capacity: Sequence[int], cuda_stream: int = 0,
                 has_router_bias: bool = False, staging_slots: int = 0, expert_format: int = EXPERTS_BF16):
        self._lib = load()
        self.shape = ModelShape(n_layers, hidden, n_experts, top_k, intermediate, max_tokens,
                                1 if has_router_bias else 0, staging_slots, expert_format)
        caps = (C.c_int32 * n_layers)(*[int(c) for c in cache_capacity])
        h = C.c_void_p()
        rc = self._lib.oled_create(C.byref(self.shape), caps, C.c_void_p(cuda_stream), C.byref(h))
        self._h = h if rc == OLED_OK else None
        if rc != OLED_OK:
            raise OledError(rc, "oled_create")
        self.expert_bytes = int(self._lib.oled_expert_blob_bytes(hidden, intermediate, expert_format))

    # -- helpers
    def _check(self, rc: int, what: str) -> None:
        if rc != OLED_OK:
            cu = self._lib.oled_last_cuda_error(self._h) if rc == ERR_CUDA else 0
            raise OledError(rc, what, cu)

    # -- entry points
    def register_router(self, layer: int, w_router_ptr: int, bias_ptr: Optional[int] = None) -> None:
        self._check(self._lib.oled_register_router(self._h, layer, w_router_ptr, bias_ptr),
                    "oled_register_router")

    def register_experts(self, layer: int, host_blob_ptr: int, expert_stride_bytes: int) -> None:
        self._check(self._lib.oled_register_experts(self._h, layer, host_blob_ptr,
                                                    expert_stride_bytes), "oled_register_experts")

    def denoise_step(self, layer: int, hidden_ptr: int, conf_ptr: int, n_tokens: int,
                     out_ptr: int) -> None:
        self._check(self._lib.oled_denoise_step(self._h, layer, hidden_ptr, conf_ptr, n_tokens,
                                                out_ptr), "oled_denoise_step")

    def denoise_step_rc(self, layer: int, hidden_ptr, conf_ptr, n_tokens: int, out_ptr) -> int:
        return self._lib.oled_denoise_step(self._h, layer, hidden_ptr, conf_ptr, n_tokens, out_ptr)

    def denoise_step_host(self, layer: int, hidden_ptr: int, conf_ptr: int, n_tokens: int,
                          out_ptr: int) -> None:
        self._check(self._lib.oled_denoise_step_host(self._h, layer, hidden_ptr, conf_ptr,
                                                     n_tokens, out_ptr), "oled_denoise_step_host")

    def denoise_iteration(self, hidden_ptr: int, conf_ptr: int, n_tokens: int, out_ptr: int) -> None:
        self._check(self._lib.oled_denoise_iteration(self._h, hidden_ptr, conf_ptr, n_tokens, out_ptr),
                    "oled_denoise_iteration")

    def denoise_iteration_host(self, hidden_ptr: int, conf_ptr: int, n_tokens: int, out_ptr: int) -> None:
        self._check(self._lib.oled_denoise_iteration_host(self._h, hidden_ptr, conf_ptr, n_tokens,
                                                          out_ptr), "oled_denoise_iteration_host")

    def stats(self, layer: int = -1) -> Stats:
        s = StatsStruct()
        self._check(self._lib.oled_stats(self._h, layer, C.byref(s)), "oled_stats")
        return Stats(*[int(getattr(s, f[0])) for f in StatsStruct._fields_])

    def debug_last(self, layer: int, n_tokens: int) -> dict:
        e, k = self.shape.n_experts, self.shape.top_k
        out = dict(ids=np.zeros((n_tokens, k), np.int32), gate=np.zeros((n_tokens, k), np.float32),
                   perm=np.zeros(n_tokens * k, np.int32), counts=np.zeros(e, np.int32),
                   scores=np.zeros(e, np.uint64), resident_before=np.zeros(e, np.uint8),
                   resident_after=np.zeros(e, np.uint8))
        self._check(self._lib.oled_debug_last(self._h, layer, *[_np_ptr(out[n]) for n in
                                                                ("ids", "gate", "perm", "counts", "scores",
                                                                 "resident_before", "resident_after")]),
                    "oled_debug_last")
        return out

    def debug_perm(self, layer: int, n_tokens: int) -> dict:
        """offsets [E+1] and pos [T*k] (the inverse of perm) of the most recent step."""
        out = dict(offsets=np.zeros(self.shape.n_experts + 1, np.int32),
                   pos=np.zeros(n_tokens * self.shape.top_k, np.int32))
        self._check(self._lib.oled_debug_perm(self._h, layer, _np_ptr(out["offsets"]), _np_ptr(out["pos"])),
                    "oled_debug_perm")
        return out

    def debug_timeline(self, layer: int) -> np.ndarray:
        """[3, TIMELINE_SLOTS] uint64: earliest entry, earliest start, latest end per kernel slot."""
        out = np.zeros((3, TIMELINE_SLOTS), np.uint64)
        self._check(self._lib.oled_debug_timeline(self._h, layer, _np_ptr(out)), "oled_debug_timeline")
        return out

    def debug_logits(self, layer: int, n_tokens: int) -> np.ndarray:
        out = np.zeros((n_tokens, self.shape.n_experts), np.float32)
        self._check(self._lib.oled_debug_logits(self._h, layer, _np_ptr(out)), "oled_debug_logits")
        return out

    def adapt_capacity(self) -> list:
        caps = np.zeros(self.shape.n_layers, np.int32)
        self._check(self._lib.oled_adapt_capacity(self._h, _np_ptr(caps)), "oled_adapt_capacity")
        return caps.tolist()

    def get_capacity(self) -> list:
        caps = np.zeros(self.shape.n_layers, np.int32)
        self._check(self._lib.oled_get_capacity(self._h, _np_ptr(caps)), "oled_get_capacity")
        return caps.tolist()

    def reset_cache(self) -> None:
        self._check(self._lib.oled_reset_cache(self._h), "oled_reset_cache")

    def residual_add(self, x_ptr: int, r_ptr: int, y_ptr: int, n: int) -> None:
        self._check(self._lib.oled_residual_add(self._h, x_ptr, r_ptr, y_ptr, n), "oled_residual_add")

    def set_option(self, option: int, value: int) -> None:
        self._check(self._lib.oled_set_option(self._h, option, value), "oled_set_option")

    def profile_read(self, reset: bool = True) -> dict:
        """Per-kernel {launches, ms, bytes, flops} collected while OPT_PROFILE was on."""
        out = {}
        for k, name in enumerate(KERNEL_NAMES):
            p = KernelProfile()
            self._check(self._lib.oled_profile_read(self._h, k, 1 if reset else 0, C.byref(p)),
                        "oled_profile_read")
            out[name] = dict(launches=int(p.launches), ms=float(p.ms), bytes=int(p.bytes),
                             flops=int(p.flops))
        return out

    def launch_count(self) -> int:
        v = C.c_uint64()
        self._check(self._lib.oled_launch_count(self._h, C.byref(v)), "oled_launch_count")
        return int(v.value)

    def synchronize(self) -> None:
        self._check(self._lib.oled_synchronize(self._h), "oled_synchronize")

    def synchronize_rc(self) -> int:
        return self._lib.oled_synchronize(self._h)

    def clear_status(self) -> None:
        self._check(self._lib.oled_clear_status(self._h), "oled_clear_status")

    def self_check_report(self):
        """(names of the violated invariants, smallest offending index or -1, guard mask)."""
        flags, index, guard = C.c_uint32(0), C.c_int32(-1), C.c_uint32(0)
        self._check(self._lib.oled_self_check_report(self._h, C.byref(flags), C.byref(index),
                                                     C.byref(guard)), "oled_self_check_report")
        names = [n for bit, n in CHECK_FLAGS.items() if flags.value & bit]
        return names, index.value, guard.value

    def policy_time(self):
        """(nanoseconds spent in the host cache policy, number of policy runs)."""
        ns, runs = C.c_uint64(), C.c_uint64()
        self._check(self._lib.oled_policy_time(self._h, C.byref(ns), C.byref(runs)), "oled_policy_time")
        return int(ns.value), int(runs.value)

    def destroy(self) -> None:
        if self._h is not None:
            self._lib.oled_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def route_noalloc(hidden_ptr, w_router_ptr, bias_ptr, conf_ptr, n_tokens: int, hidden: int,
                  n_experts: int, top_k: int, cuda_stream: int, ids_ptr, gate_ptr, counts_ptr,
                  offsets_ptr, perm_ptr) -> int:
    """``oled_route_noalloc``: routing of one step with library-internal static scratch; the
    library allocates nothing.  All pointers are device pointers; returns the status code."""
    return load().oled_route_noalloc(hidden_ptr, w_router_ptr, bias_ptr, conf_ptr, n_tokens, hidden,
                                     n_experts, top_k, C.c_void_p(cuda_stream), ids_ptr, gate_ptr,
                                     counts_ptr, offsets_ptr, perm_ptr)


class PolicySim:
    """Host-only policy simulator (``oled_policy_*``): the library's C++ policy code, no GPU."""

    def __init__(self, n_experts: int, capacity: int, pool_slots: int, policy: str = "priority", _handle=None):
        self._lib = load()
        self.n_experts = n_experts
        if _handle is None:
            h = C.c_void_p()
            rc = self._lib.oled_policy_create(n_experts, capacity, pool_slots, C.byref(h))
            if rc != OLED_OK:
                raise OledError(rc, "oled_policy_create")
            self._h = h
        else:
            self._h = _handle
        rc = self._lib.oled_policy_set_policy(self._h, POLICY_IDS[policy])
        if rc != OLED_OK:
            raise OledError(rc, "oled_policy_set_policy")

    @staticmethod
    def stack(n_experts: int, capacity: Sequence[int], staging_slots: int = 0, policy: str = "priority"):
        """Simulators of the layers of one stack sharing one slot pool sized as ``oled_create``
        sizes it (``oled_policy_create_stack``); returns (list of PolicySim, pool size)."""
        n = len(capacity)
        caps = (C.c_int32 * n)(*[int(c) for c in capacity])
        arr = (C.c_void_p * n)()
        slots = C.c_int32()
        rc = load().oled_policy_create_stack(n, n_experts, caps, staging_slots, arr, C.byref(slots))
        if rc != OLED_OK:
            raise OledError(rc, "oled_policy_create_stack")
        return [PolicySim(n_experts, int(c), 0, policy, _handle=C.c_void_p(arr[i]))
                for i, c in enumerate(capacity)], int(slots.value)

    def fills_reused(self) -> int:
        v = C.c_uint64()
        self._lib.oled_policy_fills_reused(self._h, C.byref(v))
        return int(v.value)

    @staticmethod
    def adapt(sims, total_capacity: int) -> list:
        """Layer-adaptive sizing over simulated layers (``oled_policy_adapt``)."""
        arr = (C.c_void_p * len(sims))(*[s._h for s in sims])
        caps = np.zeros(len(sims), np.int32)
        rc = load().oled_policy_adapt(arr, len(sims), total_capacity, _np_ptr(caps))
        if rc != OLED_OK:
            raise OledError(rc, "oled_policy_adapt")
        return caps.tolist()

    def step(self, counts: np.ndarray, scores: np.ndarray) -> dict:
        e = self.n_experts
        counts = np.ascontiguousarray(counts, np.int32)
        scores = np.ascontiguousarray(scores, np.uint64)
        before, after = np.zeros(e, np.uint8), np.zeros(e, np.uint8)
        slot_of = np.zeros(e, np.int32)
        nh, nm, ne = C.c_int32(), C.c_int32(), C.c_int32()
        rc = self._lib.oled_policy_step(self._h, _np_ptr(counts), _np_ptr(scores), _np_ptr(before),
                                        _np_ptr(after), _np_ptr(slot_of), C.byref(nh), C.byref(nm),
                                        C.byref(ne))
        if rc != OLED_OK:
            raise OledError(rc, "oled_policy_step")
        return dict(resident_before=before, resident_after=after, slot_of=slot_of, hits=nh.value,
                    misses=nm.value, evictions=ne.value)

    def __del__(self):
        try:
            if self._h is not None:
                self._lib.oled_policy_destroy(self._h)
                self._h = None
        except Exception:
            pass
