"""CPU oracle of the MoE denoise-step hot path.  TEST INFRASTRUCTURE ONLY.

Plain numpy, no blocking or fusion, written from the paper's definitions
(Sec. 2.1, 4.1-4.3).  Shares no code with the CUDA path and is never used by
it: only the tests, the smoke check and the benchmark's cpu-baseline /
reference legs import this package.
"""
from .moe_layer import (bf16_to_f32, fp8_e4m3_to_f32, fp8_expert_weights, gate_logits, exp_spec, topk_route, permutation,  # noqa: F401
                        expert_ffn, moe_layer_forward)
from .cache_policy import (psi, reuse_scores, priorities, retain_top_c, retain_by_value,  # noqa: F401
                           ideal_hits, apportion, AdaptiveSizer, LayerCache, LayerStats)
from .denoise import OracleStack  # noqa: F401
