"""B200-native MoE denoise step with a bounded expert cache (OLED-MoE hot path).

``synth`` (workload generator) imports without the CUDA library; ``binding`` / ``runner``
load liboled.so and raise if it has not been built — there is no CPU fallback.
"""
__all__ = ["synth", "binding", "runner", "build"]
