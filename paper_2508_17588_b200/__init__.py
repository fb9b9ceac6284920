"""HERO cached DiT step for B200: ctypes binding over the sm_100a CUDA library (libhero.so)."""
from .binding import (  # noqa: F401
    DTYPE_BF16, DTYPE_FP32, EXPORTS, Hero, HeroError, device_weights, hero_attention_bf16, hero_attention_bf16_static,
    hero_extrapolate, hero_extrapolation_error, hero_second_difference_moments,
    hero_gather_rows, hero_gemm_bf16, hero_isolated_status, hero_scatter_rows, load,
    hero_attention_bf16_static_status, hero_attention_bf16_safe, hero_attention_bf16_q_scaled, hero_gather_ln_modulate, hero_selftest_wait_timeout,
)
