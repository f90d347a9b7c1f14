"""Seeded synthetic workloads (input generators only; no method arithmetic)."""
from .gdn_inputs import (CONFIGS, GdnConfig, GdnInputs, bf16_bits_to_f32, chain_inputs,  # noqa: F401
                         epilogue_inputs, f32_to_bf16_bits, get_config, make_inputs, widen)
from .attn_inputs import ATTN_CONFIGS, AttnConfig, get_attn_config, make_attn_inputs  # noqa: F401
