"""Seeded synthetic inputs for the causal grouped-query attention workload (no arithmetic of the
method here: random tensors with the shapes of the backbone's attention layers, rounded to bf16).

q, k, v ~ N(0,1) per element, so scores scaled by 1/sqrt(d) are ~N(0,1) as after the usual q/k
normalisation.  Each (sequence, tensor) is its own Philox stream keyed by (seed, 3*b + which)."""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict

import numpy as np

from .gdn_inputs import f32_to_bf16_bits


@dataclass(frozen=True)
class AttnConfig:
    name: str
    B: int
    T: int
    Hq: int
    Hkv: int
    d: int
    seed: int

    @property
    def scale(self) -> float:
        return 1.0 / float(self.d) ** 0.5


# The prompt tiers of the paper's prefill table (2k and 10k tokens) on a 16-query-head,
# 8-key/value-head, d = 128 attention layer, plus a small case the oracle finishes in seconds.
ATTN_CONFIGS: Dict[str, AttnConfig] = {
    "attn_small": AttnConfig("attn_small", B=2, T=333, Hq=4, Hkv=2, d=128, seed=10),
    "attn_2k": AttnConfig("attn_2k", B=1, T=2048, Hq=16, Hkv=8, d=128, seed=11),
    "attn_10k": AttnConfig("attn_10k", B=1, T=10240, Hq=16, Hkv=8, d=128, seed=12),
}


def get_attn_config(name: str, **overrides) -> AttnConfig:
    cfg = ATTN_CONFIGS[name]
    return replace(cfg, **overrides) if overrides else cfg


def make_attn_inputs(cfg: AttnConfig):
    """(q, k, v) as uint16 bf16 bit patterns: q [B,T,Hq,d], k, v [B,T,Hkv,d]."""
    q = np.zeros((cfg.B, cfg.T, cfg.Hq, cfg.d), dtype=np.uint16)
    k = np.zeros((cfg.B, cfg.T, cfg.Hkv, cfg.d), dtype=np.uint16)
    v = np.zeros((cfg.B, cfg.T, cfg.Hkv, cfg.d), dtype=np.uint16)
    for b in range(cfg.B):
        for which, (dst, H) in enumerate(((q, cfg.Hq), (k, cfg.Hkv), (v, cfg.Hkv))):
            rng = np.random.Generator(np.random.Philox(key=[cfg.seed, 3 * b + which]))
            dst[b] = f32_to_bf16_bits(rng.standard_normal((cfg.T, H, cfg.d), dtype=np.float32))
    return q, k, v
