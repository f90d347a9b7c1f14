"""Seeded synthetic inputs for the gated delta-rule prefill.

This module is the only code shared by the CPU oracle's tests and the CUDA
library's tests and benchmark.  It holds none of the method's arithmetic: it only
draws random tensors with the shapes and value distributions of the five
benchmark configurations and rounds them to their storage type.

Every (sequence, head) chain is drawn from its own counter-based stream
(Philox keyed by ``(seed, sequence * H + head)``), in the fixed order
q, k, v, beta, log_alpha, initial state.  A chain can therefore be regenerated on
its own -- which is how full-size runs are spot-checked against the oracle one
chain at a time -- and the full tensors are just the chains laid side by side.

Distributions (per token and head):
  q, k       N(0,1), then L2-normalised over the feature axis (in fp32)
  v          N(0,1)
  beta       sigmoid(N(0,1))                      fp32
  log_alpha  -softplus(N(0,1)) * gate_scale       fp32 (natural log of the gate)
  S0         N(0, init_std) fp32, or absent (zeros) when init_std == 0
With ``raw=True`` the tensors are the raw projections instead, for the entry point that
runs the norms and gating itself: q, k are N(0,1) times a per-(token, head) magnitude
exp(N(0, 0.5)) and are not normalised, and the ``beta`` / ``log_alpha`` fields hold the N(0,1)
pre-activations (the call is given ``gate_scale``).
q, k, v are then rounded to the storage type (bf16 round-to-nearest-even, or kept
fp32).  bf16 tensors are returned as uint16 bit patterns.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np


@dataclass(frozen=True)
class GdnConfig:
    name: str
    B: int                      # sequences
    T: int                      # tokens per sequence (ignored when lengths is set)
    H: int
    d_k: int
    d_v: int
    dtype: str                  # storage type of q, k, v, out: "f32" or "bf16"
    gate_scale: float
    init_std: float             # 0.0 -> no initial state (zeros)
    seed: int
    chunk: int = 64
    varlen: Optional[Tuple[int, int]] = None   # (lo, hi): packed sequences, lengths ~ U{lo..hi}
    lengths: Optional[Tuple[int, ...]] = None  # explicit packed lengths (overrides varlen)
    raw: bool = False           # raw projections: q, k not normalised, gates left as pre-activations

    @property
    def packed(self) -> bool:
        return self.varlen is not None or self.lengths is not None

    def seq_lengths(self) -> List[int]:
        if self.lengths is not None:
            return list(self.lengths)
        if self.varlen is not None:
            lo, hi = self.varlen
            rng = np.random.Generator(np.random.Philox(key=[self.seed, 2**63 + 1]))
            return [int(x) for x in rng.integers(lo, hi + 1, size=self.B)]
        return [self.T] * self.B

    def total_tokens(self) -> int:
        return int(sum(self.seq_lengths()))


# The five benchmark configurations.
CONFIGS: Dict[str, GdnConfig] = {
    "tiny": GdnConfig("tiny", B=1, T=256, H=2, d_k=64, d_v=64, dtype="f32",
                      gate_scale=0.1, init_std=0.0, seed=0),
    "short": GdnConfig("short", B=1, T=2048, H=16, d_k=128, d_v=128, dtype="bf16",
                       gate_scale=0.05, init_std=0.0, seed=1),
    "long": GdnConfig("long", B=1, T=10240, H=16, d_k=128, d_v=128, dtype="bf16",
                      gate_scale=0.05, init_std=0.02, seed=2),
    "serving": GdnConfig("serving", B=8, T=0, H=16, d_k=128, d_v=128, dtype="bf16",
                         gate_scale=0.05, init_std=0.02, seed=3, varlen=(512, 8192)),
    "large": GdnConfig("large", B=4, T=32768, H=32, d_k=128, d_v=256, dtype="bf16",
                       gate_scale=0.02, init_std=0.0, seed=4),
}


def get_config(name: str, **overrides) -> GdnConfig:
    cfg = CONFIGS[name]
    return replace(cfg, **overrides) if overrides else cfg


# ---------------------------------------------------------------------------
# storage-type helpers (bit manipulation only)
# ---------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def widen(x: np.ndarray) -> np.ndarray:
    """Exact fp64 view of a stored tensor (uint16 = bf16 bits, else float)."""
    if x.dtype == np.uint16:
        return bf16_bits_to_f32(x).astype(np.float64)
    return x.astype(np.float64)


# ---------------------------------------------------------------------------
# one chain
# ---------------------------------------------------------------------------
def _store(x: np.ndarray, dtype: str) -> np.ndarray:
    return f32_to_bf16_bits(x) if dtype == "bf16" else np.ascontiguousarray(x, dtype=np.float32)


def chain_inputs(cfg: GdnConfig, n: int, h: int, length: Optional[int] = None) -> Dict[str, np.ndarray]:
    """Inputs of sequence ``n``, head ``h``: q,k [L,d_k], v [L,d_v], beta,log_alpha [L], s0 [d_k,d_v] or None."""
    L = cfg.seq_lengths()[n] if length is None else length
    rng = np.random.Generator(np.random.Philox(key=[cfg.seed, n * cfg.H + h]))
    q = rng.standard_normal((L, cfg.d_k), dtype=np.float32)
    k = rng.standard_normal((L, cfg.d_k), dtype=np.float32)
    v = rng.standard_normal((L, cfg.d_v), dtype=np.float32)
    braw = rng.standard_normal(L, dtype=np.float32)
    araw = rng.standard_normal(L, dtype=np.float32)
    if not cfg.raw:
        q /= np.linalg.norm(q, axis=-1, keepdims=True)
        k /= np.linalg.norm(k, axis=-1, keepdims=True)
        beta = (1.0 / (1.0 + np.exp(-braw.astype(np.float64)))).astype(np.float32)
        log_alpha = (-np.logaddexp(0.0, araw.astype(np.float64)) * cfg.gate_scale).astype(np.float32)
    else:
        beta, log_alpha = braw, araw
    s0 = None
    if cfg.init_std > 0.0:
        s0 = (rng.standard_normal((cfg.d_k, cfg.d_v), dtype=np.float32) * np.float32(cfg.init_std))
    if cfg.raw:     # drawn last, so that every other tensor is the same as without raw
        q *= np.exp(0.5 * rng.standard_normal((L, 1), dtype=np.float32))
        k *= np.exp(0.5 * rng.standard_normal((L, 1), dtype=np.float32))
    return {"q": _store(q, cfg.dtype), "k": _store(k, cfg.dtype), "v": _store(v, cfg.dtype),
            "beta": beta, "log_alpha": log_alpha, "s0": s0}


# ---------------------------------------------------------------------------
# whole tensors
# ---------------------------------------------------------------------------
@dataclass
class GdnInputs:
    cfg: GdnConfig
    q: np.ndarray               # [B,T,H,d_k] or packed [T,H,d_k]; float32 or uint16 (bf16 bits)
    k: np.ndarray
    v: np.ndarray
    log_alpha: np.ndarray       # [B,T,H] or [T,H] float32
    beta: np.ndarray
    initial_state: Optional[np.ndarray]   # [N,H,d_k,d_v] float32 or None
    cu_seqlens: Optional[np.ndarray]      # int32 [N+1] or None
    lengths: List[int] = field(default_factory=list)

    @property
    def T_arg(self) -> int:
        """The ``T`` argument of the library call (total tokens when packed)."""
        return int(self.q.shape[0]) if self.cu_seqlens is not None else int(self.q.shape[1])


def make_inputs(cfg: GdnConfig, threads: int = 8) -> GdnInputs:
    lengths = cfg.seq_lengths()
    N, H = cfg.B, cfg.H
    st = np.uint16 if cfg.dtype == "bf16" else np.float32
    if cfg.packed:
        Tt = int(sum(lengths))
        starts = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
        lead = (Tt,)
        cu = starts.astype(np.int32)
    else:
        lead = (N, cfg.T)
        starts = None
        cu = None
    q = np.zeros(lead + (H, cfg.d_k), dtype=st)
    k = np.zeros(lead + (H, cfg.d_k), dtype=st)
    v = np.zeros(lead + (H, cfg.d_v), dtype=st)
    la = np.zeros(lead + (H,), dtype=np.float32)
    be = np.zeros(lead + (H,), dtype=np.float32)
    s0 = np.zeros((N, H, cfg.d_k, cfg.d_v), dtype=np.float32) if cfg.init_std > 0.0 else None

    def fill(nh):
        n, h = divmod(nh, H)
        c = chain_inputs(cfg, n, h, lengths[n])
        if cfg.packed:
            sl = slice(int(starts[n]), int(starts[n + 1]))
            q[sl, h], k[sl, h], v[sl, h] = c["q"], c["k"], c["v"]
            la[sl, h], be[sl, h] = c["log_alpha"], c["beta"]
        else:
            q[n, :, h], k[n, :, h], v[n, :, h] = c["q"], c["k"], c["v"]
            la[n, :, h], be[n, :, h] = c["log_alpha"], c["beta"]
        if s0 is not None:
            s0[n, h] = c["s0"]

    if threads > 1 and N * H > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(fill, range(N * H)))
    else:
        for nh in range(N * H):
            fill(nh)
    return GdnInputs(cfg, q, k, v, la, be, s0, cu, lengths)


def epilogue_inputs(cfg: GdnConfig, lead_shape) -> Dict[str, np.ndarray]:
    """Inputs of the fused output stage for a workload: the gate tensor z ~ N(0,1) with the shape of `out`
    (``lead_shape + (H, d_v)``, stored like v) and the norm weight 1 + 0.1 N(0,1), fp32 [d_v].  One Philox
    stream keyed by the seed and a constant no chain uses."""
    rng = np.random.Generator(np.random.Philox(key=[cfg.seed, (1 << 40) + 17]))
    z = rng.standard_normal(tuple(lead_shape) + (cfg.H, cfg.d_v), dtype=np.float32)
    w = (1.0 + 0.1 * rng.standard_normal(cfg.d_v, dtype=np.float32)).astype(np.float32)
    return {"z": _store(z, cfg.dtype), "weight": w}
