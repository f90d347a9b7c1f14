"""Shared helpers of the GPU parity tests: move generated inputs to the device, run the
library through its C ABI, run the fp64 oracle on the same bits, and compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from workloads import GdnInputs, widen

# Tolerances (vs the fp64 oracle, over the whole tensor): bf16 storage with fp32
# accumulation, and the fp32 path.
BF16_REL_L2 = 5e-3
BF16_MAX_ABS = 2e-2
F32_REL_L2 = 1e-5


def to_device(x: GdnInputs, device="cuda"):
    def t(a):
        if a is None:
            return None
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).to(device)
        return torch.from_numpy(a).to(device)
    d = dict(q=t(x.q), k=t(x.k), v=t(x.v), log_alpha=t(x.log_alpha), beta=t(x.beta),
             initial_state=t(x.initial_state), cu_seqlens=t(x.cu_seqlens))
    d["out"] = torch.empty_like(d["v"])
    N = len(x.lengths)
    d["final_state"] = torch.empty((N, x.cfg.H, x.cfg.d_k, x.cfg.d_v), dtype=torch.float32, device=device)
    return d


def run_lib(fn, d, **kw):
    out, fin = fn(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["initial_state"], d["out"],
                  d["final_state"], d["cu_seqlens"], **kw)
    torch.cuda.synchronize()
    return out, fin


def run_oracle(x: GdnInputs):
    return oracle.sequential(widen(x.q), widen(x.k), widen(x.v), x.log_alpha, x.beta,
                             x.initial_state, x.cu_seqlens)


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def errors(got: np.ndarray, want: np.ndarray):
    diff = got - want
    denom = np.linalg.norm(want)
    rel = float(np.linalg.norm(diff) / denom) if denom > 0 else float(np.linalg.norm(diff))
    return rel, float(np.abs(diff).max()) if diff.size else 0.0


def assert_close(got, want, rel_tol, abs_tol=None, what=""):
    assert np.isfinite(got).all(), f"{what}: non-finite values"
    rel, mx = errors(got, want)
    assert rel <= rel_tol, f"{what}: rel-L2 {rel:.3e} > {rel_tol:.1e} (max-abs {mx:.3e})"
    if abs_tol is not None:
        assert mx <= abs_tol, f"{what}: max-abs {mx:.3e} > {abs_tol:.1e} (rel-L2 {rel:.3e})"
    return rel, mx


def _prefill_path(path):
    """gdn_chunk_prefill pinned to one implementation: 1 = fused kernel, 2 = two-kernel pipeline
    (with a freshly allocated workspace)."""
    import paper_2607_14568_b200 as gdn

    def fn(q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens=None, **kw):
        if cu_seqlens is None:
            B, T, H, d_k = q.shape
        else:
            T, H, d_k = q.shape
            B = cu_seqlens.numel() - 1
        ws = None
        if path == 2:
            nbytes = gdn.gdn_workspace_bytes(B, T, H, d_k, v.shape[-1], cu_seqlens is not None)
            ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=q.device)
            gdn.gdn_set_workspace(ws)
        gdn.lib().gdn_debug_force_path(path)
        try:
            r = gdn.gdn_chunk_prefill(q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens, **kw)
            torch.cuda.synchronize()
            assert gdn.gdn_query_status() == 0
        finally:
            gdn.lib().gdn_debug_force_path(0)
            gdn.gdn_set_workspace(None)
        return r
    return fn


prefill_fused = _prefill_path(1)
prefill_two_kernel = _prefill_path(2)
