"""Prefill on raw projections (norms and gating fused into the prepare kernel; Section "Prefill
projections: dequantize, then call the vendor") against the fp64 oracle: oracle.prologue followed by the token-by-token recurrence."""
import numpy as np
import pytest
import torch

import oracle
from workloads import get_config, make_inputs, widen
from gdn_testlib import BF16_MAX_ABS, BF16_REL_L2, assert_close, f64, to_device

pytestmark = pytest.mark.gpu


def _run_raw(gdn, d, cfg, eps, nseg=0):
    packed = d["cu_seqlens"] is not None
    if packed:
        T, H, d_k = d["q"].shape
        B = d["cu_seqlens"].numel() - 1
    else:
        B, T, H, d_k = d["q"].shape
    ws = torch.empty(max(gdn.gdn_workspace_bytes(B, T, H, d_k, cfg.d_v, packed), 256), dtype=torch.uint8, device="cuda")
    gdn.gdn_set_workspace(ws)
    gdn.lib().gdn_debug_force_segments(nseg)
    try:
        gdn.gdn_chunk_prefill_raw(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], cfg.gate_scale, eps,
                                  d["initial_state"], d["out"], d["final_state"], d["cu_seqlens"])
        torch.cuda.synchronize()
        assert gdn.gdn_query_status() == 0
    finally:
        gdn.lib().gdn_debug_force_segments(0)
        gdn.gdn_set_workspace(None)


def _oracle_raw(x, cfg, eps):
    q, k, la, be = oracle.prologue(widen(x.q), widen(x.k), x.log_alpha, x.beta, cfg.gate_scale, eps)
    return oracle.sequential(q, k, widen(x.v), la, be, x.initial_state, x.cu_seqlens)


@pytest.mark.parametrize("kw,eps,nseg", [
    (dict(B=2, T=64 * 5 + 23, H=2, init_std=0.3), 0.0, 0),
    (dict(B=1, T=64 * 20, H=2, init_std=0.0), 1e-6, 4),                       # sequence split
    (dict(B=3, T=0, H=2, init_std=0.2, lengths=(130, 64, 7)), 1e-6, 0),       # packed, ragged tails
    (dict(B=1, T=64 * 3, H=1, d_v=256, init_std=0.1, gate_scale=0.3), 0.5, 0),  # wide values, large eps
])
def test_raw_prefill_matches_oracle(kw, eps, nseg):
    import paper_2607_14568_b200 as gdn
    cfg = get_config("short", raw=True, **kw)
    x = make_inputs(cfg)
    d = to_device(x)
    _run_raw(gdn, d, cfg, eps, nseg)
    want_out, want_fin = _oracle_raw(x, cfg, eps)
    assert_close(f64(d["out"]), want_out, BF16_REL_L2, BF16_MAX_ABS, "out")
    assert_close(f64(d["final_state"]), want_fin, BF16_REL_L2, None, "final_state")


def test_raw_prefill_is_invariant_to_the_magnitude_of_q_and_k():
    """Scaling a raw q or k row by a power of two is exact in bf16 and must not change the result
    beyond fp32 rounding of the norms (eps = 0)."""
    import paper_2607_14568_b200 as gdn
    cfg = get_config("short", raw=True, B=1, T=64 * 4 + 9, H=2, init_std=0.2)
    x = make_inputs(cfg)
    d = to_device(x)
    _run_raw(gdn, d, cfg, 0.0)
    out1, fin1 = d["out"].clone(), d["final_state"].clone()
    d["q"] = (d["q"].float() * 4.0).to(torch.bfloat16)
    d["k"] = (d["k"].float() * 0.25).to(torch.bfloat16)
    _run_raw(gdn, d, cfg, 0.0)
    assert_close(f64(d["out"]), f64(out1), 2e-3, None, "out")
    assert_close(f64(d["final_state"]), f64(fin1), 1e-3, None, "final_state")


def test_zero_rows_and_missing_workspace():
    import paper_2607_14568_b200 as gdn
    cfg = get_config("short", raw=True, B=1, T=128, H=1, init_std=0.1)
    x = make_inputs(cfg)
    x.k[0, 5] = 0          # a zero key: no write at that token
    x.q[0, 9] = 0          # a zero query: a zero output row
    d = to_device(x)
    gdn.gdn_set_workspace(None)
    with pytest.raises(gdn.GdnError) as e:
        gdn.gdn_chunk_prefill_raw(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], cfg.gate_scale, 1e-6,
                                  d["initial_state"], d["out"], d["final_state"])
    assert e.value.status == 3   # GDN_ERR_WORKSPACE
    _run_raw(gdn, d, cfg, 1e-6)
    want_out, want_fin = _oracle_raw(x, cfg, 1e-6)
    assert_close(f64(d["out"]), want_out, BF16_REL_L2, BF16_MAX_ABS, "out")
    assert_close(f64(d["final_state"]), want_fin, BF16_REL_L2, None, "final_state")
    assert float(d["out"][0, 9].abs().max()) == 0.0
