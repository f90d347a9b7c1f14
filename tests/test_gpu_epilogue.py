"""Prefill with the output stage fused in (gated root-mean-square norm of every output row, inside the
kernel that produces the row; Section "Prefill projections: dequantize, then call the vendor" names the
norms and gating around the scan) against the fp64 oracle: the token-by-token recurrence followed by
oracle.epilogue."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2607_14568_b200 as gdn
from workloads import epilogue_inputs, get_config, make_inputs, widen
from gdn_testlib import BF16_MAX_ABS, BF16_REL_L2, assert_close, f64, to_device

pytestmark = pytest.mark.gpu


def _bf16_tensor(bits):
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()


def _run(x, d, e, eps, nseg=0, merged=0):
    cfg = x.cfg
    packed = d["cu_seqlens"] is not None
    ws = torch.empty(max(gdn.gdn_workspace_bytes(len(x.lengths), x.T_arg, cfg.H, cfg.d_k, cfg.d_v, packed), 4096),
                     dtype=torch.uint8, device="cuda")
    gdn.gdn_set_workspace(ws)
    gdn.lib().gdn_debug_force_segments(nseg)
    gdn.lib().gdn_debug_set_scan(merged)
    try:
        gdn.gdn_chunk_prefill_gated(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["initial_state"],
                                    _bf16_tensor(e["z"]), torch.from_numpy(e["weight"]).cuda(), eps, d["out"],
                                    d["final_state"], d["cu_seqlens"])
        assert gdn.gdn_query_status_stream() == 0
    finally:
        gdn.lib().gdn_debug_force_segments(0)
        gdn.lib().gdn_debug_set_scan(0)
        gdn.gdn_set_workspace(None)


def _oracle(x, e, eps):
    o, fin = oracle.sequential(widen(x.q), widen(x.k), widen(x.v), x.log_alpha, x.beta, x.initial_state, x.cu_seqlens)
    return o, oracle.epilogue(o, widen(e["z"]), e["weight"], eps), fin


@pytest.mark.parametrize("kw,eps,nseg,merged", [
    (dict(B=2, T=64 * 5 + 23, H=2, init_std=0.3), 1e-6, 0, 0),                 # batched, ragged tail
    (dict(B=1, T=64 * 20, H=2, init_std=0.1), 1e-5, 4, 0),                     # sequence split, three kernels
    (dict(B=1, T=64 * 20 + 5, H=2, init_std=0.1), 1e-5, 4, 1),                 # split, merged launch asked for: the
                                                                               # output stage keeps the three kernels
    (dict(B=3, T=0, H=2, init_std=0.2, lengths=(130, 64, 7)), 0.0, 0, 0),      # packed, ragged tails
    (dict(B=1, T=64 * 3, H=3, init_std=0.0), 0.5, 0, 0),                       # eps that matters
])
def test_gated_prefill_matches_oracle(kw, eps, nseg, merged):
    cfg = get_config("short", **kw)
    x = make_inputs(cfg)
    d = to_device(x)
    e = epilogue_inputs(cfg, x.q.shape[:-2])
    _run(x, d, e, eps, nseg, merged)
    o_plain, want, want_fin = _oracle(x, e, eps)
    # the norm and the gate rescale every row: the absolute bar scales with the values they produce
    scale = max(1.0, float(np.abs(want).max() / max(np.abs(o_plain).max(), 1e-30)))
    assert_close(f64(d["out"]), want, BF16_REL_L2, BF16_MAX_ABS * scale, "gated out")
    assert_close(f64(d["final_state"]), want_fin, BF16_REL_L2, BF16_MAX_ABS, "final_state")


def test_gated_prefill_rejects_what_it_does_not_support():
    cfg = get_config("short", B=1, T=128, H=1, d_v=256)
    x = make_inputs(cfg)
    d = to_device(x)
    e = epilogue_inputs(cfg, x.q.shape[:-2])
    z, w = _bf16_tensor(e["z"]), torch.from_numpy(e["weight"]).cuda()
    n0 = gdn.gdn_launch_count()
    with pytest.raises(gdn.GdnError) as err:                                   # the norm spans two value blocks
        gdn.gdn_chunk_prefill_gated(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], None, z, w, 1e-6, d["out"], None)
    assert err.value.status == 2
    cfg = get_config("short", B=1, T=128, H=1)
    x = make_inputs(cfg)
    d = to_device(x)
    e = epilogue_inputs(cfg, x.q.shape[:-2])
    z, w = _bf16_tensor(e["z"]), torch.from_numpy(e["weight"]).cuda()
    gdn.gdn_set_workspace(None)
    with pytest.raises(gdn.GdnError) as err:                                   # no scratch
        gdn.gdn_chunk_prefill_gated(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], None, z, w, 1e-6, d["out"], None)
    assert err.value.status == 3
    with pytest.raises(gdn.GdnError) as err:                                   # negative eps
        gdn.gdn_chunk_prefill_gated(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], None, z, w, -1.0, d["out"], None)
    assert err.value.status == 1
    assert gdn.gdn_launch_count() == n0
