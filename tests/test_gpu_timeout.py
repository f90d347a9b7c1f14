"""Failure detection without a GPU fault: a TMA load that never happens makes the bounded waits of
one CTA expire (about a second each); the kernel must come back by itself with GDN_ERR_TIMEOUT in
the status word, leave the context usable, and the next call must be correct."""
import pytest
import torch

import paper_2607_14568_b200 as gdn
from workloads import get_config, make_inputs

from gdn_testlib import BF16_MAX_ABS, BF16_REL_L2, assert_close, f64, prefill_two_kernel, run_oracle, to_device

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_the_context_survives():
    cfg = get_config("long", T=320, H=2, seed=95)
    x = make_inputs(cfg)
    d = to_device(x)
    L = gdn.lib()
    nbytes = gdn.gdn_workspace_bytes(cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, False)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    gdn.gdn_set_workspace(ws)
    L.gdn_debug_force_path(2)
    L.gdn_debug_force_segments(1)
    L.gdn_debug_drop_chunk(2)                        # chunk 2 of CTA (0,0,0) is never loaded
    try:
        gdn.gdn_chunk_prefill(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["initial_state"], d["out"],
                              d["final_state"])
        assert gdn.gdn_query_status() == 5           # GDN_ERR_TIMEOUT; the kernel returned on its own
    finally:
        L.gdn_debug_drop_chunk(-1)
        L.gdn_debug_force_segments(0)
        L.gdn_debug_force_path(0)
        gdn.gdn_set_workspace(None)
    assert L.gdn_debug_reset_status() == 0
    torch.cuda.synchronize()                         # no sticky CUDA error
    # the context is intact: the same problem now runs correctly
    o_ref, f_ref = run_oracle(x)
    out, fin = prefill_two_kernel(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["initial_state"], d["out"],
                                  d["final_state"])
    assert_close(f64(out), o_ref, BF16_REL_L2, BF16_MAX_ABS, "out after a timed-out call")
    assert_close(f64(fin), f_ref, BF16_REL_L2, BF16_MAX_ABS, "state after a timed-out call")


def test_expired_counter_wait_in_the_merged_kernel_is_reported_and_the_context_survives():
    """The merged scan kernel hands over between its phases through counters in global memory.  A test hook
    makes one CTA not raise its counter; the CTAs of that head that wait for it must give up after about a
    second, report GDN_ERR_TIMEOUT, run to their end, and leave the counters clean for the next call."""
    cfg = get_config("long", T=64 * 12, H=2, seed=96)
    x = make_inputs(cfg)
    d = to_device(x)
    L = gdn.lib()
    ws = torch.empty(gdn.gdn_workspace_bytes(cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, False), dtype=torch.uint8, device="cuda")
    gdn.gdn_set_workspace(ws)
    L.gdn_debug_force_path(2)
    L.gdn_debug_force_segments(3)
    L.gdn_debug_set_scan(1)
    L.gdn_debug_drop_chunk(-2)                       # CTA (0,0,0) keeps its segment summary to itself
    try:
        gdn.gdn_chunk_prefill(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["initial_state"], d["out"],
                              d["final_state"])
        assert gdn.gdn_query_status() == 5
        L.gdn_debug_drop_chunk(-1)
        assert L.gdn_debug_reset_status() == 0
        torch.cuda.synchronize()
        # same workspace, same counters: the next merged call is correct
        gdn.gdn_chunk_prefill(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["initial_state"], d["out"],
                              d["final_state"])
        assert gdn.gdn_query_status() == 0
    finally:
        L.gdn_debug_drop_chunk(-1)
        L.gdn_debug_force_segments(0)
        L.gdn_debug_set_scan(0)
        L.gdn_debug_force_path(0)
        gdn.gdn_set_workspace(None)
    o_ref, f_ref = run_oracle(x)
    assert_close(f64(d["out"]), o_ref, BF16_REL_L2, BF16_MAX_ABS, "out after a timed-out merged call")
    assert_close(f64(d["final_state"]), f_ref, BF16_REL_L2, BF16_MAX_ABS, "state after a timed-out merged call")
