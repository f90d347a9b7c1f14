"""The prefill call records into a CUDA graph: it is asynchronous on its stream, makes no host-device
copies and allocates nothing, so a captured call replays on new contents of the same buffers.  The
replays must reproduce the eager results bit for bit (same kernels, same launch configuration)."""
import pytest
import torch

from workloads import get_config, make_inputs
from gdn_testlib import to_device

pytestmark = pytest.mark.gpu


# plain two-kernel path, sequence split as three kernels, sequence split as one merged launch
@pytest.mark.parametrize("T,nseg,merged", [(64 * 6 + 11, 0, 0), (64 * 20, 4, 0), (64 * 20, 4, 1)])
def test_captured_call_replays(T, nseg, merged):
    import paper_2607_14568_b200 as gdn
    cfg = get_config("short", B=1, T=T, H=2, init_std=0.2)
    d = to_device(make_inputs(cfg))
    ws = torch.empty(gdn.gdn_workspace_bytes(1, T, 2, cfg.d_k, cfg.d_v, False), dtype=torch.uint8, device="cuda")
    gdn.gdn_set_workspace(ws)
    gdn.lib().gdn_debug_force_segments(nseg)
    gdn.lib().gdn_debug_set_scan(merged)
    try:
        def call():
            gdn.gdn_chunk_prefill(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["initial_state"], d["out"],
                                  d["final_state"])
        call()                                             # eager: reference result, one-time set-up done
        torch.cuda.synchronize()
        want_out, want_fin = d["out"].clone(), d["final_state"].clone()
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                call()
        torch.cuda.synchronize()
        d["out"].zero_(); d["final_state"].zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert gdn.gdn_query_status() == 0
        assert torch.equal(d["out"], want_out) and torch.equal(d["final_state"], want_fin)
        # new contents in the same buffers: the replay follows them
        d2 = to_device(make_inputs(get_config("short", B=1, T=T, H=2, init_std=0.2, seed=77)))
        for name in ("q", "k", "v", "log_alpha", "beta", "initial_state"):
            d[name].copy_(d2[name])
        graph.replay()
        torch.cuda.synchronize()
        got_out, got_fin = d["out"].clone(), d["final_state"].clone()
        call()
        torch.cuda.synchronize()
        assert torch.equal(got_out, d["out"]) and torch.equal(got_fin, d["final_state"])
        assert not torch.equal(got_out, want_out)
    finally:
        gdn.lib().gdn_debug_force_segments(0)
        gdn.lib().gdn_debug_set_scan(0)
        gdn.gdn_set_workspace(None)
