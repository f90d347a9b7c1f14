"""Calls of different shapes and paths follow one another on one stream without a host synchronisation in
between, sharing one workspace: the item ticket, the workspace header and the split plan of every call must
leave nothing behind for the next.  Every call is checked bit for bit against the same call made alone first
(same kernels, same launch configuration: the arithmetic order is fixed), and one of them against the oracle."""
import numpy as np
import pytest
import torch

from workloads import get_config, make_inputs
from gdn_testlib import (BF16_MAX_ABS, BF16_REL_L2, assert_close, f64, run_oracle, to_device)

pytestmark = pytest.mark.gpu

CASES = [
    dict(name="short", B=1, T=64 * 40, H=16),                    # split by the planner (few chains, many chunks)
    dict(name="short", B=2, T=64 * 5 + 17, H=3),                 # no split, ragged last chunk
    dict(name="large", B=1, T=64 * 9, H=2),                      # d_v = 256: two CTAs per chain
    dict(name="serving", B=3, H=4, varlen=(1, 700), seed=11),    # packed, lengths from 1 token up
    dict(name="short", B=1, T=64 * 24 + 5, H=8, init_std=0.3),   # split, ragged last chunk, initial state
]


def _call(gdn, d):
    gdn.gdn_chunk_prefill(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["initial_state"], d["out"],
                          d["final_state"], d["cu_seqlens"])


def test_back_to_back_calls_share_one_workspace():
    import paper_2607_14568_b200 as gdn
    xs = [make_inputs(get_config(**c)) for c in CASES]
    ds = [to_device(x) for x in xs]
    need = 0
    for x in xs:
        cfg, packed = x.cfg, x.cu_seqlens is not None
        T = int(sum(x.lengths)) if packed else cfg.T
        need = max(need, gdn.gdn_workspace_bytes(len(x.lengths), T, cfg.H, cfg.d_k, cfg.d_v, packed))
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    gdn.gdn_set_workspace(ws)
    try:
        want = []
        for d in ds:                                           # every call alone first
            _call(gdn, d)
            torch.cuda.synchronize()
            assert gdn.gdn_query_status() == 0
            want.append((d["out"].clone(), d["final_state"].clone()))
        got_ref = run_oracle(xs[4])
        assert_close(f64(want[4][0]), got_ref[0], BF16_REL_L2, BF16_MAX_ABS, "split, ragged: out")
        assert_close(f64(want[4][1]), got_ref[1], BF16_REL_L2, BF16_MAX_ABS, "split, ragged: state")
        rng = np.random.default_rng(5)
        for rnd in range(6):
            order = rng.permutation(len(ds))
            for i in order:
                ds[i]["out"].zero_(); ds[i]["final_state"].zero_()
            for i in order:                                    # no synchronisation between the calls
                _call(gdn, ds[i])
            torch.cuda.synchronize()
            assert gdn.gdn_query_status() == 0
            for i in order:
                assert torch.equal(ds[i]["out"], want[i][0]), f"round {rnd}, case {i}: out differs"
                assert torch.equal(ds[i]["final_state"], want[i][1]), f"round {rnd}, case {i}: state differs"
    finally:
        gdn.gdn_set_workspace(None)
