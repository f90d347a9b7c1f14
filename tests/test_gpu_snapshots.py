"""State snapshots at chunk boundaries (the material of a position-indexed prefix-snapshot cache,
Section "An All-GPU Engine for the Hybrid Backbone") against the fp64 oracle: snapshot i must equal
the oracle's final state of the prefix that ends at token (i + 1) * every * 64, and resuming the
prefill from a snapshot must reproduce the tail of the full run."""
import numpy as np
import pytest
import torch

import oracle
from workloads import get_config, make_inputs, widen
from gdn_testlib import BF16_MAX_ABS, BF16_REL_L2, assert_close, f64, to_device

pytestmark = pytest.mark.gpu


def _oracle_prefix_state(x, tokens):
    """Final state of the oracle run on the first `tokens` tokens of every sequence."""
    _, fin = oracle.sequential(widen(x.q[:, :tokens]), widen(x.k[:, :tokens]), widen(x.v[:, :tokens]),
                               x.log_alpha[:, :tokens], x.beta[:, :tokens], x.initial_state, None)
    return fin


def _run(gdn, d, every, nseg=0):
    B, T, H, d_k = d["q"].shape
    d_v = d["v"].shape[-1]
    n_snap = (T // 64) // every
    snaps = torch.full((B, n_snap, H, d_k, d_v), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(max(gdn.gdn_workspace_bytes(B, T, H, d_k, d_v, False), 256), dtype=torch.uint8, device="cuda")
    gdn.gdn_set_workspace(ws)
    gdn.lib().gdn_debug_force_segments(nseg)
    try:
        gdn.gdn_chunk_prefill_snapshots(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["initial_state"],
                                        d["out"], d["final_state"], every, snaps)
        torch.cuda.synchronize()
        assert gdn.gdn_query_status() == 0
    finally:
        gdn.lib().gdn_debug_force_segments(0)
        gdn.gdn_set_workspace(None)
    return snaps


@pytest.mark.parametrize("T,every,nseg", [(64 * 7 + 19, 2, 0), (64 * 8, 1, 0), (64 * 24, 3, 4), (40, 1, 0)])
def test_snapshots_match_oracle_prefix_states(T, every, nseg):
    import paper_2607_14568_b200 as gdn
    cfg = get_config("short", B=2, T=T, H=2, init_std=0.3)
    x = make_inputs(cfg)
    d = to_device(x)
    snaps = _run(gdn, d, every, nseg)
    n_snap = (T // 64) // every
    assert snaps.shape[1] == n_snap
    want_out, want_fin = oracle.sequential(widen(x.q), widen(x.k), widen(x.v), x.log_alpha, x.beta,
                                           x.initial_state, None)
    assert_close(f64(d["out"]), want_out, BF16_REL_L2, BF16_MAX_ABS, "out")
    assert_close(f64(d["final_state"]), want_fin, BF16_REL_L2, None, "final_state")
    got = f64(snaps)
    for i in range(n_snap):
        want = _oracle_prefix_state(x, (i + 1) * every * 64)
        assert_close(got[:, i], want, BF16_REL_L2, None, f"snapshot {i}")


def test_resume_from_snapshot_reproduces_the_tail():
    import paper_2607_14568_b200 as gdn
    from gdn_testlib import prefill_two_kernel
    T, every = 64 * 6 + 5, 2
    cfg = get_config("short", B=1, T=T, H=2, init_std=0.3)
    x = make_inputs(cfg)
    d = to_device(x)
    snaps = _run(gdn, d, every)
    cut = 2 * every * 64                     # snapshot 1 = state after `cut` tokens
    s0 = snaps[:, 1].contiguous()
    tail = {k: d[k][:, cut:].contiguous() for k in ("q", "k", "v", "log_alpha", "beta")}
    out2 = torch.empty_like(tail["v"])
    fin2 = torch.empty_like(d["final_state"])
    prefill_two_kernel(tail["q"], tail["k"], tail["v"], tail["log_alpha"], tail["beta"], s0, out2, fin2)
    torch.cuda.synchronize()
    # same arithmetic on the same chunk grid from the same fp32 state: bit-identical
    assert torch.equal(out2, d["out"][:, cut:])
    assert torch.equal(fin2, d["final_state"])


def test_snapshots_need_a_workspace():
    import paper_2607_14568_b200 as gdn
    cfg = get_config("short", B=1, T=128, H=1)
    d = to_device(make_inputs(cfg))
    snaps = torch.empty((1, 2, 1, cfg.d_k, cfg.d_v), dtype=torch.float32, device="cuda")
    gdn.gdn_set_workspace(None)
    with pytest.raises(gdn.GdnError) as e:
        gdn.gdn_chunk_prefill_snapshots(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["initial_state"],
                                        d["out"], d["final_state"], 1, snaps)
    assert e.value.status == 3   # GDN_ERR_WORKSPACE
