"""Single-token decode step against the fp64 oracle (the sequential recurrence with T = 1), and the
prefill -> decode hand-off through final_state."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_14568_b200 as gdn
from workloads import get_config, make_inputs, widen

from gdn_testlib import BF16_MAX_ABS, BF16_REL_L2, assert_close, f64, to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,H,dk,dv", [(1, 1, 128, 128), (3, 4, 128, 256), (5, 2, 64, 128), (64, 16, 128, 128)])
def test_decode_step_matches_oracle(B, H, dk, dv):
    cfg = get_config("long", B=B, T=1, H=H, d_k=dk, d_v=dv, init_std=0.5, seed=80 + B)
    x = make_inputs(cfg)
    d = to_device(x)
    state = d["initial_state"].clone()
    out = torch.empty((B, H, dv), dtype=torch.bfloat16, device="cuda")
    gdn.gdn_decode_step(d["q"][:, 0].contiguous(), d["k"][:, 0].contiguous(), d["v"][:, 0].contiguous(),
                        d["log_alpha"][:, 0].contiguous(), d["beta"][:, 0].contiguous(), state, out)
    torch.cuda.synchronize()
    o_ref, s_ref = oracle.sequential(widen(x.q), widen(x.k), widen(x.v), x.log_alpha, x.beta, x.initial_state)
    assert_close(f64(out), o_ref[:, 0], BF16_REL_L2, BF16_MAX_ABS, "decode out")   # one bf16 rounding of the output
    assert_close(f64(state), s_ref, 1e-5, None, "decode state")                    # fp32 arithmetic on the state


def test_prefill_then_decode_equals_longer_prefill():
    cfg = get_config("long", B=2, T=131, H=2, seed=91)
    x = make_inputs(cfg)
    d = to_device(x)
    T = cfg.T
    pre = {k: (v[:, :T - 3].contiguous() if k in ("q", "k", "v", "log_alpha", "beta") else v) for k, v in d.items()}
    pre["out"] = torch.empty_like(pre["v"])
    gdn.gdn_chunk_prefill(pre["q"], pre["k"], pre["v"], pre["log_alpha"], pre["beta"], pre["initial_state"],
                          pre["out"], pre["final_state"])
    state = pre["final_state"]
    outs = [pre["out"]]
    for t in range(T - 3, T):                       # three decode steps continue the prefill's state
        o = torch.empty((2, 2, 128), dtype=torch.bfloat16, device="cuda")
        gdn.gdn_decode_step(d["q"][:, t].contiguous(), d["k"][:, t].contiguous(), d["v"][:, t].contiguous(),
                            d["log_alpha"][:, t].contiguous(), d["beta"][:, t].contiguous(), state, o)
        outs.append(o[:, None])
    torch.cuda.synchronize()
    o_ref, s_ref = oracle.sequential(widen(x.q), widen(x.k), widen(x.v), x.log_alpha, x.beta, x.initial_state)
    assert_close(f64(torch.cat(outs, 1)), o_ref, BF16_REL_L2, BF16_MAX_ABS, "prefill+decode out")
    assert_close(f64(state), s_ref, BF16_REL_L2, BF16_MAX_ABS, "prefill+decode state")


def test_decode_error_codes():
    L = gdn.lib()
    t = torch.zeros(1 << 16, dtype=torch.float32, device="cuda")
    p = t.data_ptr()
    assert L.gdn_decode_step(None, p, p, p, p, p, p, 1, 1, 128, 128, None) == 1
    assert L.gdn_decode_step(p, p, p, p, p, p, p, 0, 1, 128, 128, None) == 1
    assert L.gdn_decode_step(p, p, p, p, p, p, p, 1, 1, 100, 128, None) == 2
    assert L.gdn_decode_step(p, p + 2, p, p, p, p, p, 1, 1, 128, 128, None) == 2
