"""GPU parity: the CUDA library, called through its C ABI, against the fp64 oracle on
the same seeded inputs, element by element."""
import numpy as np
import pytest
import torch

import paper_2607_14568_b200 as gdn
from workloads import bf16_bits_to_f32, f32_to_bf16_bits, get_config, make_inputs, widen

import oracle
from gdn_testlib import (BF16_MAX_ABS, BF16_REL_L2, F32_REL_L2, assert_close, f64, prefill_fused,
                         prefill_two_kernel, run_lib, run_oracle, to_device)

pytestmark = pytest.mark.gpu

# "fused": one kernel per call (no scratch); "two_kernel": prepare kernel + chain kernel (scratch);
# "simt": the fp32-arithmetic kernel with bf16 storage.
BF16_FNS = {"fused": prefill_fused, "two_kernel": prefill_two_kernel, "simt": gdn.gdn_chunk_prefill_bf16_simt}


def check_bf16(x, fn, what):
    d = to_device(x)
    out, fin = run_lib(fn, d)
    o_ref, f_ref = run_oracle(x)
    r1 = assert_close(f64(out), o_ref, BF16_REL_L2, BF16_MAX_ABS, what + " out")
    r2 = assert_close(f64(fin), f_ref, BF16_REL_L2, BF16_MAX_ABS, what + " final_state")
    return r1, r2


# ---- configuration 1: fp32 path, whole tensor ------------------------------------------------
def test_tiny_f32():
    x = make_inputs(get_config("tiny"))
    d = to_device(x)
    out, fin = run_lib(gdn.gdn_chunk_prefill_f32, d)
    o_ref, f_ref = run_oracle(x)
    assert_close(f64(out), o_ref, F32_REL_L2, None, "tiny out")
    assert_close(f64(fin), f_ref, F32_REL_L2, None, "tiny final_state")


@pytest.mark.parametrize("T,H,dk,dv", [(1, 1, 32, 32), (63, 2, 64, 96), (65, 1, 128, 32), (200, 3, 96, 64),
                                       (333, 2, 128, 128)])
def test_f32_ragged_shapes(T, H, dk, dv):
    cfg = get_config("tiny", T=T, H=H, d_k=dk, d_v=dv, init_std=0.5, seed=100 + T)
    x = make_inputs(cfg)
    d = to_device(x)
    out, fin = run_lib(gdn.gdn_chunk_prefill_f32, d)
    o_ref, f_ref = run_oracle(x)
    assert_close(f64(out), o_ref, F32_REL_L2, None, "out")
    assert_close(f64(fin), f_ref, F32_REL_L2, None, "final_state")


def test_f32_packed_with_empty_sequence_and_aliasing():
    cfg = get_config("tiny", B=4, H=2, d_k=64, d_v=64, lengths=(70, 0, 129, 64), init_std=0.3, seed=7)
    x = make_inputs(cfg)
    d = to_device(x)
    s0 = d["initial_state"].clone()
    d["final_state"] = d["initial_state"]            # in-place state update is allowed
    out, fin = run_lib(gdn.gdn_chunk_prefill_f32, d)
    o_ref, f_ref = run_oracle(x)
    assert_close(f64(out), o_ref, F32_REL_L2, None, "out")
    assert_close(f64(fin), f_ref, F32_REL_L2, None, "final_state")
    assert torch.equal(fin[1], s0[1])                 # the empty sequence passes its state through


def test_f32_null_states_and_split_invariance():
    cfg = get_config("tiny", T=300, H=2, seed=11)
    x = make_inputs(cfg)
    d = to_device(x)
    d["final_state"] = None
    out_a, _ = run_lib(gdn.gdn_chunk_prefill_f32, d)
    o_ref, _ = run_oracle(x)
    assert_close(f64(out_a), o_ref, F32_REL_L2, None, "out without states")
    # prefix / suffix with the state handed over == one call
    T1 = 130
    parts = []
    state = None
    for sl in (slice(0, T1), slice(T1, 300)):
        dd = {k: (v[:, sl].contiguous() if k in ("q", "k", "v", "log_alpha", "beta") else None)
              for k, v in d.items() if k in ("q", "k", "v", "log_alpha", "beta")}
        dd.update(initial_state=state, cu_seqlens=None, out=torch.empty_like(dd["v"]),
                  final_state=torch.empty((1, 2, 64, 64), device="cuda"))
        o, state = run_lib(gdn.gdn_chunk_prefill_f32, dd)
        parts.append(o)
    assert_close(f64(torch.cat(parts, 1)), o_ref, F32_REL_L2, None, "split out")


# ---- bf16 storage, reduced shapes that still span several tiles and a ragged tail ---------------
@pytest.mark.parametrize("impl", ["fused", "two_kernel", "simt"])
@pytest.mark.parametrize("T,H,dv,init", [(64, 1, 128, 0.0), (200, 2, 128, 0.02), (1000, 2, 128, 0.02),
                                         (130, 2, 256, 0.0), (1, 1, 128, 0.02)])
def test_bf16_reduced(impl, T, H, dv, init):
    cfg = get_config("long", T=T, H=H, d_v=dv, init_std=init, seed=20 + T)
    check_bf16(make_inputs(cfg), BF16_FNS[impl], f"{impl} T={T}")


@pytest.mark.parametrize("impl", ["fused", "two_kernel", "simt"])
def test_bf16_packed_ragged(impl):
    cfg = get_config("serving", B=5, H=2, lengths=(257, 64, 0, 1, 700), seed=31)
    x = make_inputs(cfg)
    (r, _), _ = check_bf16(x, BF16_FNS[impl], impl + " packed")
    # each sequence alone gives the same rows
    d = to_device(x)
    out, fin = run_lib(BF16_FNS[impl], d)
    cu = x.cu_seqlens
    for n in (0, 4):
        a, b = int(cu[n]), int(cu[n + 1])
        dd = dict(q=d["q"][None, a:b].contiguous(), k=d["k"][None, a:b].contiguous(),
                  v=d["v"][None, a:b].contiguous(), log_alpha=d["log_alpha"][None, a:b].contiguous(),
                  beta=d["beta"][None, a:b].contiguous(), initial_state=d["initial_state"][n:n + 1].contiguous(),
                  cu_seqlens=None)
        dd["out"] = torch.empty_like(dd["v"])
        dd["final_state"] = torch.empty_like(dd["initial_state"])
        o1, f1 = run_lib(BF16_FNS[impl], dd)
        assert torch.equal(o1[0], out[a:b]) and torch.equal(f1[0], fin[n])


@pytest.mark.parametrize("merged", [1, 0])
@pytest.mark.parametrize("T,nseg,gate", [(640, 2, 0.05), (1000, 3, 0.05), (2048, 5, 0.001), (4096, 16, 0.0),
                                         (333, 4, 0.02), (3000, 9, 0.0)])
def test_two_kernel_sequence_split(T, nseg, gate, merged):
    """The sequence split (segment summaries M, N; their combination; per-segment chains) against the
    oracle, including weak or no decay, where a segment's outgoing state depends fully on its
    incoming one.  merged = 1: the three phases in one launch (CTAs hand over through counters in global
    memory); merged = 0: three kernels."""
    cfg = get_config("long", T=T, H=2, gate_scale=gate, seed=60 + nseg)
    x = make_inputs(cfg)
    gdn.lib().gdn_debug_force_segments(nseg)
    gdn.lib().gdn_debug_set_scan(merged)
    try:
        check_bf16(x, prefill_two_kernel, f"split T={T} nseg={nseg} merged={merged}")
        check_bf16(x, prefill_two_kernel, f"split T={T} nseg={nseg} merged={merged}, second call")   # counters were left clean
    finally:
        gdn.lib().gdn_debug_force_segments(0)
        gdn.lib().gdn_debug_set_scan(0)


def test_two_kernel_sequence_split_wide_values_and_batch():
    """Sequence split with d_v = 256 (two value blocks share one M chain) and B = 2."""
    cfg = get_config("large", B=2, T=1100, H=2, seed=77)
    x = make_inputs(cfg)
    gdn.lib().gdn_debug_force_segments(3)
    try:
        check_bf16(x, prefill_two_kernel, "split d_v=256 B=2")
    finally:
        gdn.lib().gdn_debug_force_segments(0)


def test_bf16_special_cases():
    """beta = 0 gives pure decay of the initial state; identity padding changes nothing."""
    cfg = get_config("long", T=192, H=2, seed=41)
    x = make_inputs(cfg)
    x.beta[:] = 0.0
    d = to_device(x)
    out, fin = run_lib(gdn.gdn_chunk_prefill, d)
    G = np.exp(np.cumsum(x.log_alpha.astype(np.float64), axis=1))
    want = G[..., None] * np.einsum("bhmj,bthm->bthj", x.initial_state.astype(np.float64), widen(x.q))
    assert_close(f64(out), want, BF16_REL_L2, BF16_MAX_ABS, "pure decay out")
    assert_close(f64(fin), G[:, -1][..., None, None] * x.initial_state, BF16_REL_L2, BF16_MAX_ABS, "pure decay state")


def test_deterministic():
    x = make_inputs(get_config("short", T=640, H=4))
    d = to_device(x)
    o1, f1 = run_lib(gdn.gdn_chunk_prefill, d)
    o1, f1 = o1.clone(), f1.clone()
    o2, f2 = run_lib(gdn.gdn_chunk_prefill, d)
    assert torch.equal(o1, o2) and torch.equal(f1, f2)


# ---- the benchmark configurations at full size ----------------------------------------------------
@pytest.mark.parametrize("impl", ["fused", "two_kernel"])
@pytest.mark.parametrize("name", ["short", "long", "serving"])
def test_bf16_full_configs(name, impl):
    x = make_inputs(get_config(name))
    (ro, mo), (rs, ms) = check_bf16(x, BF16_FNS[impl], f"{name}/{impl}")
    print(f"\n{name}/{impl}: out rel-L2 {ro:.2e} max-abs {mo:.2e}; state rel-L2 {rs:.2e} max-abs {ms:.2e}")


_LARGE_ORACLE = {}


def _large_oracle(cfg, x):
    """fp64 recurrence over every (sequence, head) chain of `large`, 16 heads of one sequence at a time
    (the oracle runs one chain per host thread); computed once per test session."""
    if not _LARGE_ORACLE:
        for n in range(cfg.B):
            for h0 in range(0, cfg.H, 16):
                hs = slice(h0, min(cfg.H, h0 + 16))
                o_ref, f_ref = oracle.sequential(widen(x.q[n:n + 1, :, hs]), widen(x.k[n:n + 1, :, hs]),
                                                 widen(x.v[n:n + 1, :, hs]), x.log_alpha[n:n + 1, :, hs],
                                                 x.beta[n:n + 1, :, hs], None)
                _LARGE_ORACLE[(n, h0)] = (o_ref[0].astype(np.float32), f_ref[0])
    return _LARGE_ORACLE


@pytest.mark.parametrize("impl", ["fused", "two_kernel"])
def test_bf16_large_all_chains(impl):
    """Configuration 'large' (B=4, T=32768, H=32, d_v=256) at full size: every one of the 128 (sequence, head)
    chains is compared with the fp64 recurrence, outputs and final state (the reference outputs are kept in
    fp32, eight decimal digits, far below the bf16 tolerances)."""
    cfg = get_config("large")
    x = make_inputs(cfg, threads=16)
    d = to_device(x)
    out, fin = run_lib(BF16_FNS[impl], d)
    assert bool(torch.isfinite(out).all()) and bool(torch.isfinite(fin).all())
    ref = _large_oracle(cfg, x)
    worst = 0.0
    for (n, h0), (o_ref, f_ref) in sorted(ref.items()):
        hs = slice(h0, h0 + o_ref.shape[1])
        r, _ = assert_close(f64(out[n, :, hs]), o_ref.astype(np.float64), BF16_REL_L2, BF16_MAX_ABS,
                            f"large seq {n} heads {h0}.. out")
        assert_close(f64(fin[n, hs]), f_ref, BF16_REL_L2, BF16_MAX_ABS, f"large seq {n} heads {h0}.. state")
        worst = max(worst, r)
    print(f"\nlarge/{impl}: worst out rel-L2 over head groups {worst:.2e}")


# ---- final_state written over initial_state ------------------------------------------------------------
@pytest.mark.parametrize("impl,nseg,H,merged", [("fused", 0, 4, 0), ("two_kernel", 0, 4, 0), ("two_kernel", 3, 64, 0),
                                                ("two_kernel", 16, 16, 0), ("two_kernel", 9, 16, 1)])
def test_bf16_final_state_may_alias_initial_state(impl, nseg, H, merged):
    """The header allows final_state == initial_state.  With the sequence split the grid of the last kernel
    (H * nseg CTAs: 192 and 256 in two of the cases) does not fit the GPU in one wave, so a segment-0 CTA may well
    start after a last-segment CTA has finished; 16 heads x 9 segments run as the merged single launch.  The result
    must still be the recurrence from the given initial state."""
    cfg = get_config("long", T=1088, H=H, init_std=0.5, seed=90 + nseg)
    x = make_inputs(cfg)
    d = to_device(x)
    d["final_state"] = d["initial_state"]
    gdn.lib().gdn_debug_force_segments(nseg)
    gdn.lib().gdn_debug_set_scan(merged)
    try:
        out, fin = run_lib(BF16_FNS[impl], d)
    finally:
        gdn.lib().gdn_debug_force_segments(0)
        gdn.lib().gdn_debug_set_scan(0)
    o_ref, f_ref = run_oracle(x)
    assert_close(f64(out), o_ref, BF16_REL_L2, BF16_MAX_ABS, "aliased out")
    assert_close(f64(fin), f_ref, BF16_REL_L2, BF16_MAX_ABS, "aliased final_state")


# ---- inputs outside the usual ranges: computed as given, no clamping -----------------------------------------
@pytest.mark.parametrize("impl", ["fused", "two_kernel", "simt"])
@pytest.mark.parametrize("case", ["beta_0_1_1p5", "growing_gates", "key_norm_half", "key_norm_1p5"])
def test_bf16_unclamped_inputs(impl, case):
    """beta outside (0, 1), a few positive log gates, keys that are not unit vectors: the library applies no
    clamp and no check, so the result is still the recurrence on the values given.  Keys of norm 1.5 with
    beta near 1 make I - beta k k^T expansive (|1 - 2.25 beta| > 1); the inputs are sized so that fp64 itself
    stays bounded, and the bf16 path must stay within its usual tolerance of it."""
    cfg = get_config("long", T=300, H=2, init_std=0.02, seed=95)
    x = make_inputs(cfg)
    rng = np.random.default_rng(96)
    if case == "beta_0_1_1p5":
        x.beta[...] = rng.choice(np.array([0.0, 1.0, 1.5], dtype=np.float32), size=x.beta.shape, p=[0.3, 0.5, 0.2])
    elif case == "growing_gates":
        idx = rng.random(x.log_alpha.shape) < 0.05
        x.log_alpha[idx] = 0.03                                   # alpha > 1 on one token in twenty
    else:
        s = 0.5 if case == "key_norm_half" else 1.5
        x.k[...] = f32_to_bf16_bits(bf16_bits_to_f32(x.k) * np.float32(s))
        if s > 1:
            x.beta[...] *= 0.4                                    # keeps |1 - beta |k|^2| below one
    check_bf16(x, BF16_FNS[impl], f"{impl} {case}")


# ---- host-buffer entry point ------------------------------------------------------------------------
def test_host_entry_matches_device_entry():
    cfg = get_config("serving", B=3, H=2, lengths=(300, 64, 77), seed=51)
    x = make_inputs(cfg)
    d = to_device(x)
    out, fin = run_lib(gdn.gdn_chunk_prefill, d)
    h = to_device(x, device="cpu")
    h = {k: (v.pin_memory() if v is not None else None) for k, v in h.items()}
    nbytes = gdn.gdn_host_staging_bytes(cfg.B, x.T_arg, cfg.H, cfg.d_k, cfg.d_v)
    staging = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    o2, f2 = gdn.gdn_chunk_prefill_host(h["q"], h["k"], h["v"], h["log_alpha"], h["beta"], h["initial_state"],
                                        h["out"], h["final_state"], h["cu_seqlens"], staging)
    torch.cuda.synchronize()
    o_ref, f_ref = run_oracle(x)
    assert_close(f64(o2), o_ref, BF16_REL_L2, BF16_MAX_ABS, "host entry out vs oracle")
    assert_close(f64(f2), f_ref, BF16_REL_L2, BF16_MAX_ABS, "host entry final_state vs oracle")
    assert torch.equal(o2, out.cpu()) and torch.equal(f2, fin.cpu())      # and bit for bit the device entry point
    with pytest.raises(gdn.GdnError) as e:
        gdn.gdn_chunk_prefill_host(h["q"], h["k"], h["v"], h["log_alpha"], h["beta"], h["initial_state"],
                                   h["out"], h["final_state"], h["cu_seqlens"], staging[:1024])
    assert e.value.status == 3


@pytest.mark.parametrize("with_ws", [False, True])
def test_host_entry_long_sequence_is_pipelined_in_pieces(with_ws):
    """One long sequence goes through the host entry point in pieces of 2048 tokens with the state carried
    between them; the result must still be the recurrence over the whole sequence (ragged last piece, given
    initial state, final state returned), and two calls in a row must agree."""
    cfg = get_config("long", T=2048 * 2 + 777, H=2, seed=52)
    x = make_inputs(cfg)
    h = to_device(x, device="cpu")
    h = {k: (v.pin_memory() if v is not None else None) for k, v in h.items()}
    staging = torch.empty(gdn.gdn_host_staging_bytes(cfg.B, x.T_arg, cfg.H, cfg.d_k, cfg.d_v), dtype=torch.uint8,
                          device="cuda")
    ws = None
    if with_ws:
        ws = torch.empty(gdn.gdn_workspace_bytes(cfg.B, x.T_arg, cfg.H, cfg.d_k, cfg.d_v, False), dtype=torch.uint8,
                         device="cuda")
        gdn.gdn_set_workspace(ws)
    try:
        o1, f1 = gdn.gdn_chunk_prefill_host(h["q"], h["k"], h["v"], h["log_alpha"], h["beta"], h["initial_state"],
                                            h["out"], h["final_state"], None, staging)
        torch.cuda.synchronize()
        o1, f1 = o1.clone(), f1.clone()
        o2, f2 = gdn.gdn_chunk_prefill_host(h["q"], h["k"], h["v"], h["log_alpha"], h["beta"], h["initial_state"],
                                            h["out"], h["final_state"], None, staging)
        torch.cuda.synchronize()
        assert gdn.gdn_query_status() == 0
    finally:
        gdn.gdn_set_workspace(None)
    assert torch.equal(o1, o2) and torch.equal(f1, f2)
    want_out, want_fin = run_oracle(x)
    assert_close(f64(o1), want_out, BF16_REL_L2, BF16_MAX_ABS, "out")
    assert_close(f64(f1), want_fin, BF16_REL_L2, None, "final_state")


# ---- error behaviour ---------------------------------------------------------------------------------
def test_error_codes():
    x = make_inputs(get_config("long", T=64, H=1))
    d = to_device(x)
    n0 = gdn.gdn_launch_count()
    with pytest.raises(gdn.GdnError) as e:
        run_lib(gdn.gdn_chunk_prefill, d, chunk=32)
    assert e.value.status == 2
    L = gdn.lib()
    args = [d["q"].data_ptr(), d["k"].data_ptr(), d["v"].data_ptr(), d["log_alpha"].data_ptr(), d["beta"].data_ptr(),
            None, d["out"].data_ptr(), None, None, 1, 64, 1, 128, 128, 64, None]
    bad = list(args); bad[0] = None
    assert L.gdn_chunk_prefill(*bad) == 1
    bad = list(args); bad[9] = 0
    assert L.gdn_chunk_prefill(*bad) == 1
    bad = list(args); bad[1] = d["k"].data_ptr() + 2
    assert L.gdn_chunk_prefill(*bad) == 2
    bad = list(args); bad[12] = 100
    assert L.gdn_chunk_prefill(*bad) == 2
    assert gdn.gdn_launch_count() == n0              # nothing was launched for any of these
    assert L.gdn_chunk_prefill(*args) == 0
    torch.cuda.synchronize()
    assert gdn.gdn_launch_count() > n0


# ---- a ragged tail next to non-finite neighbours ----------------------------------------------------------
@pytest.mark.parametrize("impl", ["fused", "two_kernel", "simt"])
def test_bf16_tail_chunk_is_immune_to_what_follows_the_sequence(impl):
    """Packed input: the tile rows behind a sequence's last token are the first rows of the next sequence.  They only
    meet factors that are exactly zero, but 0 x inf is not 0 -- so the second sequence here starts with rows of inf
    and NaN in q, k and v, and the first sequence (100 tokens: a 36-token tail chunk) must still come out as the
    recurrence over its own tokens.  (The second sequence's own results are not finite, as they should be.)"""
    cfg = get_config("serving", B=2, H=2, lengths=(100, 90), seed=99)
    x = make_inputs(cfg)
    bad = np.array([0x7F80, 0xFF80, 0x7FC0], dtype=np.uint16)            # +inf, -inf, NaN in bf16
    for t in (x.q, x.k, x.v):
        t[100:140] = bad[np.arange(t[100:140].size).reshape(t[100:140].shape) % 3]
    d = to_device(x)
    out, fin = run_lib(BF16_FNS[impl], d)
    o_ref, f_ref = oracle.sequential(widen(x.q[None, :100]), widen(x.k[None, :100]), widen(x.v[None, :100]),
                                     x.log_alpha[None, :100], x.beta[None, :100], x.initial_state[:1])
    assert_close(f64(out[:100]), o_ref[0], BF16_REL_L2, BF16_MAX_ABS, impl + " first sequence out")
    assert_close(f64(fin[0]), f_ref[0], BF16_REL_L2, BF16_MAX_ABS, impl + " first sequence final_state")
