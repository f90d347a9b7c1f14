"""Causal grouped-query attention (tcgen05 kernel) against the fp64 oracle, element by element on
reduced sizes that span several tiles and a ragged tail, and on sampled rows at the full sizes."""
import numpy as np
import pytest
import torch

import oracle
from workloads import get_attn_config, make_attn_inputs, widen
from gdn_testlib import assert_close, f64

pytestmark = pytest.mark.gpu

# bf16 storage of q, k, v, the probabilities and the output; fp32 scores, softmax and accumulation
ATTN_REL_L2 = 5e-3
ATTN_MAX_ABS = 2e-2


def _dev(a):
    return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda()


def _run(cfg, q, k, v, scale=None):
    import paper_2607_14568_b200 as gdn
    dq, dk, dv = _dev(q), _dev(k), _dev(v)
    out = torch.full_like(dq, float("nan"))
    gdn.gdn_attn_causal_prefill(dq, dk, dv, out, cfg.scale if scale is None else scale)
    torch.cuda.synchronize()
    assert gdn.gdn_query_status() == 0
    return out


@pytest.mark.parametrize("kw", [
    dict(B=1, T=1, Hq=1, Hkv=1), dict(B=1, T=64, Hq=2, Hkv=1), dict(B=1, T=128, Hq=2, Hkv=2),
    dict(B=2, T=129, Hq=4, Hkv=2), dict(B=2, T=333, Hq=4, Hkv=2), dict(B=1, T=700, Hq=8, Hkv=2),
    dict(B=3, T=257, Hq=3, Hkv=3),
])
def test_reduced_sizes_match_oracle(kw):
    cfg = get_attn_config("attn_small", **kw)
    q, k, v = make_attn_inputs(cfg)
    out = _run(cfg, q, k, v)
    want = oracle.attention_causal(widen(q), widen(k), widen(v), cfg.scale)
    assert_close(f64(out), want, ATTN_REL_L2, ATTN_MAX_ABS, "out")


def test_peaked_and_flat_scores():
    """A large scale (softmax close to an argmax, the reference maximum jumps between tiles) and a
    zero scale (uniform weights: running means of v)."""
    cfg = get_attn_config("attn_small", B=1, T=520, Hq=2, Hkv=1)
    q, k, v = make_attn_inputs(cfg)
    for scale in (4.0, 0.0):
        out = _run(cfg, q, k, v, scale)
        want = oracle.attention_causal(widen(q), widen(k), widen(v), scale)
        assert_close(f64(out), want, ATTN_REL_L2, 4e-2 if scale else ATTN_MAX_ABS, f"out (scale {scale})")


def test_rising_scores_force_rescaling():
    """Keys whose score grows with position: the running maximum rises by far more than 2^8 across
    tiles, so the accumulator in tensor memory is rescaled many times."""
    cfg = get_attn_config("attn_small", B=1, T=640, Hq=1, Hkv=1)
    q, k, v = make_attn_inputs(cfg)
    qf = np.zeros((1, 640, 1, 128), dtype=np.float32)
    kf = np.zeros((1, 640, 1, 128), dtype=np.float32)
    qf[..., 0] = 1.0
    kf[0, :, 0, 0] = np.arange(640, dtype=np.float32) / 8.0        # exact in bf16 up to 256/8 steps? keep coarse
    from workloads import f32_to_bf16_bits
    q2, k2 = f32_to_bf16_bits(qf), f32_to_bf16_bits(kf)
    out = _run(cfg, q2, k2, v, 1.0)
    want = oracle.attention_causal(widen(q2), widen(k2), widen(v), 1.0)
    assert_close(f64(out), want, ATTN_REL_L2, ATTN_MAX_ABS, "out")


@pytest.mark.parametrize("name", ["attn_2k", "attn_10k"])
def test_full_sizes_on_sampled_rows(name):
    cfg = get_attn_config(name)
    q, k, v = make_attn_inputs(cfg)
    out = _run(cfg, q, k, v)
    rng = np.random.default_rng(5)
    rows = [(0, 0, 0), (0, cfg.T - 1, cfg.Hq - 1), (0, 127, 3), (0, 128, 3), (0, cfg.T - 129, 7)]
    rows += [(0, int(rng.integers(0, cfg.T)), int(rng.integers(0, cfg.Hq))) for _ in range(40)]
    want = oracle.attention_causal_rows(widen(q), widen(k), widen(v), cfg.scale, rows)
    got = np.stack([f64(out[b, i, h]) for (b, i, h) in rows])
    assert_close(got, want, ATTN_REL_L2, ATTN_MAX_ABS, "sampled rows")
    assert torch.isfinite(out.float()).all()


def test_errors():
    import paper_2607_14568_b200 as gdn
    cfg = get_attn_config("attn_small", B=1, T=64, Hq=3, Hkv=2)
    q = torch.zeros((1, 64, 3, 128), dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros((1, 64, 2, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(gdn.GdnError) as e:
        gdn.gdn_attn_causal_prefill(q, kv, kv, torch.empty_like(q))      # 3 query heads on 2 kv heads
    assert e.value.status == 2
    q64 = torch.zeros((1, 64, 2, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(gdn.GdnError) as e:
        gdn.gdn_attn_causal_prefill(q64, q64, q64, torch.empty_like(q64))  # d = 64
    assert e.value.status == 2


def test_packed_sequences():
    """Packed input: ragged lengths, an empty sequence, a one-token sequence; no leakage between sequences."""
    import paper_2607_14568_b200 as gdn
    lengths = [300, 0, 1, 129, 512, 77]
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    cfg = get_attn_config("attn_small", B=1, T=int(cu[-1]), Hq=4, Hkv=2)
    q, k, v = (a[0] for a in make_attn_inputs(cfg))          # [T, H, d]
    dq, dk, dv = _dev(q), _dev(k), _dev(v)
    out = torch.full_like(dq, float("nan"))
    gdn.gdn_attn_causal_prefill(dq, dk, dv, out, cfg.scale, cu_seqlens=torch.from_numpy(cu).cuda())
    torch.cuda.synchronize()
    assert gdn.gdn_query_status() == 0
    want = oracle.attention_causal(widen(q), widen(k), widen(v), cfg.scale, cu_seqlens=cu)
    assert_close(f64(out), want, ATTN_REL_L2, ATTN_MAX_ABS, "out")
