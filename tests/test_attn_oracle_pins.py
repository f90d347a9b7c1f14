"""Pins for the fp64 attention oracle: closed forms, invariants, brute force, and agreement of the
definition with the paper's product-softmax-product order of steps.  None retypes the oracle's
formula; each fails on a plausible mistake (off-by-one causal mask, wrong head grouping, missing
scale, softmax over the wrong axis, transposed operand)."""
import math

import numpy as np
import pytest

import oracle


def _rand(rng, B=2, T=13, Hq=4, Hkv=2, d=8):
    return (rng.standard_normal((B, T, Hq, d)), rng.standard_normal((B, T, Hkv, d)),
            rng.standard_normal((B, T, Hkv, d)))


def test_first_token_returns_its_value_and_equal_keys_give_running_means():
    rng = np.random.default_rng(0)
    q, k, v = _rand(rng)
    out = oracle.attention_causal(q, k, v, 0.3)
    for h in range(4):
        np.testing.assert_allclose(out[:, 0, h], v[:, 0, h // 2], rtol=1e-14)
    # identical keys -> identical scores -> the output is the mean of the values seen so far
    k_same = np.broadcast_to(k[:, :1], k.shape).copy()
    out = oracle.attention_causal(q, k_same, v, 0.7)
    means = np.cumsum(v, axis=1) / np.arange(1, v.shape[1] + 1)[None, :, None, None]
    for h in range(4):
        np.testing.assert_allclose(out[:, :, h], means[:, :, h // 2], rtol=1e-12, atol=1e-13)


def test_two_key_closed_form():
    # d = 1: scores are q*k*scale; with two keys the weights are a logistic function of the difference
    q = np.array([[[[1.0]], [[2.0]]]])            # [B=1, T=2, H=1, d=1]
    k = np.array([[[[0.5]], [[-1.5]]]])
    v = np.array([[[[10.0]], [[20.0]]]])
    out = oracle.attention_causal(q, k, v, 0.25)
    w1 = 1.0 / (1.0 + math.exp(-(2.0 * -1.5 - 2.0 * 0.5) * 0.25))     # weight of key 1 for query 1
    np.testing.assert_allclose(out[0, :, 0, 0], [10.0, 10.0 * (1 - w1) + 20.0 * w1], rtol=1e-14)


def test_brute_force_scalar_loops():
    rng = np.random.default_rng(1)
    q, k, v = _rand(rng, B=1, T=6, Hq=2, Hkv=1, d=3)
    out = oracle.attention_causal(q, k, v, 0.5)
    for h in range(2):
        for i in range(6):
            num = [0.0, 0.0, 0.0]
            den = 0.0
            for j in range(i + 1):
                s = sum(q[0, i, h, f] * k[0, j, 0, f] for f in range(3)) * 0.5
                w = math.exp(s)
                den += w
                for f in range(3):
                    num[f] += w * v[0, j, 0, f]
            np.testing.assert_allclose(out[0, i, h], [x / den for x in num], rtol=1e-12)


def test_invariants():
    rng = np.random.default_rng(2)
    q, k, v = _rand(rng)
    out = oracle.attention_causal(q, k, v, 0.35)
    # adding one vector to every key shifts each score row by a constant: nothing changes
    c = rng.standard_normal(k.shape[-1])
    np.testing.assert_allclose(oracle.attention_causal(q, k + c, v, 0.35), out, rtol=1e-10, atol=1e-12)
    # scaling q by a and the scale by 1/a is the same problem
    np.testing.assert_allclose(oracle.attention_causal(q * 4.0, k, v, 0.35 / 4.0), out, rtol=1e-12, atol=1e-13)
    # causality: the future does not reach the past
    k2, v2 = k.copy(), v.copy()
    k2[:, 9:] += 5.0
    v2[:, 9:] -= 3.0
    np.testing.assert_allclose(oracle.attention_causal(q, k2, v2, 0.35)[:, :9], out[:, :9], rtol=1e-14)
    assert np.abs(oracle.attention_causal(q, k2, v2, 0.35)[:, 9:] - out[:, 9:]).max() > 0.1
    # linear in v; outputs are convex combinations of the values
    np.testing.assert_allclose(oracle.attention_causal(q, k, 2 * v + 1, 0.35), 2 * out + 1, rtol=1e-12, atol=1e-12)
    # query heads of one group read the same key/value head: permuting the kv heads permutes the groups
    outp = oracle.attention_causal(q[:, :, [2, 3, 0, 1]], k[:, :, ::-1], v[:, :, ::-1], 0.35)
    np.testing.assert_allclose(outp, out[:, :, [2, 3, 0, 1]], rtol=1e-14)
    # a very large scale picks the value of the best-matching visible key
    big = oracle.attention_causal(q, k, v, 1e4)
    for i in (0, 5, 12):
        j = int(np.argmax(k[0, : i + 1, 0] @ q[0, i, 1]))
        np.testing.assert_allclose(big[0, i, 1], v[0, j, 0], rtol=1e-9, atol=1e-9)


def test_product_softmax_product_form_equals_the_definition():
    rng = np.random.default_rng(3)
    q, k, v = _rand(rng, B=2, T=37, Hq=6, Hkv=3, d=16)
    a = oracle.attention_causal(q, k, v, 1 / 4.0)
    b = oracle.attention_gemm_form(q, k, v, 1 / 4.0)
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)
    # and with torch's own routine where it is available (an independently written library path)
    torch = pytest.importorskip("torch")
    qt, kt, vt = (torch.from_numpy(x).permute(0, 2, 1, 3) for x in (q, np.repeat(k, 2, axis=2), np.repeat(v, 2, axis=2)))
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True, scale=0.25)
    np.testing.assert_allclose(a, ref.permute(0, 2, 1, 3).numpy(), rtol=1e-10, atol=1e-12)


def test_packed_sequences_are_independent():
    rng = np.random.default_rng(4)
    q, k, v = _rand(rng, B=1, T=20, Hq=2, Hkv=1, d=4)
    cu = [0, 7, 7, 20]
    packed = oracle.attention_causal(q[0], k[0], v[0], 0.4, cu_seqlens=cu)
    np.testing.assert_allclose(packed[:7], oracle.attention_causal(q[:, :7], k[:, :7], v[:, :7], 0.4)[0], rtol=1e-14)
    np.testing.assert_allclose(packed[7:], oracle.attention_causal(q[:, 7:], k[:, 7:], v[:, 7:], 0.4)[0], rtol=1e-14)
    # first token of every sequence returns its own value: nothing leaks across the boundary
    np.testing.assert_allclose(packed[7, 0], v[0, 7, 0], rtol=1e-14)


def test_rows_variant_against_full_definition_and_scalar_brute_force():
    """attention_causal_rows (the sampled-row form the full-size GPU checks use) on every row of a small
    grouped-query case: equal to attention_causal, and to scalar loops that know nothing of numpy.  A slip
    in its head grouping or in its prefix length fails here, on the CPU."""
    rng = np.random.default_rng(7)
    q, k, v = _rand(rng, B=2, T=9, Hq=6, Hkv=2, d=4)      # three query heads per key/value head
    scale = 0.4
    rows = [(b, i, h) for b in range(2) for i in range(9) for h in range(6)]
    got = oracle.attention_causal_rows(q, k, v, scale, rows)
    full = oracle.attention_causal(q, k, v, scale)
    for n, (b, i, h) in enumerate(rows):
        np.testing.assert_allclose(got[n], full[b, i, h], rtol=1e-13, atol=1e-15)
    for n, (b, i, h) in enumerate(rows[::7]):
        hk = h // 3
        den, num = 0.0, [0.0] * 4
        for j in range(i + 1):
            w = math.exp(sum(q[b, i, h, f] * k[b, j, hk, f] for f in range(4)) * scale)
            den += w
            for f in range(4):
                num[f] += w * v[b, j, hk, f]
        np.testing.assert_allclose(got[7 * n], [x / den for x in num], rtol=1e-12)
    # an out-of-order, repeated selection returns the rows in the order asked for
    pick = [(1, 8, 5), (0, 0, 0), (1, 8, 5), (0, 4, 3)]
    sub = oracle.attention_causal_rows(q, k, v, scale, pick)
    for n, (b, i, h) in enumerate(pick):
        np.testing.assert_allclose(sub[n], full[b, i, h], rtol=1e-13, atol=1e-15)
