"""Input generator: determinism, per-chain regeneration, distributions, bf16 rounding,
and the stored drift guard for the oracle on the tiny configuration."""
import os

import numpy as np
import torch

import oracle
from workloads import (CONFIGS, bf16_bits_to_f32, chain_inputs, f32_to_bf16_bits, get_config,
                       make_inputs, widen)

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "tiny_oracle_samples.txt")


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(100000) * np.exp(rng.uniform(-20, 20, 100000))).astype(np.float32)
    x[:4] = [0.0, -0.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -9]      # ties
    ours = f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    assert np.array_equal(f32_to_bf16_bits(bf16_bits_to_f32(ours)), ours)


def test_generator_is_deterministic_and_chainwise():
    cfg = get_config("short", T=192, H=3)
    a, b = make_inputs(cfg, threads=1), make_inputs(cfg, threads=4)
    for name in ("q", "k", "v", "log_alpha", "beta"):
        assert np.array_equal(getattr(a, name), getattr(b, name))
    c = chain_inputs(cfg, 0, 2)
    assert np.array_equal(a.q[0, :, 2], c["q"]) and np.array_equal(a.v[0, :, 2], c["v"])
    assert np.array_equal(a.beta[0, :, 2], c["beta"])
    assert a.initial_state is None and a.q.dtype == np.uint16


def test_distributions_and_shapes():
    cfg = get_config("long", T=4096, H=2)
    x = make_inputs(cfg)
    k = widen(x.k)
    assert np.allclose(np.linalg.norm(k, axis=-1), 1.0, atol=5e-3)        # unit keys up to bf16 rounding
    assert abs(widen(x.v).std() - 1.0) < 0.02
    assert (x.beta > 0).all() and (x.beta < 1).all() and abs(x.beta.mean() - 0.5) < 0.02
    assert (x.log_alpha < 0).all() and abs(x.log_alpha.mean() + 0.0403) < 0.002
    assert x.initial_state.shape == (1, 2, 128, 128) and abs(x.initial_state.std() - 0.02) < 0.001


def test_serving_lengths_and_packing():
    cfg = CONFIGS["serving"]
    lens = cfg.seq_lengths()
    assert len(lens) == 8 and all(512 <= n <= 8192 for n in lens) and lens == cfg.seq_lengths()
    small = get_config("serving", lengths=(70, 0, 129), B=3, H=2)
    x = make_inputs(small)
    assert list(x.cu_seqlens) == [0, 70, 70, 199] and x.q.shape == (199, 2, 128) and x.T_arg == 199
    assert np.array_equal(x.k[70:199, 1], chain_inputs(small, 2, 1)["k"])


def test_oracle_drift_guard_on_tiny():
    x = make_inputs(get_config("tiny"))
    out, fin = oracle.sequential(widen(x.q), widen(x.k), widen(x.v), x.log_alpha, x.beta, None)
    for line in open(GOLDEN):
        if line.startswith("#"):
            continue
        kind, a, b, c, val = line.split()
        a, b, c, want = int(a), int(b), int(c), float.fromhex(val)
        got = {"out": lambda: out[0, a, b, c], "state": lambda: fin[0, a, b, c],
               "norm_out": lambda: np.linalg.norm(out), "norm_state": lambda: np.linalg.norm(fin)}[kind]()
        assert abs(got - want) <= 1e-12 * max(1.0, abs(want)), line
