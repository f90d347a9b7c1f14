"""Pins for the fp64 CPU oracle: closed forms, invariants and cross-formulation
agreement.  None of these compares the oracle with its own formula retyped; each
would fail on a plausible mistake (dropped term, wrong sign, wrong mask, wrong
operator order, transposed state).

The paper prints no worked numeric example for the chunked scan (only timings and
error magnitudes), so no value-level fixture comes from it.
"""
import numpy as np
import pytest

import oracle

RTOL = 1e-12


def rel(a, b):
    d = np.linalg.norm(np.asarray(a) - np.asarray(b))
    n = np.linalg.norm(np.asarray(b))
    return d / n if n > 0 else d


def rand_problem(rng, B=1, T=40, H=2, dk=8, dv=6, gate=0.3, s0=True, normalise=True):
    q = rng.standard_normal((B, T, H, dk))
    k = rng.standard_normal((B, T, H, dk))
    if normalise:
        q /= np.linalg.norm(q, axis=-1, keepdims=True)
        k /= np.linalg.norm(k, axis=-1, keepdims=True)
    v = rng.standard_normal((B, T, H, dv))
    beta = 1 / (1 + np.exp(-rng.standard_normal((B, T, H))))
    la = -np.logaddexp(0, rng.standard_normal((B, T, H))) * gate
    S0 = rng.standard_normal((B, H, dk, dv)) * 0.5 if s0 else None
    return q, k, v, la, beta, S0


# --- P1: beta = 0 -> pure decay of the initial state (closed form) -----------------------
def test_pure_decay_closed_form():
    rng = np.random.default_rng(1)
    q, k, v, la, beta, S0 = rand_problem(rng, B=2, T=37, H=3)
    beta[:] = 0.0
    for fn in (oracle.sequential, oracle.chunked, oracle.dense):
        out, fin = fn(q, k, v, la, beta, S0)
        G = np.exp(np.cumsum(la, axis=1))                      # [B,T,H]
        want = G[..., None] * np.einsum("bhmj,bthm->bthj", S0, q)
        assert rel(out, want) < RTOL
        assert rel(fin, G[:, -1][..., None, None] * S0) < RTOL


# --- P2: alpha = 1, beta = 1, orthonormal keys -> exact write / exact overwrite ----------
def test_exact_key_write_and_overwrite():
    rng = np.random.default_rng(2)
    dk, dv, n = 8, 5, 8
    basis, _ = np.linalg.qr(rng.standard_normal((dk, dk)))
    order = [0, 1, 2, 3, 4, 5, 6, 7, 2, 5, 2]                # keys 2 and 5 are rewritten
    T = len(order)
    k = basis[:, order].T[None, :, None, :]                    # [1,T,1,dk]
    v = rng.standard_normal((1, T, 1, dv))
    q = k.copy()                                               # query the key just written
    la = np.zeros((1, T, 1))
    beta = np.ones((1, T, 1))
    last = {key: t for t, key in enumerate(order)}
    want_S = sum(np.outer(basis[:, key], v[0, t, 0]) for key, t in last.items())
    for fn in (oracle.sequential, oracle.chunked, oracle.dense):
        out, fin = fn(q, k, v, la, beta, None)
        assert rel(out, v) < RTOL                              # reading back returns the value exactly
        assert rel(fin[0, 0], want_S) < RTOL                   # rewritten keys hold only the new value
    assert n == dk


# --- P6: one token, by hand --------------------------------------------------------------
def test_single_token_closed_form():
    rng = np.random.default_rng(3)
    dk, dv = 5, 4
    q, k, v, la, beta, S0 = rand_problem(rng, B=1, T=1, H=1, dk=dk, dv=dv, normalise=False)
    kk, qq, vv = k[0, 0, 0], q[0, 0, 0], v[0, 0, 0]
    al, be = np.exp(la[0, 0, 0]), beta[0, 0, 0]
    S1 = al * (np.eye(dk) - be * np.outer(kk, kk)) @ S0[0, 0] + be * np.outer(kk, vv)
    o = S1.T @ qq
    for fn in (oracle.sequential, oracle.chunked, oracle.dense):
        out, fin = fn(q, k, v, la, beta, S0)
        assert rel(fin[0, 0], S1) < RTOL
        assert rel(out[0, 0, 0], o) < RTOL


# --- the recurrence as written with the state transposed (d_v x d_k), o = S q -----------
def test_transposed_orientation_matches():
    rng = np.random.default_rng(4)
    q, k, v, la, beta, S0 = rand_problem(rng, B=1, T=19, H=1, dk=6, dv=4, normalise=False)
    S = S0[0, 0].T.copy()                                      # d_v x d_k
    outs = []
    for t in range(q.shape[1]):
        kt, vt, qt = k[0, t, 0], v[0, t, 0], q[0, t, 0]
        S = np.exp(la[0, t, 0]) * S @ (np.eye(6) - beta[0, t, 0] * np.outer(kt, kt)) \
            + beta[0, t, 0] * np.outer(vt, kt)
        outs.append(S @ qt)
    out, fin = oracle.sequential(q, k, v, la, beta, S0)
    assert rel(out[0, :, 0], np.array(outs)) < RTOL
    assert rel(fin[0, 0], S.T) < RTOL


# --- P3/P4/P5: three formulations agree; chunk size does not matter -----------------------
@pytest.mark.parametrize("T", [1, 7, 64, 65, 150])
def test_sequential_chunked_dense_agree(T):
    rng = np.random.default_rng(10 + T)
    q, k, v, la, beta, S0 = rand_problem(rng, B=2, T=T, H=2, dk=8, dv=6, gate=0.4)
    o_seq, f_seq = oracle.sequential(q, k, v, la, beta, S0)
    for C in (1, 16, 64, T, 3):
        for form in (0, 1):
            o, f = oracle.chunked(q, k, v, la, beta, S0, chunk=C, form=form)
            assert rel(o, o_seq) < RTOL, (C, form)
            assert rel(f, f_seq) < RTOL, (C, form)
    if T <= 64:
        o, f = oracle.dense(q, k, v, la, beta, S0)
        assert rel(o, o_seq) < RTOL and rel(f, f_seq) < RTOL


def test_dense_matches_at_64_unnormalised_keys():
    rng = np.random.default_rng(5)
    q, k, v, la, beta, S0 = rand_problem(rng, B=1, T=64, H=1, dk=16, dv=8, normalise=False)
    k *= 0.3
    o1, f1 = oracle.sequential(q, k, v, la, beta, S0)
    o2, f2 = oracle.dense(q, k, v, la, beta, S0)
    o3, f3 = oracle.chunked(q, k, v, la, beta, S0, chunk=64)
    assert rel(o2, o1) < 1e-11 and rel(f2, f1) < 1e-11
    assert rel(o3, o1) < 1e-11 and rel(f3, f1) < 1e-11


# --- P7: split invariance and packed sequences -------------------------------------------
def test_split_invariance_and_packing():
    rng = np.random.default_rng(6)
    q, k, v, la, beta, S0 = rand_problem(rng, B=1, T=100, H=2, dk=8, dv=6)
    o_all, f_all = oracle.sequential(q, k, v, la, beta, S0)
    for fn in (oracle.sequential, lambda *a, **kw: oracle.chunked(*a, chunk=16, **kw)):
        T1 = 41
        o1, f1 = fn(q[:, :T1], k[:, :T1], v[:, :T1], la[:, :T1], beta[:, :T1], S0)
        o2, f2 = fn(q[:, T1:], k[:, T1:], v[:, T1:], la[:, T1:], beta[:, T1:], f1)
        assert rel(np.concatenate([o1, o2], 1), o_all) < RTOL
        assert rel(f2, f_all) < RTOL
    # packed: three sequences (one empty) == each alone
    lens = [30, 0, 70]
    cu = np.array([0, 30, 30, 100], dtype=np.int32)
    S0p = rng.standard_normal((3, 2, 8, 6))
    for fn in (oracle.sequential, lambda *a, **kw: oracle.chunked(*a, chunk=16, **kw), oracle.dense):
        o, f = fn(q[0], k[0], v[0], la[0], beta[0], S0p, cu_seqlens=cu)
        for n, (a, b) in enumerate(zip(cu[:-1], cu[1:])):
            if lens[n] == 0:
                assert np.array_equal(f[n], S0p[n])             # empty sequence: state passes through
                continue
            oo, ff = oracle.sequential(q[:, a:b], k[:, a:b], v[:, a:b], la[:, a:b], beta[:, a:b], S0p[n:n + 1])
            assert rel(o[a:b], oo[0]) < RTOL and rel(f[n], ff[0]) < RTOL


# --- P8: identity tokens (beta = 0, log_alpha = 0) change nothing ------------------------
def test_padding_invariance():
    rng = np.random.default_rng(7)
    q, k, v, la, beta, S0 = rand_problem(rng, B=1, T=50, H=2)
    pad = 14
    qp, kp, vp, lap, bp, _ = rand_problem(rng, B=1, T=pad, H=2)
    lap[:] = 0.0
    bp[:] = 0.0
    cat = lambda a, b: np.concatenate([a, b], axis=1)
    for fn in (oracle.sequential, oracle.chunked):
        o, f = fn(q, k, v, la, beta, S0)
        o2, f2 = fn(cat(q, qp), cat(k, kp), cat(v, vp), cat(la, lap), cat(beta, bp), S0)
        assert rel(o2[:, :50], o) < RTOL and rel(f2, f) < RTOL


# --- P9: linearity and equivariance -------------------------------------------------------
def test_linearity_and_head_permutation():
    rng = np.random.default_rng(8)
    q, k, v, la, beta, S0 = rand_problem(rng, B=2, T=33, H=3)
    v2 = rng.standard_normal(v.shape)
    S02 = rng.standard_normal(S0.shape)
    for fn in (oracle.sequential, oracle.chunked):
        o1, f1 = fn(q, k, v, la, beta, S0)
        o2, f2 = fn(q, k, v2, la, beta, S02)
        o3, f3 = fn(q, k, 2 * v - 3 * v2, la, beta, 2 * S0 - 3 * S02)
        assert rel(o3, 2 * o1 - 3 * o2) < 1e-11 and rel(f3, 2 * f1 - 3 * f2) < 1e-11
        o4, f4 = fn(-1.5 * q, k, v, la, beta, S0)
        assert rel(o4, -1.5 * o1) < RTOL and rel(f4, f1) < RTOL   # q scales the output only
        perm = [2, 0, 1]
        o5, f5 = fn(q[:, :, perm], k[:, :, perm], v[:, :, perm], la[:, :, perm], beta[:, :, perm], S0[:, perm])
        assert np.array_equal(o5, o1[:, :, perm]) and np.array_equal(f5, f1[:, perm])


# --- P10: orthogonal keys -> gated causal linear attention (a masked matmul) -------------
def test_orthogonal_keys_reduce_to_masked_linear_attention():
    rng = np.random.default_rng(9)
    dk, dv, T = 12, 5, 12
    basis, _ = np.linalg.qr(rng.standard_normal((dk, dk)))
    k = (basis.T * rng.uniform(0.5, 2.0, size=(dk, 1)))[None, :, None, :]   # orthogonal, not unit
    q = rng.standard_normal((1, T, 1, dk))
    v = rng.standard_normal((1, T, 1, dv))
    beta = rng.uniform(0.1, 0.9, size=(1, T, 1))
    la = -rng.uniform(0.0, 0.5, size=(1, T, 1))
    G = np.cumsum(la[0, :, 0])
    scores = (q[0, :, 0] @ k[0, :, 0].T) * np.exp(G[:, None] - G[None, :])
    scores = np.tril(scores)                                                 # i <= t, diagonal included
    want = scores @ (beta[0, :, 0, None] * v[0, :, 0])
    for fn in (oracle.sequential, oracle.chunked, oracle.dense):
        out, _ = fn(q, k, v, la, beta, None)
        assert rel(out[0, :, 0], want) < 1e-11


# --- P11: contraction bound ---------------------------------------------------------------
def test_state_norm_bound():
    rng = np.random.default_rng(11)
    q, k, v, la, beta, S0 = rand_problem(rng, B=1, T=60, H=1, dk=8, dv=6)
    bound = np.linalg.norm(S0[0, 0])
    for t in range(1, 61):
        _, f = oracle.sequential(q[:, :t], k[:, :t], v[:, :t], la[:, :t], beta[:, :t], S0)
        bound = bound + beta[0, t - 1, 0] * np.linalg.norm(v[0, t - 1, 0])
        assert np.linalg.norm(f[0, 0]) <= bound * (1 + 1e-12)


def test_oracle_rejects_bad_arguments():
    rng = np.random.default_rng(12)
    q, k, v, la, beta, S0 = rand_problem(rng, B=1, T=4, H=1)
    with pytest.raises(ValueError):
        oracle.sequential(q[0], k[0], v[0], la[0], beta[0], None, cu_seqlens=np.array([0, 3], dtype=np.int32))
    with pytest.raises(ValueError):
        oracle.chunked(q, k, v, la, beta, None, chunk=0)


# ---------------------------------------------------------------------------
# prologue (norms and gating in front of the scan)
# ---------------------------------------------------------------------------
def test_prologue_closed_forms():
    # 3-4-5 triangle: the unit vector of (3, 4) is (0.6, 0.8); of (0, -2) it is (0, -1)
    q_raw = np.array([[[3.0, 4.0]], [[0.0, -2.0]]])            # [T=2, H=1, d=2]
    k_raw = np.array([[[5.0, 12.0]], [[-8.0, 6.0]]])           # 5-12-13 and 6-8-10
    a_raw = np.array([[0.0], [np.log(np.e - 1.0)]])            # softplus = ln 2 and exactly 1
    b_raw = np.array([[0.0], [np.log(3.0)]])                   # sigmoid = 1/2 and 3/4
    q, k, la, be = oracle.prologue(q_raw, k_raw, a_raw, b_raw, gate_scale=0.25)
    np.testing.assert_allclose(q, [[[0.6, 0.8]], [[0.0, -1.0]]], rtol=1e-15, atol=0)
    np.testing.assert_allclose(k, [[[5 / 13, 12 / 13]], [[-0.8, 0.6]]], rtol=1e-15, atol=0)
    np.testing.assert_allclose(la, [[-0.25 * np.log(2.0)], [-0.25]], rtol=1e-15)
    np.testing.assert_allclose(be, [[0.5], [0.75]], rtol=1e-15)
    # eps enters under the square root: (3,4) with eps = 11 has length 6
    q2, *_ = oracle.prologue(q_raw, k_raw, a_raw, b_raw, gate_scale=1.0, eps=11.0)
    np.testing.assert_allclose(q2[0, 0], [0.5, 4.0 / 6.0], rtol=1e-15)


def test_prologue_invariants():
    rng = np.random.default_rng(21)
    q_raw = rng.standard_normal((2, 9, 3, 16)) * np.exp(rng.standard_normal((2, 9, 3, 1)))
    k_raw = rng.standard_normal((2, 9, 3, 16)) * 7.0
    a_raw = rng.standard_normal((2, 9, 3)) * 3
    b_raw = rng.standard_normal((2, 9, 3)) * 3
    q, k, la, be = oracle.prologue(q_raw, k_raw, a_raw, b_raw, gate_scale=0.05)
    np.testing.assert_allclose(np.linalg.norm(q, axis=-1), 1.0, rtol=1e-14)
    np.testing.assert_allclose(np.linalg.norm(k, axis=-1), 1.0, rtol=1e-14)
    # direction kept (cosine with the raw vector is +1), positive rescaling changes nothing
    assert ((q * q_raw).sum(-1) > 0).all()
    q3, k3, _, _ = oracle.prologue(q_raw * 3.5, k_raw * 0.01, a_raw, b_raw, gate_scale=0.05)
    np.testing.assert_allclose(q3, q, rtol=1e-13)
    np.testing.assert_allclose(k3, k, rtol=1e-13)
    # sigmoid(x) + sigmoid(-x) = 1; softplus(x) - softplus(-x) = x; gate in (0, 1]; linear in the scale
    _, _, la_neg, be_neg = oracle.prologue(q_raw, k_raw, -a_raw, -b_raw, gate_scale=0.05)
    np.testing.assert_allclose(be + be_neg, 1.0, rtol=1e-14)
    np.testing.assert_allclose((la_neg - la) / 0.05, a_raw, rtol=1e-12, atol=1e-13)
    assert (la < 0).all() and ((be > 0) & (be < 1)).all()
    _, _, la2, _ = oracle.prologue(q_raw, k_raw, a_raw, b_raw, gate_scale=0.1)
    np.testing.assert_allclose(la2, 2 * la, rtol=1e-15)
    # agrees with scipy's independently written special functions
    from scipy.special import expit, log1p, logsumexp  # noqa: F401
    np.testing.assert_allclose(be, expit(b_raw), rtol=1e-14)
    np.testing.assert_allclose(la, -0.05 * np.logaddexp(0.0, a_raw), rtol=1e-13)


# --- stage outputs of the chunked form: each against something that is not the chunked code ------------
def test_chunked_stages_against_token_loop_and_linear_algebra():
    """oracle.chunked_stages hands out g, A, P, T, W, U, Delta and the incoming state of every chunk of one
    chain.  Delta and the states are pinned by a token-by-token loop written here (the per-token correction
    delta_t and the state at each chunk boundary are what the recurrence itself produces); T by (I + A) T = I;
    g, A, P, W, U by numpy expressions of their definitions on the raw inputs; the outputs and the final state
    by the sequential oracle.  A packed batch with a ragged tail, chain (1, 1)."""
    rng = np.random.default_rng(11)
    H, dk, dv, C = 2, 8, 6, 16
    lengths = [20, 37, 5]
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    Tt = int(cu[-1])
    q, k, v, la, beta, S0 = rand_problem(rng, B=1, T=Tt, H=H, dk=dk, dv=dv)
    q, k, v, la, beta = q[0], k[0], v[0], la[0], beta[0]                 # packed [T,H,.]
    S0 = rng.standard_normal((3, H, dk, dv)) * 0.5
    n, h = 1, 1
    st = oracle.chunked_stages(q, k, v, la, beta, S0, cu, chunk=C, n=n, h=h)
    L = lengths[n]
    a, b = int(cu[n]), int(cu[n + 1])
    kk, qq, vv, aa, bb = k[a:b, h], q[a:b, h], v[a:b, h], la[a:b, h], beta[a:b, h]
    # token loop: deltas, boundary states, outputs
    S = S0[n, h].copy()
    deltas, outs, bounds = [], [], []
    for t in range(L):
        if t % C == 0:
            bounds.append(S.copy())
        S = np.exp(aa[t]) * S
        d = bb[t] * (vv[t] - S.T @ kk[t])
        S = S + np.outer(kk[t], d)
        deltas.append(d)
        outs.append(S.T @ qq[t])
    nch = (L + C - 1) // C
    assert st["length"] == L and st["g"].shape == (nch, C)
    assert rel(st["out"], np.array(outs)) < RTOL and rel(st["final_state"], S) < RTOL
    seq_out, seq_fin = oracle.sequential(q, k, v, la, beta, S0, cu)
    assert rel(st["out"], seq_out[a:b, h]) < RTOL and rel(st["final_state"], seq_fin[n, h]) < RTOL
    for c in range(nch):
        R = min(C, L - c * C)
        sl = slice(c * C, c * C + R)
        g = np.cumsum(aa[sl])
        assert rel(st["g"][c, :R], g) < RTOL
        assert rel(st["S_in"][c], bounds[c]) < RTOL
        assert rel(st["Delta"][c, :R], np.array(deltas[c * C:c * C + R])) < 1e-11
        dec = np.exp(g[:, None] - g[None, :])
        A = np.tril(bb[sl, None] * dec * (kk[sl] @ kk[sl].T), -1)
        P = np.tril(dec * (qq[sl] @ kk[sl].T), 0)
        assert rel(st["A"][c, :R, :R], A) < RTOL and rel(st["P"][c, :R, :R], P) < RTOL
        T = st["T"][c, :R, :R]
        assert np.abs((np.eye(R) + A) @ T - np.eye(R)).max() < 1e-12
        assert np.abs(np.triu(T, 1)).max() == 0.0 and np.allclose(np.diag(T), 1.0)
        assert rel(st["W"][c, :R], T @ (bb[sl, None] * np.exp(g)[:, None] * kk[sl])) < RTOL
        assert rel(st["U"][c, :R], T @ (bb[sl, None] * vv[sl])) < RTOL
        # the chunk's correction is U - W S_in (what the GPU chain forms)
        assert rel(st["Delta"][c, :R], st["U"][c, :R] - st["W"][c, :R] @ st["S_in"][c]) < 1e-11
        # rows beyond a ragged tail stay zero
        assert not st["W"][c, R:].any() and not st["T"][c, R:].any()


# --- epilogue (gated root-mean-square norm behind the scan) --------------------------------------------
def test_epilogue_closed_forms():
    import math
    # rows (3, 4) and (6, 8, 0, 0): mean squares 12.5 and 25; gates 0, ln 3 (silu = ln 3 * 3/4) and large
    o = np.array([[3.0, 4.0]])
    out = oracle.epilogue(o, np.array([[math.log(3.0), 0.0]]), np.array([1.0, 1.0]))
    np.testing.assert_allclose(out, [[3.0 / math.sqrt(12.5) * math.log(3.0) * 0.75, 0.0]], rtol=1e-14)
    o = np.array([[6.0, 8.0, 0.0, 0.0]])
    z = np.array([[40.0, -40.0, 1.0, 2.0]])                # silu(40) = 40 to 1e-16, silu(-40) = -40 e^-40
    out = oracle.epilogue(o, z, np.array([2.0, 3.0, 5.0, 7.0]))
    np.testing.assert_allclose(out[0, 0], 6.0 / 5.0 * 2.0 * 40.0, rtol=1e-14)
    np.testing.assert_allclose(out[0, 1], 8.0 / 5.0 * 3.0 * (-40.0 * math.exp(-40.0) / (1 + math.exp(-40.0))), rtol=1e-12)
    assert out[0, 2] == 0.0 and out[0, 3] == 0.0
    # eps under the root: mean square 25 + eps 11 = 36
    out = oracle.epilogue(o, np.full((1, 4), 40.0), np.ones(4), eps=11.0)
    np.testing.assert_allclose(out[0, :2], [40.0, 8.0 / 6.0 * 40.0], rtol=1e-14)


def test_epilogue_invariants_and_scalar_loops():
    import math
    rng = np.random.default_rng(21)
    o = rng.standard_normal((2, 5, 3, 8))
    z = rng.standard_normal((2, 5, 3, 8))
    w = rng.standard_normal(8)
    out = oracle.epilogue(o, z, w, eps=1e-3)
    assert out.shape == o.shape
    # scalar loops that know nothing of numpy broadcasting
    for idx in [(0, 0, 0), (1, 4, 2), (0, 3, 1)]:
        row, gate = o[idx], z[idx]
        ms = sum(x * x for x in row) / 8 + 1e-3
        for j in range(8):
            want = row[j] / math.sqrt(ms) * w[j] * gate[j] / (1.0 + math.exp(-gate[j]))
            assert abs(out[idx][j] - want) <= 1e-13 * max(1.0, abs(want))
    # the norm removes the scale of o (eps = 0), every row has unit mean square before weight and gate
    a = oracle.epilogue(o, z, w)
    b = oracle.epilogue(o * 7.5, z, w)
    assert rel(a, b) < RTOL
    unit = oracle.epilogue(o, np.full(o.shape, 60.0), np.ones(8)) / 60.0
    np.testing.assert_allclose((unit * unit).mean(axis=-1), 1.0, rtol=1e-12)
    # linear in the weight; rows and heads are independent
    assert rel(oracle.epilogue(o, z, 2.0 * w), 2.0 * a) < RTOL
    assert rel(oracle.epilogue(o[:, 2:3, 1:2], z[:, 2:3, 1:2], w), a[:, 2:3, 1:2]) < RTOL
    # silu(z) + silu(-z) = z (2 sigma(z) - 1) ... pinned through silu(z) - silu(-z) = z
    c = oracle.epilogue(o, -z, w)
    assert rel(a - c, oracle.epilogue(o, np.full(o.shape, 60.0), w) / 60.0 * z) < 1e-12
