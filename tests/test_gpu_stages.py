"""Stage-gated parity (Section "Porting the Vision Tower, Stage by Stage": no stage is trusted until it
matches its own reference).  The intermediates of the CUDA path -- the scratch items the prepare kernel
writes (gate vectors, -W^T, (T diag beta)^T, P) and the fused kernel's dump of chunk 0 (T, W, the
correction Delta, the state update, the two output terms) -- are compared element by element with the
matching intermediates of the fp64 chunked oracle, each with the tolerance of the roundings that stage
contains.  A mistake in one step shows up at that step, not as a diffuse end-to-end error."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2607_14568_b200 as gdn
from workloads import get_config, make_inputs, widen

from gdn_testlib import errors, prefill_fused, to_device

pytestmark = pytest.mark.gpu

HEADER, ITEM = 4096, 34048          # workspace header and bytes per (chunk slot, head) item
LOG2E = 1.4426950408889634


def _bf16(raw_u16):
    return (raw_u16.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _unswizzle(img_bytes, rows, cols):
    """rows x cols bf16 image in 128-byte rows with 16-byte pieces XOR-ed by (row & 7), blocks of 64 rows x 64
    columns laid out [row block][column block] -> fp64 [rows, cols]."""
    u16 = np.frombuffer(img_bytes, dtype=np.uint16)
    out = np.empty((rows, cols))
    for rb in range(rows // 64):
        for cb in range(cols // 64):
            blk = u16[((rb * (cols // 64) + cb) * 4096):][:4096].reshape(64, 8, 8)     # [row][piece][8]
            for r in range(64):
                for piece in range(8):
                    out[rb * 64 + r, cb * 64 + 8 * piece: cb * 64 + 8 * piece + 8] = _bf16(blk[r, piece ^ (r & 7)])
    return out


def _close(got, want, rel_tol, what):
    assert np.isfinite(got).all(), what
    rel, mx = errors(got, want)
    assert rel <= rel_tol, f"{what}: rel-L2 {rel:.3e} > {rel_tol:.1e} (max-abs {mx:.3e})"


@pytest.mark.parametrize("T", [64, 130, 192])
def test_prepare_kernel_items_against_oracle_stages(T):
    cfg = get_config("long", T=T, H=2, init_std=0.3, seed=300 + T)
    x = make_inputs(cfg)
    d = to_device(x)
    ws = torch.zeros(gdn.gdn_workspace_bytes(1, T, cfg.H, cfg.d_k, cfg.d_v, False), dtype=torch.uint8, device="cuda")
    gdn.gdn_set_workspace(ws)
    gdn.lib().gdn_debug_force_path(2)
    try:
        gdn.gdn_chunk_prefill(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["initial_state"], d["out"],
                              d["final_state"])
        assert gdn.gdn_query_status_stream() == 0
    finally:
        gdn.lib().gdn_debug_force_path(0)
        gdn.gdn_set_workspace(None)
    raw = ws.cpu().numpy().tobytes()
    for h in range(cfg.H):
        st = oracle.chunked_stages(widen(x.q), widen(x.k), widen(x.v), x.log_alpha, x.beta, x.initial_state, None,
                                   chunk=64, n=0, h=h)
        beta = x.beta[0, :, h].astype(np.float64)
        for c in range((T + 63) // 64):
            R = min(64, T - 64 * c)
            item = raw[HEADER + (c * cfg.H + h) * ITEM:][:ITEM]          # slot of chunk c of sequence 0 is c
            gates = np.frombuffer(item[32768:32768 + 1280], dtype=np.float32).astype(np.float64)
            g = st["g"][c, :R]
            b = beta[64 * c: 64 * c + R]
            np.testing.assert_allclose(gates[0:R], g * LOG2E, rtol=2e-6, atol=2e-6)       # step a, fp32 sums
            np.testing.assert_allclose(gates[64:64 + R], b, rtol=0, atol=0)
            np.testing.assert_allclose(gates[128:128 + R], np.exp(g), rtol=1e-5)
            np.testing.assert_allclose(gates[192:192 + R], np.exp(g[-1] - g), rtol=1e-5)
            np.testing.assert_allclose(gates[256], np.exp(g[-1]), rtol=1e-5)
            if R < 64:          # identity padding: beta = 0 and no further decay
                assert not gates[64 + R:128].any()
                np.testing.assert_allclose(gates[R:64], g[-1] * LOG2E, rtol=2e-6, atol=2e-6)
            # step b1: P, one bf16 rounding of an fp32 value
            P = _unswizzle(item[24576:32768], 64, 64)
            _close(P[:R, :R], st["P"][c, :R, :R], 3e-3, f"P chunk {c} head {h}")
            assert not np.triu(P[:R, :R], 1).any()
            # step b2: (T diag beta)^T, fp32 solve (merges through 11-bit products) then one bf16 rounding
            T2 = _unswizzle(item[16384:24576], 64, 64).T                  # image rows are columns of T
            _close(T2[:R, :R], st["T"][c, :R, :R] * b[None, :], 3e-3, f"T diag(beta) chunk {c} head {h}")
            assert not np.triu(T2[:R, :R], 1).any()
            # step b3: -W^T, product of bf16 operands (one of them the rounded T diag(beta e^g)), rounded once more
            Wt = _unswizzle(item[0:16384], 128, 64)
            _close(-Wt.T[:R], st["W"][c, :R], 4e-3, f"W chunk {c} head {h}")
            assert not Wt.T[R:].any()                                     # padded rows contribute nothing


@pytest.mark.parametrize("T", [64, 40, 200])
def test_fused_kernel_stage_dump_of_chunk_0(T):
    cfg = get_config("long", T=T, H=1, init_std=0.3, seed=400 + T)
    x = make_inputs(cfg)
    d = to_device(x)
    dump = torch.zeros(8 * 16384, dtype=torch.float32, device="cuda")
    L = gdn.lib()
    L.gdn_debug_set_dump.argtypes = [ctypes.c_void_p]
    L.gdn_debug_set_dump(ctypes.c_void_p(dump.data_ptr()))
    try:
        prefill_fused(d["q"], d["k"], d["v"], d["log_alpha"], d["beta"], d["initial_state"], d["out"], d["final_state"])
    finally:
        L.gdn_debug_set_dump(None)
    t = dump.cpu().numpy().astype(np.float64)
    st = oracle.chunked_stages(widen(x.q), widen(x.k), widen(x.v), x.log_alpha, x.beta, x.initial_state, None,
                               chunk=64, n=0, h=0)
    R = min(64, T)
    k = widen(x.k)[0, :R, 0]
    q = widen(x.q)[0, :R, 0]
    g = st["g"][0, :R]
    S0 = st["S_in"][0]
    Tm = t[1 * 16384:][:4096].reshape(64, 64)
    np.testing.assert_allclose(Tm[:R, :R], st["T"][0, :R, :R], rtol=0, atol=2e-3 * np.abs(st["T"][0]).max())  # TF32 merges
    _close(Tm[:R, :R], st["T"][0, :R, :R], 1e-3, "T")
    Wt = t[2 * 16384:][:8192].reshape(128, 64)
    _close(Wt.T[:R], st["W"][0, :R], 3e-3, "W")
    Dt = t[3 * 16384:][:8192].reshape(128, 64)
    _close(Dt.T[:R], st["Delta"][0, :R], 4e-3, "Delta = U - W S")
    dSt = t[4 * 16384:][:16384].reshape(128, 128)                         # [j][m]
    dS = (np.exp(g[-1] - g)[:, None] * k).T @ st["Delta"][0, :R]          # [m][j]
    _close(dSt.T, dS, 5e-3, "state update K~^T Delta")
    O1t = t[5 * 16384:][:8192].reshape(128, 64)
    _close(O1t.T[:R], q @ S0, 3e-3, "Q S")
    O2t = t[6 * 16384:][:8192].reshape(128, 64)
    _close(O2t.T[:R], st["P"][0, :R, :R] @ st["Delta"][0, :R], 4e-3, "P Delta")
