"""ctypes front end of the fp64 CPU oracle (test infrastructure only).

Every function takes numpy arrays of any float dtype, widens them exactly to
fp64, and returns ``(out, final_state)`` as fp64 arrays.  Layouts are those of
the C file: ``q,k [B,T,H,d_k]``, ``v [B,T,H,d_v]``, ``log_alpha,beta [B,T,H]``,
``initial_state [N,H,d_k,d_v]``; with ``cu_seqlens`` the tensors are packed
``[T_total,H,.]`` and ``N = len(cu_seqlens) - 1``.

  sequential  the token-by-token recurrence (the definition; Section "A chunked
              delta-rule scan for the recurrent layers")
  chunked     the intra-/inter-chunk form of the same section (form=1: its
              S' = M S + N variant)
  dense       the whole sequence as one general linear system (brute force)
  chunked_stages  the chunked form for one (sequence, head) chain, also returning its per-chunk
              intermediates (g, A, P, T, W, U, Delta, incoming state): stage-by-stage references in the
              sense of Section "Porting the Vision Tower, Stage by Stage"
  prologue    the per-position kernels in front of the scan (Section "Prefill projections: dequantize, then call the vendor":
              norms and gating batched over the chunk): L2 norm of q and k over the feature
              axis, beta = sigmoid(b), log_alpha = -softplus(a) * gate_scale.  The paper names
              these kernels without printing formulas; the forms here are the reading the
              benchmark inputs were drawn with.  Plain numpy, fp64.
  epilogue    the per-position kernels behind the scan (same section: "norms ... gating" are batched
              over the chunk): a root-mean-square norm of each output row over the value axis with a
              learned weight vector, multiplied by the SiLU of a gate tensor.  Again the paper prints no
              formula; this is the reading recorded for the fused output stage.  Plain numpy, fp64.
"""
from __future__ import annotations

import ctypes

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int32)
        common = [dp, dp, dp, dp, dp, dp, dp, dp, ip] + [ctypes.c_int] * 5
        lib.gdn_oracle_sequential.argtypes = common
        lib.gdn_oracle_dense.argtypes = common
        lib.gdn_oracle_chunked.argtypes = common + [ctypes.c_int, ctypes.c_int]
        lib.gdn_oracle_chunked_stages.argtypes = common + [ctypes.c_int] * 3 + [dp] * 8
        for f in (lib.gdn_oracle_sequential, lib.gdn_oracle_dense, lib.gdn_oracle_chunked,
                  lib.gdn_oracle_chunked_stages, lib.gdn_oracle_num_threads):
            f.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().gdn_oracle_num_threads())


def _f64(x):
    return np.ascontiguousarray(np.asarray(x), dtype=np.float64)


def _ptr(x):
    return None if x is None else x.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _prepare(q, k, v, log_alpha, beta, initial_state, cu_seqlens):
    q, k, v, a, b = (_f64(x) for x in (q, k, v, log_alpha, beta))
    if cu_seqlens is None:
        if q.ndim != 4:
            raise ValueError("q must be [B,T,H,d_k] without cu_seqlens")
        B, T, H, dk = q.shape
        N = B
        cu = None
    else:
        if q.ndim != 3:
            raise ValueError("q must be packed [T,H,d_k] with cu_seqlens")
        T, H, dk = q.shape
        cu = np.ascontiguousarray(np.asarray(cu_seqlens), dtype=np.int32)
        B = N = cu.shape[0] - 1
    dv = v.shape[-1]
    if k.shape != q.shape or v.shape[:-1] != q.shape[:-1]:
        raise ValueError("q, k, v shapes disagree")
    if a.shape != q.shape[:-1] or b.shape != q.shape[:-1]:
        raise ValueError("gate shapes disagree with q")
    s0 = None
    if initial_state is not None:
        s0 = _f64(initial_state)
        if s0.shape != (N, H, dk, dv):
            raise ValueError("initial_state must be [N,H,d_k,d_v]")
    out = np.empty(v.shape, dtype=np.float64)
    fin = np.empty((N, H, dk, dv), dtype=np.float64)
    return (q, k, v, a, b, s0, out, fin, cu), (B, T, H, dk, dv)


def _call(fn, arrs, dims, *extra):
    q, k, v, a, b, s0, out, fin, cu = arrs
    cup = None if cu is None else cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    rc = fn(_ptr(q), _ptr(k), _ptr(v), _ptr(a), _ptr(b), _ptr(s0), _ptr(out), _ptr(fin),
            cup, *dims, *extra)
    if rc != 0:
        raise ValueError(f"oracle rejected its arguments (code {rc})")
    return out, fin


def sequential(q, k, v, log_alpha, beta, initial_state=None, cu_seqlens=None):
    arrs, dims = _prepare(q, k, v, log_alpha, beta, initial_state, cu_seqlens)
    return _call(_load().gdn_oracle_sequential, arrs, dims)


def chunked(q, k, v, log_alpha, beta, initial_state=None, cu_seqlens=None, chunk=64, form=0):
    arrs, dims = _prepare(q, k, v, log_alpha, beta, initial_state, cu_seqlens)
    return _call(_load().gdn_oracle_chunked, arrs, dims, int(chunk), int(form))


def chunked_stages(q, k, v, log_alpha, beta, initial_state=None, cu_seqlens=None, chunk=64, n=0, h=0):
    """The chunked form (form 0) of chain (n, h) with its intermediates.  Returns a dict of fp64 arrays, nch =
    number of chunks of the sequence: g [nch,C], A, P, T [nch,C,C], W [nch,C,d_k], U, Delta [nch,C,d_v],
    S_in [nch,d_k,d_v] (the state each chunk starts from), out [len,d_v], final_state [d_k,d_v], length.
    Rows beyond the length of a tail chunk are zero."""
    arrs, dims = _prepare(q, k, v, log_alpha, beta, initial_state, cu_seqlens)
    B, T, H, dk, dv = dims
    cu = arrs[8]
    length = int(cu[n + 1] - cu[n]) if cu is not None else T
    tok0 = int(cu[n]) if cu is not None else n * T
    C = int(chunk)
    nch = (length + C - 1) // C
    z = lambda *shape: np.zeros(shape, dtype=np.float64)
    st = dict(g=z(nch, C), A=z(nch, C, C), P=z(nch, C, C), T=z(nch, C, C), W=z(nch, C, dk), U=z(nch, C, dv),
              Delta=z(nch, C, dv), S_in=z(nch, dk, dv))
    out, fin = _call(_load().gdn_oracle_chunked_stages, arrs, dims, C, int(n), int(h),
                     *[_ptr(st[name]) for name in ("g", "A", "P", "T", "W", "U", "Delta", "S_in")])
    flat = out.reshape(-1, H, dv)
    st.update(out=flat[tok0:tok0 + length, h].copy(), final_state=fin[n, h].copy(), length=length)
    return st


def dense(q, k, v, log_alpha, beta, initial_state=None, cu_seqlens=None):
    arrs, dims = _prepare(q, k, v, log_alpha, beta, initial_state, cu_seqlens)
    return _call(_load().gdn_oracle_dense, arrs, dims)


def prologue(q_raw, k_raw, a_raw, b_raw, gate_scale, eps=0.0):
    """(q, k, log_alpha, beta) in fp64 from raw projections:
    x / sqrt(sum_f x_f^2 + eps) per (token, head) for q and k, 1 / (1 + e^{-b}), -ln(1 + e^{a}) * gate_scale."""
    q_raw, k_raw, a_raw, b_raw = _f64(q_raw), _f64(k_raw), _f64(a_raw), _f64(b_raw)
    q = q_raw / np.sqrt((q_raw * q_raw).sum(axis=-1, keepdims=True) + float(eps))
    k = k_raw / np.sqrt((k_raw * k_raw).sum(axis=-1, keepdims=True) + float(eps))
    beta = 1.0 / (1.0 + np.exp(-b_raw))
    log_alpha = -np.log(1.0 + np.exp(a_raw)) * float(gate_scale)
    return q, k, log_alpha, beta


def epilogue(o, z, weight, eps=0.0):
    """Gated output norm per (token, head) over the value axis (last axis, length d_v):
    o / sqrt(mean_j o_j^2 + eps) * weight * silu(z),  silu(z) = z / (1 + e^{-z});  weight has shape [d_v]."""
    o, z, weight = _f64(o), _f64(z), _f64(weight)
    if z.shape != o.shape or weight.shape != (o.shape[-1],):
        raise ValueError("z must have the shape of o and weight the length of its last axis")
    rms = np.sqrt((o * o).mean(axis=-1, keepdims=True) + float(eps))
    return o / rms * weight * (z / (1.0 + np.exp(-z)))
