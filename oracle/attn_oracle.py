"""fp64 CPU oracle for causal softmax attention with grouped queries (test infrastructure only).

Sections "The layout trick" and "Prefill attention: finding and removing the O(N^2) wall" of the
paper rewrite the prefill attention of the softmax layers as per-head matrix products: scores S = Q K^T for the whole chunk, a column softmax that normalises
only the causally valid prefix and zeroes the tail, then a second product with V; several query
heads share one key/value head by addressing the same K/V block.

  attention_causal     the definition, one (query row, head) at a time: softmax over keys 0..i
  attention_causal_rows  the same definition for a list of (sequence, position, head) triples
  attention_gemm_form  the paper's order of steps: full rectangular score product, masked softmax
                       that normalises the valid prefix and writes exact zeros beyond it, full
                       rectangular product with V
Layouts: q [B,T,Hq,d], k, v [B,T,Hkv,d], out [B,T,Hq,d]; query head h reads key/value head
h // (Hq // Hkv).  `scale` multiplies the scores (the usual choice is 1/sqrt(d)).  With cu_seqlens the
tensors are packed [T,H,d] and every sequence attends to itself only.  Plain numpy.
"""
from __future__ import annotations

import numpy as np


def _f64(x):
    return np.ascontiguousarray(np.asarray(x), dtype=np.float64)


def _check(q, k, v):
    if q.ndim != 4 or k.ndim != 4 or v.shape != k.shape or q.shape[:2] != k.shape[:2] or q.shape[3] != k.shape[3]:
        raise ValueError("q [B,T,Hq,d], k, v [B,T,Hkv,d] expected")
    if q.shape[2] % k.shape[2] != 0:
        raise ValueError("Hq must be a multiple of Hkv")


def attention_causal(q, k, v, scale, cu_seqlens=None):
    q, k, v = _f64(q), _f64(k), _f64(v)
    if cu_seqlens is not None:          # packed [T,H,d]: every sequence on its own
        cu = [int(x) for x in np.asarray(cu_seqlens)]
        out = np.zeros(q.shape[:-1] + (v.shape[-1],))
        for a, b in zip(cu[:-1], cu[1:]):
            if b > a:
                out[a:b] = attention_causal(q[None, a:b], k[None, a:b], v[None, a:b], scale)[0]
        return out
    _check(q, k, v)
    B, T, Hq, d = q.shape
    group = Hq // k.shape[2]
    out = np.zeros((B, T, Hq, v.shape[3]))
    for b in range(B):
        for h in range(Hq):
            kh, vh = k[b, :, h // group], v[b, :, h // group]
            for i in range(T):
                s = (kh[: i + 1] @ q[b, i, h]) * float(scale)      # scores of query i against keys 0..i
                p = np.exp(s - s.max())
                out[b, i, h] = (p / p.sum()) @ vh[: i + 1]
    return out


def attention_causal_rows(q, k, v, scale, rows):
    """attention_causal for the listed (b, i, h) triples only: returns [len(rows), d] (full-size spot checks)."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    _check(q, k, v)
    group = q.shape[2] // k.shape[2]
    out = np.zeros((len(rows), v.shape[3]))
    for n, (b, i, h) in enumerate(rows):
        s = (k[b, : i + 1, h // group] @ q[b, i, h]) * float(scale)
        p = np.exp(s - s.max())
        out[n] = (p / p.sum()) @ v[b, : i + 1, h // group]
    return out


def attention_gemm_form(q, k, v, scale):
    q, k, v = _f64(q), _f64(k), _f64(v)
    _check(q, k, v)
    B, T, Hq, d = q.shape
    group = Hq // k.shape[2]
    out = np.zeros((B, T, Hq, v.shape[3]))
    for b in range(B):
        for h in range(Hq):
            kh, vh = k[b, :, h // group], v[b, :, h // group]
            S = (q[b, :, h] @ kh.T) * float(scale)                 # the full rectangle, garbage above the diagonal
            P = np.zeros_like(S)
            for i in range(T):                                     # normalise the valid prefix, zero the tail
                row = S[i, : i + 1]
                e = np.exp(row - row.max())
                P[i, : i + 1] = e / e.sum()
            out[b, :, h] = P @ vh                                  # full rectangle again: the tail multiplies zeros
    return out
