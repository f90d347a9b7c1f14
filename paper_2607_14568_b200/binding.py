"""ctypes binding of libgdn.so.  Names and argument order follow include/gdn.h.

Tensors are ``torch`` tensors (used only for device memory and streams); they are
passed as raw pointers.  ``T`` is taken from the tensors: ``q`` is ``[B,T,H,d_k]``,
or packed ``[T,H,d_k]`` when ``cu_seqlens`` (an int32 tensor with one entry more
than there are sequences) is given.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libgdn.so")
_lib = None


class GdnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({gdn_status_string(status)})")


def lib_path() -> str:
    return _LIB_PATH


def lib():
    """The loaded library; raises if it has not been built (no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with "
                               "`python -m paper_2607_14568_b200.build` (there is no CPU fallback)")
        L = ctypes.CDLL(_LIB_PATH)
        vp, ip, i, sz = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        prefill = [vp] * 8 + [ip] + [i] * 6 + [vp]
        for name in ("gdn_chunk_prefill", "gdn_chunk_prefill_f32", "gdn_chunk_prefill_bf16_simt",
                     "gdn_chunk_prefill_noalloc"):
            getattr(L, name).argtypes = prefill
            getattr(L, name).restype = i
        L.gdn_chunk_prefill_host.argtypes = [vp] * 8 + [ip] + [i] * 6 + [vp, sz, vp]
        L.gdn_chunk_prefill_host.restype = i
        L.gdn_host_staging_bytes.argtypes = [i] * 5
        L.gdn_host_staging_bytes.restype = sz
        L.gdn_decode_step.argtypes = [vp] * 7 + [i] * 4 + [vp]
        L.gdn_decode_step.restype = i
        L.gdn_chunk_prefill_snapshots.argtypes = [vp] * 8 + [i] * 7 + [vp, vp]
        L.gdn_chunk_prefill_snapshots.restype = i
        L.gdn_chunk_prefill_raw.argtypes = [vp] * 5 + [ctypes.c_float] * 2 + [vp] * 4 + [i] * 6 + [vp]
        L.gdn_chunk_prefill_raw.restype = i
        L.gdn_chunk_prefill_gated.argtypes = [vp] * 8 + [ctypes.c_float] + [vp] * 3 + [i] * 6 + [vp]
        L.gdn_chunk_prefill_gated.restype = i
        L.gdn_attn_causal_prefill.argtypes = [vp] * 5 + [i] * 5 + [ctypes.c_float, vp]
        L.gdn_attn_causal_prefill.restype = i
        L.gdn_workspace_bytes.argtypes = [i] * 7
        L.gdn_workspace_bytes.restype = sz
        L.gdn_set_workspace.argtypes = [vp, sz]
        L.gdn_set_workspace.restype = i
        L.gdn_debug_force_path.argtypes = [i]
        L.gdn_debug_force_path.restype = None
        L.gdn_debug_drop_chunk.argtypes = [i]
        L.gdn_debug_drop_chunk.restype = None
        L.gdn_debug_reset_status.argtypes = []
        L.gdn_debug_reset_status.restype = i
        L.gdn_debug_set_timing.argtypes = [i]
        L.gdn_debug_set_timing.restype = i
        L.gdn_debug_get_timing.argtypes = [ctypes.POINTER(ctypes.c_float)]
        L.gdn_debug_get_timing.restype = i
        L.gdn_debug_force_segments.argtypes = [i]
        L.gdn_debug_force_segments.restype = None
        L.gdn_debug_set_scan.argtypes = [i]
        L.gdn_debug_set_scan.restype = None
        L.gdn_query_status.argtypes = []
        L.gdn_query_status.restype = i
        L.gdn_query_status_stream.argtypes = [vp]
        L.gdn_query_status_stream.restype = i
        L.gdn_debug_set_l2_hints.argtypes = [i]
        L.gdn_debug_set_l2_hints.restype = None
        L.gdn_debug_set_chain_stamps.argtypes = [vp]
        L.gdn_debug_set_chain_stamps.restype = None
        L.gdn_debug_set_dump.argtypes = [vp]
        L.gdn_debug_set_dump.restype = None
        L.gdn_launch_count.argtypes = []
        L.gdn_launch_count.restype = ctypes.c_ulonglong
        L.gdn_status_string.argtypes = [i]
        L.gdn_status_string.restype = ctypes.c_char_p
        _lib = L
    return _lib


def gdn_status_string(status: int) -> str:
    return lib().gdn_status_string(int(status)).decode()


def gdn_workspace_bytes(B: int, T: int, H: int, d_k: int, d_v: int, packed: bool = False, chunk: int = 64) -> int:
    return int(lib().gdn_workspace_bytes(B, T, H, d_k, d_v, int(chunk), 1 if packed else 0))


_workspace_ref = None


def gdn_set_workspace(workspace: Optional[torch.Tensor]) -> None:
    """Hands the library a CUDA tensor to use as scratch (or None to remove it).  The binding
    keeps a reference so the memory outlives the calls that use it."""
    global _workspace_ref
    if workspace is None:
        rc = lib().gdn_set_workspace(None, 0)
    else:
        if workspace.device.type != "cuda" or not workspace.is_contiguous():
            raise ValueError("workspace must be a contiguous CUDA tensor")
        rc = lib().gdn_set_workspace(ctypes.c_void_p(workspace.data_ptr()),
                                     workspace.numel() * workspace.element_size())
    if rc != 0:
        raise GdnError(rc, "gdn_set_workspace")
    _workspace_ref = workspace


def gdn_query_status() -> int:
    """Synchronises the device and returns the kernels' status word (0 = ok)."""
    return int(lib().gdn_query_status())


def gdn_query_status_stream(stream=None) -> int:
    """Waits for `stream` only (default: torch's current stream) and returns the kernels' status word."""
    return int(lib().gdn_query_status_stream(_stream(stream)))


def gdn_launch_count() -> int:
    return int(lib().gdn_launch_count())


def gdn_host_staging_bytes(B: int, T: int, H: int, d_k: int, d_v: int) -> int:
    return int(lib().gdn_host_staging_bytes(B, T, H, d_k, d_v))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _dims(q, v, cu_seqlens):
    if cu_seqlens is None:
        B, T, H, d_k = q.shape
    else:
        T, H, d_k = q.shape
        B = cu_seqlens.numel() - 1
    return int(B), int(T), int(H), int(d_k), int(v.shape[-1])


def _check(ts, dtype, device_type):
    for name, t, dt in ts:
        if t is None:
            continue
        if not t.is_contiguous():
            raise ValueError(f"{name} must be contiguous")
        if t.dtype != dt:
            raise ValueError(f"{name} must be {dt}, got {t.dtype}")
        if t.device.type != device_type:
            raise ValueError(f"{name} must live on {device_type}, got {t.device}")


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _prefill(fn_name, io_dtype, q, k, v, log_alpha, beta, initial_state, out, final_state,
             cu_seqlens, chunk, stream):
    f32 = torch.float32
    _check([("q", q, io_dtype), ("k", k, io_dtype), ("v", v, io_dtype), ("out", out, io_dtype),
            ("log_alpha", log_alpha, f32), ("beta", beta, f32), ("initial_state", initial_state, f32),
            ("final_state", final_state, f32), ("cu_seqlens", cu_seqlens, torch.int32)], io_dtype, "cuda")
    B, T, H, d_k, d_v = _dims(q, v, cu_seqlens)
    if k.shape != q.shape or v.shape[:-1] != q.shape[:-1] or out.shape != v.shape:
        raise ValueError("q, k, v, out shapes disagree")
    if log_alpha.shape != q.shape[:-1] or beta.shape != q.shape[:-1]:
        raise ValueError("gate shapes disagree with q")
    for name, s in (("initial_state", initial_state), ("final_state", final_state)):
        if s is not None and tuple(s.shape) != (B, H, d_k, d_v):
            raise ValueError(f"{name} must be [B,H,d_k,d_v]")
    rc = getattr(lib(), fn_name)(_ptr(q), _ptr(k), _ptr(v), _ptr(log_alpha), _ptr(beta), _ptr(initial_state),
                                 _ptr(out), _ptr(final_state), _ptr(cu_seqlens), B, T, H, d_k, d_v,
                                 int(chunk), _stream(stream))
    if rc != 0:
        raise GdnError(rc, fn_name)
    return out, final_state


def gdn_chunk_prefill(q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens=None,
                      chunk: int = 64, stream=None):
    """bf16 q/k/v/out; see ``gdn_chunk_prefill`` in include/gdn.h."""
    return _prefill("gdn_chunk_prefill", torch.bfloat16, q, k, v, log_alpha, beta, initial_state, out,
                    final_state, cu_seqlens, chunk, stream)


def gdn_chunk_prefill_f32(q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens=None,
                          chunk: int = 64, stream=None):
    """fp32 q/k/v/out, fp32 arithmetic; see include/gdn.h."""
    return _prefill("gdn_chunk_prefill_f32", torch.float32, q, k, v, log_alpha, beta, initial_state, out,
                    final_state, cu_seqlens, chunk, stream)


def gdn_chunk_prefill_bf16_simt(q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens=None,
                                chunk: int = 64, stream=None):
    """bf16 q/k/v/out through the fp32-arithmetic kernel; see include/gdn.h."""
    return _prefill("gdn_chunk_prefill_bf16_simt", torch.bfloat16, q, k, v, log_alpha, beta, initial_state,
                    out, final_state, cu_seqlens, chunk, stream)


def gdn_chunk_prefill_noalloc(q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens=None,
                              chunk: int = 64, stream=None):
    """gdn_chunk_prefill on the library's built-in 64 MiB scratch: for callers that have no way to
    allocate device memory (see include/gdn.h).  Raises GdnError with status 6 when the problem
    does not fit.  Make the first call on a device outside stream capture; do not overlap calls."""
    return _prefill("gdn_chunk_prefill_noalloc", torch.bfloat16, q, k, v, log_alpha, beta, initial_state,
                    out, final_state, cu_seqlens, chunk, stream)


def gdn_chunk_prefill_snapshots(q, k, v, log_alpha, beta, initial_state, out, final_state, snapshot_every_chunks,
                                snapshots, chunk: int = 64, stream=None):
    """gdn_chunk_prefill (batched input) that also writes the state after every ``snapshot_every_chunks``
    chunks into ``snapshots`` [B, n_snap, H, d_k, d_v] fp32.  Needs gdn_set_workspace.  See include/gdn.h."""
    f32, bf = torch.float32, torch.bfloat16
    _check([("q", q, bf), ("k", k, bf), ("v", v, bf), ("out", out, bf), ("log_alpha", log_alpha, f32),
            ("beta", beta, f32), ("initial_state", initial_state, f32), ("final_state", final_state, f32),
            ("snapshots", snapshots, f32)], bf, "cuda")
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    n_snap = (T // 64) // int(snapshot_every_chunks)
    if tuple(snapshots.shape) != (B, n_snap, H, d_k, d_v):
        raise ValueError("snapshots must be [B, (T//64)//every, H, d_k, d_v]")
    rc = lib().gdn_chunk_prefill_snapshots(_ptr(q), _ptr(k), _ptr(v), _ptr(log_alpha), _ptr(beta),
                                           _ptr(initial_state), _ptr(out), _ptr(final_state), int(B), int(T), int(H),
                                           int(d_k), int(d_v), int(chunk), int(snapshot_every_chunks),
                                           _ptr(snapshots), _stream(stream))
    if rc != 0:
        raise GdnError(rc, "gdn_chunk_prefill_snapshots")
    return out, final_state, snapshots


def gdn_chunk_prefill_raw(q_raw, k_raw, v, a_raw, b_raw, gate_scale, norm_eps, initial_state, out, final_state,
                          cu_seqlens=None, chunk: int = 64, stream=None):
    """gdn_chunk_prefill on raw projections: the L2 norms of q, k and the gates sigmoid(b_raw),
    -softplus(a_raw) * gate_scale are computed inside the kernels.  Needs gdn_set_workspace.  See include/gdn.h."""
    f32, bf = torch.float32, torch.bfloat16
    _check([("q_raw", q_raw, bf), ("k_raw", k_raw, bf), ("v", v, bf), ("out", out, bf), ("a_raw", a_raw, f32),
            ("b_raw", b_raw, f32), ("initial_state", initial_state, f32), ("final_state", final_state, f32),
            ("cu_seqlens", cu_seqlens, torch.int32)], bf, "cuda")
    B, T, H, d_k, d_v = _dims(q_raw, v, cu_seqlens)
    if k_raw.shape != q_raw.shape or v.shape[:-1] != q_raw.shape[:-1] or out.shape != v.shape:
        raise ValueError("q, k, v, out shapes disagree")
    if a_raw.shape != q_raw.shape[:-1] or b_raw.shape != q_raw.shape[:-1]:
        raise ValueError("gate shapes disagree with q")
    for name, s in (("initial_state", initial_state), ("final_state", final_state)):
        if s is not None and tuple(s.shape) != (B, H, d_k, d_v):
            raise ValueError(f"{name} must be [B,H,d_k,d_v]")
    rc = lib().gdn_chunk_prefill_raw(_ptr(q_raw), _ptr(k_raw), _ptr(v), _ptr(a_raw), _ptr(b_raw), float(gate_scale),
                                     float(norm_eps), _ptr(initial_state), _ptr(out), _ptr(final_state),
                                     _ptr(cu_seqlens), B, T, H, d_k, d_v, int(chunk), _stream(stream))
    if rc != 0:
        raise GdnError(rc, "gdn_chunk_prefill_raw")
    return out, final_state


def gdn_chunk_prefill_gated(q, k, v, log_alpha, beta, initial_state, gate_z, norm_weight, norm_eps, out, final_state,
                            cu_seqlens=None, chunk: int = 64, stream=None):
    """gdn_chunk_prefill with the output stage fused in: out = o / sqrt(mean o^2 + norm_eps) * norm_weight * silu(gate_z)
    per (token, head); gate_z bf16 like out, norm_weight fp32 [d_v].  Needs gdn_set_workspace.  See include/gdn.h."""
    f32, bf = torch.float32, torch.bfloat16
    _check([("q", q, bf), ("k", k, bf), ("v", v, bf), ("out", out, bf), ("gate_z", gate_z, bf), ("log_alpha", log_alpha, f32),
            ("beta", beta, f32), ("initial_state", initial_state, f32), ("final_state", final_state, f32),
            ("norm_weight", norm_weight, f32), ("cu_seqlens", cu_seqlens, torch.int32)], bf, "cuda")
    B, T, H, d_k, d_v = _dims(q, v, cu_seqlens)
    if k.shape != q.shape or v.shape[:-1] != q.shape[:-1] or out.shape != v.shape or gate_z.shape != out.shape:
        raise ValueError("q, k, v, gate_z, out shapes disagree")
    if log_alpha.shape != q.shape[:-1] or beta.shape != q.shape[:-1] or tuple(norm_weight.shape) != (d_v,):
        raise ValueError("gate or weight shapes disagree with q, v")
    rc = lib().gdn_chunk_prefill_gated(_ptr(q), _ptr(k), _ptr(v), _ptr(log_alpha), _ptr(beta), _ptr(initial_state),
                                       _ptr(gate_z), _ptr(norm_weight), float(norm_eps), _ptr(out), _ptr(final_state),
                                       _ptr(cu_seqlens), B, T, H, d_k, d_v, int(chunk), _stream(stream))
    if rc != 0:
        raise GdnError(rc, "gdn_chunk_prefill_gated")
    return out, final_state


def gdn_attn_causal_prefill(q, k, v, out, scale=None, cu_seqlens=None, stream=None):
    """Causal softmax attention with grouped queries: q, out [B,T,Hq,d], k, v [B,T,Hkv,d] bf16 on the device
    (packed [T,H,d] with int32 cu_seqlens [B+1]); scale defaults to 1/sqrt(d).  See include/gdn_attn.h."""
    bf = torch.bfloat16
    _check([("q", q, bf), ("k", k, bf), ("v", v, bf), ("out", out, bf), ("cu_seqlens", cu_seqlens, torch.int32)],
           bf, "cuda")
    nd = 4 if cu_seqlens is None else 3
    if q.dim() != nd or k.dim() != nd or v.shape != k.shape or out.shape != q.shape or q.shape[:-2] != k.shape[:-2] \
            or q.shape[-1] != k.shape[-1]:
        raise ValueError("q, out [B,T,Hq,d] and k, v [B,T,Hkv,d] expected (packed: [T,H,d])")
    if cu_seqlens is None:
        B, T = q.shape[0], q.shape[1]
    else:
        B, T = cu_seqlens.numel() - 1, q.shape[0]
    Hq, d = q.shape[-2], q.shape[-1]
    if scale is None:
        scale = 1.0 / float(d) ** 0.5
    rc = lib().gdn_attn_causal_prefill(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(cu_seqlens), int(B), int(T), int(Hq),
                                       int(k.shape[-2]), int(d), float(scale), _stream(stream))
    if rc != 0:
        raise GdnError(rc, "gdn_attn_causal_prefill")
    return out


def gdn_decode_step(q, k, v, log_alpha, beta, state, out, stream=None):
    """One token per sequence: q, k [B,H,d_k], v, out [B,H,d_v] bf16; log_alpha, beta [B,H] fp32;
    state [B,H,d_k,d_v] fp32, updated in place.  See include/gdn.h."""
    f32, bf = torch.float32, torch.bfloat16
    _check([("q", q, bf), ("k", k, bf), ("v", v, bf), ("out", out, bf), ("log_alpha", log_alpha, f32),
            ("beta", beta, f32), ("state", state, f32)], bf, "cuda")
    B, H, d_k = q.shape
    d_v = v.shape[-1]
    if k.shape != q.shape or tuple(v.shape) != (B, H, d_v) or out.shape != v.shape:
        raise ValueError("q, k, v, out shapes disagree")
    if tuple(log_alpha.shape) != (B, H) or tuple(beta.shape) != (B, H) or tuple(state.shape) != (B, H, d_k, d_v):
        raise ValueError("gate or state shapes disagree with q, v")
    rc = lib().gdn_decode_step(_ptr(q), _ptr(k), _ptr(v), _ptr(log_alpha), _ptr(beta), _ptr(state), _ptr(out),
                               int(B), int(H), int(d_k), int(d_v), _stream(stream))
    if rc != 0:
        raise GdnError(rc, "gdn_decode_step")
    return out, state


def gdn_chunk_prefill_host(q, k, v, log_alpha, beta, initial_state, out, final_state, cu_seqlens,
                           staging: torch.Tensor, chunk: int = 64, stream=None):
    """Host (CPU, ideally pinned) tensors in and out; ``staging`` is a CUDA uint8 tensor of at
    least ``gdn_host_staging_bytes`` bytes.  Work is enqueued on ``stream``; synchronise it before
    reading ``out``."""
    f32, bf = torch.float32, torch.bfloat16
    _check([("q", q, bf), ("k", k, bf), ("v", v, bf), ("out", out, bf), ("log_alpha", log_alpha, f32),
            ("beta", beta, f32), ("initial_state", initial_state, f32), ("final_state", final_state, f32),
            ("cu_seqlens", cu_seqlens, torch.int32)], bf, "cpu")
    if staging.device.type != "cuda" or not staging.is_contiguous():
        raise ValueError("staging must be a contiguous CUDA tensor")
    B, T, H, d_k, d_v = _dims(q, v, cu_seqlens)
    rc = lib().gdn_chunk_prefill_host(_ptr(q), _ptr(k), _ptr(v), _ptr(log_alpha), _ptr(beta),
                                      _ptr(initial_state), _ptr(out), _ptr(final_state), _ptr(cu_seqlens),
                                      B, T, H, d_k, d_v, int(chunk), _ptr(staging),
                                      staging.numel() * staging.element_size(), _stream(stream))
    if rc != 0:
        raise GdnError(rc, "gdn_chunk_prefill_host")
    return out, final_state
