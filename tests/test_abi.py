"""The C-ABI library builds, loads without a GPU, and exports every symbol its header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2607_14568_b200 import build
    return build.build()


def declared_functions():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if not fn.endswith(".h"):
            continue
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(gdn_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_header_symbols_exported(libpath):
    names = declared_functions()
    assert "gdn_chunk_prefill" in names and len(names) >= 6
    lib = ctypes.CDLL(libpath)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/ but not exported"


def test_binding_has_the_same_names(libpath):
    import paper_2607_14568_b200 as gdn
    for n in declared_functions():
        assert hasattr(gdn, n), f"binding lacks {n}"
    assert gdn.gdn_status_string(0) == "ok" and gdn.gdn_status_string(5)
    assert gdn.gdn_host_staging_bytes(1, 64, 1, 128, 128) > 0
    assert gdn.gdn_host_staging_bytes(0, 64, 1, 128, 128) == 0


def test_host_entry_rejects_bad_arguments_without_a_gpu(libpath):
    """Argument checks of the host-buffer entry point run before any CUDA call."""
    import numpy as np
    lib = ctypes.CDLL(libpath)
    lib.gdn_chunk_prefill_host.restype = ctypes.c_int
    buf = np.zeros(64 * 128, dtype=np.uint16)
    p = buf.ctypes.data_as(ctypes.c_void_p)
    vp = ctypes.c_void_p
    # NULL staging -> invalid argument
    rc = lib.gdn_chunk_prefill_host(p, p, p, p, p, None, p, None, None, 1, 64, 1, 128, 128, 64, None,
                                    ctypes.c_size_t(0), None)
    assert rc == 1
    # staging too small -> workspace error (pointer is never dereferenced)
    rc = lib.gdn_chunk_prefill_host(p, p, p, p, p, None, p, None, None, 1, 64, 1, 128, 128, 64, vp(256),
                                    ctypes.c_size_t(16), None)
    assert rc == 3
    cu = np.array([0, 70], dtype=np.int32)
    rc = lib.gdn_chunk_prefill_host(p, p, p, p, p, None, p, None, cu.ctypes.data_as(vp), 1, 64, 1, 128, 128, 64,
                                    vp(256), ctypes.c_size_t(1 << 30), None)
    assert rc == 1   # cu_seqlens[B] != T


def test_widened_entry_points_reject_bad_arguments_without_a_gpu(libpath):
    """The argument checks of the attention, snapshot and raw-projection entry points come before any
    CUDA call, so they can be exercised on a machine without a GPU (pointers are never dereferenced)."""
    lib = ctypes.CDLL(libpath)
    vp, f = ctypes.c_void_p, ctypes.c_float
    p = vp(4096)                                                    # aligned, never dereferenced
    attn = lib.gdn_attn_causal_prefill
    attn.restype = ctypes.c_int
    attn.argtypes = [vp] * 5 + [ctypes.c_int] * 5 + [f, vp]
    assert attn(p, p, p, p, None, -1, 64, 2, 1, 128, 0.1, None) == 1       # negative B
    assert attn(p, p, p, p, None, 1, 64, 2, 1, 128, -0.1, None) == 1       # negative scale
    assert attn(p, p, p, p, None, 1, 64, 2, 1, 128, float("nan"), None) == 1
    assert attn(None, p, p, p, None, 1, 64, 2, 1, 128, 0.1, None) == 1     # null q
    assert attn(vp(4100), p, p, p, None, 1, 64, 2, 1, 128, 0.1, None) == 2  # misaligned
    assert attn(p, p, p, p, None, 1, 64, 3, 2, 128, 0.1, None) == 2        # 3 query heads on 2 kv heads
    assert attn(p, p, p, p, None, 1, 64, 2, 1, 64, 0.1, None) == 2         # d = 64
    assert attn(p, p, p, p, None, 0, 64, 2, 1, 128, 0.1, None) == 0        # empty batch: nothing to do
    raw = lib.gdn_chunk_prefill_raw
    raw.restype = ctypes.c_int
    raw.argtypes = [vp] * 5 + [f, f] + [vp] * 4 + [ctypes.c_int] * 6 + [vp]
    assert raw(p, p, p, p, p, -1.0, 0.0, None, p, None, None, 1, 64, 1, 128, 128, 64, None) == 1   # negative gate scale
    assert raw(p, p, p, p, p, 0.05, -1.0, None, p, None, None, 1, 64, 1, 128, 128, 64, None) == 1  # negative eps
    assert raw(p, p, p, p, p, 0.05, 0.0, None, p, None, None, 1, 64, 1, 128, 128, 32, None) == 2   # chunk != 64
    assert raw(p, p, p, p, p, 0.05, 0.0, None, p, None, None, 1, 64, 1, 64, 64, 64, None) == 2     # d = 64
    assert raw(p, p, p, p, p, 0.05, 0.0, None, p, None, None, 1, 64, 1, 128, 128, 64, None) == 3   # no workspace set
    snap = lib.gdn_chunk_prefill_snapshots
    snap.restype = ctypes.c_int
    snap.argtypes = [vp] * 8 + [ctypes.c_int] * 7 + [vp, vp]
    assert snap(p, p, p, p, p, None, p, None, 1, 128, 1, 128, 128, 64, 0, p, None) == 1            # every 0 chunks
    assert snap(p, p, p, p, p, None, p, None, 1, 128, 1, 128, 128, 64, 1, None, None) == 1         # no snapshot buffer
    assert snap(p, p, p, p, p, None, p, None, 1, 128, 1, 128, 128, 64, 1, p, None) == 3            # no workspace set


def test_workspace_query_takes_the_chunk_and_rejects_unsupported_tilings(libpath):
    lib = ctypes.CDLL(libpath)
    lib.gdn_workspace_bytes.restype = ctypes.c_size_t
    lib.gdn_workspace_bytes.argtypes = [ctypes.c_int] * 7
    full = lib.gdn_workspace_bytes(1, 10240, 16, 128, 128, 64, 0)
    assert full > 160 * 16 * 34048                                 # items of every (chunk, head) plus the split scratch
    assert lib.gdn_workspace_bytes(1, 10240, 16, 128, 128, 32, 0) == 0      # only 64-token chunks
    assert lib.gdn_workspace_bytes(1, 10240, 16, 64, 64, 64, 0) == 0        # sizes of the fp32 path need no scratch
    packed = lib.gdn_workspace_bytes(8, 34000, 16, 128, 128, 64, 1)
    assert 0 < packed < full * 4
