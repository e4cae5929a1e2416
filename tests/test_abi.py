"""The C-ABI library loads and exports every symbol the header declares (no GPU, no compute)."""
import os
import re

import pytest

from paper_2512_12990_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "slicemoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(slicemoe_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_header_symbols():
    from paper_2512_12990_b200 import build
    build.build()
    L = B.lib()
    declared = _declared_symbols()
    assert len(declared) >= 18
    for name in declared:
        assert hasattr(L, name), f"{name} declared in slicemoe.h but not exported"
    assert sorted(B.EXPORTS) == declared


def test_host_only_entry_points():
    assert B.lib().slicemoe_version() >= 100
    assert B.strerror(0) == "ok"
    assert "invalid" in B.strerror(B.E_INVALID_ARG)
    assert "unknown" in B.strerror(-99)
    assert B.slicemoe_plane_bytes(1408, 2048) == 1441792
    assert B.slicemoe_meta_count(1408, 2048, 128) == 22528
    assert B.slicemoe_plane_bytes(0, 5) == 0
    sh = B.make_shape(2048, 1408, 64, 6, 128, 2, 1408)
    assert B.slicemoe_workspace_bytes(sh) > 12288 * 4


def test_argument_errors_are_codes_not_faults():
    """Bad arguments are rejected on the host before any CUDA call."""
    import ctypes
    L = B.lib()
    one = ctypes.c_void_p(16)     # never dereferenced: the checks come first
    assert L.slicemoe_pack(None, 16, 128, 128, 8, 4, one, one, one, one, None) == B.E_INVALID_ARG
    assert L.slicemoe_pack(one, 16, 128, 128, 8, 3, one, one, one, one, None) == B.E_UNSUPPORTED
    assert L.slicemoe_pack(one, 15, 128, 128, 8, 4, one, one, one, one, None) == B.E_INVALID_ARG
    assert L.slicemoe_pack(one, 16, 192, 128, 8, 4, one, one, one, one, None) == B.E_INVALID_ARG
    assert L.slicemoe_pack(one, 16, 128, 48, 8, 4, one, one, one, one, None) == B.E_UNSUPPORTED
    assert L.slicemoe_route_topk(one, 1, 8, 9, None, 0, 2.0, 0, one, one, None, None) == B.E_INVALID_ARG
    assert L.slicemoe_route_topk(one, 0, 8, 2, None, 0, 2.0, 0, one, one, None, None) == B.E_INVALID_ARG
    assert L.slicemoe_route_topk(one, 1, 1024, 2, None, 0, 2.0, 0, one, one, None, None) == B.E_UNSUPPORTED
    assert L.slicemoe_route_topk(one, 1, 64, 17, None, 0, 2.0, 0, one, one, None, None) == B.E_INVALID_ARG
    sh = B.make_shape(2048, 1408, 64, 6, 128)
    big = 1 << 24
    ws = ctypes.c_void_p(4096)
    assert L.slicemoe_expert_ffn(ctypes.byref(sh), one, one, 1, one, one, one, one, ws, 16, None) == B.E_INVALID_ARG
    assert L.slicemoe_expert_ffn(ctypes.byref(sh), None, one, 1, one, one, one, one, ws, big, None) == B.E_INVALID_ARG
    assert L.slicemoe_expert_ffn(ctypes.byref(sh), one, one, 0, one, one, one, one, ws, big, None) == B.E_INVALID_ARG
    bad = B.make_shape(2048, 1408, 64, 6, 128, b_high=6, b_low=4)
    assert L.slicemoe_expert_ffn(ctypes.byref(bad), one, one, 1, one, one, one, one, ws, big, None) == B.E_UNSUPPORTED
    bad = B.make_shape(2000, 1408, 64, 6, 128)
    assert L.slicemoe_expert_ffn(ctypes.byref(bad), one, one, 1, one, one, one, one, ws, big, None) == B.E_INVALID_ARG
    bad = B.make_shape(2048, 1408, 4, 6, 128)
    assert L.slicemoe_expert_ffn(ctypes.byref(bad), one, one, 1, one, one, one, one, ws, big, None) == B.E_INVALID_ARG
    bad = B.make_shape(8192, 1408, 64, 6, 128)
    assert L.slicemoe_expert_ffn(ctypes.byref(bad), one, one, 1, one, one, one, one, ws, big, None) == B.E_UNSUPPORTED
    bad = B.make_shape(2048, 4096, 64, 6, 128)             # 6 * 4096 > 12288
    assert L.slicemoe_expert_ffn(ctypes.byref(bad), one, one, 1, one, one, one, one, ws, big, None) == B.E_UNSUPPORTED
    q = B.make_shape(2048, 1408, 60, 4, 128, 1, 5632, True)
    assert L.slicemoe_layer(ctypes.byref(q), one, one, None, one, 1, one, one, one, one, ws, big, None) == B.E_INVALID_ARG
    assert L.slicemoe_layer(ctypes.byref(q), one, None, one, one, 1, one, one, one, one, ws, big, None) == B.E_INVALID_ARG
    assert L.slicemoe_layer_flags(ctypes.byref(q), one, one, None, one, 1, one, one, one, one, ws, big, 1, None) == B.E_INVALID_ARG
    assert L.slicemoe_stream_probe(ctypes.byref(q), one, None, one, one, 1, None, None, None) == B.E_INVALID_ARG  # shared missing
    assert L.slicemoe_stream_probe(ctypes.byref(sh), None, None, one, one, 1, None, None, None) == B.E_INVALID_ARG
    assert L.slicemoe_trace_read(None, 0, None) == B.E_UNSUPPORTED      # the ordinary build carries no time stamps
    assert L.slicemoe_workspace_init(None, big, None) == B.E_INVALID_ARG
    assert L.slicemoe_get_status(None, None, None) == B.E_INVALID_ARG
    assert L.slicemoe_workspace_set_wait(None, 1000, 0, None) == B.E_INVALID_ARG
    assert L.slicemoe_workspace_set_wait(ctypes.c_void_p(8), 1000, 0, None) == B.E_INVALID_ARG   # not 256-byte aligned
    assert L.slicemoe_dbsc_create(-1, 1, 1, -1.0, 10) is None
    assert L.slicemoe_dbsc_request(None, 0, 0, 0, 0, None, None, None) == B.E_INVALID_ARG
