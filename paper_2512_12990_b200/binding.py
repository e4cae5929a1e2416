"""Thin ctypes binding over libslicemoe.so: argument marshalling only.

Function names and argument order follow include/slicemoe.h.  Device buffers are torch CUDA
tensors (torch is used for device memory and streams, nothing else); every step of the path
runs in the library's kernels.  There is no fallback: if the library is missing or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import (POINTER, Structure, c_char_p, c_double, c_float, c_int, c_int32, c_int64, c_size_t,
                    c_uint8, c_uint16, c_void_p)

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libslicemoe.so")
_lib = None

OK = 0
E_INVALID_ARG, E_UNSUPPORTED, E_CUDA, E_NOMEM = -1, -2, -3, -4
STATUS_BAD_EXPERT_ID, STATUS_WAIT_TIMEOUT, STATUS_MISSING_LSB = 1, 2, 4
MAX_TOP_K, MAX_SHARED = 16, 4
DBSC_NSTATS = 12
DBSC_STAT_NAMES = ("requests", "msb_hit", "msb_miss", "lsb_hit", "lsb_miss", "lsb_skipped", "bytes_fetched",
                   "high_exec", "low_exec", "win_bytes_fetched", "win_bytes_full", "bytes_used")

# every symbol include/slicemoe.h declares
EXPORTS = (
    "slicemoe_strerror", "slicemoe_version", "slicemoe_last_cuda_error", "slicemoe_plane_bytes", "slicemoe_meta_count", "slicemoe_pack",
    "slicemoe_unpack_plane", "slicemoe_unpack_meta", "slicemoe_compact_bytes", "slicemoe_compact_plane", "slicemoe_expand_plane", "slicemoe_route_topk", "slicemoe_workspace_bytes",
    "slicemoe_workspace_init", "slicemoe_workspace_set_wait", "slicemoe_get_status", "slicemoe_expert_ffn", "slicemoe_layer", "slicemoe_layer_flags",
    "slicemoe_decode_step_host", "slicemoe_stream_probe", "slicemoe_trace_read", "slicemoe_layer_static", "slicemoe_layer_routed", "slicemoe_prefill_workspace_bytes", "slicemoe_prefill_layer",
    "slicemoe_dbsc_create", "slicemoe_dbsc_destroy", "slicemoe_dbsc_request",
    "slicemoe_dbsc_assign", "slicemoe_dbsc_stats", "slicemoe_dbsc_contains",
    "slicemoe_dbsc_prefill_layer", "slicemoe_dbsc_prefill_end", "slicemoe_dbsc_bias", "slicemoe_cumsum_select",
    "slicemoe_cost_paper_hw", "slicemoe_cost_step", "slicemoe_dbsc_log_evictions", "slicemoe_dbsc_drain_evicted",
    "slicemoe_tier_sizes", "slicemoe_tier_store_expert", "slicemoe_tier_create", "slicemoe_tier_destroy",
    "slicemoe_tier_cache", "slicemoe_tier_request", "slicemoe_tier_sync", "slicemoe_tier_stats",
)


class SliceMoEError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = ""
        if code == E_CUDA:
            detail = ": " + lib().slicemoe_last_cuda_error().decode()
        super().__init__(f"{where}: {strerror(code)} ({code}){detail}")


class CostHw(Structure):
    _fields_ = [("dram_pj_per_bit", c_double), ("flash_pj_per_bit", c_double), ("dram_gbps", c_double),
                ("flash_gbps", c_double), ("tops", c_double), ("tops_per_watt", c_double)]


class Shape(Structure):
    _fields_ = [("hidden", c_int32), ("inter", c_int32), ("n_experts", c_int32), ("top_k", c_int32),
                ("group", c_int32), ("b_high", c_int32), ("b_low", c_int32), ("n_shared", c_int32),
                ("shared_inter", c_int32), ("shared_sigmoid_gate", c_int32)]


class Mat(Structure):
    _fields_ = [("msb", c_void_p), ("lsb", c_void_p), ("scale", c_void_p), ("zp", c_void_p),
                ("N", c_int32), ("K", c_int32)]


class Expert(Structure):
    _fields_ = [("gate", Mat), ("up", Mat), ("down", Mat)]


def lib() -> ctypes.CDLL:
    """Loads the C-ABI library on first use; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} not found: build it with `python -m paper_2512_12990_b200.build` "
                          "(there is no fallback path)")
    L = ctypes.CDLL(_LIB_PATH)
    L.slicemoe_strerror.restype = c_char_p
    L.slicemoe_strerror.argtypes = [c_int]
    L.slicemoe_version.restype = c_int
    L.slicemoe_last_cuda_error.restype = c_char_p
    L.slicemoe_plane_bytes.restype = c_size_t
    L.slicemoe_plane_bytes.argtypes = [c_int, c_int]
    L.slicemoe_meta_count.restype = c_size_t
    L.slicemoe_meta_count.argtypes = [c_int, c_int, c_int]
    L.slicemoe_pack.argtypes = [c_void_p, c_int, c_int, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p,
                                c_void_p, c_void_p]
    L.slicemoe_compact_bytes.restype = c_size_t
    L.slicemoe_compact_bytes.argtypes = [c_int, c_int, c_int]
    L.slicemoe_compact_plane.argtypes = [c_void_p, c_int, c_int, c_int, c_void_p, c_void_p]
    L.slicemoe_expand_plane.argtypes = [c_void_p, c_int, c_int, c_int, c_void_p, c_void_p]
    L.slicemoe_unpack_plane.argtypes = [c_void_p, c_int, c_int, c_void_p, c_void_p]
    L.slicemoe_unpack_meta.argtypes = [c_void_p, c_void_p, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p]
    L.slicemoe_route_topk.argtypes = [c_void_p, c_int, c_int, c_int, c_void_p, c_int, c_float, c_int, c_void_p,
                                      c_void_p, c_void_p, c_void_p]
    L.slicemoe_workspace_bytes.restype = c_size_t
    L.slicemoe_workspace_bytes.argtypes = [POINTER(Shape)]
    L.slicemoe_workspace_init.argtypes = [c_void_p, c_size_t, c_void_p]
    L.slicemoe_get_status.argtypes = [c_void_p, POINTER(c_int), c_void_p]
    L.slicemoe_workspace_set_wait.argtypes = [c_void_p, ctypes.c_ulonglong, ctypes.c_uint, c_void_p]
    L.slicemoe_expert_ffn.argtypes = [POINTER(Shape), c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p,
                                      c_void_p, c_void_p, c_size_t, c_void_p]
    L.slicemoe_layer.argtypes = [POINTER(Shape), c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p,
                                 c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    L.slicemoe_layer_flags.argtypes = [POINTER(Shape), c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p,
                                       c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, ctypes.c_uint, c_void_p]
    L.slicemoe_trace_read.argtypes = [c_void_p, c_int, POINTER(c_int)]
    L.slicemoe_stream_probe.argtypes = [POINTER(Shape), c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p,
                                        c_void_p]
    L.slicemoe_layer_static.argtypes = [POINTER(Shape), c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p,
                                        c_void_p, c_void_p, c_void_p, c_void_p]
    L.slicemoe_decode_step_host.argtypes = [POINTER(Shape), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                            c_void_p, c_int, c_float, c_int, c_void_p, c_void_p, c_size_t,
                                            c_void_p]
    L.slicemoe_layer_routed.argtypes = [POINTER(Shape), c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_void_p,
                                        c_int, c_float, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                        c_size_t, c_void_p]
    L.slicemoe_prefill_workspace_bytes.restype = c_size_t
    L.slicemoe_prefill_workspace_bytes.argtypes = [POINTER(Shape), c_int]
    L.slicemoe_prefill_layer.argtypes = [POINTER(Shape), c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p,
                                         c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]
    L.slicemoe_dbsc_create.restype = c_void_p
    L.slicemoe_dbsc_create.argtypes = [c_int64, c_int64, c_int64, c_double, c_int]
    L.slicemoe_dbsc_destroy.restype = None
    L.slicemoe_dbsc_destroy.argtypes = [c_void_p]
    L.slicemoe_dbsc_request.argtypes = [c_void_p, c_int, c_int, c_int, c_int, POINTER(c_int), POINTER(c_int),
                                        POINTER(c_int64)]
    L.slicemoe_dbsc_assign.argtypes = [c_void_p, c_int, c_int, c_void_p, c_void_p, c_int, c_void_p]
    L.slicemoe_dbsc_stats.argtypes = [c_void_p, POINTER(c_int64)]
    L.slicemoe_dbsc_contains.argtypes = [c_void_p, c_int, c_int, POINTER(c_int), POINTER(c_int)]
    L.slicemoe_dbsc_prefill_layer.argtypes = [c_void_p, c_int, c_void_p, c_void_p, c_int64, c_int, c_double]
    L.slicemoe_dbsc_prefill_end.argtypes = [c_void_p]
    L.slicemoe_dbsc_bias.argtypes = [c_void_p, c_int, c_int, c_float, c_void_p]
    L.slicemoe_dbsc_log_evictions.argtypes = [c_void_p, c_int]
    L.slicemoe_dbsc_drain_evicted.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int]
    L.slicemoe_tier_sizes.argtypes = [POINTER(Shape), POINTER(c_size_t), POINTER(c_size_t), POINTER(c_size_t), POINTER(c_size_t)]
    L.slicemoe_tier_store_expert.argtypes = [POINTER(Shape), c_void_p, c_void_p, c_void_p, c_void_p]
    L.slicemoe_tier_create.restype = c_void_p
    L.slicemoe_tier_create.argtypes = [POINTER(Shape), c_int, c_void_p, c_void_p, c_size_t, c_void_p, c_void_p, c_size_t, c_double,
                                       c_int, c_void_p]
    L.slicemoe_tier_destroy.argtypes = [c_void_p]
    L.slicemoe_tier_destroy.restype = None
    L.slicemoe_tier_cache.restype = c_void_p
    L.slicemoe_tier_cache.argtypes = [c_void_p]
    L.slicemoe_tier_request.argtypes = [c_void_p, c_int, c_int, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p]
    L.slicemoe_tier_sync.argtypes = [c_void_p, c_void_p, c_void_p]
    L.slicemoe_tier_stats.argtypes = [c_void_p, POINTER(c_int64), POINTER(c_int64), POINTER(c_int64)]
    L.slicemoe_cumsum_select.argtypes = [c_void_p, c_void_p, c_int, c_int, c_double, c_void_p]
    L.slicemoe_cost_paper_hw.argtypes = [POINTER(CostHw)]
    L.slicemoe_cost_paper_hw.restype = None
    L.slicemoe_cost_step.argtypes = [POINTER(CostHw), c_int64, c_int64, c_int64, POINTER(c_double), POINTER(c_double)]
    _lib = L
    return L


def strerror(code: int) -> str:
    return lib().slicemoe_strerror(code).decode()


def _check(rc: int, where: str) -> None:
    if rc != OK:
        raise SliceMoEError(rc, where)


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return c_void_p(s.cuda_stream)


def make_shape(hidden, inter, n_experts, top_k, group, n_shared=0, shared_inter=0, shared_sigmoid_gate=False,
               b_high=8, b_low=4) -> Shape:
    return Shape(hidden, inter, n_experts, top_k, group, b_high, b_low, n_shared, shared_inter,
                 1 if shared_sigmoid_gate else 0)


# ---- sizes ---------------------------------------------------------------------------------------
def slicemoe_plane_bytes(N: int, K: int) -> int:
    return lib().slicemoe_plane_bytes(N, K)


def slicemoe_meta_count(N: int, K: int, group: int) -> int:
    return lib().slicemoe_meta_count(N, K, group)


# ---- pack ----------------------------------------------------------------------------------------
class PackedMat:
    """Device buffers of one packed matrix (physical layout) and its Mat descriptor."""

    def __init__(self, N, K, group, msb, lsb, scale, zp):
        self.N, self.K, self.group = N, K, group
        self.msb, self.lsb, self.scale, self.zp = msb, lsb, scale, zp

    def desc(self) -> Mat:
        return Mat(self.msb.data_ptr(), self.lsb.data_ptr() if self.lsb is not None else None,
                   self.scale.data_ptr(), self.zp.data_ptr(), self.N, self.K)


def slicemoe_pack(W, group: int, b_high: int = 8, b_low: int = 4, stream=None, out: PackedMat | None = None) -> PackedMat:
    """W: CUDA float32 [N, K] contiguous.  Allocates the outputs with torch unless `out` is given."""
    import torch
    assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous() and W.dim() == 2
    N, K = W.shape
    if out is None:
        nb = max(int(slicemoe_plane_bytes(N, K)), 1)
        nm = max(int(slicemoe_meta_count(N, K, group)) if group > 0 else 1, 1)
        out = PackedMat(N, K, group,
                        torch.empty(nb, dtype=torch.uint8, device=W.device),
                        torch.empty(nb, dtype=torch.uint8, device=W.device),
                        torch.empty(nm, dtype=torch.int16, device=W.device),
                        torch.empty(nm, dtype=torch.uint8, device=W.device))
    rc = lib().slicemoe_pack(_ptr(W), N, K, group, b_high, b_low, _ptr(out.msb), _ptr(out.lsb), _ptr(out.scale),
                             _ptr(out.zp), _stream(stream))
    _check(rc, "slicemoe_pack")
    return out


def slicemoe_unpack_plane(plane, N: int, K: int, stream=None):
    import torch
    out = torch.empty((N, K), dtype=torch.uint8, device=plane.device)
    _check(lib().slicemoe_unpack_plane(_ptr(plane), N, K, _ptr(out), _stream(stream)), "slicemoe_unpack_plane")
    return out


def slicemoe_unpack_meta(scale, zp, N: int, K: int, group: int, stream=None):
    """Returns (scale fp16 [N, K/group], zp uint8 [N, K/group]) row-major."""
    import torch
    ng = K // group
    s = torch.empty((N, ng), dtype=torch.float16, device=scale.device)
    z = torch.empty((N, ng), dtype=torch.uint8, device=scale.device)
    _check(lib().slicemoe_unpack_meta(_ptr(scale), _ptr(zp), N, K, group, _ptr(s), _ptr(z), _stream(stream)),
           "slicemoe_unpack_meta")
    return s, z


# ---- route ---------------------------------------------------------------------------------------
def slicemoe_route_topk(logits, k: int, bias=None, renorm: bool = False, tau: float = 2.0, rank_high: int = 0,
                        want_prec: bool = True, stream=None):
    """logits CUDA float32 [T, E].  Returns (ids int32 [T,k], weights float32 [T,k], prec_req uint8 [T,k] | None)."""
    import torch
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous() and logits.dim() == 2
    T, E = logits.shape
    kk = max(k, 1)
    ids = torch.empty((T, kk), dtype=torch.int32, device=logits.device)
    w = torch.empty((T, kk), dtype=torch.float32, device=logits.device)
    pr = torch.empty((T, kk), dtype=torch.uint8, device=logits.device) if want_prec else None
    rc = lib().slicemoe_route_topk(_ptr(logits), T, E, k, _ptr(bias), 1 if renorm else 0, tau, rank_high,
                                   _ptr(ids), _ptr(w), _ptr(pr), _stream(stream))
    _check(rc, "slicemoe_route_topk")
    return ids, w, pr


# ---- workspace -----------------------------------------------------------------------------------
def slicemoe_workspace_bytes(shape: Shape) -> int:
    return lib().slicemoe_workspace_bytes(ctypes.byref(shape))


def new_workspace(shape: Shape, device="cuda", stream=None):
    import torch
    nbytes = slicemoe_workspace_bytes(shape)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    assert ws.data_ptr() % 256 == 0
    _check(lib().slicemoe_workspace_init(_ptr(ws), nbytes, _stream(stream)), "slicemoe_workspace_init")
    return ws


def slicemoe_workspace_set_wait(ws, wait_cycles: int, extra_arrivals: int = 0, stream=None):
    _check(lib().slicemoe_workspace_set_wait(_ptr(ws), wait_cycles, extra_arrivals, _stream(stream)),
           "slicemoe_workspace_set_wait")


def slicemoe_get_status(ws, stream=None) -> int:
    out = c_int(0)
    _check(lib().slicemoe_get_status(_ptr(ws), ctypes.byref(out), _stream(stream)), "slicemoe_get_status")
    return out.value


# ---- expert tables ---------------------------------------------------------------------------------
def expert_table(experts, device="cuda"):
    """experts: list of dict(gate=PackedMat, up=PackedMat, down=PackedMat) -> CUDA uint8 tensor holding the
    slicemoe_expert array (keep the PackedMats alive as long as the table is used)."""
    import torch
    arr = (Expert * len(experts))()
    for i, e in enumerate(experts):
        arr[i] = Expert(e["gate"].desc(), e["up"].desc(), e["down"].desc())
    raw = bytes(arr)
    host = torch.frombuffer(bytearray(raw), dtype=torch.uint8)
    return host.to(device)


# ---- FFN -----------------------------------------------------------------------------------------
def slicemoe_expert_ffn(shape: Shape, experts_tbl, x, ids, prec, weights, ws, y=None, stream=None):
    """x CUDA bf16 [T, hidden]; ids int32, prec uint8, weights float32 [T, k].  Returns y float32 [T, hidden]."""
    import torch
    T = x.shape[0]
    if y is None:
        y = torch.empty((T, shape.hidden), dtype=torch.float32, device=x.device)
    rc = lib().slicemoe_expert_ffn(ctypes.byref(shape), _ptr(experts_tbl), _ptr(x), T, _ptr(ids), _ptr(prec),
                                   _ptr(weights), _ptr(y), _ptr(ws), ws.numel(), _stream(stream))
    _check(rc, "slicemoe_expert_ffn")
    return y


LISTS_RESIDENT = 1
COOPERATIVE = 2


def slicemoe_layer(shape: Shape, experts_tbl, shared_tbl, shared_gate_vec, x, ids, prec, weights, ws, y=None,
                   stream=None, flags=0):
    """flags = 0 calls slicemoe_layer, anything else slicemoe_layer_flags."""
    import torch
    T = x.shape[0]
    if y is None:
        y = torch.empty((T, shape.hidden), dtype=torch.float32, device=x.device)
    if flags:
        rc = lib().slicemoe_layer_flags(ctypes.byref(shape), _ptr(experts_tbl), _ptr(shared_tbl), _ptr(shared_gate_vec),
                                        _ptr(x), T, _ptr(ids), _ptr(prec), _ptr(weights), _ptr(y), _ptr(ws),
                                        ws.numel(), flags, _stream(stream))
        _check(rc, "slicemoe_layer_flags")
        return y
    rc = lib().slicemoe_layer(ctypes.byref(shape), _ptr(experts_tbl), _ptr(shared_tbl), _ptr(shared_gate_vec),
                              _ptr(x), T, _ptr(ids), _ptr(prec), _ptr(weights), _ptr(y), _ptr(ws), ws.numel(),
                              _stream(stream))
    _check(rc, "slicemoe_layer")
    return y


def slicemoe_stream_probe(shape: Shape, experts_tbl, shared_tbl, ids, prec, dependent=True, bytes_out=None,
                          status_out=None, stream=None):
    """ids, prec: CUDA int32 / uint8 [top_k].  bytes_out: CUDA int64 [1] (added to) or None; status_out: CUDA
    int32 [1] or None."""
    rc = lib().slicemoe_stream_probe(ctypes.byref(shape), _ptr(experts_tbl), _ptr(shared_tbl), _ptr(ids), _ptr(prec),
                                     1 if dependent else 0, _ptr(bytes_out), _ptr(status_out), _stream(stream))
    _check(rc, "slicemoe_stream_probe")


def slicemoe_layer_static(shape: Shape, experts_tbl, shared_tbl, shared_gate_vec, x, ids, prec, weights, y, stream=None):
    """slicemoe_layer without a caller workspace: the library's built-in scratch array is used.  `y` (CUDA
    float32 [T, hidden]) is required, because nothing may be allocated on this path - not by the library and
    not by this binding."""
    rc = lib().slicemoe_layer_static(ctypes.byref(shape), _ptr(experts_tbl), _ptr(shared_tbl), _ptr(shared_gate_vec),
                                     _ptr(x), x.shape[0], _ptr(ids), _ptr(prec), _ptr(weights), _ptr(y),
                                     _stream(stream))
    _check(rc, "slicemoe_layer_static")
    return y


def slicemoe_layer_routed(shape: Shape, experts_tbl, shared_tbl, shared_gate_vec, x, logits, ws, bias=None, renorm=False,
                          tau=2.0, rank_high=0, y=None, want_lists=True, stream=None):
    """Routing and layer in one launch per token.  Returns (y, ids, prec, weights); the lists are None unless
    want_lists."""
    import torch
    T = x.shape[0]
    k = shape.top_k
    if y is None:
        y = torch.empty((T, shape.hidden), dtype=torch.float32, device=x.device)
    ids = torch.empty((T, k), dtype=torch.int32, device=x.device) if want_lists else None
    prec = torch.empty((T, k), dtype=torch.uint8, device=x.device) if want_lists else None
    w = torch.empty((T, k), dtype=torch.float32, device=x.device) if want_lists else None
    rc = lib().slicemoe_layer_routed(ctypes.byref(shape), _ptr(experts_tbl), _ptr(shared_tbl), _ptr(shared_gate_vec),
                                     _ptr(x), T, _ptr(logits), _ptr(bias), 1 if renorm else 0, tau, rank_high, _ptr(ids),
                                     _ptr(prec), _ptr(w), _ptr(y), _ptr(ws), ws.numel(), _stream(stream))
    _check(rc, "slicemoe_layer_routed")
    return y, ids, prec, w


def slicemoe_decode_step_host(shape: Shape, experts_tbl, shared_tbl, shared_gate_vec, x_host, logits_host, y_host,
                              ws, bias=None, renorm=False, tau=2.0, rank_high=0, stream=None):
    """x_host: pinned CPU bf16 [hidden]; logits_host: pinned CPU float32 [E], or None when x_host is one pinned
    byte buffer holding x (bf16 [hidden]) and then the logits (float32 [E]); y_host: pinned CPU float32
    [hidden] (written).  Synchronises the stream."""
    rc = lib().slicemoe_decode_step_host(ctypes.byref(shape), _ptr(experts_tbl), _ptr(shared_tbl),
                                         _ptr(shared_gate_vec), c_void_p(x_host.data_ptr()),
                                         None if logits_host is None else c_void_p(logits_host.data_ptr()), _ptr(bias), 1 if renorm else 0, tau,
                                         rank_high, c_void_p(y_host.data_ptr()), _ptr(ws), ws.numel(),
                                         _stream(stream))
    _check(rc, "slicemoe_decode_step_host")
    return y_host


def slicemoe_prefill_workspace_bytes(shape: Shape, T: int) -> int:
    return int(lib().slicemoe_prefill_workspace_bytes(ctypes.byref(shape), T))


def new_prefill_workspace(shape: Shape, T: int, device="cuda"):
    import torch
    n = slicemoe_prefill_workspace_bytes(shape, T)
    if n == 0:
        raise SliceMoEError(E_INVALID_ARG, "slicemoe_prefill_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def slicemoe_prefill_layer(shape: Shape, experts_tbl, shared_tbl, shared_gate_vec, x, ids, weights, expert_prec, ws,
                           y=None, status=None, stream=None):
    """x: CUDA bf16 [T, hidden]; ids/weights: CUDA [T, k]; expert_prec: CUDA uint8 [E].  Returns (y, status) with
    status a CUDA int32 [1] tensor (read it after synchronising)."""
    import torch
    T = x.shape[0]
    if y is None:
        y = torch.empty((T, shape.hidden), dtype=torch.float32, device=x.device)
    if status is None:
        status = torch.empty(1, dtype=torch.int32, device=x.device)
    rc = lib().slicemoe_prefill_layer(ctypes.byref(shape), _ptr(experts_tbl), _ptr(shared_tbl), _ptr(shared_gate_vec),
                                      _ptr(x), T, _ptr(ids), _ptr(weights), _ptr(expert_prec), _ptr(y), _ptr(ws),
                                      ws.numel(), _ptr(status), _stream(stream))
    _check(rc, "slicemoe_prefill_layer")
    return y, status


# ---- host DBSC -------------------------------------------------------------------------------------
class Dbsc:
    """Host slice cache (slicemoe_dbsc_*).  No GPU needed."""

    def __init__(self, capacity_bytes: int, msb_bytes: int, lsb_bytes: int, miss_budget: float | None = None,
                 warmup_steps: int = 10):
        self._h = lib().slicemoe_dbsc_create(capacity_bytes, msb_bytes, lsb_bytes,
                                             -1.0 if miss_budget is None else float(miss_budget), warmup_steps)
        if not self._h:
            raise SliceMoEError(E_INVALID_ARG, "slicemoe_dbsc_create")

    def close(self):
        if self._h:
            lib().slicemoe_dbsc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def request(self, step: int, layer: int, expert: int, need_lsb: bool):
        mh, lh, fb = c_int(0), c_int(0), c_int64(0)
        prec = lib().slicemoe_dbsc_request(self._h, step, layer, expert, 1 if need_lsb else 0, ctypes.byref(mh),
                                           ctypes.byref(lh), ctypes.byref(fb))
        if prec < 0:
            raise SliceMoEError(prec, "slicemoe_dbsc_request")
        return prec, bool(mh.value), (None if lh.value < 0 else bool(lh.value)), fb.value

    def assign(self, step: int, layer: int, ids, prec_req):
        """ids: numpy int32 [n]; prec_req: numpy uint8 [n] -> numpy uint8 [n]."""
        import numpy as np
        ids = np.ascontiguousarray(ids, dtype=np.int32)
        prec_req = np.ascontiguousarray(prec_req, dtype=np.uint8)
        out = np.empty(ids.shape, dtype=np.uint8)
        rc = lib().slicemoe_dbsc_assign(self._h, step, layer, ids.ctypes.data_as(c_void_p),
                                        prec_req.ctypes.data_as(c_void_p), ids.size, out.ctypes.data_as(c_void_p))
        _check(rc, "slicemoe_dbsc_assign")
        return out

    def bias(self, layer: int, n_experts: int, delta: float):
        """Cache-Prior bias of a layer: numpy float32 [n_experts]."""
        import numpy as np
        out = np.empty(n_experts, dtype=np.float32)
        _check(lib().slicemoe_dbsc_bias(self._h, layer, n_experts, delta, out.ctypes.data_as(c_void_p)), "slicemoe_dbsc_bias")
        return out

    def stats(self) -> dict:
        buf = (c_int64 * DBSC_NSTATS)()
        _check(lib().slicemoe_dbsc_stats(self._h, buf), "slicemoe_dbsc_stats")
        return dict(zip(DBSC_STAT_NAMES, list(buf)))

    def prefill_layer(self, layer: int, ids, scores, n_experts: int, tau: float):
        """Predictive cache warmup, one prefilled layer: ids / scores numpy [T, k] (the layer's routing result)."""
        import numpy as np
        ids = np.ascontiguousarray(ids, dtype=np.int32)
        scores = np.ascontiguousarray(scores, dtype=np.float32)
        if ids.shape != scores.shape:
            raise SliceMoEError(E_INVALID_ARG, "slicemoe_dbsc_prefill_layer")
        rc = lib().slicemoe_dbsc_prefill_layer(self._h, layer, ids.ctypes.data_as(c_void_p),
                                               scores.ctypes.data_as(c_void_p), ids.size, n_experts, float(tau))
        _check(rc, "slicemoe_dbsc_prefill_layer")

    def prefill_end(self):
        _check(lib().slicemoe_dbsc_prefill_end(self._h), "slicemoe_dbsc_prefill_end")

    def contains(self, layer: int, expert: int):
        a, b = c_int(0), c_int(0)
        _check(lib().slicemoe_dbsc_contains(self._h, layer, expert, ctypes.byref(a), ctypes.byref(b)),
               "slicemoe_dbsc_contains")
        return bool(a.value), bool(b.value)


# ---- routing baseline and cost model (host) ---------------------------------------------------------
def slicemoe_cumsum_select(probs, cached, k: int, p: float):
    """probs: numpy float32 [E]; cached: numpy bool/uint8 [E] -> numpy int32 [k]."""
    import numpy as np
    probs = np.ascontiguousarray(probs, dtype=np.float32)
    cached = np.ascontiguousarray(cached, dtype=np.uint8)
    out = np.empty(k, dtype=np.int32)
    rc = lib().slicemoe_cumsum_select(probs.ctypes.data_as(c_void_p), cached.ctypes.data_as(c_void_p), probs.size, k, p,
                                      out.ctypes.data_as(c_void_p))
    _check(rc, "slicemoe_cumsum_select")
    return out


def paper_hw() -> CostHw:
    hw = CostHw()
    lib().slicemoe_cost_paper_hw(ctypes.byref(hw))
    return hw


def slicemoe_cost_step(flash_bytes: int, dram_bytes: int, macs: int, hw: CostHw | None = None):
    """(energy in joules, latency in seconds) of one step under the cost model of Section 5."""
    hw = hw or paper_hw()
    e, t = c_double(0), c_double(0)
    _check(lib().slicemoe_cost_step(ctypes.byref(hw), flash_bytes, dram_bytes, macs, ctypes.byref(e), ctypes.byref(t)),
           "slicemoe_cost_step")
    return e.value, t.value


def slicemoe_compact_plane(plane, N: int, K: int, bits: int, stream=None):
    """plane: CUDA uint8 [N*K/2] (physical layout) -> CUDA uint8 [N*K*bits/8], the dense bit stream."""
    import torch
    out = torch.empty(lib().slicemoe_compact_bytes(N, K, bits), dtype=torch.uint8, device=plane.device)
    _check(lib().slicemoe_compact_plane(_ptr(plane), N, K, bits, _ptr(out), _stream(stream)), "slicemoe_compact_plane")
    return out


def slicemoe_expand_plane(compact, N: int, K: int, bits: int, stream=None):
    """The inverse: CUDA uint8 [N*K*bits/8] -> CUDA uint8 [N*K/2] in the physical plane layout."""
    import torch
    out = torch.empty(N * K // 2, dtype=torch.uint8, device=compact.device)
    _check(lib().slicemoe_expand_plane(_ptr(compact), N, K, bits, _ptr(out), _stream(stream)), "slicemoe_expand_plane")
    return out


class _BorrowedDbsc(Dbsc):
    """A Dbsc whose handle belongs to someone else: same methods, nothing is destroyed."""

    def __init__(self, handle):
        self._h = handle

    def close(self):
        self._h = None


# ---- second memory tier --------------------------------------------------------------------------------
def slicemoe_tier_sizes(shape: Shape):
    """(msb_record, lsb_record, slot_bytes, staging_bytes) of a shape: the records as stored, the slot and the
    staging buffer on the device."""
    m, l, sl, sg = c_size_t(0), c_size_t(0), c_size_t(0), c_size_t(0)
    _check(lib().slicemoe_tier_sizes(ctypes.byref(shape), ctypes.byref(m), ctypes.byref(l), ctypes.byref(sl),
                                     ctypes.byref(sg)), "slicemoe_tier_sizes")
    return m.value, l.value, sl.value, sg.value


class Tier:
    """slicemoe_tier_*: a pool of slice slots in device memory over a store in pinned host memory.

    `layers`: list (per layer) of lists (per expert) of dict(gate=PackedMat, up=..., down=...) on the device; their
    records are copied into one pinned host buffer (the slow store), after which the caller may drop them.  All
    memory is allocated here, in the binding, with torch; the library allocates none."""

    def __init__(self, shape: Shape, layers, pool_slots: int, miss_budget: float | None = None, warmup_steps: int = 10,
                 device="cuda"):
        import torch
        self.shape, self.n_layers, self.n_experts = shape, len(layers), len(layers[0])
        m, l, slot, stg = slicemoe_tier_sizes(shape)
        self.msb_record, self.lsb_record, self.slot_bytes = m, l, slot
        self.staging = torch.empty(stg, dtype=torch.uint8, device=device) if stg else None
        self.store = torch.empty((self.n_layers * self.n_experts, m + l), dtype=torch.uint8).pin_memory()
        for li, experts in enumerate(layers):
            for e, ex in enumerate(experts):
                rec = Expert(ex["gate"].desc(), ex["up"].desc(), ex["down"].desc())
                rc = lib().slicemoe_tier_store_expert(ctypes.byref(shape), ctypes.byref(rec),
                                                      c_void_p(self.store[li * self.n_experts + e].data_ptr()),
                                                      _ptr(self.staging), _stream(None))
                _check(rc, "slicemoe_tier_store_expert")
        torch.cuda.synchronize()
        self.pool = torch.empty(pool_slots * slot, dtype=torch.uint8, device=device)
        self.tables = torch.empty(self.n_layers * self.n_experts * ctypes.sizeof(Expert), dtype=torch.uint8, device=device)
        self.copy_stream = torch.cuda.Stream(device=device)
        self._h = lib().slicemoe_tier_create(ctypes.byref(shape), self.n_layers, c_void_p(self.store.data_ptr()),
                                             _ptr(self.pool), self.pool.numel(), _ptr(self.tables), _ptr(self.staging),
                                             0 if self.staging is None else self.staging.numel(),
                                             -1.0 if miss_budget is None else float(miss_budget), warmup_steps,
                                             _stream(None))
        if not self._h:
            raise SliceMoEError(E_INVALID_ARG, "slicemoe_tier_create")

    def close(self):
        if getattr(self, "_h", None):
            lib().slicemoe_tier_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def layer_table(self, layer: int):
        """The device expert table of a layer (a view into the tier's table array)."""
        n = self.n_experts * ctypes.sizeof(Expert)
        return self.tables[layer * n:(layer + 1) * n]

    def request(self, step: int, layer: int, ids, prec_req, compute_stream=None):
        """ids int32 [n], prec_req uint8 [n] (numpy, host) -> prec uint8 [n]; enqueues the copies and the waits."""
        import numpy as np
        ids = np.ascontiguousarray(ids, dtype=np.int32)
        prec_req = np.ascontiguousarray(prec_req, dtype=np.uint8)
        out = np.empty(ids.shape, dtype=np.uint8)
        rc = lib().slicemoe_tier_request(self._h, step, layer, ids.ctypes.data_as(c_void_p),
                                         prec_req.ctypes.data_as(c_void_p), ids.size, out.ctypes.data_as(c_void_p),
                                         _stream(compute_stream), c_void_p(self.copy_stream.cuda_stream))
        _check(rc, "slicemoe_tier_request")
        return out

    def cache(self):
        """The tier's own host cache (owned by the tier; valid while the tier is)."""
        return _BorrowedDbsc(lib().slicemoe_tier_cache(self._h))

    def sync(self, compute_stream=None):
        """Makes the pool hold what the cache's books hold (after a warm-up through self.cache())."""
        _check(lib().slicemoe_tier_sync(self._h, _stream(compute_stream), c_void_p(self.copy_stream.cuda_stream)),
               "slicemoe_tier_sync")

    def stats(self) -> dict:
        b, c, f = c_int64(0), c_int64(0), c_int64(0)
        _check(lib().slicemoe_tier_stats(self._h, ctypes.byref(b), ctypes.byref(c), ctypes.byref(f)), "slicemoe_tier_stats")
        out = (c_int64 * DBSC_NSTATS)()
        _check(lib().slicemoe_dbsc_stats(lib().slicemoe_tier_cache(self._h), out), "slicemoe_dbsc_stats")
        d = {k: int(v) for k, v in zip(DBSC_STAT_NAMES, out)}
        d.update(bytes_copied=b.value, copies=c.value, free_slots=f.value)
        return d
