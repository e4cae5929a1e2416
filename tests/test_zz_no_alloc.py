"""slicemoe_layer_static: the entry point for callers that may not allocate device memory (a plug-in
that only receives buffers, code under a memory pool that owns the whole device, a context where the
runtime forbids cudaMalloc).  It must give what slicemoe_layer gives with a caller workspace, call
after call, although every call reuses the same built-in scratch array.

Collected last on purpose: a failure here cannot hide the result of any other test."""
import numpy as np
import pytest

from oracle import moe
from paper_2512_12990_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_workspace_entry_point_twice():
    import torch
    from paper_2512_12990_b200 import binding as B
    sh = synth.Shape("na", 384, 256, 6, 3, 64, n_shared=1, shared_inter=128, shared_sigmoid_gate=True, seed=4242)
    L = H.Layer(sh, range(sh.n_experts))
    T = 3
    xbits, x64 = H.x_inputs(sh, T, "x-noalloc")
    x = H.to_dev_bf16(xbits)
    y_static = torch.empty((T, sh.hidden), dtype=torch.float32, device="cuda")
    for call in range(2):                       # two calls in a row: the second starts from the first one's leftovers
        logits = synth.router_logits_normal(sh.seed, ("logits-noalloc", call), T, sh.n_experts)
        ids, w, _ = moe.route_topk(logits, sh.top_k)
        prec = moe.precision_request(w, 2.0, rank_high=1 + call)
        args = (torch.from_numpy(ids).cuda(), torch.from_numpy(prec).cuda(), torch.from_numpy(w.astype(np.float32)).cuda())
        y_ws = B.slicemoe_layer(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x, *args, L.ws)
        y_static.fill_(float("nan"))
        B.slicemoe_layer_static(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x, *args, y_static)
        torch.cuda.synchronize()
        a, b = y_static.cpu().numpy(), y_ws.cpu().numpy()
        assert np.isfinite(a).all()
        for t in range(T):
            H.assert_close(a[t], b[t], f"call {call} token {t}: static scratch vs caller workspace")
        # the summation order is fixed and both paths run the same kernel on the same grid: the same bits
        assert np.array_equal(a, b)
        y_ref = moe.layer(x64, L.oracle_list(), ids, prec, w, shared=L.oracle_shared, shared_gate_vec=L.gate_vec)
        for t in range(T):
            H.assert_close(a[t], y_ref[t], f"call {call} token {t}: static scratch vs oracle")


def test_static_scratch_entry_point_refuses_what_does_not_fit():
    """A layer beyond the built-in array's size is refused on the host; nothing is launched."""
    import ctypes
    from paper_2512_12990_b200 import binding as B
    one = ctypes.c_void_p(256)
    too_wide = B.make_shape(8192, 1408, 64, 6, 128)
    too_many = B.make_shape(2048, 4096, 64, 6, 128)
    lib = B.lib()
    for shape in (too_wide, too_many):
        rc = lib.slicemoe_layer_static(ctypes.byref(shape), one, None, None, one, 1, one, one, one, one, None)
        assert rc == B.E_UNSUPPORTED
    assert lib.slicemoe_layer_static(None, one, None, None, one, 1, one, one, one, one, None) == B.E_INVALID_ARG
