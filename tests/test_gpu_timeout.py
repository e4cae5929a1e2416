"""The time-out path of the decode kernel, exercised without hanging or faulting anything: the workspace is
told to treat the intermediate vector that the CTAs exchange between the two phases as never complete,
and that no device-side wait may last longer than about a millisecond.  The kernel has to return by itself,
report SLICEMOE_STATUS_WAIT_TIMEOUT, and the same workspace has to work again once it is re-initialised."""
import time

import numpy as np
import pytest

from oracle import moe
from paper_2512_12990_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_wait_timeout_is_reported_and_the_workspace_recovers():
    import torch
    from paper_2512_12990_b200 import binding as B
    sh = synth.SHAPES["tiny"]
    layer = H.Layer(sh, range(sh.n_experts))
    logits = synth.router_logits_normal(sh.seed, ("timeout-logits",), 1, sh.n_experts)
    ids, w, _ = moe.route_topk(logits, sh.top_k)
    prec = (ids >= 4).astype(np.uint8)
    xbits, x64 = H.x_inputs(sh, 1, "timeout-x")
    x = H.to_dev_bf16(xbits)
    args = (torch.from_numpy(ids.astype(np.int32)).cuda(), torch.from_numpy(prec).cuda(),
            torch.from_numpy(w.astype(np.float32)).cuda())
    y_ref = moe.expert_ffn(x64, layer.oracle_list(), ids, prec, w)

    # a normal call first
    y = B.slicemoe_expert_ffn(layer.cshape, layer.experts_tbl, x, *args, layer.ws)
    torch.cuda.synchronize()
    assert B.slicemoe_get_status(layer.ws) == 0
    H.assert_close(y.cpu().numpy(), y_ref, "before the time-out")

    # one arrival that never comes, and a limit of 2 million cycles (about a millisecond)
    B.slicemoe_workspace_set_wait(layer.ws, 2_000_000, extra_arrivals=1)
    y_bad = torch.full((1, sh.hidden), 7.0, dtype=torch.float32, device="cuda")
    t0 = time.time()
    B.slicemoe_expert_ffn(layer.cshape, layer.experts_tbl, x, *args, layer.ws, y=y_bad)
    torch.cuda.synchronize()
    assert time.time() - t0 < 5.0, "the kernel must return by itself"
    status = B.slicemoe_get_status(layer.ws)
    assert status & B.STATUS_WAIT_TIMEOUT
    assert torch.all(y_bad == 7.0), "the output is not written when h was never complete"

    # re-initialised, the workspace works again (and the limit is back to its default)
    B.lib().slicemoe_workspace_init(layer.ws.data_ptr(), layer.ws.numel(), None)
    y2 = B.slicemoe_expert_ffn(layer.cshape, layer.experts_tbl, x, *args, layer.ws)
    torch.cuda.synchronize()
    assert B.slicemoe_get_status(layer.ws) == 0
    assert torch.equal(y2, y), "same bits as before the time-out"
