"""Two independent device paths on the same packed weights: the batch-1 decode kernel (integer mma.sync on the raw
nibble planes, fixed-point activations) and the prefill kernel (tcgen05 on fp16 tiles of q - zp) must agree within
the FFN tolerance on many seeded shapes - hidden up to the decode limit, every group size, top-k up to 16, up to
four shared experts, one and two output row blocks per CTA, 1 to 130 tokens.  Each path is compared with the float64 oracle in
its own test file; this file widens the set of shapes beyond what the oracle can cover in seconds."""
import numpy as np
import pytest

from tests import helpers as H

pytestmark = pytest.mark.gpu


def _cases():
    rng = np.random.default_rng(20251212)
    out = []
    for i in range(100):
        hidden = int(rng.choice([128, 256, 640, 1024, 2048, 2432, 3072, 4096]))
        group = int(rng.choice([32, 64, 128]))
        k = int(rng.choice([1, 2, 4, 6, 8, 16]))
        E = int(k + rng.integers(0, 6))
        n_shared = int(rng.choice([0, 1, 2, 4]))
        cap = 12288
        inter = int(rng.choice([128, 256, 384, 640, 768, 1408]))
        shared_inter = int(rng.choice([128, 256, 512, 1408])) if n_shared else 0
        while k * inter + n_shared * shared_inter > cap:
            if inter > 128:
                inter -= 128
            else:
                shared_inter -= 128
        gated = bool(rng.integers(0, 2)) and n_shared > 0
        T = int(rng.choice([1, 3, 3, 130]))
        out.append((i, hidden, inter, E, k, group, n_shared, shared_inter, gated, T))
    return out


def _heavy_cases():
    """Shapes that wrap the decode kernel's staging rings: wide slots (several 2048-column chunks per slot), small
    groups (large units), many slots, two output row blocks per CTA."""
    rng = np.random.default_rng(20251213)
    out = []
    for i in range(60):
        hidden = int(rng.choice([2048, 2432, 3072, 4096]))
        group = int(rng.choice([32, 32, 64, 128]))
        k = int(rng.choice([1, 2, 3, 4, 6, 8]))
        E = int(k + rng.integers(0, 3))
        n_shared = int(rng.choice([0, 1, 2, 4]))
        inter = int(rng.choice([1024, 1408, 2176, 2560, 4096]))
        shared_inter = int(rng.choice([1408, 2176, 5632])) if n_shared else 0
        while k * inter + n_shared * shared_inter > 12288:
            if n_shared > 1:
                n_shared -= 1
            elif inter > 1024:
                inter -= 128
            elif shared_inter > 128:
                shared_inter -= 128
            else:
                k -= 1
        E = max(E, k)
        gated = bool(rng.integers(0, 2)) and n_shared > 0
        out.append((1000 + i, hidden, inter, E, k, group, n_shared, shared_inter, gated, int(rng.choice([1, 2]))))
    return out


@pytest.mark.parametrize("case", _cases() + _heavy_cases(), ids=lambda c: f"{c[0]}-h{c[1]}-i{c[2]}-E{c[3]}-k{c[4]}-g{c[5]}-s{c[6]}x{c[7]}-T{c[9]}")
def test_decode_and_prefill_paths_agree(case):
    import torch
    from paper_2512_12990_b200 import binding as B
    i, hidden, inter, E, k, group, n_shared, shared_inter, gated, T = case
    gen = torch.Generator(device="cuda")
    gen.manual_seed(7000 + i)
    cs = B.make_shape(hidden, inter, E, k, group, n_shared, shared_inter, gated)

    def pack3(width):
        return {name: B.slicemoe_pack(torch.randn(shape, device="cuda", generator=gen) * 0.02, group)
                for name, shape in (("gate", (width, hidden)), ("up", (width, hidden)), ("down", (hidden, width)))}

    experts = [pack3(inter) for _ in range(E)]
    shared = [pack3(shared_inter) for _ in range(n_shared)]
    et = B.expert_table(experts)
    st = B.expert_table(shared) if shared else None
    gv = torch.randn(hidden, device="cuda", generator=gen) * 0.02 if gated else None
    x = torch.randn((T, hidden), device="cuda", generator=gen).to(torch.bfloat16)
    logits = torch.randn((T, E), device="cuda", generator=gen)
    ids, w, _ = B.slicemoe_route_topk(logits, k, renorm=True)
    eprec = (torch.rand(E, device="cuda", generator=gen) < 0.5).to(torch.uint8)
    prec = eprec[ids.long()].contiguous()
    ws = B.new_workspace(cs)
    y_dec = B.slicemoe_layer(cs, et, st, gv, x, ids, prec, w, ws)
    for _ in range(8):   # fixed summation order and no race on the staging ring: every run gives the same bits
        assert torch.equal(B.slicemoe_layer(cs, et, st, gv, x, ids, prec, w, ws), y_dec)
    pws = B.new_prefill_workspace(cs, T)
    y_pre, status = B.slicemoe_prefill_layer(cs, et, st, gv, x, ids, w, eprec, pws)
    y_pre = y_pre.clone()
    for _ in range(4):
        assert torch.equal(B.slicemoe_prefill_layer(cs, et, st, gv, x, ids, w, eprec, pws)[0], y_pre)
    torch.cuda.synchronize()
    assert B.slicemoe_get_status(ws) == 0 and int(status.item()) == 0
    a, b = y_dec.cpu().numpy(), y_pre.cpu().numpy()
    assert np.isfinite(a).all() and np.isfinite(b).all()
    for t in range(T):
        H.assert_close(b[t], a[t], f"token {t}")
