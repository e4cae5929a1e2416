"""slicemoe_expert_ffn / slicemoe_layer on the GPU against the float64 oracle, through the C ABI.

Tolerance: relative L2 error <= 1e-3 and max-abs error <= 2e-3 x output RMS."""
import numpy as np
import pytest

from oracle import moe
from paper_2512_12990_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _torch():
    import torch
    return torch


def _dev(a, dtype=None):
    t = _torch().from_numpy(np.ascontiguousarray(a)).cuda()
    return t


def _run_layer(L: H.Layer, xbits, ids, prec, w, use_layer=True):
    from paper_2512_12990_b200 import binding as B
    torch = _torch()
    x = H.to_dev_bf16(xbits)
    args = (_dev(ids.astype(np.int32)), _dev(prec.astype(np.uint8)), _dev(w.astype(np.float32)))
    if use_layer:
        y = B.slicemoe_layer(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x, *args, L.ws)
    else:
        y = B.slicemoe_expert_ffn(L.cshape, L.experts_tbl, x, *args, L.ws)
    torch.cuda.synchronize()
    status = B.slicemoe_get_status(L.ws)
    return y.cpu().numpy(), status


def test_tiny_config_single_token_mixed_precision():
    """Config 1: hidden 256, 8 experts x 128, top-2, group 64; experts 0-3 run 4-bit, 4-7 run 8-bit."""
    sh = synth.SHAPES["tiny"]
    L = H.Layer(sh, range(sh.n_experts))
    # find a token whose top-2 holds one expert of each precision
    for t in range(64):
        logits = synth.router_logits_normal(sh.seed, ("logits", t), 1, sh.n_experts)
        ids, w, _ = moe.route_topk(logits, sh.top_k)
        if (ids[0] >= 4).sum() == 1:
            break
    prec = (ids >= 4).astype(np.uint8)
    xbits, x64 = H.x_inputs(sh, 1)
    y, status = _run_layer(L, xbits, ids, prec, w, use_layer=False)
    y_ref = moe.expert_ffn(x64, L.oracle_list(), ids, prec, w)
    assert status == 0
    H.assert_close(y, y_ref, "tiny T=1")
    # the precision flag is honoured: all-8-bit differs from the mixed result by the oracle's amount
    y8, _ = _run_layer(L, xbits, ids, np.ones_like(prec), w, use_layer=False)
    y8_ref = moe.expert_ffn(x64, L.oracle_list(), ids, np.ones_like(prec), w)
    H.assert_close(y8, y8_ref, "tiny all 8-bit")
    assert np.linalg.norm(y8_ref - y_ref) > 50 * np.linalg.norm(y - y_ref)


def test_tiny_config_eight_tokens_all_experts_and_determinism():
    sh = synth.SHAPES["tiny"]
    L = H.Layer(sh, range(sh.n_experts))
    T = 8
    logits = synth.router_logits_normal(sh.seed, ("logits8",), T, sh.n_experts)
    ids, w, _ = moe.route_topk(logits, sh.top_k)
    ids[:, 0] = np.arange(8)                     # every expert appears
    ids[:, 1] = (np.arange(8) + 3) % 8
    prec = (ids >= 4).astype(np.uint8)
    xbits, x64 = H.x_inputs(sh, T, "x8")
    y, status = _run_layer(L, xbits, ids, prec, w, use_layer=False)
    y_ref = moe.expert_ffn(x64, L.oracle_list(), ids, prec, w)
    assert status == 0
    for t in range(T):
        H.assert_close(y[t], y_ref[t], f"tiny token {t}")
    y2, _ = _run_layer(L, xbits, ids, prec, w, use_layer=False)
    assert np.array_equal(y, y2), "fixed summation order: two runs must be bit-identical"
    # x = 0 -> y = 0 exactly
    y0, _ = _run_layer(L, np.zeros_like(xbits), ids, prec, w, use_layer=False)
    assert np.array_equal(y0, np.zeros_like(y0))


@pytest.mark.parametrize("group", [32, 64, 128])
@pytest.mark.parametrize("hidden,inter", [(128, 128), (384, 640), (2176, 128)])
def test_small_shapes_groups_and_ragged_tiles(group, hidden, inter):
    """Shapes that exercise one tile, odd tile counts and a K larger than one ring stage."""
    sh = synth.Shape("s", hidden, inter, 5, 3, group, n_shared=1, shared_inter=256, seed=2000 + group)
    L = H.Layer(sh, range(5))
    ids = np.array([[4, 0, 2]], dtype=np.int32)
    prec = np.array([[1, 0, 1]], dtype=np.uint8)
    w = np.array([[0.5, 0.3, 0.2]])
    xbits, x64 = H.x_inputs(sh, 1)
    y, status = _run_layer(L, xbits, ids, prec, w)
    y_ref = moe.layer(x64, L.oracle_list(), ids, prec, w, shared=L.oracle_shared)
    assert status == 0
    H.assert_close(y, y_ref, f"g{group} {hidden}x{inter}")


def test_dsv2_decode_layer_config():
    """Config 2: hidden 2048, 64 x 1408, top-6, 2 shared (8-bit), group 128; of the 6 selected the 3
    with the lowest gating weight run 4-bit."""
    sh = synth.SHAPES["dsv2"]
    logits = synth.router_logits_normal(sh.seed, ("logits",), 1, sh.n_experts)
    ids, w, _ = moe.route_topk(logits, sh.top_k)
    prec = moe.precision_request(w, 2.0, rank_high=3)
    L = H.Layer(sh, ids[0])
    xbits, x64 = H.x_inputs(sh, 1)
    y, status = _run_layer(L, xbits, ids, prec, w)
    y_ref = moe.layer(x64, L.oracle_list(), ids, prec, w, shared=L.oracle_shared)
    assert status == 0
    rel, mx = H.assert_close(y, y_ref, "dsv2 layer")
    print(f"dsv2 layer: rel_l2={rel:.2e} max_abs/rms={mx:.2e}")
    # routed part alone through slicemoe_expert_ffn
    yr, _ = _run_layer(L, xbits, ids, prec, w, use_layer=False)
    H.assert_close(yr, moe.expert_ffn(x64, L.oracle_list(), ids, prec, w), "dsv2 routed")
    # GPU routing + GPU FFN chained on the device
    from paper_2512_12990_b200 import binding as B
    torch = _torch()
    ids_d, w_d, pr_d = B.slicemoe_route_topk(torch.from_numpy(logits).cuda(), sh.top_k, rank_high=3)
    y2 = B.slicemoe_layer(L.cshape, L.experts_tbl, L.shared_tbl, None, H.to_dev_bf16(xbits), ids_d, pr_d, w_d, L.ws)
    torch.cuda.synchronize()
    assert np.array_equal(ids_d.cpu().numpy(), ids) and np.array_equal(pr_d.cpu().numpy(), prec)
    H.assert_close(y2.cpu().numpy(), y_ref, "dsv2 chained")


def test_qwen_decode_layer_config():
    """Config 3: hidden 2048, 60 x 1408, top-4, one shared expert 5632 scaled by sigmoid(v.x);
    per-expert precision Bernoulli(0.6) for 4-bit."""
    sh = synth.SHAPES["qwen"]
    logits = synth.router_logits_normal(sh.seed, ("logits",), 1, sh.n_experts)
    ids, w, _ = moe.route_topk(logits, sh.top_k)
    four_bit = synth.rng(sh.seed, "prec").random(sh.n_experts) < 0.6
    prec = (~four_bit[ids]).astype(np.uint8)
    L = H.Layer(sh, ids[0])
    xbits, x64 = H.x_inputs(sh, 1)
    y, status = _run_layer(L, xbits, ids, prec, w)
    y_ref = moe.layer(x64, L.oracle_list(), ids, prec, w, shared=L.oracle_shared, shared_gate_vec=L.gate_vec)
    assert status == 0
    rel, mx = H.assert_close(y, y_ref, "qwen layer")
    print(f"qwen layer: rel_l2={rel:.2e} max_abs/rms={mx:.2e}")
    # host-buffer entry point (pinned host in/out) gives the same result
    from paper_2512_12990_b200 import binding as B
    torch = _torch()
    xh = torch.from_numpy(xbits.view(np.int16).copy()).view(torch.bfloat16)[0].pin_memory()
    lh = torch.from_numpy(logits[0].copy()).pin_memory()
    yh = torch.empty(sh.hidden, dtype=torch.float32).pin_memory()
    B.slicemoe_decode_step_host(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, xh, lh, yh, L.ws, tau=2.0,
                                rank_high=0)
    y4 = moe.layer(x64, L.oracle_list(), ids, np.zeros_like(prec), w, shared=L.oracle_shared, shared_gate_vec=L.gate_vec)
    H.assert_close(yh.numpy(), y4[0], "qwen host step (all routed 4-bit)")
    # pageable host buffers take the staged path (pinned y is written by the kernel directly): same bits
    yp = torch.empty(sh.hidden, dtype=torch.float32)
    B.slicemoe_decode_step_host(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, xh.clone(), lh.clone(), yp, L.ws,
                                tau=2.0, rank_high=0)
    assert torch.equal(yp, yh)
    # x and the logits in ONE pinned buffer (logits_host = None): a single host-to-device copy, same bits
    both = torch.empty(2 * sh.hidden + 4 * sh.n_experts, dtype=torch.uint8).pin_memory()
    both[:2 * sh.hidden] = xh.view(torch.uint8)
    both[2 * sh.hidden:] = lh.view(torch.uint8)
    y1 = torch.empty(sh.hidden, dtype=torch.float32).pin_memory()
    B.slicemoe_decode_step_host(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, both, None, y1, L.ws, tau=2.0,
                                rank_high=0)
    assert torch.equal(y1, yh)


def test_bad_expert_id_is_skipped_and_reported():
    sh = synth.SHAPES["tiny"]
    L = H.Layer(sh, range(sh.n_experts))
    ids = np.array([[3, 99]], dtype=np.int32)
    prec = np.array([[1, 1]], dtype=np.uint8)
    w = np.array([[0.7, 0.3]])
    xbits, x64 = H.x_inputs(sh, 1)
    y, status = _run_layer(L, xbits, ids, prec, w, use_layer=False)
    from paper_2512_12990_b200 import binding as B
    assert status & B.STATUS_BAD_EXPERT_ID
    y_ref = moe.expert_ffn(x64, L.oracle_list(), ids[:, :1], prec[:, :1], w[:, :1])
    H.assert_close(y, y_ref, "bad id skipped")
    # all ids bad -> zero output, workspace still usable afterwards
    y, status = _run_layer(L, xbits, np.array([[-1, 8]], dtype=np.int32), prec, w, use_layer=False)
    assert status & B.STATUS_BAD_EXPERT_ID and np.array_equal(y, np.zeros_like(y))
    y, status = _run_layer(L, xbits, ids[:, :1].repeat(2, 1), prec, w, use_layer=False)
    assert status == 0


@pytest.mark.parametrize("name", ["dsv2", "qwen"])
def test_layer_routed_is_route_then_layer_in_one_launch(name):
    """slicemoe_layer_routed: the lists it reports are those of slicemoe_route_topk, bit for bit, and y equals
    slicemoe_layer run on them, bit for bit; and y is within tolerance of the oracle."""
    from paper_2512_12990_b200 import binding as B
    torch = _torch()
    sh = synth.SHAPES[name]
    T = 3
    logits = synth.router_logits_normal(sh.seed, ("routed-logits",), T, sh.n_experts)
    bias = synth.normal_f32(sh.seed, ("routed-bias",), (sh.n_experts,), 0.5)
    ids_o, w_o, _ = moe.route_topk(logits, sh.top_k, bias=bias, renorm=True)
    L = H.Layer(sh, set(ids_o.ravel().tolist()))
    xbits, x64 = H.x_inputs(sh, T, "routed-x")
    x = H.to_dev_bf16(xbits)
    dl, db = _dev(logits), _dev(bias)
    kw = dict(bias=db, renorm=True, tau=0.2, rank_high=1)
    ids, w, pr = B.slicemoe_route_topk(dl, sh.top_k, **kw)
    y_sep = B.slicemoe_layer(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x, ids, pr, w, L.ws)
    y_fused, ids_f, pr_f, w_f = B.slicemoe_layer_routed(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x, dl, L.ws, **kw)
    torch.cuda.synchronize()
    assert B.slicemoe_get_status(L.ws) == 0
    assert torch.equal(ids, ids_f) and torch.equal(pr, pr_f) and torch.equal(w, w_f)
    assert torch.equal(y_sep, y_fused)
    assert np.array_equal(ids.cpu().numpy(), ids_o)
    prec = pr.cpu().numpy()
    assert prec[:, 0].all() and 0 < prec.sum() < prec.size      # rank_high = 1; tau splits the rest
    y_ref = moe.layer(x64, L.oracle_list(), ids_o, prec, w_o, shared=L.oracle_shared, shared_gate_vec=L.gate_vec)
    for t in range(T):
        H.assert_close(y_fused[t].cpu().numpy(), y_ref[t], f"{name} routed token {t}")
    # without the lists
    y2, i2, _, _ = B.slicemoe_layer_routed(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x, dl, L.ws,
                                           want_lists=False, **kw)
    torch.cuda.synchronize()
    assert i2 is None and torch.equal(y2, y_fused)


def test_decode_reports_an_expert_without_lsb_planes_asked_for_8_bits():
    """No fault and a status bit (the output is documented as invalid); asked for 4 bits the same table is fine."""
    from paper_2512_12990_b200 import binding as B
    torch = _torch()
    sh = synth.SHAPES["tiny"]
    L = H.Layer(sh, range(sh.n_experts))
    stripped = []
    for e in range(sh.n_experts):
        mats = L.packed[e]
        if e == 1:
            mats = {k: B.PackedMat(m.N, m.K, m.group, m.msb, None, m.scale, m.zp) for k, m in mats.items()}
        stripped.append(mats)
    tbl = B.expert_table(stripped)
    ids = np.array([[1, 6]], dtype=np.int32)
    w = np.array([[0.6, 0.4]], dtype=np.float32)
    xbits, x64 = H.x_inputs(sh, 1, "nolsb-x")
    x = H.to_dev_bf16(xbits)
    y = B.slicemoe_expert_ffn(L.cshape, tbl, x, _dev(ids), _dev(np.array([[1, 1]], dtype=np.uint8)), _dev(w), L.ws)
    torch.cuda.synchronize()
    assert B.slicemoe_get_status(L.ws) == B.STATUS_MISSING_LSB
    assert torch.isfinite(y).all()
    ws2 = B.new_workspace(L.cshape)
    prec = np.array([[0, 1]], dtype=np.uint8)
    y = B.slicemoe_expert_ffn(L.cshape, tbl, x, _dev(ids), _dev(prec), _dev(w), ws2)
    torch.cuda.synchronize()
    assert B.slicemoe_get_status(ws2) == 0
    H.assert_close(y.cpu().numpy(), moe.expert_ffn(x64, L.oracle_list(), ids, prec, w.astype(np.float64)), "4-bit from MSB only")


def test_maximum_sizes_of_the_decode_kernel():
    """hidden 4096 (the limit), top-16 (the limit) of 20 experts x 640 plus 4 shared experts (the limit) x 512:
    the intermediate widths sum to 12288, exactly the capacity of the workspace; one more column is refused."""
    from paper_2512_12990_b200 import binding as B
    torch = _torch()
    sh = synth.Shape("max", 4096, 640, 20, 16, 128, n_shared=4, shared_inter=512, shared_sigmoid_gate=True, seed=2900)
    assert sh.top_k * sh.inter + sh.n_shared * sh.shared_inter == 12288
    logits = synth.router_logits_normal(sh.seed, ("max-logits",), 1, sh.n_experts)
    ids, w, _ = moe.route_topk(logits, sh.top_k)
    L = H.Layer(sh, ids.ravel().tolist())
    prec = (np.arange(sh.top_k)[None, :] % 3 == 0).astype(np.uint8)
    xbits, x64 = H.x_inputs(sh, 1, "max-x")
    y, status = _run_layer(L, xbits, ids, prec, w)
    assert status == 0
    y_ref = moe.layer(x64, L.oracle_list(), ids, prec, w, shared=L.oracle_shared, shared_gate_vec=L.gate_vec)
    H.assert_close(y, y_ref, "maximum sizes")
    # beyond the limits: refused on the host, nothing launched
    x = H.to_dev_bf16(xbits)
    args = (_dev(ids.astype(np.int32)), _dev(prec), _dev(w.astype(np.float32)))
    wide = B.make_shape(4096, 768, 20, 16, 128, 4, 512, True)          # 16 * 768 + 4 * 512 > 12288
    with pytest.raises(B.SliceMoEError) as ei:
        B.slicemoe_layer(wide, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x, *args, L.ws)
    assert ei.value.code == B.E_UNSUPPORTED
    tall = B.make_shape(4224, 640, 20, 16, 128, 4, 512, True)          # hidden > 4096
    with pytest.raises(B.SliceMoEError) as ei:
        B.slicemoe_layer(tall, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x, *args, L.ws)
    assert ei.value.code == B.E_UNSUPPORTED
    torch.cuda.synchronize()
    assert B.slicemoe_get_status(L.ws) == 0


@pytest.mark.parametrize("name", ["tiny", "dsv2", "qwen"])
def test_resident_lists_give_the_same_bits(name):
    """slicemoe_layer_flags(SLICEMOE_LISTS_RESIDENT): the kernel plans and requests the routed tiles before the
    work ahead of it has finished.  A chain of launches over several tokens (each launch overlaps the one before)
    must give, bit for bit, what slicemoe_layer gives - and what the oracle gives within the tolerance."""
    from paper_2512_12990_b200 import binding as B
    torch = _torch()
    sh = synth.SHAPES[name]
    T = 6
    logits = synth.router_logits_normal(sh.seed, ("resident-logits",), T, sh.n_experts)
    ids, w, _ = moe.route_topk(logits, sh.top_k)
    prec = (np.arange(sh.top_k)[None, :] < (1 + np.arange(T)[:, None]) % (sh.top_k + 1)).astype(np.uint8)
    L = H.Layer(sh, sorted(set(ids.ravel().tolist())))
    xbits, x64 = H.x_inputs(sh, T, "resident-x")
    x = H.to_dev_bf16(xbits)
    args = (_dev(ids.astype(np.int32)), _dev(prec), _dev(w.astype(np.float32)))
    torch.cuda.synchronize()   # the lists are complete before anything of the chain is enqueued
    y0 = B.slicemoe_layer(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x, *args, L.ws)
    y1 = B.slicemoe_layer(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x, *args, L.ws,
                          flags=B.LISTS_RESIDENT)
    torch.cuda.synchronize()
    assert B.slicemoe_get_status(L.ws) == 0
    assert torch.equal(y0, y1)
    y_ref = moe.layer(x64, L.oracle_list(), ids, prec, w, shared=L.oracle_shared, shared_gate_vec=L.gate_vec)
    H.assert_close(y1.cpu().numpy(), y_ref, f"{name} resident lists")
    # as a cooperative grid (the driver guarantees co-residency): the same bits again
    y2 = B.slicemoe_layer(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x, *args, L.ws, flags=B.COOPERATIVE)
    y3 = B.slicemoe_layer(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x, *args, L.ws,
                          flags=B.COOPERATIVE | B.LISTS_RESIDENT)
    torch.cuda.synchronize()
    assert B.slicemoe_get_status(L.ws) == 0
    assert torch.equal(y0, y2) and torch.equal(y0, y3)
    # an unknown flag is refused
    with pytest.raises(B.SliceMoEError):
        B.slicemoe_layer(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x, *args, L.ws, flags=4)


@pytest.mark.parametrize("name", ["tiny", "dsv2", "qwen"])
def test_stream_probe_moves_the_algorithmic_bytes(name):
    """slicemoe_stream_probe has to request exactly the bytes the oracle's byte count gives for the list
    (it is the ruler the decode kernel is measured against), in both launch modes, without a wait running out."""
    from paper_2512_12990_b200 import binding as B
    torch = _torch()
    sh = synth.SHAPES[name]
    logits = synth.router_logits_normal(sh.seed, ("probe-logits",), 1, sh.n_experts)
    ids, _, _ = moe.route_topk(logits, sh.top_k)
    prec = (np.arange(sh.top_k) < (sh.top_k + 1) // 2).astype(np.uint8)
    L = H.Layer(sh, sorted(set(ids.ravel().tolist())))
    olist = L.oracle_list()
    mats = ("gate", "up", "down")
    want = sum(moe.algorithmic_bytes(olist[int(e)][m], int(pr)) for e, pr in zip(ids[0], prec) for m in mats)
    want += sum(moe.algorithmic_bytes(ex[m], 1) for ex in (L.oracle_shared or []) for m in mats)
    got = torch.zeros(1, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ids_d, prec_d = _dev(ids[0].astype(np.int32)), _dev(prec)
    for dependent in (True, False, True):
        B.slicemoe_stream_probe(L.cshape, L.experts_tbl, L.shared_tbl, ids_d, prec_d, dependent, got, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert int(got.item()) == 3 * want


@pytest.mark.parametrize("name,rank_high", [("dsv2", 3), ("qwen", 2)])
@pytest.mark.parametrize("token", [0, 1, 2])
def test_full_size_decode_three_tokens_three_precision_mixes(name, rank_high, token):
    """Configs 2 and 3 at full size, element by element against the oracle: three independently drawn tokens
    (routing, activations, and so the experts that are read), each at the benchmark's mix, with every routed expert
    at 8 bits, with every routed expert at 4 bits, and with the same expert in two slots at different precisions."""
    sh = synth.SHAPES[name]
    logits = synth.router_logits_normal(sh.seed, ("full-logits", token), 1, sh.n_experts)
    ids, w, _ = moe.route_topk(logits, sh.top_k)
    L = H.Layer(sh, ids[0], layer=token)
    xbits, x64 = H.x_inputs(sh, 1, f"full-x{token}")
    mixes = {"mixed": moe.precision_request(w, 2.0, rank_high=rank_high), "all 8-bit": np.ones_like(ids, dtype=np.uint8),
             "all 4-bit": np.zeros_like(ids, dtype=np.uint8)}
    outs = {}
    for label, prec in mixes.items():
        y, status = _run_layer(L, xbits, ids, prec, w)
        y_ref = moe.layer(x64, L.oracle_list(), ids, prec, w, shared=L.oracle_shared, shared_gate_vec=L.gate_vec)
        assert status == 0
        H.assert_close(y, y_ref, f"{name} token {token} {label}")
        outs[label] = y_ref
    # the mixes are different computations: the oracle's results are further apart than the tolerance
    assert np.linalg.norm(outs["all 8-bit"] - outs["all 4-bit"]) > 1e-2 * np.linalg.norm(outs["all 8-bit"])
    # the same expert twice: slot 1 repeats slot 0's expert, at the other precision and with its own weight
    ids2 = ids.copy()
    ids2[0, 1] = ids2[0, 0]
    prec2 = mixes["mixed"].copy()
    prec2[0, 0], prec2[0, 1] = 1, 0
    y, status = _run_layer(L, xbits, ids2, prec2, w)
    y_ref = moe.layer(x64, L.oracle_list(), ids2, prec2, w, shared=L.oracle_shared, shared_gate_vec=L.gate_vec)
    assert status == 0
    H.assert_close(y, y_ref, f"{name} token {token} same expert twice")


@pytest.mark.parametrize("b_high,b_low", [(6, 3), (4, 2)])
@pytest.mark.parametrize("name", ["tiny", "dsv2"])
def test_narrower_slice_formats_decode(name, b_high, b_low):
    """MAT63 and MAT42 (Section 4.2, Table 1) through pack and the decode kernel: the layer at the mixed precision
    list, all from both slices and all from the MSB slice alone, against the oracle run with the same widths."""
    sh = synth.SHAPES[name]
    logits = synth.router_logits_normal(sh.seed, ("narrow-logits", b_high), 1, sh.n_experts)
    ids, w, _ = moe.route_topk(logits, sh.top_k)
    L = H.Layer(sh, ids[0], b_high=b_high, b_low=b_low)
    xbits, x64 = H.x_inputs(sh, 1, f"narrow-x{b_high}")
    half = (np.arange(sh.top_k)[None, :] < (sh.top_k + 1) // 2).astype(np.uint8)
    refs = {}
    for label, prec in (("mixed", half), ("both slices", np.ones_like(half)), ("MSB only", np.zeros_like(half))):
        y, status = _run_layer(L, xbits, ids, prec, w)
        y_ref = moe.layer(x64, L.oracle_list(), ids, prec, w, shared=L.oracle_shared, shared_gate_vec=L.gate_vec)
        assert status == 0
        H.assert_close(y, y_ref, f"{name} MAT{b_high}{b_low} {label}")
        refs[label] = y_ref
    # the low-bit result really is a different (coarser) model
    assert np.linalg.norm(refs["both slices"] - refs["MSB only"]) > 2e-2 * np.linalg.norm(refs["both slices"])
