"""slicemoe_prefill_layer (many tokens, grouped dense contraction on the tensor cores) against the float64
oracle, through the C ABI.  Same tolerance as the decode path: relative L2 error <= 1e-3 and max-abs error
<= 2e-3 x output RMS, per token."""
import numpy as np
import pytest

from oracle import amat, moe
from paper_2512_12990_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _torch():
    import torch
    return torch


def _dev(a):
    return _torch().from_numpy(np.ascontiguousarray(a)).cuda()


def _prefill(L: H.Layer, xbits, ids, w, expert_prec):
    from paper_2512_12990_b200 import binding as B
    torch = _torch()
    T = xbits.shape[0]
    ws = B.new_prefill_workspace(L.cshape, T)
    x = H.to_dev_bf16(xbits)
    y, status = B.slicemoe_prefill_layer(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, x,
                                         _dev(ids.astype(np.int32)), _dev(w.astype(np.float32)),
                                         _dev(expert_prec.astype(np.uint8)), ws)
    torch.cuda.synchronize()
    return y.cpu().numpy(), int(status.item())


def _oracle(L: H.Layer, x64, ids, w, expert_prec):
    prec = expert_prec[ids]
    return moe.layer(x64, L.oracle_list(), ids, prec, w, shared=L.oracle_shared, shared_gate_vec=L.gate_vec)


def _small_shape(group, n_shared, gated, seed):
    return synth.Shape(f"pf_small_g{group}", 256, 128, 8, 2, group, n_shared=n_shared, shared_inter=256 if n_shared else 0,
                       shared_sigmoid_gate=gated, n_layers=1, seed=seed)


@pytest.mark.parametrize("group,n_shared,gated", [(64, 0, False), (128, 1, True), (32, 2, False)])
def test_small_layers_every_token(group, n_shared, gated):
    """300 tokens over 8 experts: several 128-row tiles with ragged tails, one expert without any token,
    mixed per-expert precision; every token compared."""
    sh = _small_shape(group, n_shared, gated, 4100 + group)
    L = H.Layer(sh, range(sh.n_experts))
    T = 300
    logits = synth.router_logits_normal(sh.seed, ("pf-logits",), T, sh.n_experts)
    logits[:, 5] = -30.0                       # expert 5 is never selected
    ids, w, _ = moe.route_topk(logits, sh.top_k)
    assert not (ids == 5).any()
    expert_prec = (np.arange(sh.n_experts) % 2).astype(np.uint8)
    xbits, x64 = H.x_inputs(sh, T, "pf-x")
    y, status = _prefill(L, xbits, ids, w, expert_prec)
    assert status == 0
    y_ref = _oracle(L, x64, ids, w, expert_prec)
    for t in range(T):
        H.assert_close(y[t], y_ref[t], f"token {t}")
    # run to run bit-identical although the row a (token, expert) pair takes may differ
    y2, _ = _prefill(L, xbits, ids, w, expert_prec)
    assert np.array_equal(y, y2)
    # the precision list is honoured: flipping it changes the result by the oracle's amount
    y_flip, _ = _prefill(L, xbits, ids, w, 1 - expert_prec)
    y_flip_ref = _oracle(L, x64, ids, w, 1 - expert_prec)
    H.assert_close(y_flip, y_flip_ref, "flipped precision")
    assert np.linalg.norm(y_flip_ref - y_ref) > 50 * np.linalg.norm(y - y_ref)


@pytest.mark.parametrize("b_high,b_low", [(6, 3), (4, 2)])
def test_narrower_slice_formats_prefill(b_high, b_low):
    """MAT63 and MAT42 (Section 4.2, Table 1) through pack and the prefill kernel: 200 tokens, mixed per-expert
    precision and its flip, every token against the oracle run with the same widths."""
    sh = _small_shape(64, 1, True, 4300 + b_high)
    L = H.Layer(sh, range(sh.n_experts), b_high=b_high, b_low=b_low)
    T = 200
    logits = synth.router_logits_normal(sh.seed, ("pf-narrow-logits",), T, sh.n_experts)
    ids, w, _ = moe.route_topk(logits, sh.top_k)
    expert_prec = (np.arange(sh.n_experts) % 2).astype(np.uint8)
    xbits, x64 = H.x_inputs(sh, T, "pf-narrow-x")
    for ep in (expert_prec, 1 - expert_prec):
        y, status = _prefill(L, xbits, ids, w, ep)
        assert status == 0
        y_ref = _oracle(L, x64, ids, w, ep)
        for t in range(T):
            H.assert_close(y[t], y_ref[t], f"MAT{b_high}{b_low} token {t}")


def test_single_token_and_agreement_with_decode_kernel():
    """T = 1 (one ragged tile per expert) and T = 5: the prefill path and the batch-1 decode path agree
    with the oracle and therefore with each other."""
    from paper_2512_12990_b200 import binding as B
    torch = _torch()
    sh = synth.SHAPES["tiny"]
    L = H.Layer(sh, range(sh.n_experts))
    expert_prec = (np.arange(sh.n_experts) >= 4).astype(np.uint8)
    for T in (1, 5):
        logits = synth.router_logits_normal(sh.seed, ("pf-logits", T), T, sh.n_experts)
        ids, w, _ = moe.route_topk(logits, sh.top_k)
        xbits, x64 = H.x_inputs(sh, T, f"pf-x{T}")
        y, status = _prefill(L, xbits, ids, w, expert_prec)
        assert status == 0
        y_ref = _oracle(L, x64, ids, w, expert_prec)
        prec = expert_prec[ids]
        y_dec = B.slicemoe_layer(L.cshape, L.experts_tbl, L.shared_tbl, L.gate_vec_dev, H.to_dev_bf16(xbits),
                                 _dev(ids.astype(np.int32)), _dev(prec), _dev(w.astype(np.float32)), L.ws)
        torch.cuda.synchronize()
        for t in range(T):
            H.assert_close(y[t], y_ref[t], f"prefill T={T} token {t}")
            H.assert_close(y_dec[t].cpu().numpy(), y_ref[t], f"decode T={T} token {t}")


def test_bad_expert_id_is_reported_and_skipped():
    from paper_2512_12990_b200 import binding as B
    sh = synth.SHAPES["tiny"]
    L = H.Layer(sh, range(sh.n_experts))
    T = 4
    logits = synth.router_logits_normal(sh.seed, ("pf-bad",), T, sh.n_experts)
    ids, w, _ = moe.route_topk(logits, sh.top_k)
    xbits, x64 = H.x_inputs(sh, T, "pf-bad-x")
    expert_prec = np.ones(sh.n_experts, dtype=np.uint8)
    bad = ids.copy()
    bad[2, 1] = sh.n_experts + 3
    y, status = _prefill(L, xbits, bad, w, expert_prec)
    assert status & B.STATUS_BAD_EXPERT_ID
    # the bad pair is skipped, the rest is computed
    w_skip = w.copy()
    w_skip[2, 1] = 0.0
    y_ref = _oracle(L, x64, ids, w_skip, expert_prec)
    for t in range(T):
        H.assert_close(y[t], y_ref[t], f"token {t}")


def test_argument_checks():
    from paper_2512_12990_b200 import binding as B
    sh = synth.SHAPES["tiny"]
    cs = B.make_shape(sh.hidden, sh.inter, sh.n_experts, sh.top_k, sh.group)
    assert B.slicemoe_prefill_workspace_bytes(cs, 0) == 0
    assert B.slicemoe_prefill_workspace_bytes(cs, 16) > 0
    odd = B.make_shape(sh.hidden, 96, sh.n_experts, sh.top_k, sh.group)
    assert B.slicemoe_prefill_workspace_bytes(odd, 16) == 0
    L = H.Layer(sh, [0, 1])
    torch = _torch()
    x = torch.zeros((4, sh.hidden), dtype=torch.bfloat16, device="cuda")
    ids = torch.zeros((4, sh.top_k), dtype=torch.int32, device="cuda")
    w = torch.zeros((4, sh.top_k), dtype=torch.float32, device="cuda")
    ep = torch.zeros(sh.n_experts, dtype=torch.uint8, device="cuda")
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.SliceMoEError) as ei:
        B.slicemoe_prefill_layer(L.cshape, L.experts_tbl, None, None, x, ids, w, ep, small)
    assert ei.value.code == B.E_INVALID_ARG


# ---- the full-size prefill layer ------------------------------------------------------------------------
class _QwenPrefill:
    """2048 tokens, 60 experts x 1408, top-4, one gated shared expert of 5632; experts of even popularity rank
    are held at 4 bits, of odd rank at 8 bits.  Experts are drawn and packed on the GPU; the oracle works on the
    planes read back (slicemoe_pack is compared with the oracle's quantiser in test_gpu_pack.py)."""

    def __init__(self):
        torch = _torch()
        from paper_2512_12990_b200 import binding as B
        sh = self.sh = synth.SHAPES["qwen_prefill"]
        self.cshape = B.make_shape(sh.hidden, sh.inter, sh.n_experts, sh.top_k, sh.group, sh.n_shared,
                                   sh.shared_inter, sh.shared_sigmoid_gate)
        self.packed = [H.device_expert(sh.seed, ("prefill", e), sh.hidden, sh.inter, sh.group) for e in range(sh.n_experts)]
        self.packed_shared = [H.device_expert(sh.seed, ("prefill", "shared0"), sh.hidden, sh.shared_inter, sh.group)]
        self.experts_tbl = B.expert_table(self.packed)
        self.shared_tbl = B.expert_table(self.packed_shared)
        self.gate_vec = synth.normal_f32(sh.seed, ("gate_vec", 0), (sh.hidden,), 0.02)
        self.gate_vec_dev = torch.from_numpy(self.gate_vec).cuda()
        self.T = 2048
        logits, perm = synth.zipf_gumbel_logits(sh.seed, ("prefill-logits",), self.T, sh.n_experts, 1.0)
        self.ids, self.w, _ = moe.route_topk(logits, sh.top_k, renorm=True)
        self.expert_prec = np.zeros(sh.n_experts, dtype=np.uint8)
        self.expert_prec[perm[1::2]] = 1          # perm[r] = expert of popularity rank r
        self.perm = perm
        self.xbits, self.x64 = H.x_inputs(sh, self.T, "prefill-x")

    def oracle_rows(self, rows, monkeypatch):
        """Float64 layer output of the token rows `rows`: oracle.moe.layer as it stands, token by token.  It
        dequantises an expert anew for every (token, slot); so that this ends in reasonable time the oracle's own
        dequantiser is memoised for the duration (same function, same results, a bounded cache keyed by the matrix
        object and the precision) - no arithmetic happens on the test's side."""
        from collections import OrderedDict
        from oracle import amat
        real, cache = amat.dequant, OrderedDict()

        def memoised(mat, prec):
            key = (id(mat), int(prec))
            if key in cache:
                cache.move_to_end(key)
                return cache[key]
            cache[key] = real(mat, prec)
            if len(cache) > 30:
                cache.popitem(last=False)
            return cache[key]

        monkeypatch.setattr(amat, "dequant", memoised)
        rows = np.asarray(rows)
        # tokens that share their first expert next to each other: more of the cache's entries are used again
        order = np.lexsort((rows, self.ids[rows, 0]))
        experts = {int(e): H.oracle_expert_from_device(self.packed[int(e)]) for e in np.unique(self.ids[rows])}
        shared = [H.oracle_expert_from_device(self.packed_shared[0])]
        prec = self.expert_prec[self.ids]
        y = np.empty((len(rows), self.sh.hidden))
        for i in order:
            t = rows[i:i + 1]
            y[i] = moe.layer(self.x64[t], experts, self.ids[t], prec[t], self.w[t], shared=shared,
                             shared_gate_vec=self.gate_vec)[0]
        monkeypatch.setattr(amat, "dequant", real)
        return y


@pytest.fixture(scope="module")
def qwen_prefill():
    return _QwenPrefill()


def test_full_size_prefill_layer_sampled_tokens(qwen_prefill, monkeypatch):
    from paper_2512_12990_b200 import binding as B
    torch = _torch()
    q = qwen_prefill
    counts = np.bincount(q.ids.ravel(), minlength=q.sh.n_experts)
    assert counts.min() > 0 and counts.max() > 10 * counts.min(), "every expert is used, load is Zipf-skewed"
    ws = B.new_prefill_workspace(q.cshape, q.T)
    x = H.to_dev_bf16(q.xbits)
    args = (_dev(q.ids.astype(np.int32)), _dev(q.w.astype(np.float32)), _dev(q.expert_prec))
    y, status = B.slicemoe_prefill_layer(q.cshape, q.experts_tbl, q.shared_tbl, q.gate_vec_dev, x, *args, ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    y = y.cpu().numpy()
    assert np.isfinite(y).all()
    # 64+ token rows: one routed to each of the 60 experts (head and tail of the popularity order alike), the
    # first and last token and the tile boundaries of the shared expert
    rows = {0, 127, 128, 1000, 1777, 2047}
    for e in range(q.sh.n_experts):
        rows.add(int(np.nonzero((q.ids == e).any(1))[0][0]))
    rows = sorted(rows)
    assert len(rows) >= 40
    extra = [t for t in range(5, q.T, 61) if t not in rows][:max(0, 64 - len(rows))]
    rows = sorted(rows + extra)
    assert len(rows) >= 64 and set(np.unique(q.ids[rows])) == set(range(q.sh.n_experts))
    y_ref = q.oracle_rows(rows, monkeypatch)
    worst = 0.0
    for i, t in enumerate(rows):
        rel, _ = H.assert_close(y[t], y_ref[i], f"token {t}")
        worst = max(worst, rel)
    print(f"prefill: {len(rows)} sampled tokens, worst rel-L2 {worst:.2e}")
    # bit-reproducible
    y2, _ = B.slicemoe_prefill_layer(q.cshape, q.experts_tbl, q.shared_tbl, q.gate_vec_dev, x, *args, ws)
    torch.cuda.synchronize()
    assert np.array_equal(y, y2.cpu().numpy())
    # property that holds at any size: a token's result does not depend on the rest of the batch
    sel = np.array([0, 127, 128, 1000, 1777, 2047])
    ws_s = B.new_prefill_workspace(q.cshape, len(sel))
    y_s, _ = B.slicemoe_prefill_layer(q.cshape, q.experts_tbl, q.shared_tbl, q.gate_vec_dev,
                                      H.to_dev_bf16(q.xbits[sel]), _dev(q.ids[sel].astype(np.int32)),
                                      _dev(q.w[sel].astype(np.float32)), _dev(q.expert_prec), ws_s)
    torch.cuda.synchronize()
    assert np.array_equal(y_s.cpu().numpy(), y[sel])


def test_expert_without_lsb_planes_runs_from_the_msb_slice_and_reports_it():
    """expert_prec = 1 for an expert whose LSB planes are absent: no fault; the expert runs MSB-only and the
    status word says so (same contract as the decode path)."""
    from paper_2512_12990_b200 import binding as B
    sh = synth.SHAPES["tiny"]
    L = H.Layer(sh, range(sh.n_experts))
    stripped = []
    for e in range(sh.n_experts):
        mats = L.packed[e]
        if e == 2:   # expert 2 keeps only its MSB planes
            mats = {k: B.PackedMat(m.N, m.K, m.group, m.msb, None, m.scale, m.zp) for k, m in mats.items()}
        stripped.append(mats)
    tbl = B.expert_table(stripped)
    T = 40
    logits = synth.router_logits_normal(sh.seed, ("pf-nolsb",), T, sh.n_experts)
    logits[:, 2] += 3.0                       # expert 2 is selected often
    ids, w, _ = moe.route_topk(logits, sh.top_k)
    assert (ids == 2).sum() > 10
    xbits, x64 = H.x_inputs(sh, T, "pf-nolsb-x")
    ws = B.new_prefill_workspace(L.cshape, T)
    args = (H.to_dev_bf16(xbits), _dev(ids.astype(np.int32)), _dev(w.astype(np.float32)))
    ones = np.ones(sh.n_experts, dtype=np.uint8)
    y, status = B.slicemoe_prefill_layer(L.cshape, tbl, None, None, *args, _dev(ones), ws)
    _torch().cuda.synchronize()
    assert int(status.item()) == B.STATUS_MISSING_LSB
    eff = ones.copy()
    eff[2] = 0                                # what actually ran
    y_ref = _oracle(L, x64, ids, w, eff)
    for t in range(T):
        H.assert_close(y[t].cpu().numpy(), y_ref[t], f"token {t}")
    # asked correctly, nothing is reported
    y2, status2 = B.slicemoe_prefill_layer(L.cshape, tbl, None, None, *args, _dev(eff), ws)
    _torch().cuda.synchronize()
    assert int(status2.item()) == 0 and np.array_equal(y2.cpu().numpy(), y.cpu().numpy())


def test_large_batch_more_tokens_than_any_tile_count_assumption():
    """4,100 tokens on the tiny layer (33 tiles per expert on average, ragged): sampled tokens against the oracle,
    and the first 300 rows equal a 300-token call bit for bit."""
    sh = synth.SHAPES["tiny"]
    L = H.Layer(sh, range(sh.n_experts))
    T = 4100
    logits = synth.router_logits_normal(sh.seed, ("pf-big",), T, sh.n_experts)
    ids, w, _ = moe.route_topk(logits, sh.top_k)
    ep = (np.arange(sh.n_experts) < 4).astype(np.uint8)
    xbits, x64 = H.x_inputs(sh, T, "pf-big-x")
    y, status = _prefill(L, xbits, ids, w, ep)
    assert status == 0
    for t in (0, 1, 299, 300, 2048, 4095, 4099):
        y_ref = _oracle(L, x64[t:t + 1], ids[t:t + 1], w[t:t + 1], ep)
        H.assert_close(y[t], y_ref[0], f"token {t}")
    y300, _ = _prefill(L, xbits[:300], ids[:300], w[:300], ep)
    assert np.array_equal(y300, y[:300])


def test_wide_layer_beyond_the_decode_limits():
    """The prefill path has no cap on hidden or on the sum of intermediate widths: hidden 4224 (above the decode
    kernel's 4096), top-3 of 6 experts x 256, group 64."""
    sh = synth.Shape("pf_wide", 4224, 256, 6, 3, 64, n_shared=1, shared_inter=384, shared_sigmoid_gate=False, n_layers=1,
                     seed=4300)
    L = H.Layer.__new__(H.Layer)  # the decode workspace of H.Layer refuses this shape: build the parts by hand
    import torch
    from paper_2512_12990_b200 import binding as B
    L.shape = sh
    L.cshape = B.make_shape(sh.hidden, sh.inter, sh.n_experts, sh.top_k, sh.group, sh.n_shared, sh.shared_inter, False)
    L.oracle_experts, L.packed = {}, {}

    def make(tag, inter):
        W = synth.expert_weights(sh.seed, 0, tag, sh.hidden, inter)
        o = {k: amat.pack_matrix(W[k], sh.group) for k in ("gate", "up", "down")}
        d = {k: B.slicemoe_pack(torch.from_numpy(W[k]).cuda(), sh.group) for k in ("gate", "up", "down")}
        return o, d

    for e in range(sh.n_experts):
        L.oracle_experts[e], L.packed[e] = make(e, sh.inter)
    L.experts_tbl = B.expert_table([L.packed[e] for e in range(sh.n_experts)])
    so, sd = make("shared0", sh.shared_inter)
    L.oracle_shared, L.packed_shared = [so], [sd]
    L.shared_tbl = B.expert_table(L.packed_shared)
    L.gate_vec, L.gate_vec_dev = None, None
    T = 150
    logits = synth.router_logits_normal(sh.seed, ("pf-wide",), T, sh.n_experts)
    ids, w, _ = moe.route_topk(logits, sh.top_k, renorm=True)
    ep = np.array([1, 0, 1, 1, 0, 0], dtype=np.uint8)
    xbits, x64 = H.x_inputs(sh, T, "pf-wide-x")
    y, status = _prefill(L, xbits, ids, w, ep)
    assert status == 0
    y_ref = _oracle(L, x64, ids, w, ep)
    for t in range(T):
        H.assert_close(y[t], y_ref[t], f"token {t}")
