"""Pins for oracle/moe.py: routing and the mixed-precision FFN against brute force, closed
forms, invariants and a hand-computed case."""
import itertools
import math

import numpy as np
import pytest

from oracle import amat, moe
from paper_2512_12990_b200 import synth


# ----------------------------------------------------------------------------- routing
def _brute_topk(key, k):
    """All-pairs ranking: rank of e = #(strictly larger keys) + #(equal keys with lower index)."""
    E = len(key)
    rank = [sum(1 for j in range(E) if key[j] > key[e] or (key[j] == key[e] and j < e)) for e in range(E)]
    out = [None] * k
    for e in range(E):
        if rank[e] < k:
            out[rank[e]] = e
    return out


def test_topk_brute_force_and_ties():
    g = np.random.default_rng(5)
    for E, k in [(8, 2), (7, 7), (16, 5), (64, 6), (60, 4)]:
        logits = g.standard_normal((6, E)).astype(np.float32)
        logits[1, 3] = logits[1, 1]                       # exact ties
        logits[2, :] = 0.25                               # all equal -> ids 0..k-1
        ids, w, p = moe.route_topk(logits, k)
        for t in range(6):
            assert ids[t].tolist() == _brute_topk(logits[t].tolist(), k)
        assert ids[2].tolist() == list(range(k))
        assert np.allclose(p.sum(1), 1.0, atol=1e-12)
        assert (w.sum(1) <= 1 + 1e-12).all()
        # weights are the softmax probabilities of the chosen experts (math.exp evaluation)
        for t in range(6):
            den = math.fsum(math.exp(float(v) - float(logits[t].max())) for v in logits[t])
            for j in range(k):
                assert w[t, j] == pytest.approx(math.exp(float(logits[t, ids[t, j]]) - float(logits[t].max())) / den, rel=1e-12)
        ids_r, w_r, _ = moe.route_topk(logits, k, renorm=True)
        assert np.array_equal(ids_r, ids)
        assert np.allclose(w_r.sum(1), 1.0, atol=1e-12)
        assert np.allclose(w_r * w.sum(1, keepdims=True), w, rtol=1e-12)


def test_topk_k_equals_E_is_permutation_and_bias_semantics():
    g = np.random.default_rng(6)
    E, k = 12, 4
    logits = g.standard_normal((5, E)).astype(np.float32)
    ids, _, _ = moe.route_topk(logits, E)
    assert all(sorted(r.tolist()) == list(range(E)) for r in ids)
    ids0, w0, _ = moe.route_topk(logits, k)
    ids_b0, w_b0, _ = moe.route_topk(logits, k, bias=np.zeros(E, np.float32))
    assert np.array_equal(ids0, ids_b0) and np.array_equal(w0, w_b0)
    S = [2, 5, 7, 9, 11]
    bias = np.zeros(E, np.float32)
    bias[S] = 1e30
    ids_b, w_b, p_b = moe.route_topk(logits, k, bias=bias)
    assert all(set(r.tolist()) <= set(S) for r in ids_b)
    # bias affects selection only: weights are the unbiased probabilities of whoever was chosen
    _, _, p = moe.route_topk(logits, k)
    assert np.array_equal(p, p_b)
    assert np.array_equal(w_b, np.take_along_axis(p, ids_b.astype(np.int64), 1))
    # the float32 add decides ties: 1e30 + logit == 1e30 for every boosted expert -> index order
    assert all(r.tolist() == S[:k] for r in ids_b)
    # permutation invariance of the selected set
    perm = g.permutation(E)
    ids_p, _, _ = moe.route_topk(logits[:, perm], k)
    for t in range(5):
        assert set(perm[ids_p[t]].tolist()) == set(ids0[t].tolist())
    # NaN counts as -inf
    logits[0, 0] = np.nan
    ids_n, w_n, _ = moe.route_topk(logits, E)
    assert ids_n[0, -1] == 0 and w_n[0, -1] == 0.0


def test_precision_request():
    p = np.array([[0.5, 0.2, 0.19, 0.01], [0.1, 0.1, 0.05, 0.05]])
    assert moe.precision_request(p, 0.2).tolist() == [[1, 1, 0, 0], [0, 0, 0, 0]]
    assert moe.precision_request(p, 2.0, rank_high=3).tolist() == [[1, 1, 1, 0], [1, 1, 1, 0]]
    assert moe.precision_request(p, 0.5, rank_high=0).tolist() == [[1, 0, 0, 0], [0, 0, 0, 0]]


# ----------------------------------------------------------------------------- FFN
def _mat(scale, zp, q, group):
    q = np.asarray(q, dtype=np.uint8)
    msb, lsb = q >> 4, q & 15
    return dict(scale=np.asarray(scale, dtype=np.float16), zp=np.asarray(zp, dtype=np.uint8),
                msb=msb, lsb=lsb, group=group)


def test_silu_closed_forms():
    t = np.linspace(-20, 20, 81)
    assert moe.silu(np.array([0.0]))[0] == 0.0
    assert np.allclose(moe.silu(t) - moe.silu(-t), t, atol=1e-12)
    assert moe.silu(np.array([2.0]))[0] == pytest.approx(2.0 / (1.0 + math.exp(-2.0)), rel=1e-15)
    assert moe.silu(np.array([40.0]))[0] == pytest.approx(40.0, rel=1e-12)


def test_ffn_hand_case():
    """hidden 2, inter 1, group 2 (gate/up) and group 1 (down); everything computable on paper.
    gate: s=.25 zp=82 q=(90,115): high (2, 8.25), low (0, 8).  up: s=.5 zp=16 q=(18,15): high
    (1, -.5), low (8*(1-1), 8*(0-1)) = (0, -8).  down: s=1 zp=(0; 17) q=(2; 1): high (2; -16),
    low (16*(0-0); 16*(0-1)) = (0; -16).  x = (2, 1)."""
    ex = dict(gate=_mat([[0.25]], [[82]], [[90, 115]], 2),
              up=_mat([[0.5]], [[16]], [[18, 15]], 2),
              down=_mat([[1.0], [1.0]], [[0], [17]], [[2], [1]], 1))
    x = np.array([[2.0, 1.0]])
    g_hi, u_hi = 2 * 2 + 8.25, 2 * 1 - 0.5
    h_hi = g_hi / (1 + math.exp(-g_hi)) * u_hi
    y_hi = [2 * h_hi, -16 * h_hi]
    g_lo, u_lo = 0 * 2 + 8 * 1, 0 * 2 - 8 * 1
    h_lo = g_lo / (1 + math.exp(-g_lo)) * u_lo
    y_lo = [0 * h_lo, -16 * h_lo]
    ids = np.array([[0, 0]], dtype=np.int32)
    w = np.array([[0.75, 0.125]])
    y = moe.expert_ffn(x, [ex], ids, np.array([[1, 0]], dtype=np.uint8), w)
    expect = [0.75 * y_hi[0] + 0.125 * y_lo[0], 0.75 * y_hi[1] + 0.125 * y_lo[1]]
    assert y[0].tolist() == pytest.approx(expect, rel=1e-13)
    # shared expert with sigmoid gate
    v = np.array([0.5, -0.25], dtype=np.float32)
    c = 1 / (1 + math.exp(-(0.5 * 2 - 0.25 * 1)))
    y2 = moe.layer(x, [ex], ids, np.array([[1, 0]], dtype=np.uint8), w, shared=[ex], shared_gate_vec=v)
    assert y2[0].tolist() == pytest.approx([expect[0] + c * y_hi[0], expect[1] + c * y_hi[1]], rel=1e-13)
    y3 = moe.layer(x, [ex], ids, np.array([[1, 0]], dtype=np.uint8), w, shared=[ex, ex])
    assert y3[0].tolist() == pytest.approx([expect[0] + 2 * y_hi[0], expect[1] + 2 * y_hi[1]], rel=1e-13)


def _tiny_layer(seed=1001, hidden=64, inter=48, E=4, group=16):
    experts = []
    for e in range(E):
        W = synth.expert_weights(seed, 0, e, hidden, inter)
        experts.append({k: amat.pack_matrix(W[k], group) for k in ("gate", "up", "down")})
    return experts


def _dense_loops(x, s, zp, codes, group, code_scale):
    """Scalar-loop dequant + matvec with exact summation (math.fsum); an independent evaluation."""
    N, K = codes.shape
    out = []
    for n in range(N):
        terms = []
        for k in range(K):
            g = k // group
            terms.append(float(s[n, g]) * code_scale * (int(codes[n, k]) - int(zp[n, g])) * float(x[k]))
        out.append(math.fsum(terms))
    return np.array(out)


def test_ffn_matches_independent_dense_evaluation():
    """All flags 1 == dense FFN on the 8-bit dequantised weights; all flags 0 == dense FFN on the
    4-bit ones; evaluated here with scalar loops and exact summation, not the oracle's matmul."""
    hidden, inter, E, group = 64, 48, 4, 16
    experts = _tiny_layer(hidden=hidden, inter=inter, E=E, group=group)
    x = synth.bf16_to_f64(synth.activations_bf16(1001, ("x",), (1, hidden)))
    for prec in (1, 0):
        ex = experts[2]
        def mv(mat, vec):
            if prec:
                codes = mat["msb"].astype(int) * 16 + mat["lsb"]
                return _dense_loops(vec, mat["scale"], mat["zp"], codes, group, 1.0)
            return _dense_loops(vec, mat["scale"], mat["zp"] // 16, mat["msb"], group, 16.0)
        g = mv(ex["gate"], x[0])
        u = mv(ex["up"], x[0])
        h = np.array([gi / (1 + math.exp(-gi)) * ui for gi, ui in zip(g, u)])
        y_ref = mv(ex["down"], h)
        y = moe.expert_ffn(x, experts, np.array([[2]], np.int32), np.array([[prec]], np.uint8), np.array([[1.0]]))
        assert np.allclose(y[0], y_ref, rtol=1e-11, atol=1e-14)
        assert np.linalg.norm(y[0]) > 0


def test_ffn_invariants():
    hidden, inter, E, group = 64, 48, 4, 16
    experts = _tiny_layer(hidden=hidden, inter=inter, E=E, group=group)
    x = synth.bf16_to_f64(synth.activations_bf16(1001, ("x",), (2, hidden)))
    ids = np.array([[1, 3], [0, 2]], np.int32)
    prec = np.array([[1, 0], [0, 1]], np.uint8)
    w = np.array([[0.6, 0.3], [0.2, 0.1]])
    y = moe.expert_ffn(x, experts, ids, prec, w)
    assert y.shape == (2, hidden)
    # x = 0 -> y = 0
    assert np.array_equal(moe.expert_ffn(np.zeros_like(x), experts, ids, prec, w), np.zeros_like(y))
    # linear in the combine weights
    y2 = moe.expert_ffn(x, experts, ids, prec, 2.5 * w)
    assert np.allclose(y2, 2.5 * y, rtol=1e-13)
    ya = moe.expert_ffn(x, experts, ids[:, :1], prec[:, :1], w[:, :1])
    yb = moe.expert_ffn(x, experts, ids[:, 1:], prec[:, 1:], w[:, 1:])
    assert np.allclose(ya + yb, y, rtol=1e-12, atol=1e-15)
    # precision flag matters, and by about the size the slice identity predicts (not zero, not huge)
    y_all8 = moe.expert_ffn(x, experts, ids, np.ones_like(prec), w)
    y_all4 = moe.expert_ffn(x, experts, ids, np.zeros_like(prec), w)
    rel = np.linalg.norm(y_all8 - y_all4) / np.linalg.norm(y_all8)
    assert 1e-3 < rel < 0.5
    # per-token independence
    y_t1 = moe.expert_ffn(x[1:], experts, ids[1:], prec[1:], w[1:])
    assert np.array_equal(y_t1[0], y[1])
    # non-square shapes: a transposed operand cannot go unnoticed
    assert experts[0]["gate"]["msb"].shape == (inter, hidden)
    assert experts[0]["down"]["msb"].shape == (hidden, inter)


def test_algorithmic_bytes_of_a_1408_wide_expert():
    """1408-wide expert at group 128: 8-bit 8,853,504 B, 4-bit 4,528,128 B (3 matrices)."""
    mat_gu = dict(msb=np.zeros((1408, 2048), np.uint8), group=128)
    mat_d = dict(msb=np.zeros((2048, 1408), np.uint8), group=128)
    b8 = 2 * moe.algorithmic_bytes(mat_gu, 1) + moe.algorithmic_bytes(mat_d, 1)
    b4 = 2 * moe.algorithmic_bytes(mat_gu, 0) + moe.algorithmic_bytes(mat_d, 0)
    assert (b8, b4) == (8853504, 4528128)
