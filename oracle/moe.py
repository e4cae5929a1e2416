"""Oracle: routing and the mixed-precision expert FFN.  Test infrastructure only.

Section 4.1 of the paper: experts whose gating score makes them critical request both slices
and run at full precision; the others run from the MSB slice alone.  The FFN result is defined
by the dequantised weights, so the oracle is that definition in float64.
"""
from __future__ import annotations

import numpy as np

from . import amat


def softmax64(logits: np.ndarray) -> np.ndarray:
    """Softmax over the last axis in float64; NaN logits count as -inf."""
    z = np.asarray(logits, dtype=np.float64).copy()
    z[np.isnan(z)] = -np.inf
    m = z.max(axis=-1, keepdims=True)
    e = np.exp(z - m)
    return e / e.sum(axis=-1, keepdims=True)


def route_topk(logits: np.ndarray, k: int, bias: np.ndarray | None = None, renorm: bool = False):
    """Top-k gating (Section 1) with an optional cache-priority bias (Section 2.1: Cache-Prior
    boosts the gating scores of cached experts).

    logits float32 [T, E]; bias float32 [E] or None.
      p    = softmax(logits) over all E experts               (float64, bias NOT included)
      key  = float32(logits) + float32(bias)                  (one float32 add; NaN -> -inf)
      ids  = the k largest keys, ties -> lower expert index, listed by descending key
      w    = p[ids], divided by their sum when renorm
    Returns (ids int32 [T, k], w float64 [T, k], p float64 [T, E]).
    """
    logits = np.asarray(logits, dtype=np.float32)
    T, E = logits.shape
    assert 1 <= k <= E
    key = logits.copy()
    if bias is not None:
        key = (key + np.asarray(bias, dtype=np.float32)[None, :]).astype(np.float32)
    key[np.isnan(key)] = -np.inf
    p = softmax64(logits)
    ids = np.empty((T, k), dtype=np.int32)
    for t in range(T):
        order = np.argsort(-key[t].astype(np.float64), kind="stable")   # ties keep index order
        ids[t] = order[:k]
    w = np.take_along_axis(p, ids.astype(np.int64), axis=1)
    if renorm:
        w = w / w.sum(axis=1, keepdims=True)
    return ids, w, p


def precision_request(p_selected: np.ndarray, tau: float, rank_high: int = 0) -> np.ndarray:
    """Precision on demand (Section 4.1): a selected expert is critical, and requests MSB+LSB
    (flag 1), when its gating score is high; otherwise it requests the MSB slice only (flag 0).

    The paper does not print its threshold; the reading here: critical iff the (unbiased,
    un-renormalised) softmax probability >= tau, or the expert is among the first `rank_high`
    of the selection (a fixed top-n allocation, the conventional scheme the paper contrasts
    with).  p_selected [T, k] listed by descending selection key."""
    T, k = p_selected.shape
    flags = (p_selected >= tau)
    if rank_high > 0:
        flags = flags | (np.arange(k)[None, :] < rank_high)
    return flags.astype(np.uint8)


def silu(t: np.ndarray) -> np.ndarray:
    return t / (1.0 + np.exp(-t))


def expert_ffn_one(x64: np.ndarray, expert: dict, prec: int) -> np.ndarray:
    """One SwiGLU expert on one token at one precision (Section 4.1):
        Wd ( silu(Wg x) * (Wu x) ),  W = dequantised at `prec` (1 = MSB+LSB, 0 = MSB only).
    expert = dict(gate=mat, up=mat, down=mat), mat as returned by amat.pack_matrix."""
    Wg = amat.dequant(expert["gate"], prec)
    Wu = amat.dequant(expert["up"], prec)
    Wd = amat.dequant(expert["down"], prec)
    h = silu(Wg @ x64) * (Wu @ x64)
    return Wd @ h


def expert_ffn(x64: np.ndarray, experts, ids: np.ndarray, prec: np.ndarray, w: np.ndarray) -> np.ndarray:
    """Routed part of the MoE layer:  y[t] = sum_j w[t, j] * FFN_{ids[t, j]}(x[t]) at prec[t, j].

    x64 [T, hidden] float64 (the bf16 activations, exactly); experts: sequence indexable by id.
    Returns float64 [T, hidden]."""
    T = x64.shape[0]
    k = ids.shape[1]
    y = np.zeros((T, expert_out_dim(experts, ids)), dtype=np.float64)
    for t in range(T):
        for j in range(k):
            e = int(ids[t, j])
            y[t] += float(w[t, j]) * expert_ffn_one(x64[t], experts[e], int(prec[t, j]))
    return y


def expert_out_dim(experts, ids) -> int:
    e = experts[int(ids.reshape(-1)[0])]
    return e["down"]["msb"].shape[0]


def layer(x64, experts, ids, prec, w, shared=(), shared_gate_vec=None) -> np.ndarray:
    """Whole MoE layer: routed experts plus always-on shared experts at full precision.

    The shared experts are part of the two evaluated model architectures, not of the paper's
    method: each adds FFN_8bit(x) with weight 1, or with weight sigmoid(v . x) when a gate
    vector v (float32 [hidden]) is given."""
    y = expert_ffn(x64, experts, ids, prec, w)
    for t in range(x64.shape[0]):
        for sh in shared:
            c = 1.0
            if shared_gate_vec is not None:
                c = 1.0 / (1.0 + np.exp(-float(np.asarray(shared_gate_vec, dtype=np.float64) @ x64[t])))
            y[t] += c * expert_ffn_one(x64[t], sh, 1)
    return y


def algorithmic_bytes(mat: dict, prec: int) -> int:
    """Bytes a decode step must read for one matrix: the slice planes used (4 bits per weight
    each) plus the fp16 scale and u8 zero-point per group."""
    N, K = mat["msb"].shape
    planes = 2 if prec else 1
    return planes * (N * K // 2) + (N * K // mat["group"]) * 3
