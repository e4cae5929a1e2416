"""Oracle: the cache-aware routing baselines the paper compares with (Section 2.1; Section 6.1, "Baseline MoE
Acceleration").  Test infrastructure only.

Cache-Prior boosts the gating scores of experts already in DRAM; Cumsum takes a candidate set from the top gating
scores and prefers the cached ones among it.  The paper gives neither formula (they are the cited work's).
Readings:
  * Cache-Prior: a constant `delta` is added to the router logit of every expert whose MSB slice is resident,
    for SELECTION only (the combine weights stay the unbiased softmax probabilities): exactly the `bias` input of
    route_topk;
  * Cumsum: experts in descending probability (ties: lower index); the candidate set is the shortest prefix whose
    probabilities sum to at least `p`, and never fewer than k experts; of the candidates the cached ones are taken
    first, each group in descending probability, until k are selected.
"""
from __future__ import annotations

import numpy as np


def cache_prior_bias(cached_msb, delta: float) -> np.ndarray:
    """cached_msb: bool [E].  float32 [E] bias for route_topk."""
    return np.where(np.asarray(cached_msb, dtype=bool), np.float32(delta), np.float32(0.0)).astype(np.float32)


def cumsum_select(probs, cached, k: int, p: float) -> np.ndarray:
    """probs float [E], cached bool [E] -> int32 [k] selected experts, cached candidates first."""
    probs = np.asarray(probs, dtype=np.float64)
    E = probs.shape[0]
    order = sorted(range(E), key=lambda e: (-probs[e], e))
    n, acc = 0, 0.0
    while n < E and (n < k or acc < p):
        acc += probs[order[n]]
        n += 1
    cand = order[:n]
    cached = np.asarray(cached, dtype=bool)
    picked = [e for e in cand if cached[e]] + [e for e in cand if not cached[e]]
    return np.array(picked[:k], dtype=np.int32)
