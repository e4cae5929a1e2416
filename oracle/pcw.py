"""Oracle: Predictive Cache Warmup (Section 4.3, "Predictive Cache Warmup (PCW)").  Test infrastructure only.

What the paper fixes: during prefill the unified cache is reshaped; slices with low gating scores
are discarded first, starting from LSB slices; once those are gone, MSB slices with low prefill
access frequency are evicted; the single-head threshold of the precision selection decides which
experts keep high-bit precision; when prefill ends the cache is re-ordered by accumulated access
frequency so that its LRU state matches the experts expected early in decode.

Readings where the paper is silent (stated once, used by both this oracle and the host code):
  * an expert's access frequency is the number of prompt tokens routed to it, its gating score the
    mean, over those tokens, of the score the router gave it (float64 sum in token order / count);
  * prefill loads every expert it uses, so every (layer, expert) with frequency > 0 is a candidate
    for its MSB slice; it is a candidate for its LSB slice only if its score >= tau, the threshold
    that makes an expert critical in decode;
  * if the candidates exceed the capacity, LSB slices go first in ascending (score, frequency,
    layer, expert) order, then MSB slices in ascending (frequency, score, layer, expert) order,
    until the rest fits;
  * the final order: MSB slices ascending by the same MSB key, the last one being the most recently
    used; LSB slices ascending by the LSB key, the first one being the next LSB victim.
The definition below is one-shot over all layers; evicting progressively, layer by layer, whenever
the cache overflows yields the same state (the victim is always the minimum of one total order).
"""
from __future__ import annotations

import numpy as np


def prefill_stats(ids: np.ndarray, scores: np.ndarray, n_experts: int):
    """ids int [T, k], scores float32 [T, k] of one layer -> (freq int64 [E], mean float64 [E], 0 where unused)."""
    flat = np.asarray(ids).reshape(-1)
    freq = np.bincount(flat, minlength=n_experts).astype(np.int64)
    ssum = np.bincount(flat, weights=np.asarray(scores, dtype=np.float64).reshape(-1), minlength=n_experts)
    mean = np.zeros(n_experts, dtype=np.float64)
    used = freq > 0
    mean[used] = ssum[used] / freq[used]
    return freq, mean


def warm_state(freq, mean, capacity: int, msb_bytes: int, lsb_bytes: int, tau: float):
    """freq, mean: [n_layers][n_experts].  Returns (msb_order, lsb_order), lists of (layer, expert) with the
    next victim first."""
    msb, lsb = [], []
    for l in range(len(freq)):
        for e in range(len(freq[l])):
            if freq[l][e] > 0:
                msb.append((int(freq[l][e]), float(mean[l][e]), l, e))
                if mean[l][e] >= tau:
                    lsb.append((float(mean[l][e]), int(freq[l][e]), l, e))
    msb.sort()
    lsb.sort()
    used = len(msb) * msb_bytes + len(lsb) * lsb_bytes
    while used > capacity and lsb:
        lsb.pop(0)
        used -= lsb_bytes
    while used > capacity and msb:
        msb.pop(0)
        used -= msb_bytes
    return [(l, e) for _, _, l, e in msb], [(l, e) for _, _, l, e in lsb]
