"""Pins for oracle/pcw.py: Predictive Cache Warmup (Section 4.3) on a hand-worked example, against a
layer-by-layer simulation written independently here, and on the invariants the eviction rule implies."""
import numpy as np
import pytest

from oracle import moe, pcw
from oracle.dbsc import SliceCache
from paper_2512_12990_b200 import synth

M, L = 10, 6
TAU = 0.3
# two layers x four experts; expected orders below were worked out by hand from Section 4.3's rule
FREQ = [[5, 0, 2, 3], [1, 4, 4, 0]]
MEAN = [[0.5, 0.0, 0.1, 0.35], [0.2, 0.4, 0.3, 0.0]]
MSB_ALL = [(1, 0), (0, 2), (0, 3), (1, 2), (1, 1), (0, 0)]   # ascending frequency, ties by score
LSB_ALL = [(1, 2), (0, 3), (1, 1), (0, 0)]                   # score >= 0.3, ascending score


@pytest.mark.parametrize("cap,msb,lsb", [
    (84, MSB_ALL, LSB_ALL),                 # 6 x 10 + 4 x 6 fits exactly
    (83, MSB_ALL, LSB_ALL[1:]),             # one byte short: the lowest-score LSB slice goes
    (75, MSB_ALL, LSB_ALL[2:]),
    (60, MSB_ALL, []),                      # all LSB slices go before any MSB slice
    (59, MSB_ALL[1:], []),                  # then the least frequent MSB slice
    (45, MSB_ALL[2:], []),
    (9, [], []),
])
def test_hand_worked_example(cap, msb, lsb):
    got_msb, got_lsb = pcw.warm_state(FREQ, MEAN, cap, M, L, TAU)
    assert got_msb == msb and got_lsb == lsb


def test_prefill_stats_on_a_hand_example():
    ids = np.array([[0, 1], [0, 2], [3, 0]])
    sc = np.array([[0.5, 0.25], [0.25, 0.125], [0.0625, 0.75]], dtype=np.float32)
    freq, mean = pcw.prefill_stats(ids, sc, 5)
    assert freq.tolist() == [3, 1, 1, 1, 0]
    assert mean.tolist() == [0.5, 0.25, 0.125, 0.0625, 0.0]   # (0.5 + 0.25 + 0.75) / 3 = 0.5 exactly


def _streaming(freq, mean, cap, tau):
    """Section 4.3 read literally: layers arrive one by one; whenever the content exceeds the capacity the
    lowest LSB slice (by score) is dropped, and when none is left the least frequent MSB slice."""
    msb, lsb = {}, {}
    for l in range(len(freq)):
        for e in range(len(freq[l])):
            if freq[l][e] > 0:
                msb[(l, e)] = (freq[l][e], mean[l][e], l, e)
                if mean[l][e] >= tau:
                    lsb[(l, e)] = (mean[l][e], freq[l][e], l, e)
        while len(msb) * M + len(lsb) * L > cap:
            if lsb:
                del lsb[min(lsb, key=lsb.get)]
            else:
                del msb[min(msb, key=msb.get)]
    return sorted(msb, key=msb.get), sorted(lsb, key=lsb.get)


@pytest.mark.parametrize("seed", range(12))
def test_one_shot_definition_equals_layer_by_layer_eviction(seed):
    g = np.random.default_rng(seed)
    nl, ne = int(g.integers(1, 7)), int(g.integers(2, 12))
    freq = g.integers(0, 5, size=(nl, ne))                         # many ties
    mean = np.where(freq > 0, g.integers(0, 9, size=(nl, ne)) / 8.0, 0.0)  # ties in the scores too
    total = int((freq > 0).sum()) * M + int(((mean >= TAU) & (freq > 0)).sum()) * L
    for cap in sorted({0, M - 1, M, total // 3, total // 2, total - 1, total, total + 5}):
        one = pcw.warm_state(freq, mean, cap, M, L, TAU)
        assert one == _streaming(freq.tolist(), mean.tolist(), cap, TAU)
        msb, lsb = one
        used = len(msb) * M + len(lsb) * L
        assert used <= cap
        assert set(lsb) <= set(msb)
        n_msb_cand = int((freq > 0).sum())
        if len(msb) < n_msb_cand:
            assert not lsb, "an MSB slice was dropped while an LSB slice was kept"
            assert used + M > cap, "more was evicted than needed"
        # order: the next victim first
        keys = [(freq[l][e], mean[l][e], l, e) for l, e in msb]
        assert keys == sorted(keys)
        assert all(mean[l][e] >= TAU for l, e in lsb)


def _early_decode_fetch(cache, ids, preq, steps):
    before = cache.stats["bytes_fetched"]
    for s in range(steps):
        for l in range(ids.shape[1]):
            for j in range(ids.shape[2]):
                cache.request(s, l, int(ids[s, l, j]), bool(preq[s, l, j]))
    return cache.stats["bytes_fetched"] - before


def test_warm_cache_beats_naive_initial_states_in_early_decode():
    """Section 4.3: Empty, Last-layer-only and Random retention perform poorly in early decode; a cache warmed
    from prefill hotness starts with the right slices.  Prompt and decode trace share the per-layer popularity."""
    seed, NL, E, K, T, tau = 77, 8, 32, 4, 256, 0.2
    msb_b, lsb_b = 1100, 1000
    cap = int(0.3 * NL * E * (msb_b + lsb_b))
    pl = synth.prefill_trace_logits(seed, T, NL, E)
    freq, mean = [], []
    for l in range(NL):
        ids, w, _ = moe.route_topk(pl[l], K)
        f, m = pcw.prefill_stats(ids, w, E)
        freq.append(f); mean.append(m)
    dl = synth.decode_trace_logits(seed, 16, NL, E)
    d_ids = np.empty((16, NL, K), dtype=np.int64)
    d_req = np.empty((16, NL, K), dtype=bool)
    for s in range(16):
        for l in range(NL):
            ids, w, _ = moe.route_topk(dl[s, l][None, :], K)
            d_ids[s, l], d_req[s, l] = ids[0], w[0] >= tau

    def fresh():
        return SliceCache(cap, msb_b, lsb_b)

    warm = fresh()
    warm.install(*pcw.warm_state(freq, mean, cap, msb_b, lsb_b, tau))
    last = fresh()                                    # what prefill leaves behind without any policy: the last layers
    for l in range(NL):
        for e in range(E):
            if freq[l][e] > 0:
                last.request(0, l, e, True)
    rnd = fresh()
    g = np.random.default_rng(5)
    cand = [(l, e) for l in range(NL) for e in range(E) if freq[l][e] > 0]
    keep = [cand[i] for i in g.permutation(len(cand))[: cap // (msb_b + lsb_b)]]
    rnd.install(keep, keep)
    # the first four steps are where cold misses dominate; over all 16 the steady-state misses dilute the gap
    caches = [("warm", warm), ("empty", fresh()), ("last", last), ("random", rnd)]
    first4 = {name: _early_decode_fetch(c, d_ids, d_req, 4) for name, c in caches}
    later = {name: _early_decode_fetch(c, d_ids[4:], d_req[4:], 12) for name, c in caches}
    print(first4, later)
    assert first4["warm"] < 0.8 * min(first4["empty"], first4["last"], first4["random"]), first4
    assert first4["warm"] + later["warm"] < min(first4[n] + later[n] for n in ("empty", "last", "random"))
