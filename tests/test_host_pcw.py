"""Predictive Cache Warmup in the host C++ cache (slicemoe_dbsc_prefill_layer / _end) against the oracle's
one-shot definition: same content, same eviction order (checked through the decode trace that follows)."""
import numpy as np
import pytest

from oracle import moe, pcw
from oracle.dbsc import SliceCache
from paper_2512_12990_b200 import binding as B
from paper_2512_12990_b200 import synth

MSB_B, LSB_B = 1100, 1000


def _prompt(seed, NL, E, K, T):
    pl = synth.prefill_trace_logits(seed, T, NL, E)
    out = []
    for l in range(NL):
        ids, w, _ = moe.route_topk(pl[l], K)
        out.append((ids.astype(np.int32), w.astype(np.float32)))
    return out


def _decode(seed, NS, NL, E, K, tau):
    dl = synth.decode_trace_logits(seed, NS, NL, E)
    ids = np.empty((NS, NL, K), dtype=np.int32)
    req = np.empty((NS, NL, K), dtype=np.uint8)
    for s in range(NS):
        for l in range(NL):
            i, w, _ = moe.route_topk(dl[s, l][None, :], K)
            ids[s, l], req[s, l] = i[0], w[0] >= tau
    return ids, req


@pytest.mark.parametrize("frac", [0.05, 0.3, 0.7, 2.0])
@pytest.mark.parametrize("seed,NL,E,K,T", [(3, 6, 16, 2, 40), (4, 26, 64, 6, 128)])
def test_warm_state_and_the_decode_that_follows_match_the_oracle(seed, NL, E, K, T, frac):
    tau = 0.2
    cap = int(frac * NL * E * (MSB_B + LSB_B))
    prompt = _prompt(seed, NL, E, K, T)
    host = B.Dbsc(cap, MSB_B, LSB_B)
    freq, mean = [], []
    for l, (ids, w) in enumerate(prompt):
        host.prefill_layer(l, ids, w, E, tau)
        assert host.stats()["bytes_used"] <= cap          # reshaped progressively: never over capacity
        f, m = pcw.prefill_stats(ids, w, E)
        freq.append(f); mean.append(m)
    host.prefill_end()
    msb, lsb = pcw.warm_state(freq, mean, cap, MSB_B, LSB_B, tau)
    orc = SliceCache(cap, MSB_B, LSB_B)
    orc.install(msb, lsb)
    for l in range(NL):
        for e in range(E):
            assert host.contains(l, e) == orc.contains(l, e), (l, e)
    st = host.stats()
    assert st["bytes_used"] == orc.used and st["requests"] == 0 and st["bytes_fetched"] == 0
    # the eviction ORDER shows in what the following decode steps hit, miss and evict
    d_ids, d_req = _decode(seed, 12, NL, E, K, tau)
    for s in range(12):
        for l in range(NL):
            for j in range(K):
                assert host.request(s, l, int(d_ids[s, l, j]), bool(d_req[s, l, j])) == \
                    orc.request(s, l, int(d_ids[s, l, j]), bool(d_req[s, l, j])), (s, l, j)
    st = host.stats()
    for k_host, k_orc in [("requests", "requests"), ("msb_hit", "msb_hit"), ("lsb_miss", "lsb_miss"),
                          ("bytes_fetched", "bytes_fetched"), ("high_exec", "high_exec")]:
        assert st[k_host] == orc.stats[k_orc]


def test_slices_cached_before_the_prompt_go_first_and_reordering_is_by_frequency():
    cap = 4 * MSB_B
    c = B.Dbsc(cap, MSB_B, LSB_B)
    c.request(0, 9, 0, True)                   # left over from an earlier run: MSB + LSB of (9, 0)
    ids = np.array([[1, 2], [1, 2], [1, 3]], dtype=np.int32)
    sc = np.array([[0.6, 0.3], [0.6, 0.3], [0.6, 0.1]], dtype=np.float32)
    c.prefill_layer(0, ids, sc, 4, 0.5)        # candidates: MSB of 1 (f3), 2 (f2), 3 (f1); LSB of 1
    # 3 MSB + 1 LSB fit (100 bytes to spare) once the stale (9, 0) slices are gone
    assert c.contains(9, 0) == (False, False)
    assert c.contains(0, 1) == (True, True) and c.contains(0, 2) == (True, False) and c.contains(0, 3) == (True, False)
    c.prefill_end()
    # a new MSB slice needs room: the LSB slice goes first (just enough), then the least frequent MSB slice (expert 3)
    c.request(0, 5, 0, False)
    assert c.contains(0, 1) == (True, False) and c.contains(0, 3) == (True, False)
    c.request(0, 5, 1, False)
    assert c.contains(0, 3) == (False, False) and c.contains(0, 2) == (True, False)
    c.request(0, 5, 2, False)
    assert c.contains(0, 2) == (False, False) and c.contains(0, 1) == (True, False)


def test_argument_checks():
    c = B.Dbsc(10 * MSB_B, MSB_B, LSB_B)
    ids = np.array([[0, 4]], dtype=np.int32)
    sc = np.ones((1, 2), dtype=np.float32)
    with pytest.raises(B.SliceMoEError) as ei:
        c.prefill_layer(0, ids, sc, 4, 0.2)     # id 4 outside [0, 4)
    assert ei.value.code == B.E_INVALID_ARG
    with pytest.raises(B.SliceMoEError):
        c.prefill_layer(-1, ids, sc, 8, 0.2)
    L = B.lib()
    assert L.slicemoe_dbsc_prefill_layer(None, 0, None, None, 0, 4, 0.2) == B.E_INVALID_ARG
    assert L.slicemoe_dbsc_prefill_end(None) == B.E_INVALID_ARG
    c.prefill_layer(0, np.zeros((0, 2), np.int32), np.zeros((0, 2), np.float32), 4, 0.2)   # an empty prompt is fine
    c.prefill_end()
    assert c.stats()["bytes_used"] == 0
