"""The host C++ slice cache (slicemoe_dbsc_*) against the oracle on hand traces and random traces."""
import random

import numpy as np
import pytest

from oracle.dbsc import SliceCache
from paper_2512_12990_b200 import binding as B

M, L = 10, 6


def test_hand_trace_matches_section_4_1_rules():
    c = B.Dbsc(2 * M + 2 * L, M, L)
    assert c.request(0, 0, 0, True) == (1, False, False, M + L)
    assert c.request(0, 0, 1, True) == (1, False, False, M + L)
    assert c.request(1, 0, 0, True) == (1, True, True, 0)
    c.request(2, 0, 2, False)                      # both LSB entries are evicted before any MSB
    assert c.contains(0, 0) == (True, False) and c.contains(0, 1) == (True, False) and c.contains(0, 2) == (True, False)
    assert c.request(3, 0, 0, True) == (1, True, False, L)   # evicts LRU MSB (expert 1), not its own
    assert c.contains(0, 1) == (False, False) and c.contains(0, 0) == (True, True)
    assert c.request(4, 0, 7, False) == (0, False, None, M)
    c.close()


@pytest.mark.parametrize("budget", [None, 0.05, 0.3])
def test_random_traces_match_oracle(budget):
    rnd = random.Random(17)
    for trial in range(5):
        cap = rnd.randrange(0, 40) * 7
        o = SliceCache(cap, M, L, miss_budget=budget, warmup_steps=10)
        c = B.Dbsc(cap, M, L, miss_budget=budget, warmup_steps=10)
        for step in range(300):
            for _ in range(3):
                layer, e, need = rnd.randrange(3), int(rnd.paretovariate(1.1)) % 12, rnd.random() < 0.35
                assert c.request(step, layer, e, need) == o.request(step, layer, e, need)
        st = c.stats()
        for k in ("requests", "msb_hit", "msb_miss", "lsb_hit", "lsb_miss", "lsb_skipped", "bytes_fetched",
                  "high_exec", "low_exec", "win_bytes_fetched", "win_bytes_full"):
            assert st[k] == o.stats[k], k
        assert st["bytes_used"] == o.used <= cap
        c.close()


def test_assign_batch_equals_requests():
    ids = np.array([5, 3, 5, 9, 1, 3], dtype=np.int32)
    req = np.array([1, 0, 1, 1, 0, 1], dtype=np.uint8)
    a = B.Dbsc(3 * M + L, M, L)
    b = SliceCache(3 * M + L, M, L)
    for step in range(4):
        out = a.assign(step, 2, ids, req)
        ref = [b.request(step, 2, int(e), bool(r))[0] for e, r in zip(ids, req)]
        assert out.tolist() == ref
    a.close()


def test_eviction_log_names_exactly_what_left_the_cache():
    """slicemoe_dbsc_log_evictions / _drain_evicted: what a holder of the slices themselves has to release."""
    import ctypes
    from ctypes import c_void_p
    from paper_2512_12990_b200 import binding as B
    rng = np.random.default_rng(21)
    msb_b, lsb_b, E, NL = 100, 60, 9, 2
    c = B.Dbsc(4 * msb_b + 2 * lsb_b, msb_b, lsb_b)
    assert B.lib().slicemoe_dbsc_log_evictions(c._h, 1) == 0
    held = set()
    lay, exp, isl = (np.zeros(8, np.int32), np.zeros(8, np.int32), np.zeros(8, np.uint8))
    for step in range(200):
        l, e, need = int(rng.integers(0, NL)), int(rng.integers(0, E)), bool(rng.random() < 0.5)
        c.request(step, l, e, need)
        while True:
            n = B.lib().slicemoe_dbsc_drain_evicted(c._h, lay.ctypes.data_as(c_void_p), exp.ctypes.data_as(c_void_p),
                                                    isl.ctypes.data_as(c_void_p), 8)
            assert n >= 0
            for i in range(n):
                key = (int(lay[i]), int(exp[i]), int(isl[i]))
                assert key in held, "only slices that were resident are evicted"
                held.remove(key)
            if n < 8:
                break
        has_m, has_l = c.contains(l, e)
        if has_m:
            held.add((l, e, 0))
        if has_l:
            held.add((l, e, 1))
        # the holder's view equals the cache's
        for ll in range(NL):
            for ee in range(E):
                m_, l_ = c.contains(ll, ee)
                assert ((ll, ee, 0) in held) == m_ and ((ll, ee, 1) in held) == l_
    assert B.lib().slicemoe_dbsc_drain_evicted(None, None, None, None, 0) == B.E_INVALID_ARG
