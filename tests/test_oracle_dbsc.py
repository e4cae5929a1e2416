"""Pins for oracle/dbsc.py: hand-written traces of the slice cache rules of Section 4.1."""
import random

from oracle.dbsc import SliceCache

M, L = 10, 6        # bytes of an MSB slice (with scales/zero-points) and of an LSB slice


def test_msb_is_lru():
    c = SliceCache(3 * M, M, L)
    for e in (0, 1, 2):
        prec, mh, lh, fetched = c.request(0, 0, e, False)
        assert (prec, mh, lh, fetched) == (0, False, None, M)
    assert c.request(1, 0, 0, False)[1] is True          # touch 0 -> LRU order is now 1, 2, 0
    c.request(2, 0, 3, False)                            # evicts 1
    assert c.contains(0, 1) == (False, False)
    assert c.contains(0, 2)[0] and c.contains(0, 0)[0] and c.contains(0, 3)[0]
    c.request(3, 0, 4, False)                            # evicts 2
    assert not c.contains(0, 2)[0] and c.contains(0, 0)[0]
    assert c.used == 3 * M


def test_lsb_evicted_before_any_msb_and_fifo_among_lsb():
    c = SliceCache(2 * M + 2 * L, M, L)
    assert c.request(0, 0, 0, True) == (1, False, False, M + L)
    assert c.request(0, 0, 1, True) == (1, False, False, M + L)
    assert c.used == 2 * M + 2 * L
    # an LSB hit gives 8-bit execution without traffic and does not refresh its position
    assert c.request(1, 0, 0, True) == (1, True, True, 0)
    # a new MSB needs 10 bytes: both LSB entries go (oldest first), no MSB is touched
    c.request(2, 0, 2, False)
    assert c.contains(0, 0) == (True, False)
    assert c.contains(0, 1) == (True, False)
    assert c.contains(0, 2) == (True, False)
    assert c.used == 3 * M
    # critical expert with cached MSB and absent LSB reports (hit, miss); its LSB insertion must
    # evict the least-recently-used MSB (expert 1: 0 was touched at step 1), never its own MSB
    prec, mh, lh, fetched = c.request(3, 0, 0, True)
    assert (prec, mh, lh, fetched) == (1, True, False, L)
    assert c.contains(0, 1) == (False, False)
    assert c.contains(0, 0) == (True, True)
    assert c.used <= c.capacity


def test_lsb_fifo_order():
    c = SliceCache(2 * M + 2 * L + 4, M, L)
    c.request(0, 0, 0, True)
    c.request(0, 0, 1, True)
    c.request(1, 0, 0, True)                             # LSB hit on 0: no refresh
    c.request(2, 0, 2, False)                            # 4 bytes free, needs 10: evicts LSB(0) only
    assert c.contains(0, 0) == (True, False)             # oldest-inserted LSB went first, despite its later hit
    assert c.contains(0, 1) == (True, True)
    assert c.contains(0, 2) == (True, False)
    c2 = SliceCache(2 * M + 2 * L + 2, M, L)
    c2.request(0, 0, 0, True)
    c2.request(0, 0, 1, True)
    c2.request(2, 1, 5, True)                            # 2 bytes free; MSB(5) needs 10 -> evict LSB(0), LSB(1);
    assert c2.contains(0, 0) == (False, False)           # then LSB(5) needs 6 with 4 free -> evict LRU MSB(0)
    assert c2.contains(0, 1) == (True, False)
    assert c2.contains(1, 5) == (True, True)
    assert c2.used == 2 * M + L


def test_unified_across_layers_and_capacity_never_exceeded():
    rnd = random.Random(1)
    c = SliceCache(7 * M + 3 * L + 1, M, L)
    for step in range(400):
        layer, e = rnd.randrange(4), rnd.randrange(6)
        c.request(step, layer, e, rnd.random() < 0.3)
        assert c.used <= c.capacity
        assert c.used == len(c.msb) * M + len(c.lsb) * L
    # same expert id in two layers are different entries
    c = SliceCache(2 * M, M, L)
    c.request(0, 0, 3, False)
    assert c.request(0, 1, 3, False)[1] is False
    assert c.request(1, 0, 3, False)[1] is True


def test_too_small_cache_still_serves():
    c = SliceCache(L - 1, M, L)
    assert c.request(0, 0, 0, True) == (1, False, False, M + L)
    assert c.used == 0
    assert c.request(1, 0, 0, True) == (1, False, False, M + L)
    # slices are independent entries: room for an LSB but not for an MSB keeps the LSB alone
    c = SliceCache(M - 1, M, L)
    assert c.request(0, 0, 0, True) == (1, False, False, M + L)
    assert c.contains(0, 0) == (False, True) and c.used == L
    assert c.request(1, 0, 0, True) == (1, False, True, M)


def test_miss_budget_after_warmup_window():
    c = SliceCache(100 * M, M, L, miss_budget=0.05, warmup_steps=10)
    # inside the window every LSB miss is fetched
    for step in range(10):
        assert c.request(step, 0, step, True)[0] == 1
    assert c.stats["win_bytes_full"] == 0
    # first request after the window: nothing counted yet -> fetched
    assert c.request(10, 0, 50, True) == (1, False, False, M + L)
    # running miss rate is now 1.0 > 5 %: an LSB miss is not fetched, expert runs MSB-only
    prec, mh, lh, fetched = c.request(10, 0, 51, True)
    assert (prec, mh, lh, fetched) == (0, False, False, M)
    assert c.stats["lsb_skipped"] == 1
    # hits pull the rate down; LSB hits are still served at full precision meanwhile
    assert c.request(11, 0, 50, True) == (1, True, True, 0)
    for step in range(12, 400):
        c.request(step, 0, 50, True)
    assert c.stats["win_bytes_fetched"] / c.stats["win_bytes_full"] < 0.05
    assert c.request(400, 0, 52, True)[0] == 1
    st = c.stats
    assert st["requests"] == st["high_exec"] + st["low_exec"]
    assert st["requests"] == st["msb_hit"] + st["msb_miss"]
