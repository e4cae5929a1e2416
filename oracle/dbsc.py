"""Oracle: Dynamic Bit-Sliced Caching bookkeeping (Section 4.1).  Test infrastructure only.

What the paper fixes: MSB and LSB slices of an expert are cached independently and each
produces its own hit/miss; a critical expert requests both slices, a non-critical one the MSB
slice only; full precision is used when both slices are available, MSB-only computation
otherwise; MSB slices follow standard LRU; LSB slices have the lowest priority and are evicted
first; one cache is shared by all layers (Section 6.1, cache implementation); the miss-rate
constraint activates after the first 10 decode steps.

Readings where the paper is silent (stated once, used by both this oracle and the host code):
  * capacity and sizes are in bytes; scales and zero-points are charged to the MSB slice;
  * among LSB entries eviction is oldest-inserted first, and an LSB hit does not refresh it;
  * a missed slice is fetched and inserted (MSB at the most-recently-used end), evicting LSB
    entries first, then MSB entries from the least-recently-used end; slices of the expert
    being served are never evicted by its own request; a slice larger than what can be freed
    is used but not kept;
  * miss budget (optional): once `step >= warmup_steps`, if the running miss rate
    (bytes fetched / bytes of the same requests at full precision, counted from the end of the
    warm-up window) exceeds the budget, an LSB miss is not fetched and the expert runs MSB-only.
"""
from __future__ import annotations

from collections import OrderedDict


class SliceCache:
    def __init__(self, capacity_bytes: int, msb_bytes: int, lsb_bytes: int,
                 miss_budget: float | None = None, warmup_steps: int = 10):
        self.capacity = int(capacity_bytes)
        self.msb_bytes = int(msb_bytes)
        self.lsb_bytes = int(lsb_bytes)
        self.miss_budget = miss_budget
        self.warmup_steps = warmup_steps
        self.msb = OrderedDict()      # key -> None; first = least recently used
        self.lsb = OrderedDict()      # key -> None; first = oldest inserted
        self.used = 0
        self.stats = dict(requests=0, msb_hit=0, msb_miss=0, lsb_hit=0, lsb_miss=0,
                          lsb_skipped=0, bytes_fetched=0, high_exec=0, low_exec=0,
                          win_bytes_fetched=0, win_bytes_full=0)

    # -- internals -------------------------------------------------------------------------
    def _make_room(self, need: int, protect) -> bool:
        """Evict until `need` bytes are free.  LSB entries first (oldest first), then MSB entries
        (least recently used first); entries in `protect` are skipped."""
        if need > self.capacity:
            return False
        while self.capacity - self.used < need:
            victim = None
            for key in self.lsb:
                if ("L",) + key not in protect:
                    victim = ("L", key)
                    break
            if victim is None:
                for key in self.msb:
                    if ("M",) + key not in protect:
                        victim = ("M", key)
                        break
            if victim is None:
                return False
            if victim[0] == "L":
                del self.lsb[victim[1]]
                self.used -= self.lsb_bytes
            else:
                del self.msb[victim[1]]
                self.used -= self.msb_bytes
        return True

    def _over_budget(self, step: int) -> bool:
        if self.miss_budget is None or step < self.warmup_steps:
            return False
        full = self.stats["win_bytes_full"]
        return full > 0 and self.stats["win_bytes_fetched"] / full > self.miss_budget

    # -- the one operation -------------------------------------------------------------------
    def request(self, step: int, layer: int, expert: int, need_lsb: bool):
        """Serve one selected expert.  Returns (prec, msb_hit, lsb_hit, bytes_fetched) with prec 1
        = MSB+LSB execution, 0 = MSB-only; lsb_hit is None when the LSB slice was not requested."""
        key = (layer, expert)
        st = self.stats
        st["requests"] += 1
        fetched = 0
        protect = {("M",) + key, ("L",) + key}
        # MSB slice: standard LRU
        if key in self.msb:
            self.msb.move_to_end(key)
            msb_hit = True
            st["msb_hit"] += 1
        else:
            msb_hit = False
            st["msb_miss"] += 1
            fetched += self.msb_bytes
            if self._make_room(self.msb_bytes, protect):
                self.msb[key] = None
                self.used += self.msb_bytes
        # LSB slice: only for critical experts
        lsb_hit = None
        prec = 0
        if need_lsb:
            if key in self.lsb:
                lsb_hit = True
                st["lsb_hit"] += 1
                prec = 1
            else:
                lsb_hit = False
                if self._over_budget(step):
                    st["lsb_skipped"] += 1
                else:
                    st["lsb_miss"] += 1
                    fetched += self.lsb_bytes
                    prec = 1
                    if self._make_room(self.lsb_bytes, protect):
                        self.lsb[key] = None
                        self.used += self.lsb_bytes
        st["bytes_fetched"] += fetched
        st["high_exec" if prec else "low_exec"] += 1
        if step >= self.warmup_steps:
            st["win_bytes_fetched"] += fetched
            st["win_bytes_full"] += self.msb_bytes + self.lsb_bytes
        return prec, msb_hit, lsb_hit, fetched

    def install(self, msb_order, lsb_order):
        """Replaces the content: (layer, expert) lists with the next victim first (the state a cache warmup
        leaves behind).  Statistics are untouched."""
        self.msb = OrderedDict((tuple(k), None) for k in msb_order)
        self.lsb = OrderedDict((tuple(k), None) for k in lsb_order)
        self.used = len(self.msb) * self.msb_bytes + len(self.lsb) * self.lsb_bytes
        assert self.used <= self.capacity

    def contains(self, layer: int, expert: int):
        key = (layer, expert)
        return key in self.msb, key in self.lsb
