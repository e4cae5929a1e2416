"""Pins of the cost-model oracle and the routing-baseline oracle: hand-computed values from the constants the paper
prints in Section 5, limiting cases, and brute force on tiny inputs."""
import itertools

import numpy as np
import pytest

from oracle import cost, routing


def test_cost_model_hand_values():
    # 1 MB from Flash and nothing else: 8e6 bits x (103 + 1.5) pJ = 0.836 mJ; 8e6 bits / 10 Gbps = 0.8 ms
    e, t = cost.step_cost(1_000_000, 0, 0)
    assert e == pytest.approx(8e6 * 104.5e-12, rel=1e-12)
    assert t == pytest.approx(8e-4, rel=1e-12)
    # 13 MB from DRAM only: 1.04e8 bits x 1.5 pJ = 0.156 mJ; 1.04e8 / 104e9 = 1 ms
    e, t = cost.step_cost(0, 13_000_000, 0)
    assert e == pytest.approx(1.04e8 * 1.5e-12, rel=1e-12)
    assert t == pytest.approx(1e-3, rel=1e-12)
    # 8.2e9 multiply-accumulates: 1.64e10 ops / 16.4 TOPS = 1 ms; / 3.18e12 ops per joule
    e, t = cost.step_cost(0, 0, 8_200_000_000)
    assert t == pytest.approx(1e-3, rel=1e-12)
    assert e == pytest.approx(1.64e10 / 3.18e12, rel=1e-12)


def test_cost_model_structure():
    # Flash is serial, DRAM and compute overlap
    _, t = cost.step_cost(1_000_000, 13_000_000, 4_100_000_000)
    assert t == pytest.approx(8e-4 + 1e-3, rel=1e-12)          # DRAM-bound part
    _, t = cost.step_cost(1_000_000, 13_000_000, 16_400_000_000)
    assert t == pytest.approx(8e-4 + 2e-3, rel=1e-12)          # compute-bound part
    # energy is additive and a Flash bit costs (103 + 1.5) / 1.5 = 69.7 times a DRAM bit
    e1, _ = cost.step_cost(1000, 0, 0)
    e2, _ = cost.step_cost(0, 1000, 0)
    assert e1 / e2 == pytest.approx(104.5 / 1.5, rel=1e-12)
    ea, _ = cost.step_cost(5, 7, 11)
    parts = cost.step_cost(5, 0, 0)[0] + cost.step_cost(0, 7, 0)[0] + cost.step_cost(0, 0, 11)[0]
    assert ea == pytest.approx(parts, rel=1e-12)
    # other hardware numbers are honoured
    hw = dict(cost.PAPER, flash_gbps=20.0)
    assert cost.step_cost(1_000_000, 0, 0, hw)[1] == pytest.approx(4e-4, rel=1e-12)


def test_cache_prior_bias():
    b = routing.cache_prior_bias([True, False, True, False], 0.75)
    assert b.dtype == np.float32 and b.tolist() == [0.75, 0.0, 0.75, 0.0]


def test_cumsum_hand_cases():
    probs = [0.40, 0.25, 0.15, 0.10, 0.06, 0.04]
    none = [False] * 6
    # nothing cached: plain top-k, whatever p is
    assert routing.cumsum_select(probs, none, 2, 0.5).tolist() == [0, 1]
    assert routing.cumsum_select(probs, none, 2, 0.95).tolist() == [0, 1]
    # p = 0.85 -> candidates {0, 1, 2, 3} (0.40 + 0.25 + 0.15 = 0.80 < 0.85, + 0.10 = 0.90): cached 3 comes first
    assert routing.cumsum_select(probs, [False, False, False, True, True, False], 2, 0.85).tolist() == [3, 0]
    # expert 4 is cached too but outside the candidate set
    assert routing.cumsum_select(probs, [False, False, False, False, True, False], 2, 0.85).tolist() == [0, 1]
    # never fewer than k candidates
    assert routing.cumsum_select(probs, [False, True, False, False, False, False], 3, 0.1).tolist() == [1, 0, 2]
    # ties go to the lower index
    assert routing.cumsum_select([0.25, 0.25, 0.25, 0.25], [False] * 4, 2, 0.3).tolist() == [0, 1]


def test_cumsum_brute_force_properties():
    rng = np.random.default_rng(5)
    for _ in range(200):
        E, k = 7, int(rng.integers(1, 4))
        probs = rng.dirichlet(np.ones(E))
        cached = rng.random(E) < 0.4
        p = float(rng.uniform(0.1, 0.99))
        sel = routing.cumsum_select(probs, cached, k, p).tolist()
        assert len(sel) == k == len(set(sel))
        order = sorted(range(E), key=lambda e: -probs[e])
        # the candidate set by its definition: every prefix of the ranking that satisfies both conditions
        n = next(m for m in range(1, E + 1) if m >= k and probs[order[:m]].sum() >= p - 1e-15 or m == E)
        cand = set(order[:n])
        assert set(sel) <= cand
        # no unselected cached candidate while an uncached one was selected; within a class, by probability
        for a, b in itertools.product(cand - set(sel), sel):
            if cached[a] == cached[b]:
                assert probs[a] <= probs[b]
            else:
                assert not cached[a]
