"""The host-side cost model and routing baselines of the library (plain C++, no GPU) against their oracles."""
import numpy as np
import pytest

from oracle import cost, routing
from oracle.dbsc import SliceCache


def test_cost_step_matches_oracle():
    from paper_2512_12990_b200 import binding as B
    hw = B.paper_hw()
    assert (hw.dram_pj_per_bit, hw.flash_pj_per_bit, hw.dram_gbps, hw.flash_gbps, hw.tops, hw.tops_per_watt) == (
        1.5, 103.0, 104.0, 10.0, 16.4, 3.18)
    rng = np.random.default_rng(11)
    for _ in range(200):
        f, d, m = (int(v) for v in rng.integers(0, 10**10, 3))
        e, t = B.slicemoe_cost_step(f, d, m)
        eo, to = cost.step_cost(f, d, m)
        assert e == pytest.approx(eo, rel=1e-13) and t == pytest.approx(to, rel=1e-13)
    hw.flash_gbps = 20.0
    assert B.slicemoe_cost_step(1_000_000, 0, 0, hw)[1] == pytest.approx(cost.step_cost(1_000_000, 0, 0, dict(cost.PAPER, flash_gbps=20.0))[1])
    hw.flash_gbps = 0.0
    with pytest.raises(B.SliceMoEError):
        B.slicemoe_cost_step(1, 1, 1, hw)
    with pytest.raises(B.SliceMoEError):
        B.slicemoe_cost_step(-1, 1, 1)


def test_cumsum_select_matches_oracle():
    from paper_2512_12990_b200 import binding as B
    rng = np.random.default_rng(12)
    for _ in range(300):
        E = int(rng.integers(2, 70))
        k = int(rng.integers(1, min(E, 8) + 1))
        probs = rng.dirichlet(np.ones(E) * 0.3).astype(np.float32)
        if rng.random() < 0.3:
            probs[rng.integers(0, E, 3)] = probs[0]       # exact ties
        cached = rng.random(E) < 0.4
        p = float(rng.uniform(0.05, 1.0))
        got = B.slicemoe_cumsum_select(probs, cached, k, p)
        want = routing.cumsum_select(probs, cached, k, p)
        assert got.tolist() == want.tolist()
    with pytest.raises(B.SliceMoEError):
        B.slicemoe_cumsum_select(np.ones(4, np.float32), np.zeros(4, np.uint8), 5, 0.5)


def test_cache_prior_bias_follows_the_cache_state():
    from paper_2512_12990_b200 import binding as B
    msb_b, lsb_b, E = 100, 60, 12
    c_host, c_orc = B.Dbsc(5 * msb_b + 2 * lsb_b, msb_b, lsb_b), SliceCache(5 * msb_b + 2 * lsb_b, msb_b, lsb_b)
    rng = np.random.default_rng(13)
    for step in range(60):
        layer, e, need = int(rng.integers(0, 3)), int(rng.integers(0, E)), bool(rng.random() < 0.5)
        c_host.request(step, layer, e, need)
        c_orc.request(step, layer, e, need)
        for l in range(3):
            cached = [c_orc.contains(l, x)[0] for x in range(E)]
            assert c_host.bias(l, E, 0.75).tolist() == routing.cache_prior_bias(cached, 0.75).tolist()
