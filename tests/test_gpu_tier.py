"""The second memory tier (slicemoe_tier_*): all slices live in pinned host memory, a small pool of slots on the
device holds what the slice cache decides to keep, misses are copied in on a side stream.  Decode steps of a
three-layer model run through it; every precision list is compared with the oracle cache and every layer output
with the oracle layer - which only comes out right if the right bytes are in the slots the tables point to."""
import numpy as np
import pytest

from oracle import moe
from oracle.dbsc import SliceCache
from paper_2512_12990_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("b_high,b_low", [(8, 4), (6, 3), (4, 2)])
def test_decode_through_the_tier_matches_the_oracle(b_high, b_low):
    import torch
    from paper_2512_12990_b200 import binding as B
    NL, N_STEPS, tau = 3, 14, 0.3
    sh = synth.Shape("tier", 256, 128, 8, 2, 64, n_shared=1, shared_inter=256, shared_sigmoid_gate=True, n_layers=NL,
                     seed=5150)
    E, k = sh.n_experts, sh.top_k
    layers = [H.Layer(sh, range(E), layer=l, b_high=b_high, b_low=b_low) for l in range(NL)]
    m, l_, slot, staging = B.slicemoe_tier_sizes(layers[0].cshape)
    w = sh.hidden * sh.inter
    # in the store a slice takes its own width: b_low bits per weight (+ scales and zero-points), b_high - b_low bits
    assert m == 3 * (w * b_low // 8 + 3 * (w // sh.group)) and l_ == 3 * (w * (b_high - b_low) // 8)
    assert slot % 256 == 0 and slot >= 3 * (w // 2 + 3 * (w // sh.group)) and (staging == 0) == (b_low == 4)
    pool_slots = 1 + 4 * k + 3                       # 7 cached slots for 48 slices: evictions every step
    tier = B.Tier(layers[0].cshape, [[L.packed[e] for e in range(E)] for L in layers], pool_slots)
    # the originals are no longer needed - and must not be what the kernel reads
    for L in layers:
        for e in range(E):
            for mat in L.packed[e].values():
                mat.msb.zero_(); mat.lsb.zero_(); mat.scale.zero_(); mat.zp.zero_()
    orc = SliceCache((pool_slots - 1 - 2 * k) * slot, slot, slot)      # slot 0 and 2k slots in transit are set aside
    logits = synth.decode_trace_logits(sh.seed, N_STEPS, NL, E, s=1.1, p_repeat=0.3)
    n8 = n4 = 0
    for s in range(N_STEPS):
        for l, L in enumerate(layers):
            lg = np.ascontiguousarray(logits[s, l][None, :])
            ids_d, w_d, _ = B.slicemoe_route_topk(torch.from_numpy(lg).cuda(), k)
            ids_o, w_o, _ = moe.route_topk(lg, k)
            assert np.array_equal(ids_d.cpu().numpy(), ids_o)
            req = moe.precision_request(w_o, tau)
            prec = tier.request(s, l, ids_o[0], req[0])
            prec_o = [orc.request(s, l, int(ids_o[0, j]), bool(req[0, j]))[0] for j in range(k)]
            assert prec.tolist() == prec_o
            n8 += int(prec.sum()); n4 += int(k - prec.sum())
            xbits, x64 = H.x_inputs(sh, 1, f"tier-x{s}-{l}")
            y = B.slicemoe_layer(L.cshape, tier.layer_table(l), L.shared_tbl, L.gate_vec_dev, H.to_dev_bf16(xbits), ids_d,
                                 torch.from_numpy(prec[None, :].copy()).cuda(), w_d, L.ws)
            torch.cuda.synchronize()
            assert B.slicemoe_get_status(L.ws) == 0
            y_ref = moe.layer(x64, L.oracle_list(), ids_o, prec[None, :], w_o, shared=L.oracle_shared,
                              shared_gate_vec=L.gate_vec)
            H.assert_close(y.cpu().numpy(), y_ref, f"step {s} layer {l}")
    st = tier.stats()
    assert n8 > 0 and n4 > 0
    for key in ("requests", "msb_hit", "msb_miss", "lsb_hit", "lsb_miss", "high_exec", "low_exec"):
        assert st[key] == orc.stats[key], key
    # one copy per miss - except where a slice of the list was pushed out by an earlier entry of the same list and is
    # asked for again a moment later: the cache counts a miss, the bytes are still in their slot
    misses = st["msb_miss"] + st["lsb_miss"]
    assert misses - 2 * k * 3 <= st["copies"] <= misses
    assert st["copies"] * l_ <= st["bytes_copied"] <= st["copies"] * m
    assert st["msb_miss"] > 3 * k * NL, "the pool is small enough to keep missing after the first steps"
    assert 0 <= st["free_slots"] <= pool_slots - 1
    # an expert that was never requested, or was evicted, points at the stand-in slot: defined bytes (zeros), no fault
    tbl = np.frombuffer(tier.tables.cpu().numpy().tobytes(), dtype=np.uint64).reshape(NL * E, -1)
    pool_lo, pool_hi = tier.pool.data_ptr(), tier.pool.data_ptr() + tier.pool.numel()
    msb_ptrs = tbl[:, 0]
    assert ((msb_ptrs >= pool_lo) & (msb_ptrs < pool_hi)).all()
    assert (msb_ptrs == pool_lo).sum() >= NL * E - (pool_slots - 1)
    assert 0 <= st["free_slots"]
    tier.close()


def test_tier_argument_checks():
    from paper_2512_12990_b200 import binding as B
    import ctypes
    sh = B.make_shape(256, 128, 8, 2, 64)
    L = B.lib()
    assert L.slicemoe_tier_sizes(None, None, None, None, None) == B.E_INVALID_ARG
    assert not L.slicemoe_tier_create(ctypes.byref(sh), 1, None, None, 0, None, None, 0, -1.0, 10, None)
    assert L.slicemoe_tier_request(None, 0, 0, None, None, 0, None, None, None) == B.E_INVALID_ARG
    assert L.slicemoe_tier_stats(None, None, None, None) == B.E_INVALID_ARG
    L.slicemoe_tier_destroy(None)


def test_cache_warmup_reaches_the_tier():
    """Predictive Cache Warmup (Section 4.3) through the tier: the prompt's routing reshapes the tier's own cache,
    slicemoe_tier_sync brings the pool in line with it, and the decode steps that follow hit what was warmed.
    Every decode precision list and layer output is compared with the oracle chain (pcw.warm_state installed in
    the oracle cache)."""
    import torch
    from oracle import pcw
    from paper_2512_12990_b200 import binding as B
    NL, T_PROMPT, N_DEC, tau = 3, 64, 6, 0.3
    sh = synth.Shape("tier-pcw", 256, 128, 8, 2, 64, n_shared=0, shared_inter=0, shared_sigmoid_gate=False, n_layers=NL,
                     seed=5151)
    E, k = sh.n_experts, sh.top_k
    layers = [H.Layer(sh, range(E), layer=l) for l in range(NL)]
    _, _, slot, _ = B.slicemoe_tier_sizes(layers[0].cshape)
    pool_slots = 1 + 2 * k + 12                      # 12 cached slots for 48 slices
    tier = B.Tier(layers[0].cshape, [[L.packed[e] for e in range(E)] for L in layers], pool_slots)
    cap = 12 * slot
    orc = SliceCache(cap, slot, slot)
    cache = tier.cache()
    freq, mean = [], []
    for l in range(NL):
        logits = synth.zipf_gumbel_logits(sh.seed, ("tier-prompt", l), T_PROMPT, E, 1.1)[0]
        ids_o, w_o, _ = moe.route_topk(logits, k)
        cache.prefill_layer(l, ids_o, w_o.astype(np.float32), E, tau)
        f, m = pcw.prefill_stats(ids_o, w_o.astype(np.float32), E)
        freq.append(f); mean.append(m)
    cache.prefill_end()
    orc.install(*pcw.warm_state(freq, mean, cap, slot, slot, tau))
    tier.sync()
    st0 = tier.stats()
    assert st0["copies"] == len(orc.msb) + len(orc.lsb) == 12 and st0["requests"] == 0
    dec = synth.decode_trace_logits(sh.seed, N_DEC, NL, E, s=1.1, p_repeat=0.3)
    for s in range(N_DEC):
        for l, L in enumerate(layers):
            lg = np.ascontiguousarray(dec[s, l][None, :])
            ids_o, w_o, _ = moe.route_topk(lg, k)
            req = moe.precision_request(w_o, tau)
            prec = tier.request(s, l, ids_o[0], req[0])
            prec_o = [orc.request(s, l, int(ids_o[0, j]), bool(req[0, j]))[0] for j in range(k)]
            assert prec.tolist() == prec_o
            xbits, x64 = H.x_inputs(sh, 1, f"tier-pcw-x{s}-{l}")
            y = B.slicemoe_layer(L.cshape, tier.layer_table(l), None, None, H.to_dev_bf16(xbits),
                                 torch.from_numpy(ids_o.astype(np.int32)).cuda(), torch.from_numpy(prec[None, :].copy()).cuda(),
                                 torch.from_numpy(w_o.astype(np.float32)).cuda(), L.ws)
            torch.cuda.synchronize()
            assert B.slicemoe_get_status(L.ws) == 0
            H.assert_close(y.cpu().numpy(), moe.expert_ffn(x64, L.oracle_list(), ids_o, prec[None, :], w_o), f"step {s} layer {l}")
    st = tier.stats()
    for key in ("requests", "msb_hit", "msb_miss", "lsb_hit", "lsb_miss"):
        assert st[key] == orc.stats[key], key
    assert st["msb_hit"] > 0, "the warmed slices are hit"
    tier.close()
