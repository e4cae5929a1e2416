"""Config 4: a DeepSeek-V2-Lite-shaped decode stack - 26 MoE layers, 256 batch-1 decode steps with Zipf(1.1)
expert popularity and temporal reuse, a unified slice cache of 30 % of the 8-bit expert bytes on the host.

Checked here: routing of all 6,656 (step, layer) rows on the GPU against the oracle (bit-exact ids), the
host cache (C++) against the oracle cache over the whole trace (identical precision lists and counters),
and the layer output of sampled (step, layer) pairs against the float64 oracle."""
import numpy as np
import pytest

from oracle import moe
from oracle.dbsc import SliceCache
from paper_2512_12990_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

TAU = 0.25            # an expert is critical (asks for both slices) when its gating probability is >= TAU
N_STEPS = 256


def _expert_slice_bytes(sh):
    w = sh.hidden * sh.inter
    msb = 3 * (w // 2 + (w // sh.group) * 3)      # three MSB planes + scales and zero-points
    lsb = 3 * (w // 2)
    return msb, lsb


def test_decode_stack_routing_cache_and_sampled_layers():
    import torch
    from paper_2512_12990_b200 import binding as B
    sh = synth.SHAPES["dsv2_stack"]
    L, E, k = sh.n_layers, sh.n_experts, sh.top_k
    logits = synth.decode_trace_logits(sh.seed, N_STEPS, L, E, s=1.1, p_repeat=0.5)
    flat = logits.reshape(-1, E)

    # ---- routing: one call for every (step, layer) row ----
    ids_d, w_d, pr_d = B.slicemoe_route_topk(torch.from_numpy(flat).cuda(), k, tau=TAU)
    torch.cuda.synchronize()
    ids_g, w_g, req_g = ids_d.cpu().numpy(), w_d.cpu().numpy(), pr_d.cpu().numpy()
    ids, w, _ = moe.route_topk(flat, k)
    assert np.array_equal(ids_g, ids)
    assert np.allclose(w_g, w, rtol=2e-6, atol=1e-9)
    req = moe.precision_request(w, TAU)
    clear = np.abs(w - TAU) > 1e-6            # the request is decided in fp32 on the GPU: compare away from the edge
    assert np.array_equal(req_g[clear], req[clear]) and clear.mean() > 0.999
    # exactly, in the kernel's precision: the oracle's rule on the float32 weights the kernel returned
    assert np.array_equal(req_g, moe.precision_request(w_g, np.float32(TAU)))
    crit = req_g.sum(1)
    assert 0.5 < crit.mean() < 1.0 and crit.max() <= 3        # "0-2 critical experts, below one on average"
    # temporal reuse: about half of the (step, layer) rows repeat the previous step's expert set
    same = (ids.reshape(N_STEPS, L, k)[1:] == ids.reshape(N_STEPS, L, k)[:-1]).all(2).mean()
    assert 0.4 < same < 0.65

    # ---- host slice cache over the whole trace: C++ against the oracle ----
    msb_b, lsb_b = _expert_slice_bytes(sh)
    cap = int(0.30 * L * E * (msb_b + lsb_b))
    c_host, c_orc = B.Dbsc(cap, msb_b, lsb_b), SliceCache(cap, msb_b, lsb_b)
    ids3, req3 = ids_g.reshape(N_STEPS, L, k), req_g.reshape(N_STEPS, L, k)
    prec3 = np.zeros_like(req3)
    for t in range(N_STEPS):
        for l in range(L):
            prec3[t, l] = c_host.assign(t, l, ids3[t, l], req3[t, l])
            for j in range(k):
                pr, _, _, _ = c_orc.request(t, l, int(ids3[t, l, j]), bool(req3[t, l, j]))
                assert pr == prec3[t, l, j]
    st = c_host.stats()
    for key, val in c_orc.stats.items():
        assert st[key] == val, key
    assert st["bytes_used"] <= cap
    miss_rate = st["bytes_fetched"] / (st["requests"] * (msb_b + lsb_b))
    print(f"stack: miss rate {miss_rate:.3f} (bytes fetched / 8-bit bytes requested), msb hit "
          f"{st['msb_hit'] / st['requests']:.3f}, 8-bit executions {st['high_exec'] / st['requests']:.3f}")
    assert 0.0 < miss_rate < 0.6 and st["msb_hit"] > st["msb_miss"]
    c_host.close()

    # ---- sampled (step, layer) pairs through slicemoe_layer: every layer at step 0, steps 1-9, every 16th step ----
    # The experts of a sampled pair are drawn and packed on the GPU; the oracle works on the planes read back.
    samples = [(0, l) for l in range(L)] + [(t, t % L) for t in range(1, 10)] + [(t, t % L) for t in range(16, N_STEPS, 16)]
    cshape = B.make_shape(sh.hidden, sh.inter, E, k, sh.group, sh.n_shared, sh.shared_inter, False)
    ws = B.new_workspace(cshape)
    worst = 0.0
    for (t, l) in samples:
        need = [int(e) for e in ids3[t, l]]
        packed = {e: H.device_expert(sh.seed, ("stack", l, e), sh.hidden, sh.inter, sh.group) for e in need}
        decoy = H.device_expert(sh.seed, ("stack", l, "decoy"), sh.hidden, sh.inter, sh.group)
        shared = [H.device_expert(sh.seed, ("stack", l, "shared", j), sh.hidden, sh.shared_inter, sh.group)
                  for j in range(sh.n_shared)]
        tbl = B.expert_table([packed.get(e, decoy) for e in range(E)])
        stbl = B.expert_table(shared)
        xbits, x64 = H.x_inputs(sh, 1, ("x-stack", t, l))
        row = (t * L + l)
        y = B.slicemoe_layer(cshape, tbl, stbl, None, H.to_dev_bf16(xbits), ids_d[row:row + 1],
                             torch.from_numpy(prec3[t, l:l + 1].copy()).cuda(), w_d[row:row + 1], ws)
        torch.cuda.synchronize()
        assert B.slicemoe_get_status(ws) == 0
        o_experts = {e: H.oracle_expert_from_device(packed[e]) for e in need}
        o_shared = [H.oracle_expert_from_device(sx) for sx in shared]
        y_ref = moe.layer(x64, o_experts, ids3[t, l:l + 1], prec3[t, l:l + 1], w[row:row + 1], shared=o_shared)
        rel, mx = H.assert_close(y.cpu().numpy(), y_ref, f"stack step {t} layer {l}")
        worst = max(worst, rel)
    print(f"stack: {len(samples)} sampled (step, layer) pairs, worst rel-L2 {worst:.2e}")


def test_prefill_then_decode_chain_against_the_oracle():
    """Section 4.3 end to end on the device: a prompt goes through every layer's prefill kernel (all experts from
    both slices: prefill is high-bit, Section 6.3) while the host cache is reshaped from the prompt's routing;
    at the end of prefill the cache is re-ordered, and the decode steps that follow take their precision lists
    from it.  Every stage is compared with the oracle chain: routing (ids exact), prefill outputs of sampled
    tokens, the warm cache state, every decode precision list, and every decode layer output."""
    import torch
    from oracle import pcw
    from paper_2512_12990_b200 import binding as B
    NL, T_PROMPT, N_DEC, tau = 4, 96, 8, 0.35
    sh = synth.Shape("chain", 256, 128, 8, 2, 64, n_shared=1, shared_inter=256, shared_sigmoid_gate=False, n_layers=NL,
                     seed=4711)
    E, k = sh.n_experts, sh.top_k
    layers = [H.Layer(sh, range(E), layer=l) for l in range(NL)]
    msb_b, lsb_b = _expert_slice_bytes(sh)
    cap = int(0.5 * NL * E * (msb_b + lsb_b))
    c_host, c_orc = B.Dbsc(cap, msb_b, lsb_b), SliceCache(cap, msb_b, lsb_b)

    # ---- prefill, layer by layer ----
    all8 = np.ones(E, dtype=np.uint8)
    ws_p = B.new_prefill_workspace(layers[0].cshape, T_PROMPT)
    freq, mean = [], []
    for l, L in enumerate(layers):
        logits = synth.zipf_gumbel_logits(sh.seed, ("chain-prompt", l), T_PROMPT, E, 1.1)[0]
        ids_d, w_d, _ = B.slicemoe_route_topk(torch.from_numpy(logits).cuda(), k)
        ids_o, w_o, _ = moe.route_topk(logits, k)
        ids_g, w_g = ids_d.cpu().numpy(), w_d.cpu().numpy()
        assert np.array_equal(ids_g, ids_o)
        xbits, x64 = H.x_inputs(sh, T_PROMPT, f"chain-px{l}")
        y, status = B.slicemoe_prefill_layer(L.cshape, L.experts_tbl, L.shared_tbl, None, H.to_dev_bf16(xbits), ids_d, w_d,
                                             torch.from_numpy(all8).cuda(), ws_p)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        rows = [0, 17, 63, 64, T_PROMPT - 1]
        y_ref = moe.layer(x64[rows], L.oracle_list(), ids_o[rows], np.ones_like(ids_o[rows], dtype=np.uint8), w_o[rows],
                          shared=L.oracle_shared)
        for i, t in enumerate(rows):
            H.assert_close(y.cpu().numpy()[t], y_ref[i], f"prefill layer {l} token {t}")
        # the host cache sees what the device routed; the oracle chain what the oracle routed
        c_host.prefill_layer(l, ids_g, w_g, E, tau)
        f, m = pcw.prefill_stats(ids_o, w_o.astype(np.float32), E)
        freq.append(f)
        mean.append(m)
    c_host.prefill_end()
    c_orc.install(*pcw.warm_state(freq, mean, cap, msb_b, lsb_b, tau))
    for l in range(NL):
        for e in range(E):
            assert c_host.contains(l, e) == c_orc.contains(l, e), (l, e)

    # ---- decode with the warmed cache in the loop ----
    dec_logits = synth.decode_trace_logits(sh.seed, N_DEC, NL, E, s=1.1, p_repeat=0.5)
    n8 = n4 = 0
    for s in range(N_DEC):
        for l, L in enumerate(layers):
            lg = np.ascontiguousarray(dec_logits[s, l][None, :])
            ids_d, w_d, req_d = B.slicemoe_route_topk(torch.from_numpy(lg).cuda(), k, tau=tau)
            ids_o, w_o, _ = moe.route_topk(lg, k)
            assert np.array_equal(ids_d.cpu().numpy(), ids_o)
            req_g, req_o = req_d.cpu().numpy(), moe.precision_request(w_o, tau)
            assert np.all(np.abs(w_o - tau) > 1e-5), "the seeded trace keeps clear of the threshold"
            assert np.array_equal(req_g, req_o)
            # the host cache is fed by the device's routing, the oracle cache by the oracle's
            prec = c_host.assign(s, l, ids_d.cpu().numpy()[0], req_g[0])
            prec_o = [c_orc.request(s, l, int(ids_o[0, j]), bool(req_o[0, j]))[0] for j in range(k)]
            assert prec.tolist() == prec_o
            n8 += int(prec.sum())
            n4 += int(k - prec.sum())
            xbits, x64 = H.x_inputs(sh, 1, f"chain-dx{s}-{l}")
            y = B.slicemoe_layer(L.cshape, L.experts_tbl, L.shared_tbl, None, H.to_dev_bf16(xbits), ids_d,
                                 torch.from_numpy(prec[None, :].copy()).cuda(), w_d, L.ws)
            torch.cuda.synchronize()
            assert B.slicemoe_get_status(L.ws) == 0
            y_ref = moe.layer(x64, L.oracle_list(), ids_o, prec[None, :], w_o, shared=L.oracle_shared)
            H.assert_close(y.cpu().numpy(), y_ref, f"decode step {s} layer {l}")
    assert n8 > 0 and n4 > 0, "both precisions occur in the decode that follows the warmup"
    st = c_host.stats()
    for key in ("requests", "msb_hit", "msb_miss", "lsb_hit", "lsb_miss", "bytes_fetched", "high_exec", "low_exec"):
        assert st[key] == c_orc.stats[key], key
