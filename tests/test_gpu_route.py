"""slicemoe_route_topk on the GPU against the oracle: ids bit-exact, weights to fp32 accuracy."""
import numpy as np
import pytest

from oracle import moe
from paper_2512_12990_b200 import synth

pytestmark = pytest.mark.gpu


def _run(logits, k, bias=None, renorm=False, tau=2.0, rank_high=0):
    import torch
    from paper_2512_12990_b200 import binding as B
    lg = torch.from_numpy(logits).cuda()
    bs = None if bias is None else torch.from_numpy(bias).cuda()
    ids, w, pr = B.slicemoe_route_topk(lg, k, bs, renorm, tau, rank_high)
    torch.cuda.synchronize()
    return ids.cpu().numpy(), w.cpu().numpy(), pr.cpu().numpy()


@pytest.mark.parametrize("T,E,k", [(1, 8, 2), (8, 8, 2), (1, 64, 6), (1, 60, 4), (37, 64, 6), (2048, 60, 4),
                                   (5, 7, 7), (3, 33, 16), (2, 512, 8), (6656, 64, 6)])
@pytest.mark.parametrize("renorm", [False, True])
def test_route_matches_oracle(T, E, k, renorm):
    logits = synth.router_logits_normal(901, ("route", T, E, k), T, E)
    ids, w, _ = _run(logits, k, renorm=renorm)
    ids_o, w_o, _ = moe.route_topk(logits, k, renorm=renorm)
    assert np.array_equal(ids, ids_o)
    assert np.allclose(w, w_o, rtol=2e-6, atol=1e-9)


def test_route_ties_bias_nan():
    E, k = 64, 6
    logits = synth.router_logits_normal(902, ("route-ties",), 8, E)
    logits[1, 40] = logits[1, 3]
    logits[1, 17] = logits[1, 3]
    logits[2, :] = 0.5
    logits[3, 5] = np.nan
    logits[4, :] = -np.inf
    logits[4, 9] = 0.0
    bias = np.zeros(E, np.float32)
    bias[[2, 5, 7, 9, 11, 20, 33, 63]] = 1e30
    for b in (None, bias, np.zeros(E, np.float32), synth.normal_f32(903, ("bias",), (E,), 0.5)):
        ids, w, _ = _run(logits, k, bias=b)
        ids_o, w_o, _ = moe.route_topk(logits, k, bias=b)
        assert np.array_equal(ids, ids_o)
        ok = np.isfinite(w_o)
        assert np.allclose(w[ok], w_o[ok], rtol=2e-6, atol=1e-9)
    ids, _, _ = _run(logits, k, bias=bias)
    rows = [0, 1, 2, 3, 5, 6, 7]                  # row 4 has -inf logits: -inf + 1e30 stays -inf
    assert all(set(ids[t].tolist()) <= {2, 5, 7, 9, 11, 20, 33, 63} for t in rows)
    ids, _, _ = _run(logits, k)
    assert ids[2].tolist() == list(range(k))


def test_precision_request_matches_oracle_away_from_threshold():
    T, E, k = 64, 64, 6
    logits = (synth.router_logits_normal(904, ("route-prec",), T, E) * 2.0).astype(np.float32)
    for tau, rank_high in [(0.2, 0), (2.0, 3), (0.1, 1), (2.0, 0)]:
        ids, w, pr = _run(logits, k, tau=tau, rank_high=rank_high)
        ids_o, w_o, _ = moe.route_topk(logits, k)
        pr_o = moe.precision_request(w_o, tau, rank_high)
        decided = np.abs(w_o - tau) > 1e-5          # the comparison is taken in fp32 on the device
        assert np.array_equal(pr[decided], pr_o[decided])
        assert decided.mean() > 0.99
        # the exact definition, in the kernel's precision: the flag is the oracle's rule applied to the float32
        # weight the kernel returns and tau as a float32 (every entry, none masked)
        assert w.dtype == np.float32
        assert np.array_equal(pr, moe.precision_request(w, np.float32(tau), rank_high))
        if rank_high:
            assert (pr[:, :rank_high] == 1).all()
