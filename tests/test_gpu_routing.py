"""The sigmoid-group routing family (Appendix A; the 8B tier: n = 8 groups, keep 4, K = 8, scale 2.5,
E = 128) through the C ABI, row by row against the oracle.  Floating point decides integers here
(which groups survive, which experts win): the kernel decides in fp32, the oracle in fp64, so a row is
compared exactly wherever the oracle's margins at the two decision boundaries exceed the fp32
rounding, and every row must at least be a valid answer for the kernel's own precision."""
import numpy as np
import pytest
import torch

import paper_2609_18063_b200 as edg
from oracle import moe_oracle as orc

pytestmark = pytest.mark.gpu


def _margins(l, bias, K, n, G):
    """fp64 margins at the group boundary and at the expert boundary of one row."""
    sig = 1.0 / (1.0 + np.exp(-l.astype(np.float64)))
    sel = sig if bias is None else sig + bias.astype(np.float64)
    per = l.shape[0] // n
    gs = np.array([np.sort(sel[g * per:(g + 1) * per])[::-1][:2].sum() for g in range(n)])
    order = np.sort(gs)[::-1]
    g_margin = order[G - 1] - order[G] if G < n else np.inf
    keep = set(sorted(range(n), key=lambda i: (-gs[i], i))[:G])
    alive = np.array([sel[e] for e in range(l.shape[0]) if e // per in keep])
    a = np.sort(alive)[::-1]
    e_margin = a[K - 1] - a[K] if K < a.shape[0] else np.inf
    return g_margin, e_margin


@pytest.mark.parametrize("E,n,G,K,T,with_bias", [(128, 8, 4, 8, 515, False), (128, 8, 4, 8, 515, True),
                                                 (256, 8, 4, 8, 130, True), (16, 2, 1, 2, 9, False)])
def test_sigmoid_group_rows_match_the_oracle(E, n, G, K, T, with_bias):
    rng = np.random.default_rng(100 + E + T)
    logits = (rng.standard_normal((T, E)) * 2.0).astype(np.float32)
    bias = (rng.uniform(-0.05, 0.05, E)).astype(np.float32) if with_bias else None
    inds = torch.full((T, K), -1, dtype=torch.int32, device="cuda")
    gates = torch.zeros((T, K), dtype=torch.float32, device="cuda")
    edg.sigmoid_group_topk_rows(torch.from_numpy(logits).cuda(), T, E, K, n, G, 2.5,
                                None if bias is None else torch.from_numpy(bias).cuda(), inds, gates)
    torch.cuda.synchronize()
    inds_h, gates_h = inds.cpu().numpy(), gates.cpu().numpy()
    exact = 0
    for t in range(T):
        want_i, want_w = orc.sigmoid_group_topk(logits[t], K, n, G, 2.5, bias)
        got = inds_h[t]
        assert np.all(np.diff(got) > 0) and got.min() >= 0 and got.max() < E          # K distinct experts, ascending
        # the gates are the renormalised raw sigmoids of whatever was selected
        sig = 1.0 / (1.0 + np.exp(-logits[t, got].astype(np.float64)))
        assert np.allclose(gates_h[t], 2.5 * sig / (sig.sum() + 1e-20), rtol=2e-6, atol=1e-7)
        assert abs(gates_h[t].sum() - 2.5) < 1e-5
        gm, em = _margins(logits[t], bias, K, n, G)
        if gm > 1e-5 and em > 1e-5:
            assert got.tolist() == want_i.tolist(), t
            assert np.allclose(gates_h[t], want_w, rtol=2e-6, atol=1e-7)
            exact += 1
    assert exact >= 0.9 * T                       # the margins rarely bind


def test_sigmoid_group_ties_go_to_the_lower_index_and_group():
    # two groups of four with identical contents: the lower group survives; inside it equal scores go to the lower index
    l = np.array([[1.0, 1.0, 0.5, 0.5, 1.0, 1.0, 0.5, 0.5]], dtype=np.float32)
    inds = torch.zeros((1, 3), dtype=torch.int32, device="cuda")
    gates = torch.zeros((1, 3), dtype=torch.float32, device="cuda")
    edg.sigmoid_group_topk_rows(torch.from_numpy(l).cuda(), 1, 8, 3, 2, 1, 2.5, None, inds, gates)
    torch.cuda.synchronize()
    want_i, want_w = orc.sigmoid_group_topk(l[0], 3, 2, 1, 2.5)
    assert inds.cpu().numpy()[0].tolist() == want_i.tolist() == [0, 1, 2]
    assert np.allclose(gates.cpu().numpy()[0], want_w, rtol=2e-6)


def test_sigmoid_group_rejects_shapes_it_cannot_route():
    z = torch.zeros((1, 8), dtype=torch.float32, device="cuda")
    i = torch.zeros((1, 8), dtype=torch.int32, device="cuda")
    g = torch.zeros((1, 8), dtype=torch.float32, device="cuda")
    for args in [(8, 2, 3, 1), (8, 2, 8, 1), (8, 5, 2, 1), (8, 2, 2, 3)]:      # (E, K, n, G): groups not dividing E, one expert a group, K beyond the survivors, G > n
        with pytest.raises(Exception):
            edg.sigmoid_group_topk_rows(z, 1, args[0], args[1], args[2], args[3], 2.5, None, i, g)


# ------------------------------------------------------------------ the full head (Sec. 3.2 "Head")

# fp32 accumulation of ~3000 fp16 x bf16 products per logit, logits of order 1.  Measured on a B200:
# at most 3.4e-7 (logits up to 3.0), i.e. a few fp32 ulps of the largest logit; the bar is ten times that.
MLP_LOGIT_TOL = 4e-6

@pytest.mark.parametrize("name,width,n_heads,variant", [("cfg2", 512, 3, "full"), ("cfg1", 64, 2, "full"),
                                                       ("cfg2", 512, 1, "no_residual"), ("cfg1", 64, 1, "no_bias")])
def test_mlp_head_matches_the_oracle(name, width, n_heads, variant):
    from workloads import synth
    from tests._gpu_util import x_dev
    cfg = synth.CONFIGS[name]
    d = edg.make_desc(cfg, n_slots=cfg.E)
    E, K, H = cfg.E, cfg.K, cfg.H
    rng = np.random.default_rng(17)
    heads = [synth.mlp_head_weights(cfg, layer, width) for layer in range(n_heads)]
    Wres = [synth.prerouter_weights(cfg, layer) for layer in range(n_heads)]
    X = synth.hidden_states(cfg, n_heads, stream=41)
    cur = np.stack([np.sort(rng.choice(E, K, replace=False)) for _ in range(n_heads)]).astype(np.int32)
    prev = np.stack([np.sort(rng.choice(E, K, replace=False)) for _ in range(n_heads)]).astype(np.int32)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    W1, W2 = dev(np.stack([h["W1"] for h in heads])), dev(np.stack([h["W2"] for h in heads]))
    b1 = None if variant == "no_bias" else dev(np.stack([h["b1"] for h in heads]))
    b2 = None if variant == "no_bias" else dev(np.stack([h["b2"] for h in heads]))
    Wr = None if variant == "no_residual" else dev(np.stack(Wres))
    inds = torch.zeros((n_heads, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((n_heads, K), dtype=torch.float32, device="cuda")
    logits = torch.zeros((n_heads, E), dtype=torch.float32, device="cuda")
    edg.prerouter_mlp_topk(d, W1, b1, W2, b2, Wr, width, x_dev(X), dev(cur), dev(prev), n_heads, inds, gates, logits)
    torch.cuda.synchronize()
    for h in range(n_heads):
        want = orc.prerouter_mlp_logits(heads[h]["W1"], None if b1 is None else heads[h]["b1"], heads[h]["W2"],
                                        None if b2 is None else heads[h]["b2"], None if Wr is None else Wres[h],
                                        X[h], cur[h], prev[h])
        got = logits[h].cpu().numpy().astype(np.float64)
        err = np.abs(got - want).max()
        print(f"mlp head {name}/{variant} head {h}: max |logit error| = {err:.3e}, max |logit| = {np.abs(want).max():.3f}")
        assert err <= MLP_LOGIT_TOL
        # the routing is the exact top-k of the GPU's own logits, and the oracle's wherever its margin allows
        gi, gw = orc.softmax_topk(got, K)
        assert inds[h].cpu().numpy().tolist() == gi.tolist()
        assert np.allclose(gates[h].cpu().numpy(), gw, rtol=1e-5, atol=1e-7)
        srt = np.sort(want)[::-1]
        if srt[K - 1] - srt[K] > 1e-3:
            assert gi.tolist() == orc.softmax_topk(want, K)[0].tolist()
    # the K-hot inputs matter: other executed routings give other logits
    logits2 = torch.zeros_like(logits)
    edg.prerouter_mlp_topk(d, W1, b1, W2, b2, Wr, width, x_dev(X), dev(prev), dev(cur), n_heads, inds, gates, logits2)
    torch.cuda.synchronize()
    assert not torch.equal(logits, logits2)
