"""Batched decode (config 4 shape) and prefill (config 5 shape, reduced token count): the grouped
tensor-core path against the oracle applied token by token."""
import numpy as np
import pytest
import torch

import paper_2609_18063_b200 as edg
from oracle import moe_oracle as orc
from paper_2609_18063_b200 import layer_io
from workloads import synth

from _gpu_util import TOL_MAX_ABS, TOL_REL_L2, device_layer, out_tensor, x_dev

pytestmark = pytest.mark.gpu


def _ffn_tokens(L, d, X_bits, inds, gates, T, use_table=True):
    if L.ws.numel() < edg.ffn_workspace_bytes(d, T):
        L.ws = layer_io.new_workspace(d, T)
    L.ws[:4096].zero_()
    y = out_tensor(d, T)
    table = torch.arange(d.E, dtype=torch.int32, device="cuda") if use_table else None
    edg.moe_expert_ffn_int4_lora(d, L.pool, table, T, inds, inds, gates, x_dev(X_bits), L.lora, y, L.ws)
    torch.cuda.synchronize()
    assert edg.workspace_status(L.ws) == 0
    return y.cpu().numpy()


def _check_tokens(L, X_bits, inds_h, gates_h, Y, tokens):
    cfg = L.cfg
    worst_abs = worst_rel = 0.0
    for t in tokens:
        ref = orc.moe_ffn(X_bits[t], inds_h[t], gates_h[t].astype(np.float64), L.expert, L.get_lora, cfg.lora_scale, cfg.group)
        worst_abs = max(worst_abs, orc.max_abs(Y[t], ref))
        worst_rel = max(worst_rel, orc.rel_l2(Y[t], ref))
    assert worst_abs <= TOL_MAX_ABS and worst_rel <= TOL_REL_L2, (worst_abs, worst_rel)
    return worst_abs, worst_rel


def test_batched_decode_cfg4_shape():
    """64 concurrent tokens, independent top-8 routing from the head, union of experts resident."""
    L = device_layer("cfg2")                      # same layer shape as cfg4; every expert resident
    cfg = synth.CONFIGS["cfg4"]
    T, K, E = cfg.T, cfg.K, cfg.E
    X = synth.hidden_states(cfg, T, stream=31)
    inds = torch.zeros((T, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((T, K), dtype=torch.float32, device="cuda")
    edg.prerouter_topk_tokens(L.desc, L.W, x_dev(X), T, inds, gates, None)
    torch.cuda.synchronize()
    inds_h, gates_h = inds.cpu().numpy(), gates.cpu().numpy()
    for t in range(0, T, 7):                      # the routing is the oracle's (fp64 gap permitting)
        l = orc.prerouter_logits(L.W_np, X[t])
        srt = np.sort(l)[::-1]
        if srt[K - 1] - srt[K] > 1e-4:
            assert inds_h[t].tolist() == orc.softmax_topk(l, K)[0].tolist()
    assert len(np.unique(inds_h)) > 150           # a wide union of experts, a few tokens each
    Y = _ffn_tokens(L, L.desc, X, inds, gates, T)
    _check_tokens(L, X, inds_h, gates_h, Y, range(0, T, 3))
    # the same call with slots given directly (no table) is bit-identical
    Y2 = _ffn_tokens(L, L.desc, X, inds, gates, T, use_table=False)
    assert np.array_equal(Y, Y2)


def test_prefill_cfg5_shape_reduced_tokens():
    """Zipf(1.1)-skewed routing from the router's own logits; ragged token count (not a tile multiple)."""
    L = device_layer("cfg2")
    cfg = synth.CONFIGS["cfg5"]
    T, K, E = 300, cfg.K, cfg.E
    X = synth.hidden_states(cfg, T, stream=32)
    logits = synth.zipf_router_logits(cfg, T)
    inds = torch.zeros((T, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((T, K), dtype=torch.float32, device="cuda")
    edg.softmax_topk_rows(L.desc, torch.from_numpy(logits).cuda(), T, inds, gates)
    torch.cuda.synchronize()
    inds_h, gates_h = inds.cpu().numpy(), gates.cpu().numpy()
    for t in range(T):
        i_ref, w_ref = orc.softmax_topk(logits[t], K)
        assert inds_h[t].tolist() == i_ref.tolist() and np.abs(gates_h[t] - w_ref).max() <= 2e-6
    counts = np.bincount(inds_h.ravel(), minlength=E)
    assert counts.max() > 64 and counts.max() > 10 * max(1, np.median(counts))     # skewed: some groups span several tiles
    Y = _ffn_tokens(L, L.desc, X, inds, gates, T)
    rng = np.random.default_rng(0)
    sample = sorted(set(rng.choice(T, 14, replace=False).tolist()) | {0, T - 1})
    _check_tokens(L, X, inds_h, gates_h, Y, sample)
    assert np.isfinite(Y).all()


def test_prefill_cfg5_full_size_sampled_tokens():
    """The full 4096-token prefill in the launch configuration the benchmark times (tiles of 128
    tokens on the tcgen05 path; the popular experts span many tiles, the unpopular ones a ragged
    fraction of one).  The oracle computes sampled tokens one by one; every output must be finite."""
    L = device_layer("cfg2")
    cfg = synth.CONFIGS["cfg5"]
    T, K, E = cfg.T, cfg.K, cfg.E
    assert T == 4096
    X = synth.hidden_states(cfg, T, stream=34)
    logits = synth.zipf_router_logits(cfg, T)
    inds = torch.zeros((T, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((T, K), dtype=torch.float32, device="cuda")
    edg.softmax_topk_rows(L.desc, torch.from_numpy(logits).cuda(), T, inds, gates)
    torch.cuda.synchronize()
    inds_h, gates_h = inds.cpu().numpy(), gates.cpu().numpy()
    counts = np.bincount(inds_h.ravel(), minlength=E)
    assert counts.max() > 8 * 128 and counts.min() < 128          # many tiles for some experts, a partial tile for others
    Y = _ffn_tokens(L, L.desc, X, inds, gates, T)
    assert np.isfinite(Y).all()
    rng = np.random.default_rng(3)
    # tokens routed to the most and to the least popular expert, plus a random sample and both ends
    hot, cold = int(np.argmax(counts)), int(np.argmin(np.where(counts > 0, counts, 1 << 30)))
    pick = {0, T - 1, int(np.nonzero((inds_h == hot).any(axis=1))[0][-1]), int(np.nonzero((inds_h == cold).any(axis=1))[0][0])}
    pick |= set(rng.choice(T, 12, replace=False).tolist())
    # an expert of middling popularity that spans a few 128-token tiles: the tokens on both sides of
    # its first tile boundary, its first and its last token (the ragged tail of its last tile)
    mid = int(np.argmin(np.where((counts > 256) & (counts < 1024), np.abs(counts - 400), 1 << 30)))
    assert 256 < counts[mid] < 1024
    toks = np.nonzero((inds_h == mid).any(axis=1))[0]          # ascending, the order of the expert's token list
    pick |= {int(toks[0]), int(toks[127]), int(toks[128]), int(toks[255]), int(toks[256]), int(toks[-1])}
    _check_tokens(L, X, inds_h, gates_h, Y, sorted(pick))
    # a second run is bit-identical (fixed reduction order, no atomics on the data path)
    Y2 = _ffn_tokens(L, L.desc, X, inds, gates, T)
    assert np.array_equal(Y, Y2)


@pytest.mark.parametrize("n_adapters", [1, 16])
def test_large_groups_on_the_small_layer_shape(n_adapters):
    """The tensor-memory path on the other supported shape: H 1024, I 256, groups of 32 (a new scale
    every chunk), rank 8 (half an MMA k-step, zero-padded), shared and per-expert adapters, ragged
    tiles (token counts that are no multiple of 16) and experts that span several tiles."""
    L = device_layer("cfg1", n_adapters)
    cfg = L.cfg
    T = 333
    X = synth.hidden_states(cfg, T, stream=35)
    rng = np.random.default_rng(7)
    pop = np.array([8.0] * 2 + [1.0] * (cfg.E - 2)); pop /= pop.sum()            # two hot experts
    inds_h = np.stack([np.sort(rng.choice(cfg.E, cfg.K, replace=False, p=pop)) for _ in range(T)]).astype(np.int32)
    gates_h = rng.dirichlet(np.ones(cfg.K), size=T).astype(np.float32)
    counts = np.bincount(inds_h.ravel(), minlength=cfg.E)
    assert T * cfg.K > 8 * cfg.E and counts.max() > 128 and (counts % 16 != 0).any()
    inds, gates = torch.from_numpy(inds_h).cuda(), torch.from_numpy(gates_h).cuda()
    Y = _ffn_tokens(L, L.desc, X, inds, gates, T)
    _check_tokens(L, X, inds_h, gates_h, Y, range(T))


def test_grouped_reduces_to_the_decode_path_and_handles_per_expert_adapters():
    L = device_layer("cfg1", 16)                  # per-expert adapters
    cfg = L.cfg
    T = 7
    X = synth.hidden_states(cfg, T, stream=33)
    X[3] = X[0]                                   # two identical tokens with identical routing
    rng = np.random.default_rng(1)
    inds_h = np.stack([np.sort(rng.choice(cfg.E, cfg.K, replace=False)) for _ in range(T)]).astype(np.int32)
    gates_h = rng.dirichlet(np.ones(cfg.K), size=T).astype(np.float32)
    inds_h[3], gates_h[3] = inds_h[0], gates_h[0]
    inds, gates = torch.from_numpy(inds_h).cuda(), torch.from_numpy(gates_h).cuda()
    Y = _ffn_tokens(L, L.desc, X, inds, gates, T)
    _check_tokens(L, X, inds_h, gates_h, Y, range(T))
    assert np.array_equal(Y[0], Y[3])
    # T = 1 (fused decode kernel) on the same token agrees with the grouped result
    y1 = _ffn_tokens(L, L.desc, X[:1], inds[:1].contiguous(), gates[:1].contiguous(), 1)
    assert orc.max_abs(y1[0], Y[0]) <= TOL_MAX_ABS and orc.rel_l2(y1[0], Y[0]) <= TOL_REL_L2
    # an out-of-range expert in one pair is skipped and flagged, the other tokens are untouched
    bad = inds_h.copy(); bad[5, 1] = cfg.E
    L.ws[:4096].zero_()
    y = out_tensor(L.desc, T)
    edg.moe_expert_ffn_int4_lora(L.desc, L.pool, torch.arange(cfg.E, dtype=torch.int32, device="cuda"), T,
                                 torch.from_numpy(bad).cuda(), None, gates, x_dev(X), L.lora, y, L.ws)
    torch.cuda.synchronize()
    assert edg.workspace_status(L.ws) == -4
    yb = y.cpu().numpy()
    assert np.array_equal(yb[0], Y[0]) and np.array_equal(yb[6], Y[6])
