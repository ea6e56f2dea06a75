"""The hot executor path on the GPU (Sec. 3.1: LRU-resident hot experts, misses fall to the on-demand
path): hits run from the hot set, misses are fetched by the SMs from the pinned-host tier into
transient slots inside the layer-step, admissions land behind the step.  Every step is compared
with the oracle (outputs, routing), the bookkeeping with the oracle's hot-set allocator."""
import dataclasses

import numpy as np
import pytest
import torch

import paper_2609_18063_b200 as edg
from oracle import moe_oracle as orc
from paper_2609_18063_b200 import layer_io
from workloads import synth

from _gpu_util import x_dev
from test_gpu_parity import _assert_close, _check_routing, _make_store

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,K,S_hot,admit_after,steps", [("cfg1", 2, 5, 1, 48), ("cfg1", 2, 3, 2, 48),
                                                          ("cfg2", 4, 24, 1, 10), ("cfg2", 8, 40, 1, 6)])
def test_hot_path_decode_matches_oracle(name, K, S_hot, admit_after, steps):
    cfg = dataclasses.replace(synth.CONFIGS[name], K=K)           # K = 4: the 35B tier's shipped profile
    store, d, hosts, slots, tables, cs, _ = _make_store(cfg, n_slots=S_hot + K)
    store.set_hot(True, admit_after)
    hot = orc.HotSetAllocator(cfg.E, S_hot, admit_after)
    W_np = synth.prerouter_weights(cfg)
    W = torch.from_numpy(W_np).cuda()
    # correlated states, so that consecutive steps share experts and the hot set earns hits
    X = synth.hidden_states_ar1(cfg, steps + 1, 0.8, stream=71)
    xd = x_dev(X)
    ws = layer_io.new_workspace(d)
    inds = torch.zeros((steps + 1, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((steps + 1, K), dtype=torch.float32, device="cuda")
    logits = torch.zeros((steps + 1, cfg.E), dtype=torch.float32, device="cuda")
    y = torch.zeros((steps, cfg.H), dtype=torch.float32, device="cuda")
    mirror = torch.full((steps + 1, K), -1, dtype=torch.int32).pin_memory()
    edg.prerouter_topk(d, W, xd[steps], 1, inds[0], gates[0], logits[0], inds_host_mirror_opt=mirror[0])
    torch.cuda.synchronize()
    for t in range(steps):
        P = mirror[t].numpy().copy()
        assert (P >= 0).all()
        got, n_miss = edg.stage_experts_to_slots(store, 0, P)
        want, adm = hot.step(P.tolist())
        assert got.tolist() == want and n_miss == sum(1 for s in want if s < 0)
        edg.moe_layer_decode(store, 0, xd[t], inds[t], gates[t], W, inds[t + 1], gates[t + 1], logits[t + 1], y[t], ws,
                             inds_next_host_mirror_opt=mirror[t + 1])
        torch.cuda.synchronize()                                  # the host needs the next routing to stage it
    assert edg.workspace_status(ws) == 0
    ih, gh, lh, yh = inds.cpu().numpy(), gates.cpu().numpy(), logits.cpu().numpy(), y.cpu().numpy()
    experts = {}
    get = lambda e: experts.setdefault(e, synth.expert_tensors(cfg, 0, e))
    lora = synth.lora_tensors(cfg, 0, 0)
    for t in range(steps):
        ref = orc.moe_ffn(X[t], ih[t], gh[t].astype(np.float64), get, lambda e: lora, cfg.lora_scale, cfg.group)
        _assert_close(yh[t], ref)
        _check_routing(lh[t + 1], ih[t + 1], gh[t + 1], W_np.astype(np.float32), X[t], K)
    hs = store.hot_stats()
    assert (hs["hits"], hs["misses"], hs["admitted"]) == (hot.hits, hot.misses, hot.admitted)
    assert hs["hits"] > 0 and hs["misses"] > 0                    # both kinds of step were exercised
    cs.synchronize()
    eos, soe = store.snapshot(0)
    assert eos.tolist()[:S_hot] == hot.expert_of_slot and soe.tolist() == hot.slot_of_expert
    assert tables[0].cpu().numpy().tolist() == soe.tolist()
    pool = slots[0].cpu()
    for sl, e in enumerate(hot.expert_of_slot):
        if e >= 0:
            assert torch.equal(pool[sl], hosts[0][e])             # admissions carried the right bytes
    store.close()


def test_hot_path_with_per_expert_adapters_and_a_bad_index():
    """Misses served from transient slots still pick the adapter of their expert; an expert id out of
    range is skipped and flagged, as on every other path."""
    cfg = dataclasses.replace(synth.CONFIGS["cfg1"], n_adapters=16)
    store, d, hosts, slots, tables, cs, _ = _make_store(cfg, n_slots=6)
    store.set_hot(True, 1)
    xb = synth.hidden_states(cfg, 2, stream=72)
    ws = layer_io.new_workspace(d)
    y = torch.zeros((cfg.H,), dtype=torch.float32, device="cuda")
    adapters = {}
    get_lora = lambda e: adapters.setdefault(e, synth.lora_tensors(cfg, 0, e))
    experts = {}
    get = lambda e: experts.setdefault(e, synth.expert_tensors(cfg, 0, e))
    for t, P in enumerate(([3, 9], [3, 11])):                    # second step: one hit (3), one miss (11)
        inds = torch.tensor(P, dtype=torch.int32, device="cuda")
        gates = torch.tensor([0.3, 0.7], dtype=torch.float32, device="cuda")
        edg.stage_experts_to_slots(store, 0, np.array(P, dtype=np.int32))
        edg.moe_layer_decode(store, 0, x_dev(xb[t]), inds, gates, None, None, None, None, y, ws)
        torch.cuda.synchronize()
        ref = orc.moe_ffn(xb[t], P, [0.3, 0.7], get, get_lora, cfg.lora_scale, cfg.group)
        _assert_close(y.cpu().numpy(), ref)
    assert store.hot_stats()["hits"] == 1
    assert edg.workspace_status(ws) == 0
    inds = torch.tensor([3, cfg.E + 5], dtype=torch.int32, device="cuda")
    edg.moe_layer_decode(store, 0, x_dev(xb[0]), inds, torch.tensor([1.0, 0.5], device="cuda"), None, None, None, None, y, ws)
    torch.cuda.synchronize()
    assert edg.workspace_status(ws) == -4
    ref = orc.moe_ffn(xb[0], [3], [1.0], get, get_lora, cfg.lora_scale, cfg.group)
    _assert_close(y.cpu().numpy(), ref)
    store.close()
