"""The shared expert inside the layer-step: y = sum_k w_k expert_k(x) + shared(x), the shared expert
running as one more expert of the same kernel launch with weight 1 and an adapter of its own
(Sec. 3.1 lists it beside the routed experts; Sec. 4 "Phase 2" puts the recovery adapter on it).
Checked against the oracle, chained and alone, with the adapter on the routed experts, on the
shared expert only (the paper's placement), and on neither."""
import dataclasses

import numpy as np
import pytest
import torch

import paper_2609_18063_b200 as edg
from oracle import moe_oracle as orc
from paper_2609_18063_b200 import layer_io
from workloads import synth

from _gpu_util import x_dev
from test_gpu_chain import _run
from test_gpu_parity import _assert_close, _check_routing, _make_store

pytestmark = pytest.mark.gpu

SHARED_ID = 1000          # stream key of the shared expert's tensors (no routed expert has this index)


def _setup(cfg, routed_lora, shared_lora):
    store, d, hosts, slots, tables, cs, keep = _make_store(cfg, n_slots=cfg.E, with_lora=routed_lora)
    for e0 in range(0, cfg.E, 64):
        edg.stage_experts_to_slots(store, 0, np.arange(e0, min(cfg.E, e0 + 64), dtype=np.int32))
    torch.cuda.synchronize()
    shared = synth.expert_tensors(cfg, 0, SHARED_ID)
    rec = torch.from_numpy(edg.pack_expert(d, shared)).cuda()
    slo_np = synth.lora_tensors(cfg, 0, SHARED_ID)
    slo, keep2 = layer_io.lora_to_device(edg.make_desc(cfg, n_adapters=1), [slo_np])
    store.set_shared_expert(0, rec, slo if shared_lora else None)
    return store, d, shared, slo_np, (rec, keep, keep2)


@pytest.mark.parametrize("name,routed_lora,shared_lora,steps", [("cfg1", True, True, 20), ("cfg1", False, True, 12),
                                                               ("cfg1", False, False, 6), ("cfg2", True, True, 8),
                                                               ("cfg2", False, True, 5)])
def test_shared_expert_in_the_layer_step(name, routed_lora, shared_lora, steps):
    cfg = synth.CONFIGS[name]
    store, d, shared, slo_np, keep = _setup(cfg, routed_lora, shared_lora)
    W_np = synth.prerouter_weights(cfg)
    W = torch.from_numpy(W_np).cuda()
    X = synth.hidden_states(cfg, steps + 1, stream=81)
    ws = layer_io.new_workspace(d)
    inds_c, gates_c, logits_c, y_c = _run(cfg, store, d, W, x_dev(X), steps, ws, True)      # chained: steps in flight
    inds_u, gates_u, logits_u, y_u = _run(cfg, store, d, W, x_dev(X), steps, ws, False)     # each step alone
    assert np.array_equal(inds_c, inds_u) and np.abs(logits_c - logits_u).max() <= 1e-5
    assert np.abs(y_c - y_u).max() <= 1e-4
    experts = {}
    get = lambda e: experts.setdefault(e, synth.expert_tensors(cfg, 0, e))
    lora = synth.lora_tensors(cfg, 0, 0)
    for t in range(steps):
        ref = orc.moe_ffn_with_shared(X[t], inds_c[t], gates_c[t].astype(np.float64), get,
                                      (lambda e: lora) if routed_lora else None, shared,
                                      slo_np if shared_lora else None, cfg.lora_scale, cfg.group)
        _assert_close(y_c[t], ref)
        _check_routing(logits_c[t + 1], inds_c[t + 1], gates_c[t + 1], W_np.astype(np.float32), X[t], cfg.K)
    # the shared expert is far above the tolerance: leaving it out cannot pass
    no_shared = orc.moe_ffn(X[0], inds_c[0], gates_c[0].astype(np.float64), get, (lambda e: lora) if routed_lora else None,
                            cfg.lora_scale, cfg.group)
    assert orc.rel_l2(no_shared, y_c[0]) > 0.2
    # taking it away again gives the routed experts alone
    store.set_shared_expert(0, None)
    inds_n, gates_n, logits_n, y_n = _run(cfg, store, d, W, x_dev(X), 2, ws, False)
    _assert_close(y_n[1], orc.moe_ffn(X[1], inds_n[1], gates_n[1].astype(np.float64), get,
                                      (lambda e: lora) if routed_lora else None, cfg.lora_scale, cfg.group))
    store.close()


def test_shared_expert_with_per_expert_adapters_and_on_the_hot_path():
    """Per-expert adapters on the routed experts, the shared expert's own adapter beside them, and the
    hot executor path underneath (misses fetched into transient slots)."""
    cfg = dataclasses.replace(synth.CONFIGS["cfg1"], n_adapters=16)
    store, d, hosts, slots, tables, cs, keep = _make_store(cfg, n_slots=7)
    store.set_hot(True, 1)
    shared = synth.expert_tensors(cfg, 0, SHARED_ID)
    rec = torch.from_numpy(edg.pack_expert(d, shared)).cuda()
    slo_np = synth.lora_tensors(cfg, 0, SHARED_ID)
    slo, keep2 = layer_io.lora_to_device(edg.make_desc(cfg, n_adapters=1), [slo_np])
    store.set_shared_expert(0, rec, slo)
    ws = layer_io.new_workspace(d)
    xb = synth.hidden_states(cfg, 3, stream=82)
    y = torch.zeros((cfg.H,), dtype=torch.float32, device="cuda")
    experts, adapters = {}, {}
    get = lambda e: experts.setdefault(e, synth.expert_tensors(cfg, 0, e))
    get_lora = lambda e: adapters.setdefault(e, synth.lora_tensors(cfg, 0, e))
    for t, P in enumerate(([2, 7], [2, 12], [7, 12])):
        edg.stage_experts_to_slots(store, 0, np.array(P, dtype=np.int32))
        edg.moe_layer_decode(store, 0, x_dev(xb[t]), torch.tensor(P, dtype=torch.int32, device="cuda"),
                             torch.tensor([0.4, 0.6], device="cuda"), None, None, None, None, y, ws)
        torch.cuda.synchronize()
        ref = orc.moe_ffn_with_shared(xb[t], P, [0.4, 0.6], get, get_lora, shared, slo_np, cfg.lora_scale, cfg.group)
        _assert_close(y.cpu().numpy(), ref)
    assert edg.workspace_status(ws) == 0 and store.hot_stats()["hits"] >= 2
    store.close()
