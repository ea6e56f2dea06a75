"""Chained layer-steps (Sec. 3.2: step t+1 consumes the routing predicted during step t) launched
back to back without host synchronisation, so that several steps are in flight at once and the
hand-off ring inside the workspace wraps around several times.  Every checked step must match the
oracle on the routing the GPU itself produced, the routing must be the exact top-k of the GPU's own
logits, and switching the chaining off must give the same indices and the same outputs."""
import numpy as np
import pytest
import torch

import paper_2609_18063_b200 as edg
from paper_2609_18063_b200 import layer_io
from oracle import moe_oracle as orc
from workloads import synth
from tests._gpu_util import x_dev, out_tensor
from tests.test_gpu_parity import _make_store, _check_routing, _assert_close

pytestmark = pytest.mark.gpu


def _run(cfg, store, d, W, xd, steps, ws, chaining):
    store.set_chaining(2 if chaining else 0)    # 2: chain whether or not the previous step is still running
    inds = torch.zeros((steps + 1, cfg.K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((steps + 1, cfg.K), dtype=torch.float32, device="cuda")
    logits = torch.zeros((steps + 1, cfg.E), dtype=torch.float32, device="cuda")
    edg.prerouter_topk(d, W, xd[steps], 1, inds[0], gates[0], logits[0])
    y = out_tensor(d, steps)
    for t in range(steps):                      # no host synchronisation inside the loop
        edg.moe_layer_decode(store, 0, xd[t], inds[t], gates[t], W, inds[t + 1], gates[t + 1], logits[t + 1], y[t], ws)
    torch.cuda.synchronize()
    assert edg.workspace_status(ws) == 0
    return inds.cpu().numpy(), gates.cpu().numpy(), logits.cpu().numpy(), y.float().cpu().numpy()


@pytest.mark.parametrize("name,steps,stride", [("cfg1", 50, 1), ("cfg2", 50, 7)])
def test_chained_steps_in_flight_match_oracle_and_unchained(name, steps, stride):
    cfg = synth.CONFIGS[name]
    store, d, hosts, slots, tables, cs, _ = _make_store(cfg, n_slots=cfg.E)
    for e0 in range(0, cfg.E, 64):              # everything resident: no staging between the steps
        edg.stage_experts_to_slots(store, 0, np.arange(e0, min(cfg.E, e0 + 64), dtype=np.int32))
    torch.cuda.synchronize()
    W_np = synth.prerouter_weights(cfg)
    W = torch.from_numpy(W_np).cuda()
    X = synth.hidden_states(cfg, steps + 1, stream=23)
    xd = x_dev(X)
    ws = layer_io.new_workspace(d)
    inds_c, gates_c, logits_c, y_c = _run(cfg, store, d, W, xd, steps, ws, True)
    inds_u, gates_u, logits_u, y_u = _run(cfg, store, d, W, xd, steps, ws, False)
    # the routing is the same in both launch modes, floats agree far inside the tolerance
    assert np.array_equal(inds_c, inds_u)
    # (the two launch forms split a head row's K range differently: same logits up to fp32 rounding)
    assert np.abs(logits_c - logits_u).max() <= 1e-5
    assert np.abs(gates_c - gates_u).max() <= 1e-5
    assert np.abs(y_c - y_u).max() <= 1e-4
    experts = {}
    get = lambda e: experts.setdefault(e, synth.expert_tensors(cfg, 0, e))
    lora = synth.lora_tensors(cfg, 0, 0)
    for t in list(range(0, steps, stride)) + [steps - 1]:
        ref = orc.moe_ffn(X[t], inds_c[t], gates_c[t].astype(np.float64), get, lambda e: lora, cfg.lora_scale, cfg.group)
        _assert_close(y_c[t], ref)
        _check_routing(logits_c[t + 1], inds_c[t + 1], gates_c[t + 1], W_np, X[t], cfg.K)
    store.close()


def test_a_hand_off_that_never_arrives_times_out_and_falls_back():
    """Failure path of the chained hand-off, provoked from the host: after a step has published its
    head's logits and routing in the workspace ring, the test wipes that ring slot (back to "not yet
    written"), so the chained next step polls for a routing that never comes.  Its bounded wait must run out, raise
    EDG_E_TIMEOUT in the status word, fall back to waiting for the previous kernel and to the routing
    that kernel wrote -- and still produce the right output.  Nothing faults or hangs."""
    cfg = synth.CONFIGS["cfg1"]
    store, d, hosts, slots, tables, cs, _ = _make_store(cfg, n_slots=cfg.E)
    edg.stage_experts_to_slots(store, 0, np.arange(cfg.E, dtype=np.int32))
    torch.cuda.synchronize()
    W_np = synth.prerouter_weights(cfg)
    W = torch.from_numpy(W_np).cuda()
    X = synth.hidden_states(cfg, 3, stream=29)
    xd = x_dev(X)
    ws = layer_io.new_workspace(d)
    store.set_chaining(2)                       # the default would launch a step that finds the GPU idle on its own
    inds = torch.zeros((3, cfg.K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((3, cfg.K), dtype=torch.float32, device="cuda")
    logits = torch.zeros((3, cfg.E), dtype=torch.float32, device="cuda")
    y = out_tensor(d, 2)
    edg.prerouter_topk(d, W, xd[2], 1, inds[0], gates[0], logits[0])
    edg.moe_layer_decode(store, 0, xd[0], inds[0], gates[0], W, inds[1], gates[1], logits[1], y[0], ws)
    torch.cuda.synchronize()
    assert edg.workspace_status(ws) == 0
    # find the ring slot that holds the published logits and wipe it
    wsf = ws.view(torch.float32)
    first = (wsf == logits[1][0]).nonzero().flatten().tolist()
    hits = [i for i in first if i + cfg.E <= wsf.numel() and torch.equal(wsf[i:i + cfg.E], logits[1])]
    assert len(hits) == 1
    ws.view(torch.int32)[hits[0]:hits[0] + cfg.E + 64] = -1     # the logits and the (expert, gate) pairs behind them
    torch.cuda.synchronize()
    edg.moe_layer_decode(store, 0, xd[1], inds[1], gates[1], W, inds[2], gates[2], logits[2], y[1], ws)   # chained
    torch.cuda.synchronize()
    assert edg.workspace_status(ws) == -6                      # EDG_E_TIMEOUT, sticky
    inds_h, gates_h, y_h = inds.cpu().numpy(), gates.cpu().numpy(), y.float().cpu().numpy()
    experts = {}
    get = lambda e: experts.setdefault(e, synth.expert_tensors(cfg, 0, e))
    lora = synth.lora_tensors(cfg, 0, 0)
    for t in range(2):
        ref = orc.moe_ffn(X[t], inds_h[t], gates_h[t].astype(np.float64), get, lambda e: lora, cfg.lora_scale, cfg.group)
        _assert_close(y_h[t], ref)
    _check_routing(logits[2].cpu().numpy(), inds_h[2], gates_h[2], W_np, X[1], cfg.K)
    store.close()


def test_default_policy_gives_the_same_results_whether_or_not_steps_overlap():
    """Default chaining policy: a step is chained only while the step before it is still in flight.
    With a host synchronisation after every step each step finds the GPU idle and is launched on its
    own; without one the steps queue up and are chained.  Indices and logits must be bit-equal in
    both regimes and equal to those with chaining off; outputs agree far inside the tolerance."""
    cfg = synth.CONFIGS["cfg1"]
    steps = 24
    store, d, hosts, slots, tables, cs, _ = _make_store(cfg, n_slots=cfg.E)
    edg.stage_experts_to_slots(store, 0, np.arange(cfg.E, dtype=np.int32))
    torch.cuda.synchronize()
    W = torch.from_numpy(synth.prerouter_weights(cfg)).cuda()
    xd = x_dev(synth.hidden_states(cfg, steps + 1, stream=31))
    ws = layer_io.new_workspace(d)

    def run(mode, sync_each):
        store.set_chaining(mode)
        inds = torch.zeros((steps + 1, cfg.K), dtype=torch.int32, device="cuda")
        gates = torch.zeros((steps + 1, cfg.K), dtype=torch.float32, device="cuda")
        logits = torch.zeros((steps + 1, cfg.E), dtype=torch.float32, device="cuda")
        edg.prerouter_topk(d, W, xd[steps], 1, inds[0], gates[0], logits[0])
        y = out_tensor(d, steps)
        for t in range(steps):
            edg.moe_layer_decode(store, 0, xd[t], inds[t], gates[t], W, inds[t + 1], gates[t + 1], logits[t + 1], y[t], ws)
            if sync_each:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        assert edg.workspace_status(ws) == 0
        return inds.cpu().numpy(), logits.cpu().numpy(), y.float().cpu().numpy()

    ref = run(0, False)
    for mode, sync_each in [(1, True), (1, False), (2, True)]:
        got = run(mode, sync_each)
        assert np.array_equal(got[0], ref[0])
        assert np.abs(got[1] - ref[1]).max() <= 1e-5
        assert np.abs(got[2] - ref[2]).max() <= 1e-4
    store.close()


@pytest.mark.parametrize("per_expert_adapters", [False, True])
def test_chained_small_layer_with_an_fp16_head(per_expert_adapters):
    """The small layer shape with an fp16 head, chained unconditionally.  With one shared adapter a
    cluster takes both routed experts one after the other; with one adapter per expert every expert
    has a cluster of its own and the adapter follows the expert.  Every step is checked against the
    oracle on the routing the GPU produced."""
    import dataclasses
    base = synth.CONFIGS["cfg1"]
    cfg = dataclasses.replace(base, pre_dtype="f16", n_adapters=base.E if per_expert_adapters else 1)
    steps = 20
    store, d, hosts, slots, tables, cs, _ = _make_store(cfg, n_slots=cfg.E)
    edg.stage_experts_to_slots(store, 0, np.arange(cfg.E, dtype=np.int32))
    torch.cuda.synchronize()
    W_np = synth.prerouter_weights(cfg)
    W = torch.from_numpy(W_np).cuda()
    X = synth.hidden_states(cfg, steps + 1, stream=37)
    xd = x_dev(X)
    ws = layer_io.new_workspace(d)
    inds_c, gates_c, logits_c, y_c = _run(cfg, store, d, W, xd, steps, ws, True)
    inds_u, gates_u, logits_u, y_u = _run(cfg, store, d, W, xd, steps, ws, False)
    assert np.array_equal(inds_c, inds_u) and np.abs(logits_c - logits_u).max() <= 1e-5 and np.abs(gates_c - gates_u).max() <= 1e-5
    assert np.abs(y_c - y_u).max() <= 1e-4
    experts, adapters = {}, {}
    get = lambda e: experts.setdefault(e, synth.expert_tensors(cfg, 0, e))
    get_lora = lambda e: adapters.setdefault(e if per_expert_adapters else 0, synth.lora_tensors(cfg, 0, e if per_expert_adapters else 0))
    for t in range(steps):
        ref = orc.moe_ffn(X[t], inds_c[t], gates_c[t].astype(np.float64), get, get_lora, cfg.lora_scale, cfg.group)
        _assert_close(y_c[t], ref)
        _check_routing(logits_c[t + 1], inds_c[t + 1], gates_c[t + 1], W_np.astype(np.float32), X[t], cfg.K)
    store.close()
