"""The full prerouter head inside the layer-step, with the feedback the paper describes (Sec. 3.2
"Head", "Feature drift"): the head's feature is the hidden state plus the K-hot vector of the routing
the layer executes at this step plus the K-hot vector of the routing it executed at the previous
step -- at decode both are the head's own earlier predictions.  A chain of steps is run through
moe_layer_decode with no host involvement in the feedback; every step's logits are recomputed by
the oracle from the routings the GPU actually executed."""
import numpy as np
import pytest
import torch

import paper_2609_18063_b200 as edg
from oracle import moe_oracle as orc
from paper_2609_18063_b200 import layer_io
from workloads import synth

from _gpu_util import x_dev
from test_gpu_parity import _assert_close, _make_store
from test_gpu_routing import MLP_LOGIT_TOL

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,width,steps", [("cfg2", 512, 24), ("cfg1", 64, 30)])
def test_mlp_head_chain_with_routing_feedback(name, width, steps):
    cfg = synth.CONFIGS[name]
    K, E = cfg.K, cfg.E
    store, d, hosts, slots, tables, cs, _ = _make_store(cfg, n_slots=E)
    for e0 in range(0, E, 64):
        edg.stage_experts_to_slots(store, 0, np.arange(e0, min(E, e0 + 64), dtype=np.int32))
    torch.cuda.synchronize()
    hw = synth.mlp_head_weights(cfg, 0, width)
    Wres_np = synth.prerouter_weights(cfg)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    t_ = {k: dev(v) for k, v in hw.items()}
    Wres = dev(Wres_np)
    store.set_mlp_head(0, t_["W1"], t_["b1"], t_["W2"], t_["b2"], Wres, width)
    X = synth.hidden_states(cfg, steps + 1, stream=95)
    xd = x_dev(X)
    ws = layer_io.new_workspace(d)
    inds = torch.zeros((steps + 1, K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((steps + 1, K), dtype=torch.float32, device="cuda")
    logits = torch.zeros((steps + 1, E), dtype=torch.float32, device="cuda")
    y = torch.zeros((steps, cfg.H), dtype=torch.float32, device="cuda")
    mirror = torch.full((steps + 1, K), -1, dtype=torch.int32).pin_memory()
    edg.prerouter_topk(d, Wres, xd[steps], 1, inds[0], gates[0], logits[0])     # routing of step 0: the linear path on a prompt state
    for t in range(steps):                                                       # no host synchronisation: the feedback stays on the device
        edg.moe_layer_decode(store, 0, xd[t], inds[t], gates[t], None, inds[t + 1], gates[t + 1], logits[t + 1], y[t], ws,
                             inds_next_host_mirror_opt=mirror[t + 1])
    torch.cuda.synchronize()
    assert edg.workspace_status(ws) == 0
    ih, gh, lh, yh = inds.cpu().numpy(), gates.cpu().numpy(), logits.cpu().numpy(), y.cpu().numpy()
    assert np.array_equal(mirror.numpy()[1:], ih[1:])
    experts = {}
    get = lambda e: experts.setdefault(e, synth.expert_tensors(cfg, 0, e))
    lora = synth.lora_tensors(cfg, 0, 0)
    decided = 0
    for t in range(steps):
        prev = ih[t - 1] if t > 0 else []                                      # nothing executed before the first step
        want = orc.prerouter_mlp_logits(hw["W1"], hw["b1"], hw["W2"], hw["b2"], Wres_np, X[t], ih[t], prev)
        got = lh[t + 1].astype(np.float64)
        assert np.abs(got - want).max() <= MLP_LOGIT_TOL, (t, np.abs(got - want).max())
        gi, gw = orc.softmax_topk(got, K)
        assert ih[t + 1].tolist() == gi.tolist() and np.allclose(gh[t + 1], gw, rtol=1e-5, atol=1e-7)
        srt = np.sort(want)[::-1]
        if srt[K - 1] - srt[K] > 1e-4:
            assert gi.tolist() == orc.softmax_topk(want, K)[0].tolist()
            decided += 1
        # the feedback matters: without the previous step's K-hot vector the logits differ
        if t > 0:
            other = orc.prerouter_mlp_logits(hw["W1"], hw["b1"], hw["W2"], hw["b2"], Wres_np, X[t], ih[t], [])
            assert np.abs(other - want).max() > 100 * MLP_LOGIT_TOL
        if t % 4 == 0 or t == steps - 1:
            _assert_close(yh[t], orc.moe_ffn(X[t], ih[t], gh[t].astype(np.float64), get, lambda e: lora, cfg.lora_scale, cfg.group))
    assert decided >= steps - 2
    # a new sequence: the feedback is cleared, the first step again sees an empty "previous" vector
    store.reset_feedback(0)
    l2 = torch.zeros((E,), dtype=torch.float32, device="cuda")
    i2 = torch.zeros((K,), dtype=torch.int32, device="cuda")
    g2 = torch.zeros((K,), dtype=torch.float32, device="cuda")
    edg.moe_layer_decode(store, 0, xd[3], inds[3], gates[3], None, i2, g2, l2, y[0], ws)
    torch.cuda.synchronize()
    want = orc.prerouter_mlp_logits(hw["W1"], hw["b1"], hw["W2"], hw["b2"], Wres_np, X[3], ih[3], [])
    assert np.abs(l2.cpu().numpy() - want).max() <= MLP_LOGIT_TOL
    # removing the head brings the linear path back
    store.set_mlp_head(0)
    edg.moe_layer_decode(store, 0, xd[3], inds[3], gates[3], Wres, i2, g2, l2, y[0], ws)
    torch.cuda.synchronize()
    assert np.abs(l2.cpu().numpy() - orc.prerouter_logits(Wres_np, X[3])).max() <= 1e-5
    store.close()
