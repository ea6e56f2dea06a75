"""Data-dependent layer-steps, the way a decoder produces them: the hidden state of step t+1 is
x(t+1) = bf16(rmsnorm(x(t) + y(t))), computed on the device, so no step can start its arithmetic
before the one before it has finished.  Parity is step-local: the GPU's own x(t) is read back and
fed to the oracle for that step only, so a rounding difference in one step cannot leak into the
bit-exact routing checks of the next.  Also here: the host mirror of the predicted routing."""
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


def _bf16_ulps(a_bits, b_bits):
    """distance in bf16 steps between two arrays of bit patterns (sign-magnitude -> ordered ints)"""
    def key(b):
        b = b.astype(np.int32)
        return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
    return np.abs(key(a_bits) - key(b_bits))


@pytest.mark.parametrize("name,steps,chaining", [("cfg1", 40, 0), ("cfg2", 12, 0), ("cfg1", 40, 1)])
def test_dependent_chain_step_local_parity(name, steps, chaining):
    cfg = synth.CONFIGS[name]
    store, d, hosts, slots, tables, cs, _ = _make_store(cfg, n_slots=cfg.E)
    for e0 in range(0, cfg.E, 64):
        edg.stage_experts_to_slots(store, 0, np.arange(e0, min(cfg.E, e0 + 64), dtype=np.int32))
    torch.cuda.synchronize()
    # chaining 1 (adaptive) would chain steps that are still in flight: with x produced between two
    # calls that breaks the chained call's contract, so the dependent chain must run unchained; the
    # parametrisation with chaining = 1 checks that a host sync per step (GPU idle) keeps it correct
    store.set_chaining(chaining)
    W_np = synth.prerouter_weights(cfg)
    W = torch.from_numpy(W_np).cuda()
    x0 = synth.hidden_states(cfg, 2, stream=61)
    xs = torch.zeros((steps + 1, cfg.H), dtype=torch.bfloat16, device="cuda")
    xs[0] = x_dev(x0[0])
    inds = torch.zeros((steps + 1, cfg.K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((steps + 1, cfg.K), dtype=torch.float32, device="cuda")
    logits = torch.zeros((steps + 1, cfg.E), dtype=torch.float32, device="cuda")
    y = torch.zeros((steps, cfg.H), dtype=torch.float32, device="cuda")
    ws = layer_io.new_workspace(d)
    edg.prerouter_topk(d, W, x_dev(x0[1]), 1, inds[0], gates[0], logits[0])
    for t in range(steps):
        edg.moe_layer_decode(store, 0, xs[t], inds[t], gates[t], W, inds[t + 1], gates[t + 1], logits[t + 1], y[t], ws)
        edg.next_hidden_state(d, xs[t], y[t], xs[t + 1], 1e-6)
        if chaining:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    assert edg.workspace_status(ws) == 0
    X = xs.view(torch.int16).cpu().numpy().view(np.uint16)
    ih, gh, lh, yh = inds.cpu().numpy(), gates.cpu().numpy(), logits.cpu().numpy(), y.cpu().numpy()
    experts = {}
    get = lambda e: experts.setdefault(e, synth.expert_tensors(cfg, 0, e))
    lora = synth.lora_tensors(cfg, 0, 0)
    assert len({tuple(r) for r in ih.tolist()}) > steps // 2          # the routing really changes from step to step
    for t in range(steps):
        ref = orc.moe_ffn(X[t], ih[t], gh[t].astype(np.float64), get, lambda e: lora, cfg.lora_scale, cfg.group)
        _assert_close(yh[t], ref)
        _check_routing(lh[t + 1], ih[t + 1], gh[t + 1], W_np.astype(np.float32), X[t], cfg.K)
        want = orc.next_hidden_state(X[t], yh[t].astype(np.float64), 1e-6)      # from the GPU's own y: step-local
        assert _bf16_ulps(X[t + 1], want).max() <= 1
        assert (X[t + 1] == want).mean() > 0.98
    rms = np.sqrt(np.mean(orc.bf16_to_f64(X[steps]) ** 2))
    assert 0.99 < rms < 1.01
    store.close()


@pytest.mark.parametrize("out_dtype", ["f16", "bf16"])
def test_next_hidden_state_reads_every_output_dtype(out_dtype):
    cfg = synth.CONFIGS["cfg1"]
    d = edg.make_desc(cfg, out_dtype=out_dtype, n_slots=cfg.E)
    rng = np.random.default_rng(3)
    xb = synth.hidden_states(cfg, 1, stream=62)[0]
    yt = torch.from_numpy((rng.standard_normal(cfg.H) * 6).astype(np.float32)).cuda().to(
        torch.float16 if out_dtype == "f16" else torch.bfloat16)
    xn = torch.zeros((cfg.H,), dtype=torch.bfloat16, device="cuda")
    edg.next_hidden_state(d, x_dev(xb), yt, xn, 1e-6)
    torch.cuda.synchronize()
    want = orc.next_hidden_state(xb, yt.float().cpu().numpy().astype(np.float64), 1e-6)
    got = xn.view(torch.int16).cpu().numpy().view(np.uint16)
    assert _bf16_ulps(got, want).max() <= 1 and (got == want).mean() > 0.98


def test_predicted_routing_is_mirrored_into_pinned_host_memory():
    """The stager's hand-off without a device-to-host copy: the kernels store the predicted indices in
    mapped pinned host memory as well.  The caller fills the mirror with -1; every entry is final once
    it is >= 0.  Both the stand-alone head and the head inside the layer-step must do it."""
    cfg = synth.CONFIGS["cfg2"]
    store, d, hosts, slots, tables, cs, _ = _make_store(cfg, n_slots=16)
    W = torch.from_numpy(np.stack([synth.prerouter_weights(cfg, l) for l in range(3)])).cuda()
    X = x_dev(synth.hidden_states(cfg, 3, stream=63))
    inds = torch.zeros((3, cfg.K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((3, cfg.K), dtype=torch.float32, device="cuda")
    mirror = torch.full((3, cfg.K), -1, dtype=torch.int32).pin_memory()
    edg.prerouter_topk(d, W, X, 3, inds, gates, None, inds_host_mirror_opt=mirror)
    torch.cuda.synchronize()
    assert (mirror.numpy() >= 0).all() and np.array_equal(mirror.numpy(), inds.cpu().numpy())
    # inside the layer-step: stage from the mirror, decode, and find the next prediction mirrored
    ws = layer_io.new_workspace(d)
    y = torch.zeros((cfg.H,), dtype=torch.float32, device="cuda")
    nxt = torch.full((cfg.K,), -1, dtype=torch.int32).pin_memory()
    i2 = torch.zeros((cfg.K,), dtype=torch.int32, device="cuda")
    g2 = torch.zeros((cfg.K,), dtype=torch.float32, device="cuda")
    edg.stage_experts_to_slots(store, 0, mirror.numpy()[0])
    edg.moe_layer_decode(store, 0, X[1], inds[0], gates[0], W[1], i2, g2, None, y, ws, inds_next_host_mirror_opt=nxt)
    # poll, as a stager would, instead of synchronising the stream
    import time
    t0 = time.time()
    while (nxt.numpy() < 0).any() and time.time() - t0 < 10.0:
        pass
    assert (nxt.numpy() >= 0).all()
    torch.cuda.synchronize()
    assert np.array_equal(nxt.numpy(), i2.cpu().numpy())
    assert np.array_equal(nxt.numpy(), inds[1].cpu().numpy())       # same head, same state as the batched call above
    store.close()


def test_exposed_wait_measurement_counts_the_waits_it_brackets():
    cfg = synth.CONFIGS["cfg1"]
    store, d, hosts, slots, tables, cs, _ = _make_store(cfg, n_slots=4)
    store.time_waits(True)
    W = torch.from_numpy(synth.prerouter_weights(cfg)).cuda()
    X = x_dev(synth.hidden_states(cfg, 9, stream=64))
    inds = torch.zeros((10, cfg.K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((10, cfg.K), dtype=torch.float32, device="cuda")
    y = torch.zeros((9, cfg.H), dtype=torch.float32, device="cuda")
    ws = layer_io.new_workspace(d)
    edg.prerouter_topk(d, W, X[8], 1, inds[0], gates[0], None)
    staged_with_copies = 0
    for t in range(8):
        torch.cuda.synchronize()
        n_miss = edg.stage_experts_to_slots(store, 0, inds[t].cpu().numpy())[1]
        staged_with_copies += 1 if n_miss else 0
        edg.moe_layer_decode(store, 0, X[t], inds[t], gates[t], W, inds[t + 1], gates[t + 1], None, y[t], ws)
    ms, n = store.exposed_wait_ms()
    assert n == staged_with_copies and n >= 1 and 0.0 <= ms < 1000.0
    assert store.exposed_wait_ms() == (0.0, 0)                       # reading resets
    store.close()


@pytest.mark.parametrize("name,steps,chaining,out_dtype", [("cfg1", 300, 2, "f32"), ("cfg2", 40, 2, "f32"), ("cfg1", 40, 0, "f32"),
                                                          ("cfg2", 12, 1, "f32"), ("cfg1", 30, 2, "f16"), ("cfg1", 30, 2, "bf16")])
def test_dependent_chain_with_the_state_produced_inside_the_layer_kernel(name, steps, chaining, out_dtype):
    """moe_layer_decode_dependent: the kernel's last reducer writes x(t+1) itself, and with chaining on
    step t+1 is already resident, has its routing and its first weights, and waits on a device flag
    for x(t+1).  No host synchronisation inside the loop (300 steps wrap the 128-slot ring twice).
    Step-local parity against the oracle on the GPU's own x(t)."""
    cfg = synth.CONFIGS[name]
    d_out = edg.make_desc(cfg, n_slots=cfg.E, out_dtype=out_dtype)
    store, d, hosts, slots, tables, cs, _ = _make_store(cfg, n_slots=cfg.E)
    store.close()
    # (a store whose descriptor carries the output type under test)
    loras = [layer_io.lora_to_device(d_out, [synth.lora_tensors(cfg, 0, a) for a in range(cfg.n_adapters)])]
    store = edg.Store(d_out, hosts, slots, tables, [loras[0][0]], cs)
    d = d_out
    for e0 in range(0, cfg.E, 64):
        edg.stage_experts_to_slots(store, 0, np.arange(e0, min(cfg.E, e0 + 64), dtype=np.int32))
    torch.cuda.synchronize()
    store.set_chaining(chaining)
    W_np = synth.prerouter_weights(cfg)
    W = torch.from_numpy(W_np).cuda()
    x0 = synth.hidden_states(cfg, 2, stream=65)
    xs = torch.zeros((steps + 1, cfg.H), dtype=torch.bfloat16, device="cuda")
    xs[0] = x_dev(x0[0])
    inds = torch.zeros((steps + 1, cfg.K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((steps + 1, cfg.K), dtype=torch.float32, device="cuda")
    logits = torch.zeros((steps + 1, cfg.E), dtype=torch.float32, device="cuda")
    ydt = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}[out_dtype]
    y = torch.zeros((steps, cfg.H), dtype=ydt, device="cuda")
    ws = layer_io.new_workspace(d)
    edg.prerouter_topk(d, W, x_dev(x0[1]), 1, inds[0], gates[0], logits[0])
    for t in range(steps):
        edg.moe_layer_decode_dependent(store, 0, xs[t], inds[t], gates[t], W, inds[t + 1], gates[t + 1], logits[t + 1],
                                       y[t], xs[t + 1], ws, 1e-6)
    torch.cuda.synchronize()
    assert edg.workspace_status(ws) == 0
    X = xs.view(torch.int16).cpu().numpy().view(np.uint16)
    ih, gh, lh = inds.cpu().numpy(), gates.cpu().numpy(), logits.cpu().numpy()
    yh = y.float().cpu().numpy()
    experts = {}
    get = lambda e: experts.setdefault(e, synth.expert_tensors(cfg, 0, e))
    lora = synth.lora_tensors(cfg, 0, 0)
    check = range(steps) if name == "cfg1" else sorted(set(range(0, steps, 5)) | {steps - 1})
    for t in range(steps):
        _check_routing(lh[t + 1], ih[t + 1], gh[t + 1], W_np.astype(np.float32), X[t], cfg.K)
        want = orc.next_hidden_state(X[t], yh[t].astype(np.float64), 1e-6)      # from the GPU's own stored y: step-local
        assert _bf16_ulps(X[t + 1], want).max() <= 1, t
        assert (X[t + 1] == want).mean() > 0.98
        if t in check and out_dtype != "bf16":
            ref = orc.moe_ffn(X[t], ih[t], gh[t].astype(np.float64), get, lambda e: lora, cfg.lora_scale, cfg.group)
            _assert_close(yh[t], ref)
    assert len({tuple(r) for r in ih.tolist()}) > min(steps // 2, 60)       # (cfg1 has only 120 possible routings)
    store.close()
