"""Parity for the code paths the configuration-shaped tests do not reach: every instantiation of the
batch-1 layer kernel (H 1024/2048 x I 256/512 x scaled blocks of 32/64 codes), the generic batch-1
kernels that serve shapes the fused kernel rejects, the fp32 variant of the batched head, zero
points that are not integers, and the hand-off ring of chained layer-steps wrapping around.  Each
case is checked against the fp64 oracle on the same seeded inputs, through the C ABI."""
import dataclasses

import numpy as np
import pytest
import torch

import paper_2609_18063_b200 as edg
from oracle import moe_oracle as orc
from paper_2609_18063_b200 import layer_io
from workloads import synth

from _gpu_util import TOL_MAX_ABS, TOL_REL_L2, DeviceLayer, out_tensor, x_dev
from test_gpu_chain import _run
from test_gpu_parity import _assert_close, _check_routing, _make_store

pytestmark = pytest.mark.gpu


def _shape(H, I, group, rank=8, pre="f16", E=16, K=2, seed=11):
    return dataclasses.replace(synth.CONFIGS["cfg1"], name=f"H{H}I{I}g{group}r{rank}", H=H, I=I, group=group, rank=rank,
                               E=E, K=K, n_slots=E, pre_dtype=pre, seed=seed)


def _resident_store(cfg):
    store, d, hosts, slots, tables, cs, keep = _make_store(cfg, n_slots=cfg.E)
    for e0 in range(0, cfg.E, 64):
        edg.stage_experts_to_slots(store, 0, np.arange(e0, min(cfg.E, e0 + 64), dtype=np.int32))
    torch.cuda.synchronize()
    return store, d, keep


def _check_steps(cfg, X, W_np, inds, gates, logits, y, steps):
    experts = {}
    get = lambda e: experts.setdefault(e, synth.expert_tensors(cfg, 0, e))
    lora = synth.lora_tensors(cfg, 0, 0)
    for t in steps:
        ref = orc.moe_ffn(X[t], inds[t], gates[t].astype(np.float64), get, lambda e: lora, cfg.lora_scale, cfg.group)
        _assert_close(y[t], ref)
        _check_routing(logits[t + 1], inds[t + 1], gates[t + 1], W_np.astype(np.float32), X[t], cfg.K)


# ------------------------------------------------------------------ every instantiation of the fused kernel

@pytest.mark.parametrize("H,I,group,pre", [(2048, 512, 32, "f16"), (2048, 256, 64, "f16"), (2048, 256, 32, "f32"),
                                          (1024, 512, 64, "f16"), (1024, 512, 32, "f16"), (1024, 256, 64, "f32"),
                                          (2048, 512, 128, "f16")])
def test_fused_kernel_shapes_chained_and_alone(H, I, group, pre):
    """Small layers (16 experts, top-2, rank 8) of every supported (H, I, block) combination: a chain of
    steps in flight (one cluster walks all four quarters of its experts) and the same steps launched
    alone (four clusters per expert), each step against the oracle."""
    cfg = _shape(H, I, group, pre=pre)
    store, d, keep = _resident_store(cfg)
    W_np = synth.prerouter_weights(cfg)
    W = torch.from_numpy(W_np).cuda()
    steps = 9
    X = synth.hidden_states(cfg, steps + 1, stream=51)
    ws = layer_io.new_workspace(d)
    inds_c, gates_c, logits_c, y_c = _run(cfg, store, d, W, x_dev(X), steps, ws, True)
    inds_u, gates_u, logits_u, y_u = _run(cfg, store, d, W, x_dev(X), steps, ws, False)
    assert np.array_equal(inds_c, inds_u) and np.abs(logits_c - logits_u).max() <= 1e-5
    assert np.abs(y_c - y_u).max() <= 1e-4
    _check_steps(cfg, X, W_np, inds_c, gates_c, logits_c, y_c, range(steps))
    store.close()


# ------------------------------------------------------------------ shapes the fused kernel does not take

@pytest.mark.parametrize("H,I,group,rank,E,K,pre", [(512, 128, 32, 8, 16, 2, "f16"), (512, 128, 32, 8, 16, 2, "f32"),
                                                   (2048, 512, 64, 32, 16, 4, "f16"), (4096, 1024, 128, 16, 8, 2, "f16")])
def test_generic_batch1_kernels_match_the_oracle(H, I, group, rank, E, K, pre):
    """H = 512 / 4096, or rank 32 at the 35B-class shape: the layer-step runs on the generic kernels
    (rank-r projections, gate/up GEMV with SiLU, down GEMV with the reduce, stand-alone head)."""
    cfg = _shape(H, I, group, rank=rank, pre=pre, E=E, K=K)
    store, d, keep = _resident_store(cfg)
    W_np = synth.prerouter_weights(cfg)
    W = torch.from_numpy(W_np).cuda()
    steps = 4
    X = synth.hidden_states(cfg, steps + 1, stream=52)
    ws = layer_io.new_workspace(d)
    inds, gates, logits, y = _run(cfg, store, d, W, x_dev(X), steps, ws, False)
    _check_steps(cfg, X, W_np, inds, gates, logits, y, range(steps))
    store.close()
    # the FFN call alone (slots given directly, no table), with and without the adapter
    L = DeviceLayer(cfg)
    sl = torch.tensor(inds[0], device="cuda")
    g = torch.tensor(gates[0], device="cuda")
    for lora in (L.lora, None):
        yy = out_tensor(L.desc)
        L.ws[:4096].zero_()
        edg.moe_expert_ffn_int4_lora(L.desc, L.pool, None, 1, sl, sl, g, x_dev(X[:1]), lora, yy, L.ws)
        torch.cuda.synchronize()
        ref = orc.moe_ffn(X[0], inds[0], gates[0].astype(np.float64), L.expert, None if lora is None else L.get_lora,
                          cfg.lora_scale, cfg.group)
        _assert_close(yy[0].cpu().numpy(), ref)


def test_batched_head_with_fp32_weights():
    """prerouter_topk_tokens with an fp32 head (the fp32-FMA kernel; the fp16 head takes MMA tiles):
    20 tokens = two blocks of 8 and a ragged block of 4."""
    cfg = synth.CONFIGS["cfg1"]
    d = edg.make_desc(cfg, n_slots=cfg.E)
    assert d.pre_dtype == edg.F32
    T = 20
    W_np = synth.prerouter_weights(cfg)
    S = synth.hidden_states(cfg, T, stream=53)
    inds = torch.full((T, cfg.K), -1, dtype=torch.int32, device="cuda")
    gates = torch.zeros((T, cfg.K), dtype=torch.float32, device="cuda")
    logits = torch.zeros((T, cfg.E), dtype=torch.float32, device="cuda")
    edg.prerouter_topk_tokens(d, torch.from_numpy(W_np).cuda(), x_dev(S), T, inds, gates, logits)
    torch.cuda.synchronize()
    decided = sum(_check_routing(logits[t].cpu().numpy(), inds[t].cpu().numpy(), gates[t].cpu().numpy(), W_np, S[t], cfg.K)
                  for t in range(T))
    assert decided >= T - 2


@pytest.mark.parametrize("H,E,K,T", [(2048, 256, 8, 20), (1024, 128, 4, 13), (1024, 256, 8, 64), (512, 128, 2, 9)])
def test_batched_head_with_fp16_weights_on_mma_tiles(H, E, K, T):
    """prerouter_topk_tokens with an fp16 head (MMA tiles, 16-byte operand loads under a shared k
    permutation): logits of every token against the oracle, ragged last block of tokens, one and two
    row tiles per CTA (E = 128 / 256), K slices of 64, 128 and 256 per warp (H = 512, 1024, 2048)."""
    cfg = dataclasses.replace(synth.CONFIGS["cfg2"], H=H, E=E, K=K, pre_dtype="f16")
    d = edg.make_desc(cfg, n_slots=E)
    assert d.pre_dtype == edg.F16
    W_np = synth.prerouter_weights(cfg)
    S = synth.hidden_states(cfg, T, stream=57)
    inds = torch.full((T, K), -1, dtype=torch.int32, device="cuda")
    gates = torch.zeros((T, K), dtype=torch.float32, device="cuda")
    logits = torch.zeros((T, E), dtype=torch.float32, device="cuda")
    edg.prerouter_topk_tokens(d, torch.from_numpy(W_np).cuda(), x_dev(S), T, inds, gates, logits)
    torch.cuda.synchronize()
    decided = sum(_check_routing(logits[t].cpu().numpy(), inds[t].cpu().numpy(), gates[t].cpu().numpy(),
                                 W_np.astype(np.float32), S[t], K) for t in range(T))
    assert decided >= T - 2


# ------------------------------------------------------------------ zero points that are not integers

class _FractionalZeroLayer(DeviceLayer):
    """A layer whose zero points are multiples of 1/4 in [0, 15.75] (7.5, 3.25, ...): still exact for
    every kernel, but no longer the integers the generator draws."""

    def expert(self, e):
        if e not in self._experts:
            ex = synth.expert_tensors(self.cfg, self.layer, e)
            rng = np.random.default_rng([77, e])
            out = {}
            for proj, (c, s, z) in ex.items():
                frac = rng.integers(0, 4, size=z.shape).astype(np.float32) * 0.25
                out[proj] = (c, s, np.minimum(z.astype(np.float32) + frac, 15.75).astype(np.float16))
            self._experts[e] = out
        return self._experts[e]


@pytest.mark.parametrize("name", ["cfg1", "fused_off"])
def test_fractional_zero_points_on_every_path(name):
    cfg = synth.CONFIGS["cfg1"] if name == "cfg1" else _shape(512, 128, 32)
    L = _FractionalZeroLayer(cfg)
    z = L.expert(3)["gate"][2].astype(np.float64)
    assert (z != np.round(z)).mean() > 0.5 and 7.5 in z and 3.25 in z
    rng = np.random.default_rng(5)
    # batch 1 (the fused kernel for cfg1, the generic kernels for the other shape)
    X = synth.hidden_states(cfg, 3, stream=54)
    for t in range(3):
        inds = np.sort(rng.choice(cfg.E, cfg.K, replace=False)).astype(np.int32)
        gates = rng.dirichlet(np.ones(cfg.K)).astype(np.float32)
        y = out_tensor(L.desc)
        L.ws[:4096].zero_()
        edg.moe_expert_ffn_int4_lora(L.desc, L.pool, None, 1, torch.tensor(inds, device="cuda"), torch.tensor(inds, device="cuda"),
                                     torch.tensor(gates, device="cuda"), x_dev(X[t:t + 1]), L.lora, y, L.ws)
        torch.cuda.synchronize()
        _assert_close(y[0].cpu().numpy(), orc.moe_ffn(X[t], inds, gates, L.expert, L.get_lora, cfg.lora_scale, cfg.group))
    if name != "cfg1":
        return
    # grouped: a few tokens per expert (mma.sync tiles), then many (tensor-memory path)
    for T in (6, 200):
        Xt = synth.hidden_states(cfg, T, stream=55)
        inds_h = np.stack([np.sort(rng.choice(cfg.E, cfg.K, replace=False)) for _ in range(T)]).astype(np.int32)
        gates_h = rng.dirichlet(np.ones(cfg.K), size=T).astype(np.float32)
        ws = layer_io.new_workspace(L.desc, T)
        y = out_tensor(L.desc, T)
        edg.moe_expert_ffn_int4_lora(L.desc, L.pool, None, T, torch.from_numpy(inds_h).cuda(), torch.from_numpy(inds_h).cuda(),
                                     torch.from_numpy(gates_h).cuda(), x_dev(Xt), L.lora, y, ws)
        torch.cuda.synchronize()
        assert edg.workspace_status(ws) == 0
        Y = y.cpu().numpy()
        for t in range(0, T, 1 if T < 10 else 9):
            _assert_close(Y[t], orc.moe_ffn(Xt[t], inds_h[t], gates_h[t].astype(np.float64), L.expert, L.get_lora,
                                            cfg.lora_scale, cfg.group))


# ------------------------------------------------------------------ the hand-off ring wraps around

@pytest.mark.parametrize("name,steps,stride", [("cfg1", 300, 1), ("cfg2", 272, 9)])
def test_chained_steps_wrap_the_hand_off_ring(name, steps, stride):
    """More chained steps than the ring has slots (128), on one workspace, launched without any host
    synchronisation: the slot a step publishes into was reset by the step that consumed it one lap
    earlier, the reduce scratch of a ring slot is reused, the head counter wraps.  Every step (cfg1) or
    a stride plus the steps on both sides of every wrap (cfg2) is checked against the oracle."""
    cfg = synth.CONFIGS[name]
    store, d, keep = _resident_store(cfg)
    W_np = synth.prerouter_weights(cfg)
    W = torch.from_numpy(W_np).cuda()
    X = synth.hidden_states(cfg, steps + 1, stream=56)
    ws = layer_io.new_workspace(d)
    inds, gates, logits, y = _run(cfg, store, d, W, x_dev(X), steps, ws, True)
    check = set(range(0, steps, stride)) | {steps - 1}
    for wrap in range(128, steps, 128):
        check |= {wrap - 2, wrap - 1, wrap, wrap + 1}
    _check_steps(cfg, X, W_np, inds, gates, logits, y, sorted(t for t in check if 0 <= t < steps))
    # a second lap on the same workspace, not chained this time, continues from the ring where it stands
    # (step 0 is routed from another "last prompt" state in the shorter run: compare from step 1)
    inds_u, gates_u, logits_u, y_u = _run(cfg, store, d, W, x_dev(X), 140, ws, False)
    assert np.array_equal(inds_u[1:], inds[1:141]) and np.abs(logits_u[1:] - logits[1:141]).max() <= 1e-5
    assert np.abs(y_u[1:] - y[1:140]).max() <= 1e-4
    store.close()
