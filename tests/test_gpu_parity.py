"""GPU parity: every C-ABI call against the fp64 CPU oracle on the same seeded inputs.

Bars: expert indices, slot maps and top-k sets bit-exact; fp32 / fp16 outputs within max abs
error 2e-2 and relative L2 1e-3 of the oracle; a bf16 store within one bf16 ulp of the oracle's
value rounded to bf16 (bf16 itself cannot hold the values to 1e-3).  Where fp32 logits decide an
integer (the top-k), the kernel's choice must be the exact top-k of its own logits everywhere and
equal the oracle's wherever the fp64 gap at the selection boundary exceeds 1e-4.
"""
import numpy as np
import pytest
import torch

import paper_2609_18063_b200 as edg
from oracle import moe_oracle as orc
from paper_2609_18063_b200 import layer_io
from workloads import synth

from _gpu_util import TOL_MAX_ABS, TOL_REL_L2, DeviceLayer, device_layer, out_tensor, x_dev

pytestmark = pytest.mark.gpu


def _assert_close(y_gpu, y_ref):
    assert np.isfinite(y_gpu).all()
    assert orc.max_abs(y_gpu, y_ref) <= TOL_MAX_ABS, orc.max_abs(y_gpu, y_ref)
    assert orc.rel_l2(y_gpu, y_ref) <= TOL_REL_L2, orc.rel_l2(y_gpu, y_ref)


def _topk_of_own_logits(l32, K):
    order = sorted(range(len(l32)), key=lambda i: (-float(l32[i]), i))
    return sorted(order[:K])


def _check_routing(l_gpu, inds_gpu, gates_gpu, W_np, s_bits, K):
    l_ref = orc.prerouter_logits(W_np, s_bits)
    assert np.abs(l_gpu.astype(np.float64) - l_ref).max() <= 1e-5                       # (A)
    assert inds_gpu.tolist() == _topk_of_own_logits(l_gpu, K)                           # (B)
    sel = l_gpu[inds_gpu].astype(np.float64)
    w = np.exp(sel - sel.max()); w /= w.sum()
    assert np.abs(gates_gpu - w).max() <= 2e-6 and abs(float(gates_gpu.sum()) - 1.0) <= 1e-6
    inds_ref, gates_ref = orc.softmax_topk(l_ref, K)
    srt = np.sort(l_ref)[::-1]
    gap = srt[K - 1] - srt[K] if K < len(l_ref) else np.inf
    if gap > 1e-4:                                                                      # (C)
        assert inds_gpu.tolist() == inds_ref.tolist()
        assert np.abs(gates_gpu - gates_ref).max() <= 1e-5
        return True
    return False


# ------------------------------------------------------------------ a1 + a2

@pytest.mark.parametrize("name", ["cfg1", "cfg2"])
def test_prerouter_topk_single_and_batched(name):
    L = device_layer(name)
    cfg, d = L.cfg, L.desc
    n = 48
    S_bits = synth.hidden_states(cfg, n, stream=7)
    s = x_dev(S_bits)
    inds = torch.full((n, cfg.K), -1, dtype=torch.int32, device="cuda")
    gates = torch.zeros((n, cfg.K), dtype=torch.float32, device="cuda")
    logits = torch.zeros((n, cfg.E), dtype=torch.float32, device="cuda")
    # one head applied to one state at a time
    for t in range(n):
        edg.prerouter_topk(d, L.W, s[t], 1, inds[t], gates[t], logits[t])
    torch.cuda.synchronize()
    decided = sum(_check_routing(logits[t].cpu().numpy(), inds[t].cpu().numpy(), gates[t].cpu().numpy(),
                                 L.W_np, S_bits[t], cfg.K) for t in range(n))
    assert decided >= n - 2
    # the single flush: several (head, state) pairs in one launch
    heads = 5
    Ws = [synth.prerouter_weights(cfg, layer) for layer in range(heads)]
    Wd = torch.from_numpy(np.stack(Ws)).cuda()
    i2 = torch.full((heads, cfg.K), -1, dtype=torch.int32, device="cuda")
    g2 = torch.zeros((heads, cfg.K), dtype=torch.float32, device="cuda")
    l2 = torch.zeros((heads, cfg.E), dtype=torch.float32, device="cuda")
    edg.prerouter_topk(d, Wd, s[:heads].contiguous(), heads, i2, g2, l2)
    torch.cuda.synchronize()
    for h in range(heads):
        _check_routing(l2[h].cpu().numpy(), i2[h].cpu().numpy(), g2[h].cpu().numpy(), Ws[h], S_bits[h], cfg.K)
    # logits are optional
    i3 = torch.full((cfg.K,), -1, dtype=torch.int32, device="cuda")
    g3 = torch.zeros((cfg.K,), dtype=torch.float32, device="cuda")
    edg.prerouter_topk(d, L.W, s[0], 1, i3, g3, None)
    torch.cuda.synchronize()
    assert torch.equal(i3, inds[0]) and torch.equal(g3, gates[0])


@pytest.mark.parametrize("E,K", [(256, 8), (16, 2), (16, 16), (64, 1), (1000, 32)])
def test_softmax_topk_rows_with_ties(E, K):
    d = edg.make_desc(synth.CONFIGS["cfg2"], E=E, K=K, n_slots=E)
    rng = np.random.default_rng(E * 100 + K)
    T = 67
    logits = rng.standard_normal((T, E)).astype(np.float32)
    logits[1::2] = np.round(logits[1::2] * 2) / 2          # many exact ties on every other row
    logits[3] = 0.0                                        # all equal
    lg = torch.from_numpy(logits).cuda()
    inds = torch.full((T, K), -1, dtype=torch.int32, device="cuda")
    gates = torch.zeros((T, K), dtype=torch.float32, device="cuda")
    edg.softmax_topk_rows(d, lg, T, inds, gates)
    torch.cuda.synchronize()
    inds, gates = inds.cpu().numpy(), gates.cpu().numpy()
    for t in range(T):
        i_ref, w_ref = orc.softmax_topk(logits[t], K)      # fp32 logits are exact in fp64: same decision
        assert inds[t].tolist() == i_ref.tolist()
        assert np.abs(gates[t] - w_ref).max() <= 2e-6
    assert inds[3].tolist() == list(range(K))


# ------------------------------------------------------------------ a4 - a6

def _run_ffn(L, d, x_bits, inds, gates, lora, T=1, use_table=False, experts="same"):
    y = out_tensor(d, T)
    slots = torch.tensor(np.asarray(inds, dtype=np.int32).reshape(T, d.K), device="cuda")
    g = torch.tensor(np.asarray(gates, dtype=np.float32).reshape(T, d.K), device="cuda")
    table = torch.arange(d.E, dtype=torch.int32, device="cuda") if use_table else None
    ex = slots if experts == "same" else experts
    L.ws[:4096].zero_()
    edg.moe_expert_ffn_int4_lora(d, L.pool, table, T, slots, ex, g, x_dev(x_bits), lora, y, L.ws)
    torch.cuda.synchronize()
    return y


def _oracle_ffn(L, x_bits, inds, gates, with_lora=True):
    cfg = L.cfg
    return orc.moe_ffn(x_bits, inds, gates, L.expert, L.get_lora if with_lora else None, cfg.lora_scale, cfg.group)


@pytest.mark.parametrize("n_adapters", [1, 16])
def test_ffn_cfg1_every_step(n_adapters):
    L = device_layer("cfg1", n_adapters)
    cfg = L.cfg
    X = synth.hidden_states(cfg, 24, stream=3)
    for t in range(24):
        l = orc.prerouter_logits(L.W_np, X[t])
        inds, gates = orc.softmax_topk(l, cfg.K)
        y = _run_ffn(L, L.desc, X[t:t + 1], inds, gates, L.lora, use_table=bool(t % 2))
        assert edg.workspace_status(L.ws) == 0
        _assert_close(y[0].cpu().numpy(), _oracle_ffn(L, X[t], inds, gates))


def test_ffn_cfg2_shape_and_gate_order():
    L = device_layer("cfg2")
    cfg = L.cfg
    X = synth.hidden_states(cfg, 3, stream=3)
    rng = np.random.default_rng(0)
    for t in range(3):
        inds = np.sort(rng.choice(cfg.E, cfg.K, replace=False)).astype(np.int32)
        gates = rng.dirichlet(np.ones(cfg.K)).astype(np.float32)
        y = _run_ffn(L, L.desc, X[t:t + 1], inds, gates, L.lora)
        ref = _oracle_ffn(L, X[t], inds, gates)
        _assert_close(y[0].cpu().numpy(), ref)
        assert 3.0 < np.std(ref) < 12.0
        # unsorted slot order is honoured too (the reduce follows the order given)
        perm = rng.permutation(cfg.K)
        y2 = _run_ffn(L, L.desc, X[t:t + 1], inds[perm], gates[perm], L.lora)
        _assert_close(y2[0].cpu().numpy(), ref)


def test_ffn_without_lora_and_lora_linearity():
    L = device_layer("cfg1")
    cfg = L.cfg
    x = synth.hidden_states(cfg, 1, stream=5)
    inds, gates = [3, 9], [0.25, 0.75]
    base = _run_ffn(L, L.desc, x, inds, gates, None)[0].cpu().numpy()
    _assert_close(base, _oracle_ffn(L, x[0], inds, gates, with_lora=False))
    d0 = L.desc_with(rank=0)
    assert np.array_equal(_run_ffn(L, d0, x, inds, gates, L.lora)[0].cpu().numpy(), base)
    # B = 0 reproduces the base bit for bit
    zero_b = [{p: (a[p][0], np.zeros_like(a[p][1])) for p in a} for a in L.adapters]
    lz, keep = layer_io.lora_to_device(L.desc, zero_b)
    assert np.array_equal(_run_ffn(L, L.desc, x, inds, gates, lz)[0].cpu().numpy(), base)
    # with the adapter on the delta is far above the parity bar, so a dropped delta cannot pass
    full = _run_ffn(L, L.desc, x, inds, gates, L.lora)[0].cpu().numpy()
    assert orc.rel_l2(base, full) > 5 * TOL_REL_L2


@pytest.mark.parametrize("out_dtype", ["f16", "bf16"])
def test_ffn_output_dtypes(out_dtype):
    L = device_layer("cfg1")
    cfg = L.cfg
    d = L.desc_with(out_dtype={"f16": edg.F16, "bf16": edg.BF16}[out_dtype])
    x = synth.hidden_states(cfg, 1, stream=6)
    inds, gates = [1, 14], [0.6, 0.4]
    ref = _oracle_ffn(L, x[0], inds, gates)
    y = _run_ffn(L, d, x, inds, gates, L.lora)[0]
    if out_dtype == "f16":
        _assert_close(y.float().cpu().numpy(), ref)
    else:
        # compared with the oracle rounded to bf16: the stored value is that rounding, or its
        # neighbour where the fp32 result sits next to a rounding boundary
        got_bits = y.view(torch.int16).cpu().numpy().view(np.uint16)
        want_bits = orc.f64_to_bf16_bits(ref)
        assert (got_bits == want_bits).mean() >= 0.98
        got = orc.bf16_to_f64(got_bits)
        assert (np.abs(got - ref) <= np.abs(ref) * 2.0 ** -8 + 1e-4).all()


@pytest.mark.parametrize("name,T", [("cfg1", 5), ("cfg2", 3)])
def test_ffn_token_batched_equals_token_by_token(name, T):
    L = device_layer(name)
    cfg = L.cfg
    X = synth.hidden_states(cfg, T, stream=9)
    rng = np.random.default_rng(T)
    inds = np.stack([np.sort(rng.choice(cfg.E, cfg.K, replace=False)) for _ in range(T)]).astype(np.int32)
    gates = rng.dirichlet(np.ones(cfg.K), size=T).astype(np.float32)
    if L.ws.numel() < edg.ffn_workspace_bytes(L.desc, T):
        L.ws = layer_io.new_workspace(L.desc, T)
    Y = _run_ffn(L, L.desc, X, inds, gates, L.lora, T=T).cpu().numpy()
    ref = orc.moe_ffn_tokens(X, inds, gates, L.expert, L.get_lora, cfg.lora_scale, cfg.group)
    _assert_close(Y, ref)


def test_ffn_out_of_range_index_raises_status_without_fault():
    L = device_layer("cfg1")
    cfg = L.cfg
    x = synth.hidden_states(cfg, 1, stream=10)
    y = _run_ffn(L, L.desc, x, [2, cfg.E], [0.5, 0.5], L.lora)       # slot == n_slots: skipped
    assert edg.workspace_status(L.ws) == -4
    ref = 0.5 * orc.expert_ffn(orc.bf16_to_f64(x[0]), L.expert(2), L.get_lora(2), cfg.lora_scale, cfg.group)
    y2 = _run_ffn(L, L.desc, x, [2, 5], [0.5, 0.0], L.lora)
    assert edg.workspace_status(L.ws) == 0
    _assert_close(y2[0].cpu().numpy(), ref)
    # host-side argument checks
    with pytest.raises(edg.EdgError) as ei:
        edg.moe_expert_ffn_int4_lora(L.desc, L.pool, None, 1, torch.zeros(2, dtype=torch.int32, device="cuda"), None,
                                     torch.zeros(2, device="cuda"), x_dev(x), L.lora, out_tensor(L.desc), L.ws, 128)
    assert ei.value.code == -7


# ------------------------------------------------------------------ a3

def _make_store(cfg, n_layers=1, n_slots=None, with_lora=True):
    S = cfg.n_slots if n_slots is None else n_slots
    d = edg.make_desc(cfg, n_slots=S)
    hosts, loras, keep = [], [], []
    for layer in range(n_layers):
        hosts.append(layer_io.host_layer(d, lambda e, layer=layer: synth.expert_tensors(cfg, layer, e)))
        lo, k = layer_io.lora_to_device(d, [synth.lora_tensors(cfg, layer, a) for a in range(cfg.n_adapters)])
        loras.append(lo); keep.append(k)
    R = edg.record_bytes(d)
    slots = torch.zeros((n_layers, S, R), dtype=torch.uint8, device="cuda")
    tables = torch.zeros((n_layers, cfg.E), dtype=torch.int32, device="cuda")
    copy_stream = torch.cuda.Stream()
    store = edg.Store(d, hosts, slots, tables, loras if with_lora else None, copy_stream)
    return store, d, hosts, slots, tables, copy_stream, keep


def test_stage_experts_matches_the_oracle_allocator_and_copies_only_misses():
    cfg = synth.CONFIGS["cfg1"]
    store, d, hosts, slots, tables, cs, _ = _make_store(cfg, n_layers=2)
    allocs = [orc.SlotAllocator(cfg.E, cfg.n_slots) for _ in range(2)]
    rng = np.random.default_rng(5)
    misses = 0
    assert (tables.cpu().numpy() == -1).all()
    for step in range(40):
        layer = step % 2
        P = np.sort(rng.choice(cfg.E, cfg.K, replace=False)).astype(np.int32)
        if step % 5 == 4:
            P = prev[layer]                                   # a repeated set: all hits
        got_slots, n_miss = edg.stage_experts_to_slots(store, layer, P)
        want_slots, copies = allocs[layer].stage(P.tolist())
        assert got_slots.tolist() == want_slots and n_miss == len(copies)
        misses += n_miss
        eos, soe = store.snapshot(layer)
        assert eos.tolist() == allocs[layer].expert_of_slot and soe.tolist() == allocs[layer].slot_of_expert
        cs.synchronize()
        # slot bytes == host record bytes for every resident expert; device table == host table
        pool = slots[layer].cpu()
        for s_, e_ in enumerate(eos.tolist()):
            if e_ >= 0:
                assert torch.equal(pool[s_], hosts[layer][e_])
        assert tables[layer].cpu().numpy().tolist() == soe.tolist()
        prev = locals().get("prev", {}); prev[layer] = P
    st = store.stats()
    assert st["misses"] == misses and st["hits"] == 40 * cfg.K - misses
    assert st["bytes_copied"] == misses * cfg.record_bytes and st["stage_calls"] == 40
    with pytest.raises(edg.EdgError) as ei:
        edg.stage_experts_to_slots(store, 0, np.arange(cfg.n_slots + 1, dtype=np.int32))
    assert ei.value.code == -3
    with pytest.raises(edg.EdgError) as ei:
        edg.stage_experts_to_slots(store, 0, np.array([1, 1], dtype=np.int32))
    assert ei.value.code == -4
    with pytest.raises(edg.EdgError) as ei:
        edg.stage_experts_to_slots(store, 2, np.array([1, 2], dtype=np.int32))
    assert ei.value.code == -4
    eos2, _ = store.snapshot(0)
    assert eos2.tolist() == allocs[0].expert_of_slot          # failed calls changed nothing
    store.close()


# ------------------------------------------------------------------ the whole layer-step

@pytest.mark.parametrize("name,n_slots,steps", [("cfg1", 4, 64), ("cfg2", 8, 6), ("cfg2", 16, 6)])
def test_moe_layer_decode_chain(name, n_slots, steps):
    """Decode steps through the store: the routing produced by step t is staged and consumed by
    step t+1.  Each step is checked against the oracle on the same inputs (step-local)."""
    cfg = synth.CONFIGS[name]
    store, d, hosts, slots, tables, cs, _ = _make_store(cfg, n_slots=n_slots)
    W_np = synth.prerouter_weights(cfg)
    W = torch.from_numpy(W_np).cuda()
    X = synth.hidden_states(cfg, steps + 1, stream=11)
    xd = x_dev(X)
    ws = layer_io.new_workspace(d)
    experts = {}
    get = lambda e: experts.setdefault(e, synth.expert_tensors(cfg, 0, e))
    lora = synth.lora_tensors(cfg, 0, 0)
    alloc = orc.SlotAllocator(cfg.E, n_slots)
    # routing of step 0 comes from a "last prompt token" state, staged synchronously
    inds = torch.zeros((steps + 2, cfg.K), dtype=torch.int32, device="cuda")
    gates = torch.zeros((steps + 2, cfg.K), dtype=torch.float32, device="cuda")
    logits = torch.zeros((steps + 2, cfg.E), dtype=torch.float32, device="cuda")
    edg.prerouter_topk(d, W, xd[steps], 1, inds[0], gates[0], logits[0])
    y = out_tensor(d, steps)
    for t in range(steps):
        torch.cuda.synchronize()
        P = inds[t].cpu().numpy()
        got_slots, n_miss = edg.stage_experts_to_slots(store, 0, P)
        want_slots, copies = alloc.stage(P.tolist())
        assert got_slots.tolist() == want_slots and n_miss == len(copies)
        edg.moe_layer_decode(store, 0, xd[t], inds[t], gates[t], W, inds[t + 1], gates[t + 1], logits[t + 1], y[t], ws)
    torch.cuda.synchronize()
    assert edg.workspace_status(ws) == 0
    inds_h, gates_h, logits_h, y_h = inds.cpu().numpy(), gates.cpu().numpy(), logits.cpu().numpy(), y.cpu().numpy()
    for t in range(steps):
        ref = orc.moe_ffn(X[t], inds_h[t], gates_h[t].astype(np.float64), get, lambda e: lora, cfg.lora_scale, cfg.group)
        _assert_close(y_h[t], ref)
        _check_routing(logits_h[t + 1], inds_h[t + 1], gates_h[t + 1], W_np, X[t], cfg.K)
    assert store.stats()["misses"] > 0
    store.close()
