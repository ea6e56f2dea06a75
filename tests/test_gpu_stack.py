"""Config-3-shaped decode through the expert stack (small: 3 layers, 5 tokens): prediction-driven
staging across layers, every layer-step checked against the oracle on the same inputs."""
import numpy as np
import pytest
import torch

import paper_2609_18063_b200 as edg
from oracle import moe_oracle as orc
from paper_2609_18063_b200 import layer_io
from paper_2609_18063_b200.decoder import StackDecoder
from workloads import synth

from _gpu_util import TOL_MAX_ABS, TOL_REL_L2

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n_slots,prefetch", [(8, True), (16, True), (8, False)])
def test_stack_decode_matches_oracle(n_slots, prefetch):
    cfg = synth.CONFIGS["cfg3"].with_(n_layers=3)
    L, T, K, E = cfg.n_layers, 5, cfg.K, cfg.E
    d = edg.make_desc(cfg, n_slots=n_slots)
    R = edg.record_bytes(d)
    experts = {}
    get = lambda l, e: experts.setdefault((l, e), synth.expert_tensors(cfg, l, e))
    hosts = [layer_io.host_layer(d, lambda e, l=l: get(l, e)) for l in range(L)]
    loras_np = [synth.lora_tensors(cfg, l, 0) for l in range(L)]
    loras, keep = zip(*[layer_io.lora_to_device(d, [ln]) for ln in loras_np])
    slots = torch.zeros((L, n_slots, R), dtype=torch.uint8, device="cuda")
    tables = torch.zeros((L, E), dtype=torch.int32, device="cuda")
    store = edg.Store(d, hosts, slots, tables, list(loras), torch.cuda.Stream())
    W_np = np.stack([synth.prerouter_weights(cfg, l) for l in range(L)])
    W = torch.from_numpy(W_np).cuda()
    X_np = np.stack([synth.hidden_states(cfg, T + 1, layer=l, stream=21) for l in range(L)])   # [L][T+1][H]
    X = layer_io.bits_to_device(X_np, torch.bfloat16)
    dec = StackDecoder(d, store, W, prefetch=prefetch)
    dec.prime(X[:, T].contiguous())
    Y = torch.zeros((T, L, cfg.H), dtype=torch.float32, device="cuda")
    logits = torch.zeros((T, L, E), dtype=torch.float32, device="cuda")
    allocs = [orc.SlotAllocator(E, n_slots) for _ in range(L)]
    routing = []
    for t in range(T):
        dec.step(t, X[:, t].contiguous(), Y[t], logits[t])
        torch.cuda.synchronize()
        routing.append((dec.inds[t % 2].cpu().numpy().copy(), dec.gates[t % 2].cpu().numpy().copy()))
    assert edg.workspace_status(dec.ws) == 0
    Yh, lg = Y.cpu().numpy(), logits.cpu().numpy()
    want_miss = 0
    for t in range(T):
        inds_t, gates_t = routing[t]
        for l in range(L):
            want_miss += len(allocs[l].stage(inds_t[l].tolist())[1])
            ref = orc.moe_ffn(X_np[l, t], inds_t[l], gates_t[l].astype(np.float64), lambda e, l=l: get(l, e),
                              lambda e, l=l: loras_np[l], cfg.lora_scale, cfg.group)
            assert orc.max_abs(Yh[t, l], ref) <= TOL_MAX_ABS and orc.rel_l2(Yh[t, l], ref) <= TOL_REL_L2
            # the head owned by layer l predicted layer (l+1) % L of the next token
            ln = (l + 1) % L
            l_ref = orc.prerouter_logits(W_np[l], X_np[l, t])
            assert np.abs(lg[t, ln] - l_ref).max() <= 1e-5
            if t + 1 < T:
                i_ref, _ = orc.softmax_topk(l_ref, K)
                srt = np.sort(l_ref)[::-1]
                if srt[K - 1] - srt[K] > 1e-4:
                    assert routing[t + 1][0][ln].tolist() == i_ref.tolist()
    assert dec.misses == want_miss == store.stats()["misses"]
    for l in range(L):
        eos, soe = store.snapshot(l)
        assert eos.tolist() == allocs[l].expert_of_slot and soe.tolist() == allocs[l].slot_of_expert
    store.close()
