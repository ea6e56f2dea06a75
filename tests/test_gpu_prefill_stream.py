"""The whole-layer executor path on the GPU (Sec. 3.1, path 4): a model of several layers served for
prefill from a store of TWO pool layers.  Layer l+1 is loaded in one copy while layer l's grouped
FFN runs; each layer's output is checked against the oracle on sampled tokens."""
import numpy as np
import pytest
import torch

import paper_2609_18063_b200 as edg
from oracle import moe_oracle as orc
from paper_2609_18063_b200 import layer_io
from workloads import synth

from _gpu_util import TOL_MAX_ABS, TOL_REL_L2, x_dev

pytestmark = pytest.mark.gpu


def test_whole_layer_prefill_double_buffer_matches_oracle():
    cfg = synth.CONFIGS["cfg1"]
    depth, T, K, E = 5, 150, cfg.K, cfg.E
    d = edg.make_desc(cfg, n_slots=E)
    R = edg.record_bytes(d)
    experts = {}
    get = lambda l, e: experts.setdefault((l, e), synth.expert_tensors(cfg, l, e))
    hosts = [layer_io.host_layer(d, lambda e, l=l: get(l, e)) for l in range(depth)]
    loras_np = [synth.lora_tensors(cfg, l, 0) for l in range(depth)]
    loras = [layer_io.lora_to_device(d, [ln]) for ln in loras_np]
    pool = torch.zeros((2, E, R), dtype=torch.uint8, device="cuda")
    tables = torch.full((2, E), -7, dtype=torch.int32, device="cuda")
    store = edg.Store(d, hosts[:2], pool, tables, None, torch.cuda.Stream())
    ws = layer_io.new_workspace(d, T)
    rng = np.random.default_rng(9)
    X = [synth.hidden_states(cfg, T, layer=l, stream=91) for l in range(depth)]
    inds_h = [np.stack([np.sort(rng.choice(E, K, replace=False)) for _ in range(T)]).astype(np.int32) for _ in range(depth)]
    gates_h = [rng.dirichlet(np.ones(K), size=T).astype(np.float32) for _ in range(depth)]
    Y = torch.zeros((depth, T, cfg.H), dtype=torch.float32, device="cuda")
    st = torch.cuda.current_stream()
    store.load_whole_layer(0, hosts[0])
    for l in range(depth):
        if l + 1 < depth:
            store.load_whole_layer((l + 1) % 2, hosts[l + 1])          # overlaps this layer's compute
        p = l % 2
        store.wait_staged(p, st)
        edg.moe_expert_ffn_int4_lora(d, pool[p], tables[p], T, torch.from_numpy(inds_h[l]).cuda(), None,
                                     torch.from_numpy(gates_h[l]).cuda(), x_dev(X[l]), loras[l][0], Y[l], ws)
        store.mark_computed(p, st)
    torch.cuda.synchronize()
    assert edg.workspace_status(ws) == 0
    Yh = Y.cpu().numpy()
    for l in range(depth):
        for t in (0, 37, T - 1):
            ref = orc.moe_ffn(X[l][t], inds_h[l][t], gates_h[l][t].astype(np.float64), lambda e, l=l: get(l, e),
                              lambda e, l=l: loras_np[l], cfg.lora_scale, cfg.group)
            assert orc.max_abs(Yh[l, t], ref) <= TOL_MAX_ABS and orc.rel_l2(Yh[l, t], ref) <= TOL_REL_L2, (l, t)
    assert tables.cpu().numpy().tolist() == [list(range(E))] * 2
    assert store.stats()["bytes_copied"] == depth * E * R
    store.close()
