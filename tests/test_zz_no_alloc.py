"""The no-allocation entry point: for callers that cannot call cudaMalloc (a plugin inside another
engine's memory plan, a loop that must not touch the allocator once started), the batch-1 FFN is
also offered with its scratch in a fixed array inside the library.  Its output must equal the
regular entry point's on the same inputs -- on two calls in a row, since the array keeps whatever
the previous call left in it.  This file is collected last on purpose."""
import numpy as np
import pytest
import torch

import paper_2609_18063_b200 as edg
from workloads import synth

from _gpu_util import TOL_MAX_ABS, TOL_REL_L2, device_layer, out_tensor, x_dev

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_the_regular_one_twice():
    from oracle import moe_oracle as orc
    L = device_layer("cfg2")
    cfg, d = L.cfg, L.desc
    rng = np.random.default_rng(42)
    X = synth.hidden_states(cfg, 2, stream=77)
    for call in range(2):
        inds = torch.tensor(np.sort(rng.choice(cfg.E, cfg.K, replace=False)).astype(np.int32), device="cuda")
        gates = torch.tensor(rng.dirichlet(np.ones(cfg.K)).astype(np.float32), device="cuda")
        x = x_dev(X[call:call + 1])
        y_ref, y_new = out_tensor(d), out_tensor(d)
        L.ws[:4096].zero_()
        edg.moe_expert_ffn_int4_lora(d, L.pool, None, 1, inds, inds, gates, x, L.lora, y_ref, L.ws)
        edg.moe_expert_ffn_int4_lora_static(d, L.pool, None, inds, inds, gates, x, L.lora, y_new)
        torch.cuda.synchronize()
        a, b = y_new[0].cpu().numpy(), y_ref[0].cpu().numpy()
        assert np.isfinite(a).all()
        assert orc.max_abs(a, b) <= TOL_MAX_ABS and orc.rel_l2(a, b) <= TOL_REL_L2
        assert np.array_equal(a, b)          # same kernel, same arithmetic: in fact bit-identical
        # ... and against the fp64 oracle, like every other entry point
        ref = orc.moe_ffn(X[call], inds.cpu().numpy(), gates.cpu().numpy().astype(np.float64), L.expert, L.get_lora,
                          cfg.lora_scale, cfg.group)
        assert orc.max_abs(a, ref) <= TOL_MAX_ABS and orc.rel_l2(a, ref) <= TOL_REL_L2
    # a shape whose scratch cannot fit the fixed array, or that the batch-1 kernel does not cover, is rejected
    bad = edg.make_desc(cfg, n_slots=cfg.E, H=4096)
    with pytest.raises(edg.EdgError) as ei:
        edg.moe_expert_ffn_int4_lora_static(bad, L.pool, None, inds, inds, gates, x, L.lora, y_new)
    assert ei.value.code in (-2, -7)
