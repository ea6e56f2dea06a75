"""Host loop of the expert stack: one token through L MoE layers with prediction-driven staging.

Orchestration only -- every arithmetic step runs in the CUDA library.  Per token the loop does what
the paper's decode timeline shows: the routing of every layer was predicted one token earlier (the
head owned by layer l, evaluated on that layer's input at token t, predicts layer (l+1) mod L at
token t+1); it is handed to the host once per token (the single flush), the stager enqueues the
copies of the missing experts on the side stream, and each layer's kernel waits only for its own
layer's copies, so later layers' copies overlap earlier layers' compute.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B
from . import layer_io


class StackDecoder:
    def __init__(self, desc: B.LayerDesc, store: B.Store, W_pre: torch.Tensor, prefetch: bool = True):
        """W_pre: device [L][E][H]; head l predicts the routing of layer (l+1) % L at the next token."""
        self.desc, self.store, self.W_pre, self.prefetch = desc, store, W_pre, prefetch
        self.L = store.n_layers
        K = desc.K
        self.inds = torch.zeros((2, self.L, K), dtype=torch.int32, device="cuda")
        self.gates = torch.zeros((2, self.L, K), dtype=torch.float32, device="cuda")
        self.inds_host = torch.zeros((self.L, K), dtype=torch.int32).pin_memory()
        self.ws = layer_io.new_workspace(desc)
        self.misses = 0

    def prime(self, x_prompt: torch.Tensor) -> None:
        """Routing of token 0 from the last prompt token's layer inputs [L][H] (prefill has no
        prediction; one batched flush over all heads)."""
        L = self.L
        tmp_i = torch.zeros((L, self.desc.K), dtype=torch.int32, device="cuda")
        tmp_g = torch.zeros((L, self.desc.K), dtype=torch.float32, device="cuda")
        B.prerouter_topk(self.desc, self.W_pre, x_prompt, L, tmp_i, tmp_g, None)
        # head l feeds layer (l+1) % L
        self.inds[0] = torch.roll(tmp_i, 1, dims=0)
        self.gates[0] = torch.roll(tmp_g, 1, dims=0)

    def step(self, t: int, X: torch.Tensor, Y: torch.Tensor, logits_out=None) -> None:
        """Token t: X device bf16 [L][H] (layer inputs), Y device [L][H] (layer outputs)."""
        cur, nxt = t % 2, (t + 1) % 2
        stream = torch.cuda.current_stream()
        # one hand-off per token: the predictions made during the previous token
        self.inds_host.copy_(self.inds[cur], non_blocking=True)
        stream.synchronize()
        ih = self.inds_host.numpy()
        if self.prefetch:
            for l in range(self.L):
                self.misses += B.stage_experts_to_slots(self.store, l, ih[l])[1]
        for l in range(self.L):
            if not self.prefetch:
                self.misses += B.stage_experts_to_slots(self.store, l, ih[l])[1]
            ln = (l + 1) % self.L
            B.moe_layer_decode(self.store, l, X[l], self.inds[cur, l], self.gates[cur, l], self.W_pre[l],
                               self.inds[nxt, ln], self.gates[nxt, ln],
                               None if logits_out is None else logits_out[ln], Y[l], self.ws)
