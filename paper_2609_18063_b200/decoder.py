"""The expert stack: one token through L MoE layers with prediction-driven staging.

A thin owner of the buffers around ``edg_stack_decode_token`` -- the per-token host loop itself (wait
for the mirrored routing, stage, enqueue the L layer-steps) runs inside the C library.  Per token
it does what the paper's decode timeline shows: the routing of every layer was predicted one token
earlier (the head owned by layer l, evaluated on that layer's input at token t, predicts layer
(l+1) mod L at token t+1); the kernels mirror it into pinned host memory, so the single hand-off of
a token needs neither a device-to-host copy nor a stream synchronisation; the stager enqueues the
copies of the missing experts on the side stream, and each layer's kernel waits only for its own
layer's copies, so later layers' copies overlap earlier layers' compute.
"""
from __future__ import annotations

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
        # host mirrors of the two routing buffers, written by the kernels themselves (-1 = not yet)
        self.mirror = torch.full((2, self.L, K), -1, dtype=torch.int32).pin_memory()
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
        self.mirror[0].copy_(self.inds[0])
        torch.cuda.current_stream().synchronize()

    def step(self, t: int, X: torch.Tensor, Y: torch.Tensor, logits_out=None) -> None:
        """Token t: X device bf16 [L][H] (layer inputs), Y device [L][H] (layer outputs)."""
        cur, nxt = t % 2, (t + 1) % 2
        self.misses += B.stack_decode_token(self.store, X, self.inds[cur], self.gates[cur], self.W_pre,
                                            self.inds[nxt], self.gates[nxt], logits_out, self.mirror[cur],
                                            self.mirror[nxt], Y, self.ws, prefetch=self.prefetch)
