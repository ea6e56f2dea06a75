"""Shared set-up for the GPU parity tests: a layer's synthetic tensors on the device."""
import functools

import numpy as np
import torch

import paper_2609_18063_b200 as edg
from paper_2609_18063_b200 import layer_io
from workloads import synth

TOL_MAX_ABS = 2e-2     # parity bar for fp32 / fp16 outputs against the fp64 oracle
TOL_REL_L2 = 1e-3


class DeviceLayer:
    """One layer of a config with every expert resident (slot e holds expert e)."""

    def __init__(self, cfg: synth.MoEConfig, layer: int = 0, out_dtype: str = "f32"):
        self.cfg, self.layer = cfg, layer
        self.desc = edg.make_desc(cfg, out_dtype=out_dtype, n_slots=cfg.E)
        self._experts = {}
        self.host = layer_io.host_layer(self.desc, self.expert)
        self.pool = self.host.cuda()
        self.W_np = synth.prerouter_weights(cfg, layer)
        self.W = torch.from_numpy(self.W_np).cuda()
        self.adapters = [synth.lora_tensors(cfg, layer, a) for a in range(cfg.n_adapters)]
        self.lora, self._keep = layer_io.lora_to_device(self.desc, self.adapters)
        self.ws = layer_io.new_workspace(self.desc, max(cfg.T, 1))

    def expert(self, e: int):
        if e not in self._experts:
            self._experts[e] = synth.expert_tensors(self.cfg, self.layer, e)
        return self._experts[e]

    def get_lora(self, e: int):
        return self.adapters[0] if self.cfg.n_adapters == 1 else self.adapters[e]

    def desc_with(self, **kw):
        d = edg.make_desc(self.cfg, n_slots=self.cfg.E)
        d.out_dtype = self.desc.out_dtype
        for k, v in kw.items():
            setattr(d, k, v)
        return d


@functools.lru_cache(maxsize=None)
def device_layer(name: str, n_adapters: int = 1, layer: int = 0) -> DeviceLayer:
    cfg = synth.CONFIGS[name].with_(n_adapters=n_adapters)
    return DeviceLayer(cfg, layer)


def x_dev(bits: np.ndarray) -> torch.Tensor:
    return layer_io.bits_to_device(bits, torch.bfloat16)


def out_tensor(desc, T=1):
    dt = {edg.F32: torch.float32, edg.F16: torch.float16, edg.BF16: torch.bfloat16}[desc.out_dtype]
    return torch.full((T, desc.H), float("nan"), dtype=dt, device="cuda")
