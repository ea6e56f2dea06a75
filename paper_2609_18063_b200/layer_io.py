"""Loading helpers: canonical expert tensors -> pinned host store, adapters -> device.

These move bytes only (repacking goes through ``edg_pack_expert``); torch is used for pinned
and device memory.
"""
from __future__ import annotations

from typing import Callable, Dict, Sequence

import numpy as np
import torch

from . import binding as B


def host_layer(desc: B.LayerDesc, get_expert: Callable[[int], Dict[str, tuple]], pin: bool = True) -> torch.Tensor:
    """All E expert records of one layer as a uint8 tensor [E][record bytes] in (pinned) host memory."""
    R = B.record_bytes(desc)
    buf = torch.empty((desc.E, R), dtype=torch.uint8, pin_memory=pin)
    view = buf.numpy()
    for e in range(desc.E):
        B.pack_expert(desc, get_expert(e), view[e])
    return buf


def bits_to_device(bits: np.ndarray, dtype: torch.dtype, device="cuda") -> torch.Tensor:
    """16-bit patterns (uint16) -> device tensor of bf16/fp16 with the same bits."""
    t = torch.from_numpy(np.ascontiguousarray(bits, dtype=np.uint16).view(np.int16).copy())
    return t.to(device).view(dtype)


def lora_to_device(desc: B.LayerDesc, adapters: Sequence[Dict[str, tuple]], device="cuda"):
    """adapters[a][proj] = (A bits [r][Kd], B bits [N][r]) -> (Lora struct, tensors to keep alive).
    len(adapters) must equal desc.n_adapters."""
    if len(adapters) != desc.n_adapters:
        raise ValueError("adapter count does not match the descriptor")
    keep = {}
    for proj in ("gate", "up", "down"):
        keep["A_" + proj] = bits_to_device(np.stack([a[proj][0] for a in adapters]), torch.bfloat16, device)
        keep["B_" + proj] = bits_to_device(np.stack([a[proj][1] for a in adapters]), torch.bfloat16, device)
    lora = B.make_lora(keep["A_gate"], keep["B_gate"], keep["A_up"], keep["B_up"], keep["A_down"], keep["B_down"])
    return lora, keep


def new_workspace(desc: B.LayerDesc, T: int = 1, device="cuda") -> torch.Tensor:
    """Zeroed device workspace for the FFN calls (the control block must start at zero)."""
    return torch.zeros(B.ffn_workspace_bytes(desc, T), dtype=torch.uint8, device=device)
