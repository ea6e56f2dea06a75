"""Seeded synthetic tensors for the streaming-MoE decode step.

Every tensor is a stream keyed by (config seed, layer, expert/adapter, tensor
id), so any single expert record can be regenerated without holding a whole
18 GB layer stack.  Formats:

* activations and LoRA factors: bf16, carried as ``uint16`` bit patterns
  (numpy has no bf16), rounded to nearest-even from float32 draws;
* prerouter weights: float32 or float16;
* expert projections: int4 codes packed two per byte in the canonical
  interchange order (row-major, byte j of a row holds k=2j in its low nibble
  and k=2j+1 in its high nibble), with one fp16 scale and one fp16 zero point
  per group of ``group`` consecutive k.

Value distributions follow the workload description: codes uniform on 0..15,
scales U(0.005, 0.02), zero points uniform integers 0..15, prerouter weights
N(0, 0.02), LoRA A ~ N(0, 0.02), B ~ N(0, 0.01), activations N(0, 1).
Nothing here computes any part of the method.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Tuple

import numpy as np

# tensor ids inside a stream key
_T_X, _T_WPRE, _T_CODES, _T_SCALES, _T_ZEROS, _T_LORA_A, _T_LORA_B, _T_LOGITS, _T_PERM, _T_MLP = range(10)
_PROJ_ID = {"gate": 0, "up": 1, "down": 2}
PROJS = ("gate", "up", "down")


@dataclass(frozen=True)
class MoEConfig:
    """Shape of one MoE layer (and of the run around it)."""

    name: str
    H: int            # hidden size
    I: int            # expert intermediate size
    E: int            # experts per layer
    K: int            # experts routed per token
    group: int        # quantisation group size along the input dimension
    rank: int         # LoRA rank
    n_slots: int      # slots per layer in the HBM pool
    seed: int
    pre_dtype: str = "f16"     # storage type of the prerouter head: "f32" | "f16"
    lora_scale: float = 2.0    # alpha / r
    n_layers: int = 1
    n_adapters: int = 1        # 1: one adapter per layer shared by all experts; E: one per expert
    T: int = 1                 # tokens per step (1 = batch-1 decode)

    def proj_shape(self, proj: str) -> Tuple[int, int]:
        """(out rows N, input dim Kd) of a projection."""
        return (self.I, self.H) if proj in ("gate", "up") else (self.H, self.I)

    @property
    def record_bytes(self) -> int:
        """Bytes of one expert: three int4 matrices plus fp16 (scale, zero) per group."""
        return 3 * self.H * self.I // 2 + 3 * (self.H * self.I // self.group) * 4

    def with_(self, **kw) -> "MoEConfig":
        return replace(self, **kw)


CONFIGS: Dict[str, MoEConfig] = {
    # tiny single layer, batch-1 decode, fp32 head
    "cfg1": MoEConfig("cfg1", H=1024, I=256, E=16, K=2, group=32, rank=8, n_slots=4, seed=0, pre_dtype="f32"),
    # one 35B-class layer, batch-1 decode
    "cfg2": MoEConfig("cfg2", H=2048, I=512, E=256, K=8, group=64, rank=16, n_slots=8, seed=1),
    # 40-layer 35B-class stack, expert part only
    "cfg3": MoEConfig("cfg3", H=2048, I=512, E=256, K=8, group=64, rank=16, n_slots=8, seed=2, n_layers=40),
    # batched decode, 64 concurrent tokens, union slot pool
    "cfg4": MoEConfig("cfg4", H=2048, I=512, E=256, K=8, group=64, rank=16, n_slots=256, seed=3, T=64),
    # prefill, 4096 tokens, Zipf(1.1) expert popularity
    "cfg5": MoEConfig("cfg5", H=2048, I=512, E=256, K=8, group=64, rank=16, n_slots=256, seed=4, T=4096),
}


def _rng(seed: int, *key: int) -> np.random.Generator:
    return np.random.default_rng([int(seed), *[int(k) for k in key]])


# ---------------------------------------------------------------- formats

def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


# ---------------------------------------------------------------- tensors

def hidden_states(cfg: MoEConfig, n: int, layer: int = 0, stream: int = 0) -> np.ndarray:
    """``n`` independent hidden-state vectors ~ N(0,1), bf16 bits, shape [n][H]."""
    g = _rng(cfg.seed, layer, stream, _T_X)
    return f32_to_bf16_bits(g.standard_normal((n, cfg.H), dtype=np.float32))


def hidden_states_ar1(cfg: MoEConfig, n: int, rho: float, layer: int = 0, stream: int = 0) -> np.ndarray:
    """Trace-like hidden states: x[t+1] = rho x[t] + sqrt(1-rho^2) eps, unit variance, bf16 bits.

    Consecutive tokens then agree on part of their routed set, as decode
    traces do; rho is calibrated by the caller against the overlap wanted.
    """
    g = _rng(cfg.seed, layer, stream, _T_X, 1)
    eps = g.standard_normal((n, cfg.H), dtype=np.float32)
    out = np.empty_like(eps)
    out[0] = eps[0]
    c = np.float32(np.sqrt(1.0 - rho * rho))
    for t in range(1, n):
        out[t] = np.float32(rho) * out[t - 1] + c * eps[t]
    return f32_to_bf16_bits(out)


def prerouter_weights(cfg: MoEConfig, layer: int = 0) -> np.ndarray:
    """Linear prerouter head [E][H] ~ N(0, 0.02), float32 or float16 per ``cfg.pre_dtype``."""
    g = _rng(cfg.seed, layer, _T_WPRE)
    w = (g.standard_normal((cfg.E, cfg.H), dtype=np.float32) * np.float32(0.02))
    if cfg.pre_dtype == "f16":
        return w.astype(np.float16)
    if cfg.pre_dtype == "f32":
        return w
    raise ValueError(f"pre_dtype {cfg.pre_dtype!r}")


def mlp_head_weights(cfg: MoEConfig, layer: int = 0, width: int = 512) -> Dict[str, np.ndarray]:
    """The MLP path of a prerouter head (fp16, the paper's export precision): W1 [width][H + 2E] and
    W2 [E][width] ~ N(0, 0.02), biases b1 [width], b2 [E] ~ N(0, 0.01)."""
    g = _rng(cfg.seed, layer, _T_MLP)
    f = cfg.H + 2 * cfg.E
    return {"W1": (g.standard_normal((width, f), dtype=np.float32) * np.float32(0.02)).astype(np.float16),
            "b1": (g.standard_normal(width, dtype=np.float32) * np.float32(0.01)).astype(np.float16),
            "W2": (g.standard_normal((cfg.E, width), dtype=np.float32) * np.float32(0.02)).astype(np.float16),
            "b2": (g.standard_normal(cfg.E, dtype=np.float32) * np.float32(0.01)).astype(np.float16)}


def expert_tensors(cfg: MoEConfig, layer: int, expert: int) -> Dict[str, Tuple[np.ndarray, np.ndarray, np.ndarray]]:
    """Canonical tensors of one expert: proj -> (packed codes u8 [N][Kd/2], scales f16 [N][Kd/g], zeros f16 [N][Kd/g])."""
    out = {}
    for proj in PROJS:
        n, kd = cfg.proj_shape(proj)
        pid = _PROJ_ID[proj]
        codes = _rng(cfg.seed, layer, expert, pid, _T_CODES).integers(0, 256, size=(n, kd // 2), dtype=np.uint8)
        scales = _rng(cfg.seed, layer, expert, pid, _T_SCALES).uniform(0.005, 0.02, size=(n, kd // cfg.group))
        zeros = _rng(cfg.seed, layer, expert, pid, _T_ZEROS).integers(0, 16, size=(n, kd // cfg.group))
        out[proj] = (codes, scales.astype(np.float16), zeros.astype(np.float16))
    return out


def lora_tensors(cfg: MoEConfig, layer: int, adapter: int = 0) -> Dict[str, Tuple[np.ndarray, np.ndarray]]:
    """LoRA factors of one adapter: proj -> (A bf16 bits [r][Kd], B bf16 bits [N][r])."""
    out = {}
    for proj in PROJS:
        n, kd = cfg.proj_shape(proj)
        pid = _PROJ_ID[proj]
        a = _rng(cfg.seed, layer, adapter, pid, _T_LORA_A).standard_normal((cfg.rank, kd), dtype=np.float32) * np.float32(0.02)
        b = _rng(cfg.seed, layer, adapter, pid, _T_LORA_B).standard_normal((n, cfg.rank), dtype=np.float32) * np.float32(0.01)
        out[proj] = (f32_to_bf16_bits(a), f32_to_bf16_bits(b))
    return out


def zipf_router_logits(cfg: MoEConfig, n: int, layer: int = 0, alpha: float = 1.1) -> np.ndarray:
    """Router logits [n][E] float32 whose top-K is a draw of K distinct experts with
    probability proportional to rank^-alpha (Gumbel perturbation of log-popularity
    over a seeded ranking of the experts)."""
    perm = _rng(cfg.seed, layer, _T_PERM).permutation(cfg.E)
    rank = np.empty(cfg.E, dtype=np.float64)
    rank[perm] = np.arange(1, cfg.E + 1)
    g = _rng(cfg.seed, layer, _T_LOGITS)
    gumbel = g.gumbel(size=(n, cfg.E))
    return (-alpha * np.log(rank)[None, :] + gumbel).astype(np.float32)
