"""CPU oracle for the streaming-MoE per-layer decode step.  TEST INFRASTRUCTURE.

A plain, slow, fp64 restatement of what the step computes, written from the
paper's definitions.  It shares no code with the CUDA library and must never
be imported by it; only the tests, the smoke check and the benchmark's CPU
baseline call it.  Inputs are stored bit patterns (bf16 as uint16, fp16,
packed int4 bytes) which are widened exactly to float64; every sum is a plain
fp64 sum in index order (numpy dot products serve as the library primitive
for the inner products).

Passages followed (section names of the paper):
  * Appendix A "Routing Math", softmax-topk and sigmoid-group blocks;
  * Sec. 3.2 "The Prerouter: Prediction Is the Routing" (linear residual path
    of the head; the prediction is consumed as the routing);
  * Sec. 3.1 "SSD Streaming Expert Layers": the staged executor path (slot
    table + take, sticky slots) and the math contract
    down(silu(gate(x)) * up(x));
  * Sec. 3.3 "Recovery LoRA: Unmerged by Design" and the Fig. 1 caption:
    y = W_int4(x) + (alpha/r) B A x as a parallel delta.

Readings taken where the paper is silent (each is listed in the design notes
of the repository): w = scale * (q - zero) with groups along the input
dimension; nibble order low-then-high; the K routed experts are reported in
ascending expert index; exact ties go to the lower index; the slot victim is
the least recently used slot that the current step does not need.

Parity pins: every function here is pinned by tests that run without a GPU
(closed forms, brute force on tiny inputs, invariants, the paper's printed
byte counts).  No function is "parity unpinned".
"""
from __future__ import annotations

import math
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np

PROJS = ("gate", "up", "down")


# ------------------------------------------------------------------ formats

def bf16_to_f64(bits) -> np.ndarray:
    """Exact value of bf16 bit patterns (uint16): bf16 is the top half of an IEEE float32."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16
    return b.view(np.float32).astype(np.float64)


def f64_to_bf16_bits(v) -> np.ndarray:
    """Nearest-even rounding of float64 values to bf16 bit patterns (used to check a bf16 store)."""
    v = np.asarray(v, dtype=np.float64)
    a = np.abs(v)
    # Going through float32 would round twice, so pick the nearest of the three bf16
    # neighbours of the float32 image directly in fp64 (ties to the even bit pattern).
    t = (a.astype(np.float32).view(np.uint32) >> 16).astype(np.int64)
    best = None
    for c in (t - 1, t, t + 1):
        c = np.clip(c, 0, 0x7F80)
        val = (c.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        err = np.abs(val - a)
        if best is None:
            best, best_err = c, err
        else:
            take = (err < best_err) | ((err == best_err) & (c % 2 == 0) & (best % 2 == 1))
            best = np.where(take, c, best)
            best_err = np.where(take, err, best_err)
    sign = (np.signbit(v).astype(np.int64)) << 15
    return (best | sign).astype(np.uint16)


def unpack_codes(packed) -> np.ndarray:
    """Canonical int4 unpacking: byte j of a row holds code k=2j (low nibble) and k=2j+1 (high nibble)."""
    p = np.asarray(packed, dtype=np.uint8)
    out = np.empty(p.shape[:-1] + (p.shape[-1] * 2,), dtype=np.uint8)
    out[..., 0::2] = p & 0x0F
    out[..., 1::2] = p >> 4
    return out


def pack_codes(codes) -> np.ndarray:
    """Inverse of :func:`unpack_codes` for codes in 0..15."""
    c = np.asarray(codes, dtype=np.uint8)
    if c.shape[-1] % 2 or (c > 15).any():
        raise ValueError("codes must be 0..15 with an even innermost length")
    return (c[..., 0::2] | (c[..., 1::2] << 4)).astype(np.uint8)


def record_bytes(H: int, I: int, group: int) -> int:
    """Bytes of one expert at int4 with an fp16 scale and an fp16 zero point per group
    (Sec. 3.1 "Problem": 1.77 MB per expert at H=2048, I=512, group 64)."""
    return 3 * (H * I // 2) + 3 * (H * I // group) * 2 * 2


# ------------------------------------------------------------------ dequantisation

def dequant(packed, scales, zeros, group: int) -> np.ndarray:
    """w[n][k] = scale[n][k // group] * (q[n][k] - zero[n][k // group]) in fp64
    (int4 affine group quantisation, Sec. 3.1 / Table "tiers")."""
    q = unpack_codes(packed).astype(np.float64)
    s = np.asarray(scales).astype(np.float64)
    z = np.asarray(zeros).astype(np.float64)
    n, kd = q.shape
    if kd % group or s.shape != (n, kd // group) or z.shape != s.shape:
        raise ValueError("group layout mismatch")
    return np.repeat(s, group, axis=1) * (q - np.repeat(z, group, axis=1))


# ------------------------------------------------------------------ routing (Appendix A)

def prerouter_logits(W_pre, s_bits) -> np.ndarray:
    """l[e] = sum_j W_pre[e][j] * s[j]: the linear residual path of the prerouter head
    applied to the hidden state (Sec. 3.2 "Head")."""
    W = np.asarray(W_pre).astype(np.float64)
    s = bf16_to_f64(s_bits)
    return np.array([np.dot(W[e], s) for e in range(W.shape[0])], dtype=np.float64)


def gelu_erf(z) -> np.ndarray:
    """Exact (erf) GELU: z * Phi(z) = 0.5 z (1 + erf(z / sqrt 2)), the activation of the prerouter's MLP
    path (Sec. 3.2 "Head")."""
    z = np.asarray(z, dtype=np.float64)
    return np.array([0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0))) for v in z.ravel()], dtype=np.float64).reshape(z.shape)


def prerouter_mlp_logits(W1, b1, W2, b2, W_res, s_bits, cur_inds, prev_inds) -> np.ndarray:
    """Sec. 3.2 "Head", the full head of one layer: fc1 -> erf-gelu -> fc2 plus the linear residual path.

    The input feature concatenates the hidden state with two K-hot vectors over the E experts: the
    experts this layer routed to at this token (``cur_inds``) and at the previous token
    (``prev_inds``): f = [s ; hot(cur) ; hot(prev)], dimension d + 2E.
        z = W1 f + b1        (W1 [D][d + 2E], D the hidden width)
        l = W2 gelu(z) + b2 + W_res s        (W2 [E][D]; W_res [E][d], the residual path, acts on the
                                              hidden state: it is what a router weight would be)
    Biases and the residual path are optional (None = absent)."""
    s = bf16_to_f64(s_bits)
    W1 = np.asarray(W1).astype(np.float64)
    W2 = np.asarray(W2).astype(np.float64)
    d = s.shape[0]
    E = W2.shape[0]
    if W1.shape[1] != d + 2 * E or W2.shape[1] != W1.shape[0]:
        raise ValueError("head shapes do not fit")
    f = np.zeros(d + 2 * E, dtype=np.float64)
    f[:d] = s
    for e in cur_inds:
        f[d + int(e)] = 1.0
    for e in prev_inds:
        f[d + E + int(e)] = 1.0
    z = np.array([np.dot(W1[r], f) for r in range(W1.shape[0])], dtype=np.float64)
    if b1 is not None:
        z = z + np.asarray(b1).astype(np.float64)
    a = gelu_erf(z)
    l = np.array([np.dot(W2[e], a) for e in range(E)], dtype=np.float64)
    if b2 is not None:
        l = l + np.asarray(b2).astype(np.float64)
    if W_res is not None:
        l = l + prerouter_logits(W_res, s_bits)
    return l


def softmax_topk(logits, K: int) -> Tuple[np.ndarray, np.ndarray]:
    """Appendix A, softmax-topk with renormalisation:
    g = softmax(l); inds = top-k(g, K); w = g[inds] / sum(g[inds]).

    The top-k is the first K of a full stable sort by descending logit (softmax
    is monotone, so ranking g and ranking l agree); equal logits go to the lower
    expert index.  The K experts are returned in ascending expert index with
    their weights aligned.
    """
    l = np.asarray(logits, dtype=np.float64)
    E = l.shape[0]
    if not 1 <= K <= E:
        raise ValueError("K out of range")
    e = np.exp(l - l.max())
    g = e / e.sum()
    order = sorted(range(E), key=lambda i: (-l[i], i))
    inds = np.array(sorted(order[:K]), dtype=np.int32)
    w = g[inds] / g[inds].sum()
    return inds, w


def sigmoid_group_topk(logits, K: int, n_groups: int, keep_groups: int, scale: float,
                       bias=None) -> Tuple[np.ndarray, np.ndarray]:
    """Appendix A, sigmoid-group routing: sigma = sigmoid(l); a group's score is the sum of
    its two largest (biased) scores; keep the best ``keep_groups`` groups; top-K among the
    survivors by (biased) score; w = scale * sigma[inds] / (sum sigma[inds] + 1e-20).
    Selection uses sigma + bias when a bias is given, weights use the raw sigmoid."""
    l = np.asarray(logits, dtype=np.float64)
    E = l.shape[0]
    sig = 1.0 / (1.0 + np.exp(-l))
    sel = sig if bias is None else sig + np.asarray(bias, dtype=np.float64)
    per = E // n_groups
    gscore = []
    for gi in range(n_groups):
        blk = sorted(sel[gi * per:(gi + 1) * per], reverse=True)
        gscore.append(blk[0] + blk[1])
    gorder = sorted(range(n_groups), key=lambda i: (-gscore[i], i))[:keep_groups]
    alive = [i for i in range(E) if (i // per) in gorder]
    order = sorted(alive, key=lambda i: (-sel[i], i))[:K]
    inds = np.array(sorted(order), dtype=np.int32)
    w = scale * sig[inds] / (sig[inds].sum() + 1e-20)
    return inds, w


# ------------------------------------------------------------------ slot pool (staged executor path)

class SlotAllocator:
    """Slot table of one layer (Sec. 3.1, "staged" path): a fixed pool of S slots, a table from
    expert to slot, sticky residency (an expert that stays routed keeps its slot and is not
    copied again) and least-recently-used eviction.

    ``stage(P)`` takes the K experts of a step in ascending index.  Experts already resident keep
    their slot.  Each missing expert, in order, takes the slot with the smallest
    (last_use, slot index) among slots that this step neither keeps nor has already assigned.
    """

    def __init__(self, E: int, S: int):
        self.E, self.S = E, S
        self.expert_of_slot = [-1] * S
        self.slot_of_expert = [-1] * E
        self.last_use = [-1] * S
        self.n = 0

    def stage(self, P: Sequence[int]) -> Tuple[List[int], List[Tuple[int, int]]]:
        """Returns (slots aligned with P, list of (expert, slot) copies to perform)."""
        P = [int(e) for e in P]
        if len(P) > self.S:
            raise ValueError("more routed experts than slots")
        if len(set(P)) != len(P) or any(e < 0 or e >= self.E for e in P):
            raise ValueError("bad expert set")
        taken = [False] * self.S
        for e in P:
            s = self.slot_of_expert[e]
            if s >= 0:
                taken[s] = True
                self.last_use[s] = self.n
        copies = []
        for e in P:
            if self.slot_of_expert[e] >= 0:
                continue
            victim = min((s for s in range(self.S) if not taken[s]), key=lambda s: (self.last_use[s], s))
            old = self.expert_of_slot[victim]
            if old >= 0:
                self.slot_of_expert[old] = -1
            self.expert_of_slot[victim] = e
            self.slot_of_expert[e] = victim
            self.last_use[victim] = self.n
            taken[victim] = True
            copies.append((e, victim))
        self.n += 1
        return [self.slot_of_expert[e] for e in P], copies


class HotSetAllocator:
    """The "hot" executor path of one layer (Sec. 3.1): a fixed pool of S_hot slots holds the
    least-recently-used-resident hot experts; a routed expert that is resident is a hit and is run
    from its slot; one that is not is a miss and is served on demand for this step (the paper's
    misses "fall to exact"), without waiting for any staging.

    Readings taken (the paper gives the path one sentence): a miss also enters the hot set for
    *later* steps once the expert has been routed ``admit_after`` times in total (1 = plain LRU
    cache; larger values make it a popularity cache), replacing the least recently used slot that
    this step neither hit nor has already given away; if every slot is spoken for, the miss is only
    served.  ``step(P)`` takes the routed experts in ascending index and returns
    (slot per expert, -1 for a miss served on demand; the (expert, slot) admissions that take
    effect after this step's compute).
    """

    def __init__(self, E: int, S_hot: int, admit_after: int = 1):
        self.E, self.S, self.admit_after = E, S_hot, admit_after
        self.expert_of_slot = [-1] * S_hot
        self.slot_of_expert = [-1] * E
        self.last_use = [-1] * S_hot
        self.uses = [0] * E
        self.n = 0
        self.hits = self.misses = self.admitted = 0

    def step(self, P: Sequence[int]) -> Tuple[List[int], List[Tuple[int, int]]]:
        P = [int(e) for e in P]
        if len(set(P)) != len(P) or any(e < 0 or e >= self.E for e in P):
            raise ValueError("bad expert set")
        for e in P:
            self.uses[e] += 1
        spoken = [False] * self.S
        now = [self.slot_of_expert[e] for e in P]           # what this step's compute sees
        for s in now:
            if s >= 0:
                spoken[s] = True
                self.last_use[s] = self.n
        admissions = []
        for e, s in zip(P, now):
            if s >= 0:
                self.hits += 1
                continue
            self.misses += 1
            if self.uses[e] < self.admit_after:
                continue
            free = [v for v in range(self.S) if not spoken[v]]
            if not free:
                continue
            victim = min(free, key=lambda v: (self.last_use[v], v))
            old = self.expert_of_slot[victim]
            if old >= 0:
                self.slot_of_expert[old] = -1
            self.expert_of_slot[victim] = e
            self.slot_of_expert[e] = victim
            self.last_use[victim] = self.n
            spoken[victim] = True
            admissions.append((e, victim))
            self.admitted += 1
        self.n += 1
        return now, admissions


# ------------------------------------------------------------------ expert FFN + LoRA + reduce

def silu(v):
    """silu(v) = v * sigmoid(v) = v / (1 + exp(-v))."""
    v = np.asarray(v, dtype=np.float64)
    return v / (1.0 + np.exp(-v))


def _proj(x: np.ndarray, tensors, lora, sigma: float, group: int) -> np.ndarray:
    """One quantised projection with its parallel LoRA branch:
    y = W x + sigma * B (A x), W dequantised (Sec. 3.3: y = W_4bit(x) + (alpha/r) B A x)."""
    packed, scales, zeros = tensors
    W = dequant(packed, scales, zeros, group)
    y = W @ x
    if lora is not None:
        A = bf16_to_f64(lora[0])
        B = bf16_to_f64(lora[1])
        y = y + sigma * (B @ (A @ x))
    return y


def expert_ffn(x: np.ndarray, expert: Dict[str, tuple], lora: Optional[Dict[str, tuple]],
               sigma: float, group: int) -> np.ndarray:
    """o = down(silu(gate(x)) * up(x)) for one expert (Sec. 3.1 "Math contract"), each of the
    three projections carrying its LoRA delta; the down adapter sees the same h as the base."""
    g = _proj(x, expert["gate"], None if lora is None else lora["gate"], sigma, group)
    u = _proj(x, expert["up"], None if lora is None else lora["up"], sigma, group)
    h = silu(g) * u
    return _proj(h, expert["down"], None if lora is None else lora["down"], sigma, group)


def moe_ffn(x_bits, inds, gates, get_expert: Callable[[int], Dict[str, tuple]],
            get_lora: Optional[Callable[[int], Dict[str, tuple]]], sigma: float, group: int) -> np.ndarray:
    """y = sum_k w_k * expert_{inds[k]}(x), summed in the order given (Appendix A weights applied
    to the expert outputs of the math contract)."""
    x = bf16_to_f64(x_bits)
    y = None
    for e, w in zip(inds, gates):
        lora = None if get_lora is None else get_lora(int(e))
        o = float(w) * expert_ffn(x, get_expert(int(e)), lora, sigma, group)
        y = o if y is None else y + o
    return y


def moe_ffn_with_shared(x_bits, inds, gates, get_expert, get_lora, shared_expert, shared_lora,
                        sigma: float, group: int) -> np.ndarray:
    """y = sum_k w_k * expert_k(x) + shared(x): the routed experts plus the layer's always-on shared
    expert (Sec. 3.1 lists it beside the routed experts; Sec. 4 "Phase 2" puts the adapter on its
    projections).  Reading taken: the shared expert obeys the same math contract and enters with
    weight 1 (the paper states no gate for it).  Summed routed experts first, the shared one last."""
    y = moe_ffn(x_bits, inds, gates, get_expert, get_lora, sigma, group) if len(inds) else None
    o = expert_ffn(bf16_to_f64(x_bits), shared_expert, shared_lora, sigma, group)
    return o if y is None else y + o


def moe_ffn_tokens(X_bits, inds, gates, get_expert, get_lora, sigma: float, group: int) -> np.ndarray:
    """Batched decode / prefill: the batch-1 definition applied token by token.
    X_bits [T][H], inds [T][K], gates [T][K] -> Y [T][H]."""
    return np.stack([moe_ffn(X_bits[t], inds[t], gates[t], get_expert, get_lora, sigma, group)
                     for t in range(len(X_bits))])


def moe_layer_decode(x_bits, inds_cur, gates_cur, W_pre_next, K: int, get_expert, get_lora,
                     sigma: float, group: int, alloc: Optional[SlotAllocator] = None):
    """One layer-step (Sec. 3.2 "Motivation", the double shift): the routing predicted one token
    earlier is consumed as is (staged set == routed set), the experts run, and the head applied to
    the same hidden state predicts the next layer-step's routing.
    Returns (y, slots or None, copies or None, inds_next, gates_next, logits_next)."""
    slots = copies = None
    if alloc is not None:
        slots, copies = alloc.stage(inds_cur)
    y = moe_ffn(x_bits, inds_cur, gates_cur, get_expert, get_lora, sigma, group)
    logits = prerouter_logits(W_pre_next, x_bits)
    inds_next, gates_next = softmax_topk(logits, K)
    return y, slots, copies, inds_next, gates_next, logits


# ------------------------------------------------------------------ chaining consecutive layer-steps (benchmark construct)

def next_hidden_state(x_bits, y, eps: float = 1e-6) -> np.ndarray:
    """x_next = bf16(rmsnorm(x + y)), unit gain, rmsnorm(v) = v / sqrt(mean(v^2) + eps): residual
    connection plus the next block's input norm.  Not a step of the paper's method; the stand-in by
    which the dependent-chain measurement makes step t+1 wait for step t's output.  Returns bf16 bits."""
    v = bf16_to_f64(x_bits) + np.asarray(y, dtype=np.float64)
    return f64_to_bf16_bits(v / math.sqrt(float(np.mean(v * v)) + eps))


# ------------------------------------------------------------------ error measures used by the parity tests

def rel_l2(a, b) -> float:
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    d = math.sqrt(float(np.sum((a - b) ** 2)))
    n = math.sqrt(float(np.sum(b ** 2)))
    return d / n if n > 0 else d


def max_abs(a, b) -> float:
    return float(np.max(np.abs(np.asarray(a, dtype=np.float64) - np.asarray(b, dtype=np.float64)))) if np.size(a) else 0.0
