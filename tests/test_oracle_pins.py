"""Pins for the CPU oracle: closed forms, brute force on tiny inputs, invariants and the sizes
the paper prints.  None of these needs a GPU, and none re-types the oracle's own formula: each
expected value comes from hand arithmetic, an independent slow loop, or a property the
mathematics fixes."""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import moe_oracle as orc
from workloads import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bf16(vals):
    return synth.f32_to_bf16_bits(np.asarray(vals, dtype=np.float32))


# ------------------------------------------------------------------ formats

def test_bf16_known_bit_patterns():
    bits = np.array([0x3F80, 0xC000, 0x4049, 0x0000, 0x3E80, 0xBF00], dtype=np.uint16)
    assert orc.bf16_to_f64(bits).tolist() == [1.0, -2.0, 3.140625, 0.0, 0.25, -0.5]


def test_bf16_rounding_ties_to_even_and_no_double_rounding():
    # 1 + 2^-8 is exactly between 1.0 (0x3F80, even) and 1+2^-7 (0x3F81): goes to even.
    assert orc.f64_to_bf16_bits([1.0 + 2.0 ** -8])[0] == 0x3F80
    assert orc.f64_to_bf16_bits([1.0 + 3 * 2.0 ** -8])[0] == 0x3F82
    # just above the tie must round up even though float32 would first round it onto the tie
    assert orc.f64_to_bf16_bits([1.0 + 2.0 ** -8 + 2.0 ** -40])[0] == 0x3F81
    assert orc.f64_to_bf16_bits([-(1.0 + 2.0 ** -8 + 2.0 ** -40)])[0] == 0xBF81
    v = np.random.default_rng(0).standard_normal(1000)
    back = orc.bf16_to_f64(orc.f64_to_bf16_bits(v))
    assert np.all(np.abs(back - v) <= np.abs(v) * 2.0 ** -8)


def test_pack_unpack_identity_and_nibble_order():
    assert orc.unpack_codes(np.array([[0x21, 0xF0]], dtype=np.uint8)).tolist() == [[1, 2, 0, 15]]
    c = np.random.default_rng(1).integers(0, 16, size=(5, 64), dtype=np.uint8)
    assert np.array_equal(orc.unpack_codes(orc.pack_codes(c)), c)
    p = np.random.default_rng(2).integers(0, 256, size=(3, 32), dtype=np.uint8)
    assert np.array_equal(orc.pack_codes(orc.unpack_codes(p)), p)


def test_record_bytes_match_the_sizes_the_paper_prints():
    g = {}
    for line in open(os.path.join(GOLDEN, "paper_sizes.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            g[k] = float(v)
    R = orc.record_bytes(int(g["H"]), int(g["I"]), int(g["group"]))
    assert R == 1_769_472
    assert round(R / 1e6, 2) == g["expert_MB"]
    assert round(R * g["E"] / 1e6) == g["layer_MB"]
    assert round(R * g["E"] * g["L"] / 1e9) == g["routed_GB"]
    assert round(R * g["E"] * g["L"] / 2 ** 30, 1) == g["routed_GiB"]
    assert round(4 * R / 1e6) == g["k4_layer_MB"]
    assert g["lora_alpha"] / g["lora_rank"] == g["lora_scale"]
    assert synth.CONFIGS["cfg2"].record_bytes == R
    assert synth.CONFIGS["cfg1"].record_bytes == orc.record_bytes(1024, 256, 32) == 491_520


# ------------------------------------------------------------------ dequant

def test_dequant_hand_worked_codes():
    # s = 2^-7, z = 8, q = 0..15  ->  w = (q - 8) / 128
    codes = np.arange(16, dtype=np.uint8)[None, :].repeat(2, axis=0)
    codes = np.concatenate([codes, codes], axis=1)                     # [2][32], one group of 32
    w = orc.dequant(orc.pack_codes(codes), np.full((2, 1), 2.0 ** -7, np.float16),
                    np.full((2, 1), 8, np.float16), 32)
    expect = [(q - 8) / 128 for q in range(16)] * 2
    assert w[0].tolist() == expect and w[1].tolist() == expect
    assert w[0][0] == -0.0625 and w[0][15] == 0.0546875
    # z = 0, s = 1 -> w = q
    w = orc.dequant(orc.pack_codes(codes), np.ones((2, 1), np.float16), np.zeros((2, 1), np.float16), 32)
    assert np.array_equal(w, codes.astype(np.float64))


def test_dequant_groups_run_along_the_input_dimension():
    codes = np.full((1, 64), 3, dtype=np.uint8)
    s = np.array([[1.0, 0.5]], np.float16)
    z = np.array([[1.0, 2.0]], np.float16)
    w = orc.dequant(orc.pack_codes(codes), s, z, 32)
    assert w[0, :32].tolist() == [2.0] * 32 and w[0, 32:].tolist() == [0.5] * 32


# ------------------------------------------------------------------ logits

def test_logits_brute_force_and_identity_head():
    rng = np.random.default_rng(3)
    W = (rng.standard_normal((5, 16)) * 0.02).astype(np.float32)
    s = _bf16(rng.standard_normal(16))
    got = orc.prerouter_logits(W, s)
    sv = orc.bf16_to_f64(s)
    for e in range(5):
        exact = sum(Fraction(float(W[e, j])) * Fraction(float(sv[j])) for j in range(16))
        assert abs(got[e] - float(exact)) <= 1e-15
    # an identity head returns the hidden state itself
    assert np.array_equal(orc.prerouter_logits(np.eye(16, dtype=np.float32), s), sv)
    # a transposed operand would fail this one: row e is e * ones
    W2 = np.arange(4, dtype=np.float32)[:, None] * np.ones((4, 16), np.float32)
    assert np.allclose(orc.prerouter_logits(W2, s), np.arange(4) * sv.sum(), rtol=0, atol=1e-12)


# ------------------------------------------------------------------ softmax top-k (Appendix A)

def _topk_by_repeated_argmax(l, K):
    l = list(map(float, l))
    left = set(range(len(l)))
    out = []
    for _ in range(K):
        best = min(left, key=lambda i: (-l[i], i))
        out.append(best)
        left.remove(best)
    return sorted(out)


def test_topk_equals_full_sort_and_selection_properties():
    rng = np.random.default_rng(4)
    for E, K in [(16, 2), (256, 8), (256, 4), (8, 8), (7, 1)]:
        for _ in range(20):
            l = rng.standard_normal(E)
            inds, w = orc.softmax_topk(l, K)
            assert inds.tolist() == _topk_by_repeated_argmax(l, K)
            assert inds.tolist() == sorted(np.argsort(-l, kind="stable")[:K].tolist())
            assert len(set(inds.tolist())) == K
            rest = np.setdiff1d(np.arange(E), inds)
            if len(rest):
                assert l[inds].min() >= l[rest].max()
            assert abs(w.sum() - 1.0) <= 1e-12 and (w > 0).all()
    inds, w = orc.softmax_topk(rng.standard_normal(12), 12)
    assert inds.tolist() == list(range(12))


def test_topk_ties_go_to_the_lower_index():
    l = np.array([0.5, 2.0, 2.0, 2.0, -1.0])
    assert orc.softmax_topk(l, 2)[0].tolist() == [1, 2]
    assert orc.softmax_topk(np.zeros(6), 3)[0].tolist() == [0, 1, 2]


def test_gates_closed_forms():
    # logits ln(1..4): softmax = [.1,.2,.3,.4]; top-2 = experts 2,3 with weights 3/7, 4/7
    inds, w = orc.softmax_topk(np.log([1.0, 2.0, 3.0, 4.0]), 2)
    assert inds.tolist() == [2, 3]
    assert np.allclose(w, [3 / 7, 4 / 7], rtol=0, atol=1e-15)
    # out of order on purpose: weights stay aligned with ascending expert index
    inds, w = orc.softmax_topk(np.log([4.0, 1.0, 2.0, 3.0]), 3)
    assert inds.tolist() == [0, 2, 3]
    assert np.allclose(w, [4 / 9, 2 / 9, 3 / 9], rtol=0, atol=1e-15)
    # softmax restricted to the selected logits, shift invariance, K = 1
    rng = np.random.default_rng(5)
    l = rng.standard_normal(64) * 3
    inds, w = orc.softmax_topk(l, 8)
    sel = [math.exp(l[i]) for i in inds]
    assert np.allclose(w, np.array(sel) / sum(sel), rtol=1e-13, atol=0)
    inds2, w2 = orc.softmax_topk(l + 123.25, 8)
    assert inds2.tolist() == inds.tolist() and np.allclose(w2, w, rtol=1e-12, atol=0)
    assert orc.softmax_topk(l, 1)[1].tolist() == [1.0]


def test_topk_permutation_equivariance():
    rng = np.random.default_rng(6)
    l = rng.standard_normal(32)
    perm = rng.permutation(32)
    inds, w = orc.softmax_topk(l, 4)
    inds_p, w_p = orc.softmax_topk(l[perm], 4)
    assert sorted(perm[inds_p].tolist()) == inds.tolist()
    back = dict(zip(perm[inds_p].tolist(), w_p.tolist()))
    assert np.allclose([back[i] for i in inds.tolist()], w, rtol=1e-13, atol=0)


def test_sigmoid_group_hand_example():
    # 2 groups of 4, keep 1 group, K=2, scale 2.5.  sigmoid(0)=.5, sigmoid(ln3)=.75, sigmoid(-ln3)=.25
    L3 = math.log(3.0)
    l = np.array([L3, L3, -L3, -L3, L3, 0.0, 0.0, 0.0])
    # group scores: 1.5 vs 1.25 -> group 0 survives; top-2 inside it are experts 0,1
    inds, w = orc.sigmoid_group_topk(l, K=2, n_groups=2, keep_groups=1, scale=2.5)
    assert inds.tolist() == [0, 1]
    assert np.allclose(w, [1.25, 1.25], rtol=0, atol=1e-12)
    # a selection bias can flip the surviving group while the weights still use the raw sigmoid
    bias = np.array([0, 0, 0, 0, 0, 0.5, 0, 0.0])
    inds, w = orc.sigmoid_group_topk(l, K=2, n_groups=2, keep_groups=1, scale=2.5, bias=bias)
    assert inds.tolist() == [4, 5]
    assert np.allclose(w, [2.5 * 0.75 / 1.25, 2.5 * 0.5 / 1.25], rtol=0, atol=1e-12)


def _sig_logit(p):
    return math.log(p / (1.0 - p))


def test_sigmoid_group_score_is_the_top2_sum_not_the_max_nor_the_group_sum():
    # Three groups of three whose sigmoids are chosen so that the three candidate group scores rank
    # the groups differently (Appendix A: a group is ranked by the sum of its two largest scores):
    #   group 0: .9  .15 .1    max .9   top-2 sum 1.05  whole sum 1.15
    #   group 1: .6  .6  .05   max .6   top-2 sum 1.2   whole sum 1.25
    #   group 2: .5  .5  .45   max .5   top-2 sum 1.0   whole sum 1.45
    # keep 1 group: top-2 sum -> group 1; the max would keep group 0; the whole sum group 2.
    sig = [.9, .15, .1, .6, .6, .05, .5, .5, .45]
    l = np.array([_sig_logit(p) for p in sig])
    inds, w = orc.sigmoid_group_topk(l, K=2, n_groups=3, keep_groups=1, scale=1.0)
    assert inds.tolist() == [3, 4]
    assert np.allclose(w, [0.5, 0.5], rtol=0, atol=1e-12)
    # keep 2 of 3 groups.  top-2 sums 1.05 / 1.2 / 1.0: groups 1 and 0.  (The max would keep {0, 1} as
    # well, the whole sum {1, 2}: expert 0 tells them apart.)
    inds, w = orc.sigmoid_group_topk(l, K=3, n_groups=3, keep_groups=2, scale=2.0)
    assert inds.tolist() == [0, 3, 4]
    assert np.allclose(w, [2.0 * .9 / 2.1, 2.0 * .6 / 2.1, 2.0 * .6 / 2.1], rtol=0, atol=1e-12)
    # keep 2 of 3 where the second survivor differs between top-2 sum and max:
    #   group 0: .7 .1 .1 (max .7, top-2 .8)   group 1: .6 .6 .1 (max .6, top-2 1.2)   group 2: .5 .45 .1 (max .5, top-2 .95)
    # top-2 sum keeps {1, 2}; the max would keep {0, 1}.  K = 4 of the six survivors by score.
    sig = [.7, .1, .1, .6, .6, .1, .5, .45, .1]
    l = np.array([_sig_logit(p) for p in sig])
    inds, w = orc.sigmoid_group_topk(l, K=4, n_groups=3, keep_groups=2, scale=2.5)
    assert inds.tolist() == [3, 4, 6, 7]
    tot = .6 + .6 + .5 + .45
    assert np.allclose(w, [2.5 * .6 / tot, 2.5 * .6 / tot, 2.5 * .5 / tot, 2.5 * .45 / tot], rtol=0, atol=1e-12)
    # an off-by-one in the number of kept groups (1 or 3 instead of 2) changes the answer:
    assert orc.sigmoid_group_topk(l, K=4, n_groups=3, keep_groups=3, scale=2.5)[0].tolist() == [0, 3, 4, 6]
    # K as large as the survivors: every expert of the kept groups, none of the dropped group
    inds, _ = orc.sigmoid_group_topk(l, K=6, n_groups=3, keep_groups=2, scale=2.5)
    assert inds.tolist() == [3, 4, 5, 6, 7, 8]


# ------------------------------------------------------------------ FFN, LoRA, reduce

def _tiny_expert(rng, H, I, g):
    ex = {}
    for proj, (n, kd) in {"gate": (I, H), "up": (I, H), "down": (H, I)}.items():
        ex[proj] = (rng.integers(0, 256, (n, kd // 2), dtype=np.uint8),
                    rng.uniform(0.005, 0.02, (n, kd // g)).astype(np.float16),
                    rng.integers(0, 16, (n, kd // g)).astype(np.float16))
    return ex


def _tiny_lora(rng, H, I, r):
    lo = {}
    for proj, (n, kd) in {"gate": (I, H), "up": (I, H), "down": (H, I)}.items():
        lo[proj] = (_bf16(rng.standard_normal((r, kd)) * 0.02), _bf16(rng.standard_normal((n, r)) * 0.01))
    return lo


def _brute_proj(x, tensors, lora, sigma, g):
    """Scalar Python loops straight from w = s (q - z) and y = W x + sigma B (A x)."""
    packed, scales, zeros = tensors
    n, half = packed.shape
    out = []
    for i in range(n):
        acc = 0.0
        for k in range(2 * half):
            byte = int(packed[i, k // 2])
            q = (byte & 15) if k % 2 == 0 else (byte >> 4)
            acc += float(scales[i, k // g]) * (q - float(zeros[i, k // g])) * x[k]
        out.append(acc)
    if lora is not None:
        A = orc.bf16_to_f64(lora[0])
        B = orc.bf16_to_f64(lora[1])
        u = [sum(A[j, k] * x[k] for k in range(len(x))) for j in range(A.shape[0])]
        out = [out[i] + sigma * sum(B[i, j] * u[j] for j in range(len(u))) for i in range(n)]
    return out


def test_expert_ffn_brute_force_tiny_layer():
    rng = np.random.default_rng(7)
    H = I = 32
    g = 32
    ex = _tiny_expert(rng, H, I, g)
    lo = _tiny_lora(rng, H, I, 2)
    x = orc.bf16_to_f64(_bf16(rng.standard_normal(H)))
    gate = _brute_proj(x, ex["gate"], lo["gate"], 2.0, g)
    up = _brute_proj(x, ex["up"], lo["up"], 2.0, g)
    h = [gv / (1.0 + math.exp(-gv)) * uv for gv, uv in zip(gate, up)]
    o = _brute_proj(h, ex["down"], lo["down"], 2.0, g)
    got = orc.expert_ffn(x, ex, lo, 2.0, g)
    assert np.allclose(got, o, rtol=1e-12, atol=1e-13)


def test_expert_ffn_constant_weights_closed_form():
    # every dequantised weight equals c = s (q - z): g = u = c sum(x), o = c I silu(g) u
    H, I, g = 64, 32, 32
    s, q, z = 0.5, 9, 7          # c = 1.0
    ex = {}
    for proj, (n, kd) in {"gate": (I, H), "up": (I, H), "down": (H, I)}.items():
        ex[proj] = (orc.pack_codes(np.full((n, kd), q, np.uint8)), np.full((n, kd // g), s, np.float16),
                    np.full((n, kd // g), z, np.float16))
    x = orc.bf16_to_f64(_bf16(np.linspace(-1, 1.5, H)))
    c = s * (q - z)
    gsum = c * x.sum()
    expect = c * I * (gsum / (1 + math.exp(-gsum))) * gsum
    got = orc.expert_ffn(x, ex, None, 2.0, g)
    assert np.allclose(got, np.full(H, expect), rtol=1e-13, atol=0)


def test_lora_pins():
    rng = np.random.default_rng(8)
    H, I, g, r = 64, 32, 32, 4
    ex = _tiny_expert(rng, H, I, g)
    lo = _tiny_lora(rng, H, I, r)
    x = orc.bf16_to_f64(_bf16(rng.standard_normal(H)))
    base = orc.expert_ffn(x, ex, None, 2.0, g)
    # B = 0 (or A = 0) reproduces the base bit for bit
    zero_b = {p: (lo[p][0], np.zeros_like(lo[p][1])) for p in lo}
    zero_a = {p: (np.zeros_like(lo[p][0]), lo[p][1]) for p in lo}
    assert np.array_equal(orc.expert_ffn(x, ex, zero_b, 2.0, g), base)
    assert np.array_equal(orc.expert_ffn(x, ex, zero_a, 2.0, g), base)
    # rank-1 one-hot adapter on the down projection only: delta = sigma * h[j] on row i
    i_row, j_col = 5, 3
    A = np.zeros((1, I), np.float32); A[0, j_col] = 1.0
    B = np.zeros((H, 1), np.float32); B[i_row, 0] = 1.0
    none = lambda n, kd: (_bf16(np.zeros((1, kd))), _bf16(np.zeros((n, 1))))
    one_hot = {"gate": none(I, H), "up": none(I, H), "down": (_bf16(A), _bf16(B))}
    gate = orc.dequant(*ex["gate"], g) @ x
    up = orc.dequant(*ex["up"], g) @ x
    h = gate / (1 + np.exp(-gate)) * up
    for sigma in (2.0, 4.0):
        d = orc.expert_ffn(x, ex, one_hot, sigma, g) - base
        expect = np.zeros(H); expect[i_row] = sigma * h[j_col]
        assert np.allclose(d, expect, rtol=1e-12, atol=1e-12)
    # the delta of a down-only adapter is linear in sigma
    down_only = {"gate": none(I, H), "up": none(I, H), "down": lo["down"]}
    d1 = orc.expert_ffn(x, ex, down_only, 1.0, g) - base
    d2 = orc.expert_ffn(x, ex, down_only, 2.0, g) - base
    assert np.allclose(d2, 2 * d1, rtol=1e-9, atol=1e-12)


def test_dropped_lora_delta_is_visible_at_the_parity_tolerance():
    cfg = synth.CONFIGS["cfg1"]
    x_bits = synth.hidden_states(cfg, 1)[0]
    ex = synth.expert_tensors(cfg, 0, 3)
    lo = synth.lora_tensors(cfg, 0, 0)
    x = orc.bf16_to_f64(x_bits)
    with_ = orc.expert_ffn(x, ex, lo, cfg.lora_scale, cfg.group)
    without = orc.expert_ffn(x, ex, None, cfg.lora_scale, cfg.group)
    assert orc.rel_l2(without, with_) > 5e-3      # five times the 1e-3 parity bar


def test_reduce_pins():
    rng = np.random.default_rng(9)
    H, I, g = 32, 32, 32
    experts = {e: _tiny_expert(rng, H, I, g) for e in range(4)}
    x_bits = _bf16(rng.standard_normal(H))
    x = orc.bf16_to_f64(x_bits)
    outs = {e: orc.expert_ffn(x, experts[e], None, 2.0, g) for e in range(4)}
    get = lambda e: experts[e]
    # one-hot gates pick one expert's output
    y = orc.moe_ffn(x_bits, [1, 3], [0.0, 1.0], get, None, 2.0, g)
    assert np.array_equal(y, outs[3])
    # equal gates give the mean
    y = orc.moe_ffn(x_bits, [0, 2], [0.5, 0.5], get, None, 2.0, g)
    assert np.allclose(y, 0.5 * (outs[0] + outs[2]), rtol=1e-15, atol=0)
    # permuting (inds, gates) together changes nothing beyond summation order
    y1 = orc.moe_ffn(x_bits, [0, 1, 2], [0.2, 0.3, 0.5], get, None, 2.0, g)
    y2 = orc.moe_ffn(x_bits, [2, 0, 1], [0.5, 0.2, 0.3], get, None, 2.0, g)
    assert np.allclose(y1, y2, rtol=1e-13, atol=1e-15)
    assert np.allclose(y1, 0.2 * outs[0] + 0.3 * outs[1] + 0.5 * outs[2], rtol=1e-13, atol=1e-15)
    # the token-batched form is the batch-1 form applied row by row
    X = _bf16(rng.standard_normal((3, H)))
    inds = [[0, 1], [2, 3], [1, 2]]
    gts = [[0.4, 0.6], [0.5, 0.5], [0.9, 0.1]]
    Y = orc.moe_ffn_tokens(X, inds, gts, get, None, 2.0, g)
    for t in range(3):
        assert np.array_equal(Y[t], orc.moe_ffn(X[t], inds[t], gts[t], get, None, 2.0, g))


# ------------------------------------------------------------------ slot pool

def test_slot_allocator_hand_worked_sequence():
    a = orc.SlotAllocator(E=8, S=3)
    assert a.stage([1, 4]) == ([0, 1], [(1, 0), (4, 1)])          # empty pool: lowest slots first
    assert a.stage([4, 6]) == ([1, 2], [(6, 2)])                  # 4 is sticky, 6 takes the unused slot
    assert a.stage([4, 5]) == ([1, 0], [(5, 0)])                  # LRU victim is slot 0 (expert 1, used at step 0)
    assert a.stage([1, 4]) == ([2, 1], [(1, 2)])                  # slot 2 (expert 6, step 1) is older than slot 0 (step 2)
    assert a.slot_of_expert[6] == -1 and a.slot_of_expert[5] == 0
    assert a.stage([1, 4]) == ([2, 1], [])                        # a repeat copies nothing


def test_slot_allocator_invariants_random_walk():
    rng = np.random.default_rng(10)
    for E, S, K in [(16, 4, 2), (256, 8, 8), (256, 32, 8), (64, 64, 8)]:
        a = orc.SlotAllocator(E, S)
        resident = set()
        for step in range(200):
            P = sorted(rng.choice(E, K, replace=False).tolist())
            before = {e: a.slot_of_expert[e] for e in resident}
            slots, copies = a.stage(P)
            assert len(set(slots)) == K and all(0 <= s < S for s in slots)
            for e, s in zip(P, slots):
                assert a.expert_of_slot[s] == e and a.slot_of_expert[e] == s
            # staged set == routed set; copies are exactly the missing experts; hits do not move
            assert sorted(e for e, _ in copies) == sorted(set(P) - resident)
            for e in set(P) & resident:
                assert a.slot_of_expert[e] == before[e]
            # an expert that stays resident never changes slot
            for e in resident:
                if a.slot_of_expert[e] >= 0:
                    assert a.slot_of_expert[e] == before[e]
            resident = {e for e in range(E) if a.slot_of_expert[e] >= 0}
            assert len(resident) == sum(1 for s in a.expert_of_slot if s >= 0) <= S
    with pytest.raises(ValueError):
        orc.SlotAllocator(16, 2).stage([1, 2, 3])
    with pytest.raises(ValueError):
        orc.SlotAllocator(16, 4).stage([1, 16])


def test_slot_allocator_full_pool_never_copies_after_warmup():
    a = orc.SlotAllocator(E=16, S=16)
    rng = np.random.default_rng(11)
    seen = set()
    for _ in range(100):
        P = sorted(rng.choice(16, 4, replace=False).tolist())
        _, copies = a.stage(P)
        assert {e for e, _ in copies} == set(P) - seen
        seen |= set(P)


# ------------------------------------------------------------------ whole layer-step

def test_layer_decode_is_the_composition_of_its_parts():
    cfg = synth.CONFIGS["cfg1"]
    x_bits = synth.hidden_states(cfg, 2)[1]
    W = synth.prerouter_weights(cfg)
    get = lambda e: synth.expert_tensors(cfg, 0, e)
    lora = synth.lora_tensors(cfg, 0, 0)
    get_lora = lambda e: lora
    inds_cur, gates_cur = orc.softmax_topk(orc.prerouter_logits(W, synth.hidden_states(cfg, 2)[0]), cfg.K)
    alloc = orc.SlotAllocator(cfg.E, cfg.n_slots)
    y, slots, copies, inds_n, gates_n, logits = orc.moe_layer_decode(
        x_bits, inds_cur, gates_cur, W, cfg.K, get, get_lora, cfg.lora_scale, cfg.group, alloc)
    assert np.array_equal(y, orc.moe_ffn(x_bits, inds_cur, gates_cur, get, get_lora, cfg.lora_scale, cfg.group))
    assert np.array_equal(logits, orc.prerouter_logits(W, x_bits))
    i2, g2 = orc.softmax_topk(logits, cfg.K)
    assert np.array_equal(inds_n, i2) and np.array_equal(gates_n, g2)
    assert sorted(e for e, _ in copies) == inds_cur.tolist() and slots == [0, 1]
    # magnitudes the tolerances were derived for: outputs of order 1-10, not 1e-3 or 1e3
    assert 1.0 < np.std(y) < 30.0


# ------------------------------------------------------------------ the MLP head (Sec. 3.2 "Head")

def test_gelu_erf_known_values_and_limits():
    # z * Phi(z) with the standard normal CDF: Phi(0) = 1/2, Phi(1) = 0.8413447460685429, Phi(-1) = 1 - Phi(1)
    g = orc.gelu_erf(np.array([0.0, 1.0, -1.0, 2.0, 8.0, -8.0]))
    assert g[0] == 0.0
    assert abs(g[1] - 0.8413447460685429) < 1e-15
    assert abs(g[2] + (1.0 - 0.8413447460685429)) < 1e-15
    assert abs(g[3] - 2.0 * 0.9772498680518208) < 1e-15
    assert abs(g[4] - 8.0) < 1e-13 and abs(g[5]) < 1e-13          # identity far right, zero far left
    # the identity gelu(z) - gelu(-z) = z holds for every z
    z = np.random.default_rng(3).standard_normal(50) * 3
    assert np.allclose(orc.gelu_erf(z) - orc.gelu_erf(-z), z, rtol=0, atol=1e-14)


def test_mlp_head_reduces_to_the_linear_head_and_to_a_column_gather():
    rng = np.random.default_rng(11)
    d, E, D, K = 32, 8, 16, 2
    s_bits = _bf16(rng.standard_normal(d))
    W1 = rng.standard_normal((D, d + 2 * E)) * 0.3
    b1 = rng.standard_normal(D) * 0.1
    W2 = rng.standard_normal((E, D)) * 0.3
    b2 = rng.standard_normal(E) * 0.1
    Wr = rng.standard_normal((E, d)) * 0.2
    cur, prev = [1, 6], [0, 6]
    # with a zero fc2 the head is the residual path alone (+ b2): the linear head that is pinned above
    l0 = orc.prerouter_mlp_logits(W1, b1, np.zeros((E, D)), None, Wr, s_bits, cur, prev)
    assert np.array_equal(l0, orc.prerouter_logits(Wr, s_bits))
    # the one-hot part of the feature picks columns of W1: brute force with an explicit concatenated vector
    s = orc.bf16_to_f64(s_bits)
    z = W1[:, :d] @ s + W1[:, d + 1] + W1[:, d + 6] + W1[:, d + E + 0] + W1[:, d + E + 6] + b1
    a = np.array([0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0))) for v in z])
    want = W2 @ a + b2 + Wr @ s
    got = orc.prerouter_mlp_logits(W1, b1, W2, b2, Wr, s_bits, cur, prev)
    assert np.allclose(got, want, rtol=0, atol=1e-12)
    # the two one-hot blocks are distinct inputs: swapping them changes the result
    assert not np.allclose(got, orc.prerouter_mlp_logits(W1, b1, W2, b2, Wr, s_bits, prev, cur))
    # hand example: d = 1, E = 1, D = 1: z = 2*1.5 + 0.25 (cur) + 0.5 (prev) - 0.75 = 3.0, l = 4 * gelu(3) + 1 + 0.5 * 1.5
    one = orc.prerouter_mlp_logits([[2.0, 0.25, 0.5]], [-0.75], [[4.0]], [1.0], [[0.5]], _bf16([1.5]), [0], [0])
    assert abs(one[0] - (4.0 * 3.0 * 0.9986501019683699 + 1.0 + 0.75)) < 1e-12


# ------------------------------------------------------------------ the benchmark's chain construct

def test_next_hidden_state_closed_forms():
    # x + y = (3, 4, 0, 0): mean square 25/4, rms 2.5 -> (1.2, 1.6, 0, 0), rounded to bf16
    x = _bf16([1.0, 1.0, 0.5, -2.0])
    y = np.array([2.0, 3.0, -0.5, 2.0])
    out = orc.next_hidden_state(x, y, eps=0.0)
    assert out.tolist() == [0x3F9A, 0x3FCD, 0x0000, 0x0000]          # 1.203125, 1.6015625 (nearest bf16 of 1.2, 1.6)
    # a constant vector normalises to ones whatever its size; the sign survives
    assert orc.next_hidden_state(_bf16([0.0] * 8), np.full(8, -7.25), eps=0.0).tolist() == [0xBF80] * 8
    # scale invariance without eps, and eps in the right place: v = (1e-3,)*4, eps = 1e-6 -> 1e-3 / sqrt(2e-6)
    rng = np.random.default_rng(11)
    xb, yv = _bf16(rng.standard_normal(64)), rng.standard_normal(64)
    a = orc.next_hidden_state(xb, yv, eps=0.0)
    xs = orc.bf16_to_f64(xb) * 4.0
    b = orc.next_hidden_state(_bf16(xs), yv * 4.0, eps=0.0)
    assert np.array_equal(a, b)
    got = orc.bf16_to_f64(orc.next_hidden_state(_bf16([0.0] * 4), np.full(4, 1e-3), eps=1e-6))
    assert np.allclose(got, 1e-3 / math.sqrt(2e-6), rtol=2.0 ** -8)


# ------------------------------------------------------------------ the hot executor path

def test_hot_set_hand_worked_sequence():
    # 3 hot slots, plain LRU admission.  Step by step, by hand:
    a = orc.HotSetAllocator(E=8, S_hot=3)
    assert a.step([1, 2]) == ([-1, -1], [(1, 0), (2, 1)])          # cold start: both served on demand, both admitted
    assert a.step([1, 5]) == ([0, -1], [(5, 2)])                   # 1 hits slot 0; 5 takes the last empty slot
    assert a.step([2, 5]) == ([1, 2], [])                          # two hits, nothing moves
    # 6 and 7 miss; slot 0 (expert 1, last used at step 1) is the LRU, then slot 1 (expert 2, used at step 2)
    # -- but slots used by THIS step are never given away: here none is, so 6 -> slot 0, 7 -> slot 1
    assert a.step([6, 7]) == ([-1, -1], [(6, 0), (7, 1)])
    assert a.expert_of_slot == [6, 7, 5] and a.slot_of_expert[1] == -1 and a.slot_of_expert[2] == -1
    # a step that hits two slots and misses two more: only one slot is free to give away
    assert a.step([0, 3, 5, 6]) == ([-1, -1, 2, 0], [(0, 1)])      # 0 takes slot 1 (expert 7); 3 is only served
    assert a.expert_of_slot == [6, 0, 5]
    assert (a.hits, a.misses, a.admitted) == (5, 7, 6)


def test_hot_set_popularity_admission_and_invariants():
    # admit_after = 3: an expert enters the hot set only on its third routing
    a = orc.HotSetAllocator(E=6, S_hot=2, admit_after=3)
    assert a.step([4]) == ([-1], [])
    assert a.step([4]) == ([-1], [])
    assert a.step([4]) == ([-1], [(4, 0)])
    assert a.step([4]) == ([0], [])
    rng = np.random.default_rng(12)
    b = orc.HotSetAllocator(E=32, S_hot=6, admit_after=2)
    for _ in range(300):
        P = sorted(rng.choice(32, 4, replace=False).tolist())
        before = list(b.slot_of_expert)
        now, adm = b.step(P)
        assert now == [before[e] for e in P]                         # this step sees the table as it was
        for e, v in adm:
            assert before[e] < 0 and v not in [s for s in now if s >= 0]    # a slot hit by this step is never given away
        res = [e for e in b.expert_of_slot if e >= 0]
        assert len(res) == len(set(res))
        for v, e in enumerate(b.expert_of_slot):
            if e >= 0:
                assert b.slot_of_expert[e] == v
        assert sum(1 for s in b.slot_of_expert if s >= 0) == len(res)
    assert b.hits + b.misses == 1200 and b.admitted <= b.misses


# ------------------------------------------------------------------ the shared expert

def test_shared_expert_is_one_more_expert_with_weight_one():
    rng = np.random.default_rng(21)
    H, I, g, r = 32, 32, 32, 4
    experts = [_tiny_expert(rng, H, I, g) for _ in range(3)]
    shared, lo, slo = _tiny_expert(rng, H, I, g), _tiny_lora(rng, H, I, r), _tiny_lora(rng, H, I, r)
    x = _bf16(rng.standard_normal(H))
    xv = orc.bf16_to_f64(x)
    # brute force: the scalar-loop projections of this file, composed by hand
    def brute_ffn(ex, lora):
        gt = _brute_proj(xv, ex["gate"], lora["gate"], 2.0, g)
        up = _brute_proj(xv, ex["up"], lora["up"], 2.0, g)
        h = np.array([a / (1.0 + math.exp(-a)) * b for a, b in zip(gt, up)])
        return np.array(_brute_proj(h, ex["down"], lora["down"], 2.0, g))
    want = 0.25 * brute_ffn(experts[0], lo) + 0.75 * brute_ffn(experts[2], lo) + brute_ffn(shared, slo)
    got = orc.moe_ffn_with_shared(x, [0, 2], [0.25, 0.75], experts.__getitem__, lambda e: lo, shared, slo, 2.0, g)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)
    # no routed expert at all: the layer is the shared expert; routed part and shared part add
    only = orc.moe_ffn_with_shared(x, [], [], experts.__getitem__, None, shared, slo, 2.0, g)
    assert np.allclose(only, brute_ffn(shared, slo), rtol=1e-12, atol=1e-12)
    routed = orc.moe_ffn(x, [0, 2], [0.25, 0.75], experts.__getitem__, lambda e: lo, 2.0, g)
    assert np.allclose(got - routed, only, rtol=1e-10, atol=1e-12)
    # the shared expert's adapter is its own: swapping it for the routed adapter changes the result
    other = orc.moe_ffn_with_shared(x, [0, 2], [0.25, 0.75], experts.__getitem__, lambda e: lo, shared, lo, 2.0, g)
    assert np.abs(other - got).max() > 1e-6
