"""The arithmetic the batch-1 kernel relies on when it feeds int4 codes to the tensor cores without
subtracting anything first, checked in numpy against what IEEE fp16 fixes.

A 32-bit word holds eight codes, code k in bits 4k..4k+3.  Masking with 0x000F000F and or-ing
0x6400 into both halves gives two fp16 numbers 1024 + q (codes 0 and 4; after a shift by 8: codes 2
and 6); masking with 0x00F000F0 and or-ing 0x5400 gives 64 + q (codes 1 and 5; 3 and 7): the nibble
sits four bits higher in the mantissa and the exponent is four lower.  A dot product over such
operands therefore carries 1024 * (sum of the activations at even positions) + 64 * (sum at odd
positions), which is removed once per scaled block."""
import numpy as np


def _halves_as_fp16(word):
    return np.array([word & 0xFFFF, word >> 16], dtype=np.uint16).view(np.float16).astype(np.float64)


def test_every_code_at_every_position_becomes_bias_plus_code():
    for k in range(8):
        for q in range(16):
            w = q << (4 * k)
            w2 = w >> 8
            words = [(w & 0x000F000F) | 0x64006400, (w & 0x00F000F0) | 0x54005400,
                     (w2 & 0x000F000F) | 0x64006400, (w2 & 0x00F000F0) | 0x54005400]
            # operand register r holds codes (r, r + 4): low half code r, high half code r + 4
            got = {}
            for r, word in enumerate(words):
                lo, hi = _halves_as_fp16(word)
                got[r], got[r + 4] = lo, hi
            for kk in range(8):
                bias = 1024.0 if kk % 2 == 0 else 64.0
                assert got[kk] == bias + (q if kk == k else 0), (k, q, kk, got[kk])


def test_block_sum_minus_bias_is_the_code_dot_product():
    rng = np.random.default_rng(7)
    for _ in range(200):
        q = rng.integers(0, 16, size=64)
        x = rng.standard_normal(64).astype(np.float16)        # what the tensor core sees
        bias = np.where(np.arange(64) % 2 == 0, 1024.0, 64.0)
        # products of two fp16 numbers are exact in fp32; sum them in fp32 in MMA order (16 at a time)
        prod = ((bias + q).astype(np.float32) * x.astype(np.float32)).astype(np.float32)
        assert np.array_equal(prod.astype(np.float64), (bias + q) * x.astype(np.float64))
        acc = np.float32(0)
        for j in range(0, 64, 16):
            acc = np.float32(acc + prod[j:j + 16].sum(dtype=np.float32))
        xe, xo = x[0::2].astype(np.float32).sum(dtype=np.float32), x[1::2].astype(np.float32).sum(dtype=np.float32)
        corrected = np.float32(acc - np.float32(np.float32(1024) * xe + np.float32(64) * xo))
        exact = float((q * x.astype(np.float64)).sum())
        # the rounding is that of fp32 sums of terms of size <= 1039 |x|
        bound = 16 * 2.0 ** -24 * float((np.abs(bias + q) * np.abs(x.astype(np.float64))).sum())
        assert abs(float(corrected) - exact) <= bound
        # ... which is far inside the tolerance on a block's contribution
        assert bound <= 2e-3 * max(1.0, float((q * np.abs(x.astype(np.float64))).sum()))
