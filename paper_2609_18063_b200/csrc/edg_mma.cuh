// int4 -> fp16 tensor-core fragments shared by the batch-1 and the grouped kernels.
//
// A 32-bit word holds 8 codes k0..k7 of one row.  (w & 0x000F000F) | 0x64006400 is the half2
// (1024 + k0, 1024 + k4), (w & 0x00F000F0) | 0x64006400 is (1024 + 16 k1, 1024 + 16 k5), and the
// same on w >> 8 gives (k2, k6) and (k3, k7); subtracting 1024 (or multiplying by 1/16 and
// subtracting 64) is exact, so the MMA sees exact integer codes.  The k slots of the
// m16n8k16 MMA are therefore used in the order (k0,k4 | k1,k5) for the first k-step of a 32-code
// chunk and (k2,k6 | k3,k7) for the second, lane t of a quad owning word t of the chunk; the
// activation operand is arranged in the same order (permute8), so a B fragment of a chunk is four
// consecutive 32-bit registers.
#pragma once

#include "edg_common.cuh"

namespace edg {

__device__ __forceinline__ uint32_t lop3_and_or(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t h2_as_u32(__half2 v) { return *reinterpret_cast<uint32_t*>(&v); }
__device__ __forceinline__ __half2 u32_as_h2(uint32_t v) { return *reinterpret_cast<__half2*>(&v); }

// One 32-bit word = codes k0..k7 of one row.  Returns the four half2 (k0,k4) (k1,k5) (k2,k6) (k3,k7)
// of q - z, exact for integer zero points.
__device__ __forceinline__ void dequant_word(uint32_t w, __half2 z2, uint32_t (&out)[4]) {
    const __half2 k1024 = __float2half2_rn(1024.f), k64 = __float2half2_rn(64.f), k16th = __float2half2_rn(0.0625f);
    const uint32_t w2 = w >> 8;
    const __half2 q04 = __hsub2(u32_as_h2(lop3_and_or(w, 0x000F000Fu, 0x64006400u)), k1024);
    const __half2 q15 = __hfma2(u32_as_h2(lop3_and_or(w, 0x00F000F0u, 0x64006400u)), k16th, __hneg2(k64));
    const __half2 q26 = __hsub2(u32_as_h2(lop3_and_or(w2, 0x000F000Fu, 0x64006400u)), k1024);
    const __half2 q37 = __hfma2(u32_as_h2(lop3_and_or(w2, 0x00F000F0u, 0x64006400u)), k16th, __hneg2(k64));
    out[0] = h2_as_u32(__hsub2(q04, z2));
    out[1] = h2_as_u32(__hsub2(q15, z2));
    out[2] = h2_as_u32(__hsub2(q26, z2));
    out[3] = h2_as_u32(__hsub2(q37, z2));
}

// d = a . b  (fresh accumulator)
__device__ __forceinline__ void mma16816_zero(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}
__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// 8 consecutive fp32 activations -> the fp16 residuals v - fp16(v), same k-slot order
__device__ __forceinline__ uint4 permute8_lo(const float (&v)[8]) {
    float r[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) r[i] = v[i] - __half2float(__float2half_rn(v[i]));
    uint4 o;
    o.x = h2_as_u32(__floats2half2_rn(r[0], r[4]));
    o.y = h2_as_u32(__floats2half2_rn(r[1], r[5]));
    o.z = h2_as_u32(__floats2half2_rn(r[2], r[6]));
    o.w = h2_as_u32(__floats2half2_rn(r[3], r[7]));
    return o;
}

// 8 consecutive activations -> fp16 in the k-slot order of the fragments: (x0,x4,x1,x5,x2,x6,x3,x7)
__device__ __forceinline__ uint4 permute8(const float (&v)[8]) {
    uint4 r;
    r.x = h2_as_u32(__floats2half2_rn(v[0], v[4]));
    r.y = h2_as_u32(__floats2half2_rn(v[1], v[5]));
    r.z = h2_as_u32(__floats2half2_rn(v[2], v[6]));
    r.w = h2_as_u32(__floats2half2_rn(v[3], v[7]));
    return r;
}

// The cheapest form: the code words masked straight into fp16 with a bias -- codes 0, 2, 4, 6 of a
// word as 1024 + q, codes 1, 3, 5, 7 as 64 + q (their nibble sits four bits higher in the
// mantissa) -- five instructions a word.  The dot product then carries 1024 * (sum of the
// activations at even positions) + 64 * (sum at odd positions), exactly representable products
// summed in fp32, which the caller subtracts per scaled block along with the zero-point term.
__device__ __forceinline__ void dequant_word_b(uint32_t w, uint32_t (&out)[4]) {
    const uint32_t w2 = w >> 8;
    out[0] = lop3_and_or(w, 0x000F000Fu, 0x64006400u);
    out[1] = lop3_and_or(w, 0x00F000F0u, 0x54005400u);
    out[2] = lop3_and_or(w2, 0x000F000Fu, 0x64006400u);
    out[3] = lop3_and_or(w2, 0x00F000F0u, 0x54005400u);
}

}  // namespace edg
