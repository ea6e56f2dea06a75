// The rank-r projections of the unmerged adapter (Sec. 3.3: delta = sigma * B (A v)) for many tokens at
// once, on the tensor cores: u = A_gate x and A_up x per token (before gate/up), u_d = A_down h per
// (token, choice) pair (before down).  With one adapter per layer the A matrices are the same for every
// token, so 8 tokens (or pairs) become the 8 columns of m16n8k16 tiles whose rows are the adapter's
// rows: an A row is read once per 8 tokens instead of once per token.  Operands are fetched 16 bytes at a
// time under a permutation of k that A and B share (lane (g, t4) takes k = 8 t4 .. 8 t4 + 7 of every
// 32-k block, words 0, 1 to one MMA and words 2, 3 to the next), K is split over the warps and summed
// through shared memory.  bf16 adapter rows and bf16 states convert to fp16 exactly in the normal
// range; the fp32 h is fed as an fp16 value plus an fp16 residual (two MMAs); accumulation is fp32.
#include "edg_common.cuh"
#include "edg_mma.cuh"

namespace edg {
namespace {

constexpr int kLtTok = 8;          // tokens (pairs) per CTA = MMA columns

// 8 bf16 (one 16-byte load) as four fp16 pairs, order kept
__device__ __forceinline__ uint4 bf16x8_as_f16x8(uint4 v) {
    uint4 o;
    o.x = h2_as_u32(__floats2half2_rn(bf16_lo(v.x), bf16_hi(v.x)));
    o.y = h2_as_u32(__floats2half2_rn(bf16_lo(v.y), bf16_hi(v.y)));
    o.z = h2_as_u32(__floats2half2_rn(bf16_lo(v.z), bf16_hi(v.z)));
    o.w = h2_as_u32(__floats2half2_rn(bf16_lo(v.w), bf16_hi(v.w)));
    return o;
}

// u_gu[t][0][proj][j] = sum_k A_proj[j][k] x[t][k]: rows 0 .. r-1 of the tiles are A_gate, r .. 2r-1 A_up.
// TILES = ceil(2r / 16) row tiles, KB = 32-k blocks per warp (H / 8 warps / 32).
template <int TILES, int KB>
__global__ void __launch_bounds__(256, 2) lora_ax_tokens_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ A_gate,
                                                               const uint16_t* __restrict__ A_up, float* __restrict__ u_gu,
                                                               int T, int H, int r) {
    const int t0 = blockIdx.x * kLtTok;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t4 = lane & 3;
    extern __shared__ float smem[];
    float* s_red = smem;                                               // [8 warps][TILES x 16 x 8]
    const int xs = H * 2 + 64;                                         // bytes per token row (padded against bank conflicts)
    uint8_t* s_xh = reinterpret_cast<uint8_t*>(s_red + 8 * TILES * 128);
    const int ksl = H / 8;                                             // k per warp = 32 KB
    constexpr int KH = KB / 2;                                         // the K slice in two passes: half the registers, two CTAs per SM

    const uint16_t* rows[TILES][2];
#pragma unroll
    for (int ti = 0; ti < TILES; ++ti) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int m = ti * 16 + g + 8 * hh;
            rows[ti][hh] = m < r ? A_gate + (size_t)m * H : (m < 2 * r ? A_up + (size_t)(m - r) * H : nullptr);
        }
    }
    uint4 a[TILES][KH][2];
    auto load_a = [&](int pass) {
#pragma unroll
        for (int ti = 0; ti < TILES; ++ti) {
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
                for (int j = 0; j < KH; ++j)
                    a[ti][j][hh] = rows[ti][hh] != nullptr ? ld_stream16(rows[ti][hh] + warp * ksl + 32 * (pass * KH + j) + 8 * t4)
                                                           : make_uint4(0, 0, 0, 0);
            }
        }
    };
    // the adapter rows of the first pass are on their way while the states are converted
    load_a(0);
    // (four loads of a thread in flight at a time: the conversion is a chain of trips to memory otherwise)
    for (int i0 = threadIdx.x; i0 < kLtTok * (H / 8); i0 += 4 * blockDim.x) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * blockDim.x, tt = i / (H / 8), c = i % (H / 8), t = t0 + tt;
            v[u] = (i < kLtTok * (H / 8) && t < T) ? *reinterpret_cast<const uint4*>(x + (size_t)t * H + c * 8) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * blockDim.x, tt = i / (H / 8), c = i % (H / 8);
            if (i < kLtTok * (H / 8)) *reinterpret_cast<uint4*>(s_xh + tt * xs + c * 16) = bf16x8_as_f16x8(v[u]);
        }
    }
    __syncthreads();

    const uint8_t* xb = s_xh + g * xs + (warp * ksl + 8 * t4) * 2;
    float c[TILES][4];
#pragma unroll
    for (int ti = 0; ti < TILES; ++ti) { c[ti][0] = 0.f; c[ti][1] = 0.f; c[ti][2] = 0.f; c[ti][3] = 0.f; }
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
        if (pass) load_a(1);
#pragma unroll
        for (int j = 0; j < KH; ++j) {
            const uint4 b = *reinterpret_cast<const uint4*>(xb + 64 * (pass * KH + j));
#pragma unroll
            for (int ti = 0; ti < TILES; ++ti) {
                const uint4 lo = bf16x8_as_f16x8(a[ti][j][0]), hi = bf16x8_as_f16x8(a[ti][j][1]);
                mma16816(c[ti], lo.x, hi.x, lo.y, hi.y, b.x, b.y);
                mma16816(c[ti], lo.z, hi.z, lo.w, hi.w, b.z, b.w);
            }
        }
    }
    // rows g / g + 8, tokens 2 t4 / 2 t4 + 1 of this warp's K slice
    float* mine = s_red + warp * TILES * 128;
#pragma unroll
    for (int ti = 0; ti < TILES; ++ti) {
        mine[ti * 128 + g * 8 + 2 * t4] = c[ti][0]; mine[ti * 128 + g * 8 + 2 * t4 + 1] = c[ti][1];
        mine[ti * 128 + (g + 8) * 8 + 2 * t4] = c[ti][2]; mine[ti * 128 + (g + 8) * 8 + 2 * t4 + 1] = c[ti][3];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < TILES * 128; i += blockDim.x) {
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) v += s_red[w * TILES * 128 + i];      // fixed order
        const int row = i >> 3, tok = i & 7;
        if (row < 2 * r && t0 + tok < T) u_gu[(size_t)(t0 + tok) * 2 * r + row] = v;
    }
}

// u_d[pair][j] = sum_i A_down[j][i] h[pair][i]; TILES = ceil(r / 16), KB = 32-k blocks per warp (I / 4 warps / 32)
template <int TILES, int KB>
__global__ void __launch_bounds__(128) lora_adh_pairs_kernel(const float* __restrict__ h, const uint16_t* __restrict__ A_down,
                                                            float* __restrict__ u_d, int P, int I, int r) {
    const int p0 = blockIdx.x * kLtTok;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t4 = lane & 3;
    extern __shared__ float smem[];
    float* s_red = smem;                                               // [4 warps][TILES x 16 x 8]
    const int hs = I * 2 + 64;                                         // bytes per pair row
    uint8_t* s_hh = reinterpret_cast<uint8_t*>(s_red + 4 * TILES * 128);   // [8][I + 32] fp16 value
    uint8_t* s_hl = s_hh + kLtTok * hs;                                 // [8][I + 32] fp16 residual
    const int ksl = I / 4;

    uint4 a[TILES][KB][2];
#pragma unroll
    for (int ti = 0; ti < TILES; ++ti) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int m = ti * 16 + g + 8 * hh;
#pragma unroll
            for (int j = 0; j < KB; ++j)
                a[ti][j][hh] = m < r ? ld_stream16(A_down + (size_t)m * I + warp * ksl + 32 * j + 8 * t4) : make_uint4(0, 0, 0, 0);
        }
    }
    for (int i = threadIdx.x; i < kLtTok * (I / 8); i += blockDim.x) {
        const int tt = i / (I / 8), c = i % (I / 8), pr = p0 + tt;
        uint4 hi = make_uint4(0, 0, 0, 0), lo = hi;
        if (pr < P) {
            const float4 v0 = *reinterpret_cast<const float4*>(h + (size_t)pr * I + c * 8);
            const float4 v1 = *reinterpret_cast<const float4*>(h + (size_t)pr * I + c * 8 + 4);
            const float f[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
            uint32_t wh[4], wl[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const __half2 hv = __floats2half2_rn(f[2 * e], f[2 * e + 1]);
                const float2 back = __half22float2(hv);
                wh[e] = h2_as_u32(hv);
                wl[e] = h2_as_u32(__floats2half2_rn(f[2 * e] - back.x, f[2 * e + 1] - back.y));
            }
            hi = make_uint4(wh[0], wh[1], wh[2], wh[3]);
            lo = make_uint4(wl[0], wl[1], wl[2], wl[3]);
        }
        *reinterpret_cast<uint4*>(s_hh + tt * hs + c * 16) = hi;
        *reinterpret_cast<uint4*>(s_hl + tt * hs + c * 16) = lo;
    }
    __syncthreads();

    const int boff = g * hs + (warp * ksl + 8 * t4) * 2;
    float c[TILES][4];
#pragma unroll
    for (int ti = 0; ti < TILES; ++ti) { c[ti][0] = 0.f; c[ti][1] = 0.f; c[ti][2] = 0.f; c[ti][3] = 0.f; }
#pragma unroll
    for (int j = 0; j < KB; ++j) {
        const uint4 bh = *reinterpret_cast<const uint4*>(s_hh + boff + 64 * j);
        const uint4 bl = *reinterpret_cast<const uint4*>(s_hl + boff + 64 * j);
#pragma unroll
        for (int ti = 0; ti < TILES; ++ti) {
            const uint4 lo = bf16x8_as_f16x8(a[ti][j][0]), hi = bf16x8_as_f16x8(a[ti][j][1]);
            mma16816(c[ti], lo.x, hi.x, lo.y, hi.y, bh.x, bh.y);
            mma16816(c[ti], lo.z, hi.z, lo.w, hi.w, bh.z, bh.w);
            mma16816(c[ti], lo.x, hi.x, lo.y, hi.y, bl.x, bl.y);
            mma16816(c[ti], lo.z, hi.z, lo.w, hi.w, bl.z, bl.w);
        }
    }
    float* mine = s_red + warp * TILES * 128;
#pragma unroll
    for (int ti = 0; ti < TILES; ++ti) {
        mine[ti * 128 + g * 8 + 2 * t4] = c[ti][0]; mine[ti * 128 + g * 8 + 2 * t4 + 1] = c[ti][1];
        mine[ti * 128 + (g + 8) * 8 + 2 * t4] = c[ti][2]; mine[ti * 128 + (g + 8) * 8 + 2 * t4 + 1] = c[ti][3];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < TILES * 128; i += blockDim.x) {
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) v += s_red[w * TILES * 128 + i];
        const int row = i >> 3, tok = i & 7;
        if (row < r && p0 + tok < P) u_d[(size_t)(p0 + tok) * r + row] = v;
    }
}

}  // namespace

// A x for all tokens with one shared adapter; false when the shape is not covered (the caller falls back)
bool launch_lora_ax_tokens(const edg_layer_desc* d, const void* x, const edg_lora* lora, float* u_gu, int T, cudaStream_t st) {
    const int r = d->rank, H = d->H;
    if (d->n_adapters != 1 || r < 8 || r % 8 != 0 || 2 * r > 32 || (H != 1024 && H != 2048)) return false;
    const uint16_t* Ag = static_cast<const uint16_t*>(lora->A_gate);
    const uint16_t* Au = static_cast<const uint16_t*>(lora->A_up);
    const int tiles = (2 * r + 15) / 16, grid = (T + kLtTok - 1) / kLtTok;
    const size_t sm = (size_t)8 * tiles * 128 * 4 + (size_t)kLtTok * (H * 2 + 64);
    const uint16_t* xx = static_cast<const uint16_t*>(x);
#define EDG_LAX(TI, KB_)                                                                                         \
    do {                                                                                                         \
        static bool conf = false;                                                                                \
        if (!conf) { cudaFuncSetAttribute(lora_ax_tokens_kernel<TI, KB_>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024); conf = true; } \
        lora_ax_tokens_kernel<TI, KB_><<<grid, 256, sm, st>>>(xx, Ag, Au, u_gu, T, H, r);                        \
    } while (0)
    if (H == 2048) { if (tiles == 1) EDG_LAX(1, 8); else EDG_LAX(2, 8); }
    else { if (tiles == 1) EDG_LAX(1, 4); else EDG_LAX(2, 4); }
#undef EDG_LAX
    return true;
}

// A_down h for all pairs with one shared adapter
bool launch_lora_adh_pairs(const edg_layer_desc* d, const edg_lora* lora, const float* h, float* u_d, int P, cudaStream_t st) {
    const int r = d->rank, I = d->I;
    if (d->n_adapters != 1 || r < 8 || r % 8 != 0 || r > 32 || (I != 256 && I != 512)) return false;
    const uint16_t* Ad = static_cast<const uint16_t*>(lora->A_down);
    const int tiles = (r + 15) / 16, grid = (P + kLtTok - 1) / kLtTok;
    const size_t sm = (size_t)4 * tiles * 128 * 4 + (size_t)2 * kLtTok * (I * 2 + 64);
    if (I == 512) { if (tiles == 1) lora_adh_pairs_kernel<1, 4><<<grid, 128, sm, st>>>(h, Ad, u_d, P, I, r); else lora_adh_pairs_kernel<2, 4><<<grid, 128, sm, st>>>(h, Ad, u_d, P, I, r); }
    else { if (tiles == 1) lora_adh_pairs_kernel<1, 2><<<grid, 128, sm, st>>>(h, Ad, u_d, P, I, r); else lora_adh_pairs_kernel<2, 2><<<grid, 128, sm, st>>>(h, Ad, u_d, P, I, r); }
    return true;
}

}  // namespace edg
