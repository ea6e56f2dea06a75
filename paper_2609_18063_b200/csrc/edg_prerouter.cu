// a1 + a2: prerouter head logits, softmax, top-k and renormalised gate weights
// (Sec. 3.2 "Head" linear path; Appendix A softmax-topk).
//
// One thread-block cluster per head: the E rows of the head are split over the CTAs of the
// cluster, every CTA writes its logits straight into the leader CTA's shared memory
// (distributed shared memory), and after one cluster barrier a single warp of the leader does
// softmax + top-k with warp shuffles.  No global scratch, no atomics, one launch.
#include <cooperative_groups.h>
#include <math_constants.h>

#include "edg_common.cuh"
#include "edg_mma.cuh"

namespace cg = cooperative_groups;

namespace edg {

constexpr int kPreCluster = 8;      // CTAs per head (portable cluster size)
constexpr int kPreWarps = 8;

struct PreParams {
    const void* W;          // [n_heads][E][H]
    const uint16_t* s;      // [n_heads][H] bf16
    int32_t* inds;          // [n_heads][K]
    float* gates;           // [n_heads][K]
    float* logits;          // [n_heads][E] or null
    int H, E, K;
    int shared_head;        // 1: every state uses head 0 (batched tokens of one layer)
    int32_t* mirror;        // [n_heads][K] in mapped pinned host memory, or null
};

template <typename WT> struct RowDot;

// fp16 head: 8 weights (16 bytes) per lane per step
template <> struct RowDot<__half> {
    static __device__ __forceinline__ float partial(const void* W, size_t row, const float* sx, int H, int lane) {
        const uint4* wp = reinterpret_cast<const uint4*>(static_cast<const __half*>(W) + row * H);
        float acc = 0.f;
#pragma unroll 8
        for (int c = lane; c < H / 8; c += 32) {
            const uint4 w = ld_stream16(wp + c);
            const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&w.x));
            const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&w.y));
            const float2 d = __half22float2(*reinterpret_cast<const __half2*>(&w.z));
            const float2 e = __half22float2(*reinterpret_cast<const __half2*>(&w.w));
            const float* x = sx + c * 8;
            acc = fmaf(a.x, x[0], acc); acc = fmaf(a.y, x[1], acc);
            acc = fmaf(b.x, x[2], acc); acc = fmaf(b.y, x[3], acc);
            acc = fmaf(d.x, x[4], acc); acc = fmaf(d.y, x[5], acc);
            acc = fmaf(e.x, x[6], acc); acc = fmaf(e.y, x[7], acc);
        }
        return acc;
    }
    static __device__ __forceinline__ float run(const void* W, size_t row, const float* sx, int H, int lane) {
        return warp_sum(partial(W, row, sx, H, lane));
    }
};

// fp32 head: 4 weights (16 bytes) per lane per step
template <> struct RowDot<float> {
    static __device__ __forceinline__ float partial(const void* W, size_t row, const float* sx, int H, int lane) {
        const uint4* wp = reinterpret_cast<const uint4*>(static_cast<const float*>(W) + row * H);
        float acc = 0.f;
#pragma unroll 4
        for (int c = lane; c < H / 4; c += 32) {
            const uint4 w = ld_stream16(wp + c);
            const float* x = sx + c * 4;
            acc = fmaf(__uint_as_float(w.x), x[0], acc); acc = fmaf(__uint_as_float(w.y), x[1], acc);
            acc = fmaf(__uint_as_float(w.z), x[2], acc); acc = fmaf(__uint_as_float(w.w), x[3], acc);
        }
        return acc;
    }
    static __device__ __forceinline__ float run(const void* W, size_t row, const float* sx, int H, int lane) {
        return warp_sum(partial(W, row, sx, H, lane));
    }
};

template <typename WT>
__global__ void __launch_bounds__(kPreWarps * 32) prerouter_kernel(PreParams p) {
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank();
    const int csize = (int)cluster.num_blocks();
    const int head = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    extern __shared__ float smem[];
    float* s_logits = smem;             // [E]   (the leader's copy collects every CTA's rows)
    float* s_x = smem + p.E;            // [H]   hidden state widened to fp32

    const uint16_t* sv = p.s + (size_t)head * p.H;
    for (int i = threadIdx.x; i < p.H; i += blockDim.x) s_x[i] = bf16_bits_to_float(sv[i]);
    __syncthreads();

    float* leader = cluster.map_shared_rank(s_logits, 0);
    const int per = (p.E + csize - 1) / csize;
    const int e0 = crank * per, e1 = min(p.E, e0 + per);
    const size_t wbase = p.shared_head ? 0 : (size_t)head * p.E;
    for (int e = e0 + warp; e < e1; e += kPreWarps) {
        const float l = RowDot<WT>::run(p.W, wbase + e, s_x, p.H, lane);
        if (lane == 0) leader[e] = l;
    }
    cluster.sync();                     // every CTA's logits have landed in the leader
    if (crank != 0) return;

    if (p.logits != nullptr)
        for (int e = threadIdx.x; e < p.E; e += blockDim.x) p.logits[(size_t)head * p.E + e] = s_logits[e];
    __syncthreads();
    if (warp == 0) {
        warp_softmax_topk(s_logits, p.E, p.K, lane, p.inds + (size_t)head * p.K, p.gates + (size_t)head * p.K);
        mirror_inds(p.mirror != nullptr ? p.mirror + (size_t)head * p.K : nullptr, p.inds + (size_t)head * p.K, p.K, lane);
    }
}

// One head, T hidden states (batched decode of one layer): a cluster handles kTokBlock tokens, so
// a row of the head is read once per token block instead of once per token.  CTA c of the cluster
// computes its share of the E rows for all tokens of the block (one warp per row, the tokens' states
// in shared memory as fp32), writes the logits into the leader's shared memory, and after the cluster
// barrier warp w of the leader does softmax + top-k for token w of the block.
constexpr int kTokBlock = 8;

template <typename WT>
__global__ void __launch_bounds__(kPreWarps * 32) prerouter_tokens_kernel(PreParams p, int T) {
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank();
    const int csize = (int)cluster.num_blocks();
    const int t0 = blockIdx.y * kTokBlock;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    extern __shared__ float smem[];
    float* s_logits = smem;                         // [kTokBlock][E]  (the leader's copy collects every CTA's rows)
    float* s_x = smem + kTokBlock * p.E;            // [kTokBlock][H]  hidden states widened to fp32
    for (int tt = 0; tt < kTokBlock; ++tt) {
        const int t = t0 + tt;
        for (int i = threadIdx.x; i < p.H; i += blockDim.x)
            s_x[tt * p.H + i] = t < T ? bf16_bits_to_float(p.s[(size_t)t * p.H + i]) : 0.f;
    }
    __syncthreads();

    float* leader = cluster.map_shared_rank(s_logits, 0);
    const int per = (p.E + csize - 1) / csize;
    const int e0 = crank * per, e1 = min(p.E, e0 + per);
    constexpr int VPL = 16 / (int)sizeof(WT);       // weights per 16-byte load
    const int n16 = p.H / VPL;                      // 16-byte pieces of a row
    for (int e = e0 + warp; e < e1; e += kPreWarps) {
        const uint4* wp = reinterpret_cast<const uint4*>(static_cast<const WT*>(p.W) + (size_t)e * p.H);
        float acc[kTokBlock];
#pragma unroll
        for (int t = 0; t < kTokBlock; ++t) acc[t] = 0.f;
        for (int c0 = 0; c0 < n16; c0 += 8 * 32) {   // 8 independent loads per lane in flight, then the arithmetic
            uint4 wr[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int c = c0 + j * 32 + lane;
                wr[j] = c < n16 ? ld_stream16(wp + c) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int c = c0 + j * 32 + lane;
                if (c >= n16) continue;
                const uint4 w = wr[j];
                float wf[8];
                if (VPL == 8) {
                    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&w.x));
                    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&w.y));
                    const float2 d = __half22float2(*reinterpret_cast<const __half2*>(&w.z));
                    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w.w));
                    wf[0] = a.x; wf[1] = a.y; wf[2] = b.x; wf[3] = b.y; wf[4] = d.x; wf[5] = d.y; wf[6] = f.x; wf[7] = f.y;
                } else {
                    wf[0] = __uint_as_float(w.x); wf[1] = __uint_as_float(w.y); wf[2] = __uint_as_float(w.z); wf[3] = __uint_as_float(w.w);
                    wf[4] = wf[5] = wf[6] = wf[7] = 0.f;
                }
#pragma unroll
                for (int t = 0; t < kTokBlock; ++t) {
                    const float* x = s_x + t * p.H + c * VPL;
                    const float4 x0 = *reinterpret_cast<const float4*>(x);
                    float a = acc[t];
                    a = fmaf(wf[0], x0.x, a); a = fmaf(wf[1], x0.y, a); a = fmaf(wf[2], x0.z, a); a = fmaf(wf[3], x0.w, a);
                    if (VPL == 8) {
                        const float4 x1 = *reinterpret_cast<const float4*>(x + 4);
                        a = fmaf(wf[4], x1.x, a); a = fmaf(wf[5], x1.y, a); a = fmaf(wf[6], x1.z, a); a = fmaf(wf[7], x1.w, a);
                    }
                    acc[t] = a;
                }
            }
        }
#pragma unroll
        for (int t = 0; t < kTokBlock; ++t) {
            const float l = warp_sum(acc[t]);
            if (lane == 0) leader[t * p.E + e] = l;
        }
    }
    cluster.sync();                     // every CTA's logits have landed in the leader
    if (crank != 0) return;

    const int t = t0 + warp;            // kPreWarps == kTokBlock: warp w finishes token w of the block
    if (warp < kTokBlock && t < T) {
        float* row = s_logits + warp * p.E;
        if (p.logits != nullptr)
            for (int e = lane; e < p.E; e += 32) p.logits[(size_t)t * p.E + e] = row[e];
        __syncwarp();
        warp_softmax_topk(row, p.E, p.K, lane, p.inds + (size_t)t * p.K, p.gates + (size_t)t * p.K);
    }
}

// The same for an fp16 head on the tensor cores: the block's 8 tokens are the 8 columns of an
// m16n8k16 tile, 16 rows of the head its rows.  A CTA takes its share of the rows two tiles at a
// time; warp w multiplies K slice w of both.  Operands are fetched 16 bytes at a time: lane (g, t4)
// reads k = 8 t4 .. 8 t4 + 7 of every 32-k block, of head rows g and g + 8 (straight from memory) and
// of token g (fp16 in shared memory, rows padded by 64 bytes against bank conflicts), and feeds words
// 0, 1 of each to one MMA and words 2, 3 to a second one -- a permutation of k that A and B share, so
// the dot products are unchanged.  All loads of a warp's slice are issued before the first MMA (one
// trip to memory); the slices are summed through shared memory, and the logits go to the leader as
// above.  fp16 of a bf16 state is exact in the normal range; products are exact in fp32 and summed
// in fp32.
constexpr int kMmaHeadKs = 256;        // k per warp and pass: 8 blocks of 32
__global__ void __launch_bounds__(kPreWarps * 32) prerouter_tokens_mma_kernel(PreParams p, int T) {
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank();
    const int csize = (int)cluster.num_blocks();
    const int t0 = blockIdx.y * kTokBlock;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t4 = lane & 3;
    extern __shared__ float smem[];
    float* s_logits = smem;                                             // [kTokBlock][E]
    float* s_red = smem + kTokBlock * p.E;                              // [kPreWarps][2 x 16 x 8] partial tiles
    const int xs = p.H * 2 + 64;                                        // bytes per token row
    uint8_t* s_xh = reinterpret_cast<uint8_t*>(s_red + kPreWarps * 256);    // [kTokBlock][H + 32] fp16
    const __half* W = static_cast<const __half*>(p.W);
    const int per = p.E / csize;                                        // rows of this CTA: a multiple of 16
    const int ksl = p.H / kPreWarps;                                    // k per warp: a multiple of 32

    // the head rows of the first pass are on their way while the tokens' states are converted
    uint4 a[2][kMmaHeadKs / 32][2];
    auto load_a = [&](int r0, int k0, bool two) {
#pragma unroll
        for (int tile = 0; tile < 2; ++tile) {
            const __half* w = W + (size_t)(r0 + (two ? 16 * tile : 0) + g) * p.H + warp * ksl + k0 + 8 * t4;
#pragma unroll
            for (int j = 0; j < kMmaHeadKs / 32; ++j) {
                const bool on = k0 + 32 * j < ksl;
                a[tile][j][0] = on ? ld_stream16(w + 32 * j) : make_uint4(0, 0, 0, 0);
                a[tile][j][1] = on ? ld_stream16(w + (size_t)8 * p.H + 32 * j) : make_uint4(0, 0, 0, 0);
            }
        }
    };
    const int r_first = crank * per;
    load_a(r_first, 0, r_first + 16 < (crank + 1) * per);
    for (int i = threadIdx.x; i < kTokBlock * (p.H / 8); i += blockDim.x) {
        const int tt = i / (p.H / 8), c = i % (p.H / 8), t = t0 + tt;
        uint4 o = make_uint4(0, 0, 0, 0);
        if (t < T) {
            const uint4 v = *reinterpret_cast<const uint4*>(p.s + (size_t)t * p.H + c * 8);
            o.x = h2_as_u32(__floats2half2_rn(bf16_lo(v.x), bf16_hi(v.x)));
            o.y = h2_as_u32(__floats2half2_rn(bf16_lo(v.y), bf16_hi(v.y)));
            o.z = h2_as_u32(__floats2half2_rn(bf16_lo(v.z), bf16_hi(v.z)));
            o.w = h2_as_u32(__floats2half2_rn(bf16_lo(v.w), bf16_hi(v.w)));
        }
        *reinterpret_cast<uint4*>(s_xh + tt * xs + c * 16) = o;
    }
    __syncthreads();

    float* leader = cluster.map_shared_rank(s_logits, 0);
    for (int r0 = r_first; r0 < (crank + 1) * per; r0 += 32) {
        const bool two = r0 + 16 < (crank + 1) * per;
        const uint8_t* xb = s_xh + g * xs + (warp * ksl + 8 * t4) * 2;
        float c[4] = {0.f, 0.f, 0.f, 0.f}, d[4] = {0.f, 0.f, 0.f, 0.f};
        for (int k0 = 0; k0 < ksl; k0 += kMmaHeadKs) {
            if (k0 > 0 || r0 > r_first) load_a(r0, k0, two);
#pragma unroll
            for (int j = 0; j < kMmaHeadKs / 32; ++j) {
                if (k0 + 32 * j < ksl) {
                    const uint4 b = *reinterpret_cast<const uint4*>(xb + (k0 + 32 * j) * 2);
                    mma16816(c, a[0][j][0].x, a[0][j][1].x, a[0][j][0].y, a[0][j][1].y, b.x, b.y);
                    mma16816(c, a[0][j][0].z, a[0][j][1].z, a[0][j][0].w, a[0][j][1].w, b.z, b.w);
                    mma16816(d, a[1][j][0].x, a[1][j][1].x, a[1][j][0].y, a[1][j][1].y, b.x, b.y);
                    mma16816(d, a[1][j][0].z, a[1][j][1].z, a[1][j][0].w, a[1][j][1].w, b.z, b.w);
                }
            }
        }
        // rows g / g + 8, tokens 2 t4 / 2 t4 + 1 of this warp's K slice, for both tiles
        float* mine = s_red + warp * 256;
        mine[g * 8 + 2 * t4] = c[0]; mine[g * 8 + 2 * t4 + 1] = c[1];
        mine[(g + 8) * 8 + 2 * t4] = c[2]; mine[(g + 8) * 8 + 2 * t4 + 1] = c[3];
        mine[128 + g * 8 + 2 * t4] = d[0]; mine[128 + g * 8 + 2 * t4 + 1] = d[1];
        mine[128 + (g + 8) * 8 + 2 * t4] = d[2]; mine[128 + (g + 8) * 8 + 2 * t4 + 1] = d[3];
        __syncthreads();
        if (threadIdx.x < 128 || two) {
            float v = 0.f;
#pragma unroll
            for (int w = 0; w < kPreWarps; ++w) v += s_red[w * 256 + threadIdx.x];
            const int row = threadIdx.x >> 3, tok = threadIdx.x & 7;      // row 0..31 over the two tiles
            leader[tok * p.E + r0 + row] = v;
        }
        __syncthreads();
    }
    cluster.sync();                     // every CTA's logits have landed in the leader
    if (crank != 0) return;

    const int t = t0 + warp;            // kPreWarps == kTokBlock: warp w finishes token w of the block
    if (warp < kTokBlock && t < T) {
        float* row = s_logits + warp * p.E;
        if (p.logits != nullptr)
            for (int e = lane; e < p.E; e += 32) p.logits[(size_t)t * p.E + e] = row[e];
        __syncwarp();
        warp_softmax_topk(row, p.E, p.K, lane, p.inds + (size_t)t * p.K, p.gates + (size_t)t * p.K);
    }
}

// a2 alone: one warp per row of given logits.
__global__ void __launch_bounds__(128) softmax_topk_rows_kernel(const float* logits, int T, int E, int K,
                                                                int32_t* inds, float* gates) {
    extern __shared__ float smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = blockIdx.x * 4 + warp;
    if (t >= T) return;
    float* work = smem + warp * E;
    for (int e = lane; e < E; e += 32) work[e] = logits[(size_t)t * E + e];
    __syncwarp();
    warp_softmax_topk(work, E, K, lane, inds + (size_t)t * K, gates + (size_t)t * K);
}

// ---------------------------------------------------------------- the full head (Sec. 3.2 "Head")
// fc1 -> erf-gelu -> fc2 plus the linear residual path, one cluster per head.  The feature is the
// hidden state followed by two K-hot vectors (this layer's experts at this token and at the previous
// one), so fc1 is a dot product over the hidden state plus a gather of 2K columns.  Phase 1: the D
// rows of fc1 are dealt to the CTAs of the cluster, a warp per row; every activation is written
// into the shared memory of all CTAs.  Phase 2: the E rows of fc2 (+ the residual row over the
// hidden state) likewise; the logits land in the leader, which does softmax + top-k.
struct MlpParams {
    const __half* W1;       // [n_heads][D][H + 2E]
    const __half* b1;       // [n_heads][D] or null
    const __half* W2;       // [n_heads][E][D]
    const __half* b2;       // [n_heads][E] or null
    const void* Wres;       // [n_heads][E][H] (fp16 or fp32) or null
    const uint16_t* s;      // [n_heads][H] bf16
    const int32_t* cur;     // [n_heads][K]
    const int32_t* prev;    // [n_heads][K]
    int32_t* inds;          // [n_heads][K]
    float* gates;           // [n_heads][K]
    float* logits;          // [n_heads][E] or null
    int H, E, K, D;
    int32_t* mirror;        // [n_heads][K] in mapped pinned host memory, or null
};

// dot product of an fp16 row of n (a multiple of 8) weights with fp32 activations, by one warp
__device__ __forceinline__ float half_row_dot(const __half* row, const float* sx, int n, int lane) {
    const uint4* wp = reinterpret_cast<const uint4*>(row);
    float acc = 0.f;
#pragma unroll 8
    for (int c = lane; c < n / 8; c += 32) {
        const uint4 w = ld_stream16(wp + c);
        const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&w.x));
        const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&w.y));
        const float2 d = __half22float2(*reinterpret_cast<const __half2*>(&w.z));
        const float2 e = __half22float2(*reinterpret_cast<const __half2*>(&w.w));
        const float* x = sx + c * 8;
        acc = fmaf(a.x, x[0], acc); acc = fmaf(a.y, x[1], acc);
        acc = fmaf(b.x, x[2], acc); acc = fmaf(b.y, x[3], acc);
        acc = fmaf(d.x, x[4], acc); acc = fmaf(d.y, x[5], acc);
        acc = fmaf(e.x, x[6], acc); acc = fmaf(e.y, x[7], acc);
    }
    return acc;                          // (not yet summed over the lanes)
}

// two rows at once against the same activations: twice the loads in flight, the activations read once
__device__ __forceinline__ void half_row_dot2(const __half* row0, const __half* row1, const float* sx, int n, int lane,
                                              float& acc0, float& acc1) {
    const uint4* wp0 = reinterpret_cast<const uint4*>(row0);
    const uint4* wp1 = reinterpret_cast<const uint4*>(row1);
    acc0 = 0.f; acc1 = 0.f;
#pragma unroll 8
    for (int c = lane; c < n / 8; c += 32) {
        const uint4 w0 = ld_stream16(wp0 + c), w1 = ld_stream16(wp1 + c);
        const float4 x0 = *reinterpret_cast<const float4*>(sx + c * 8), x1 = *reinterpret_cast<const float4*>(sx + c * 8 + 4);
        float2 a = __half22float2(*reinterpret_cast<const __half2*>(&w0.x)), b = __half22float2(*reinterpret_cast<const __half2*>(&w0.y));
        float2 d = __half22float2(*reinterpret_cast<const __half2*>(&w0.z)), e = __half22float2(*reinterpret_cast<const __half2*>(&w0.w));
        acc0 = fmaf(a.x, x0.x, acc0); acc0 = fmaf(a.y, x0.y, acc0); acc0 = fmaf(b.x, x0.z, acc0); acc0 = fmaf(b.y, x0.w, acc0);
        acc0 = fmaf(d.x, x1.x, acc0); acc0 = fmaf(d.y, x1.y, acc0); acc0 = fmaf(e.x, x1.z, acc0); acc0 = fmaf(e.y, x1.w, acc0);
        a = __half22float2(*reinterpret_cast<const __half2*>(&w1.x)); b = __half22float2(*reinterpret_cast<const __half2*>(&w1.y));
        d = __half22float2(*reinterpret_cast<const __half2*>(&w1.z)); e = __half22float2(*reinterpret_cast<const __half2*>(&w1.w));
        acc1 = fmaf(a.x, x0.x, acc1); acc1 = fmaf(a.y, x0.y, acc1); acc1 = fmaf(b.x, x0.z, acc1); acc1 = fmaf(b.y, x0.w, acc1);
        acc1 = fmaf(d.x, x1.x, acc1); acc1 = fmaf(d.y, x1.y, acc1); acc1 = fmaf(e.x, x1.z, acc1); acc1 = fmaf(e.y, x1.w, acc1);
    }
}

constexpr int kMlpWarps = 8;      // warps per CTA of the full head (16 measured no faster)

template <typename WT>
__global__ void __launch_bounds__(kMlpWarps * 32) prerouter_mlp_kernel(MlpParams p) {
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank();
    const int csize = (int)cluster.num_blocks();
    const int head = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    extern __shared__ float smem[];
    float* s_logits = smem;             // [E]   (the leader's copy collects every CTA's rows)
    float* s_x = smem + p.E;            // [H]   hidden state widened to fp32
    float* s_a = s_x + p.H;             // [D]   gelu(fc1), complete in every CTA after the first cluster barrier

    const uint16_t* sv = p.s + (size_t)head * p.H;
    for (int i = threadIdx.x; i < p.H; i += blockDim.x) s_x[i] = bf16_bits_to_float(sv[i]);
    __syncthreads();

    const int F = p.H + 2 * p.E;
    const int perD = (p.D + csize - 1) / csize;
    // the K-hot parts of the feature pick columns: lane k < K holds the k-th expert of either list
    int hc = -1, hq = -1;
    if (lane < p.K) {
        hc = p.cur[(size_t)head * p.K + lane];
        hq = p.prev[(size_t)head * p.K + lane];
        if (hc < 0 || hc >= p.E) hc = -1;
        if (hq < 0 || hq >= p.E) hq = -1;
    }
    const int rend = min(p.D, (crank + 1) * perD);
    for (int r = crank * perD + warp; r < rend; r += 2 * kMlpWarps) {      // two rows of this warp at a time
        const int r1 = r + kMlpWarps;
        const bool two = r1 < rend;
        const __half* row0 = p.W1 + ((size_t)head * p.D + r) * F;
        const __half* row1 = two ? row0 + (size_t)kMlpWarps * F : row0;
        // (the gathered columns are fetched together with the rows, not after them)
        const __half gc0 = hc >= 0 ? row0[p.H + hc] : __float2half(0.f), gq0 = hq >= 0 ? row0[p.H + p.E + hq] : __float2half(0.f);
        const __half gc1 = hc >= 0 ? row1[p.H + hc] : __float2half(0.f), gq1 = hq >= 0 ? row1[p.H + p.E + hq] : __float2half(0.f);
        float z0, z1;
        half_row_dot2(row0, row1, s_x, p.H, lane, z0, z1);
        z0 = warp_sum(z0 + __half2float(gc0) + __half2float(gq0));
        z1 = warp_sum(z1 + __half2float(gc1) + __half2float(gq1));
        if (p.b1 != nullptr) {
            z0 += __half2float(p.b1[(size_t)head * p.D + r]);
            if (two) z1 += __half2float(p.b1[(size_t)head * p.D + r1]);
        }
        const float a0 = 0.5f * z0 * (1.f + erff(z0 * 0.70710678118654752f));
        const float a1 = 0.5f * z1 * (1.f + erff(z1 * 0.70710678118654752f));
        if (lane < csize) {
            float* dst = cluster.map_shared_rank(s_a, lane);
            dst[r] = a0;
            if (two) dst[r1] = a1;
        }
    }
    cluster.sync();                     // every CTA holds all D activations

    float* leader = cluster.map_shared_rank(s_logits, 0);
    const int perE = (p.E + csize - 1) / csize;
    for (int e = crank * perE + warp; e < min(p.E, (crank + 1) * perE); e += kMlpWarps) {
        // (both dot products' loads are issued before either sum is reduced)
        float l = half_row_dot(p.W2 + ((size_t)head * p.E + e) * p.D, s_a, p.D, lane);
        if (p.Wres != nullptr) l += RowDot<WT>::partial(p.Wres, (size_t)head * p.E + e, s_x, p.H, lane);
        l = warp_sum(l);
        if (p.b2 != nullptr) l += __half2float(p.b2[(size_t)head * p.E + e]);
        if (lane == 0) leader[e] = l;
    }
    cluster.sync();                     // every CTA's logits have landed in the leader
    if (crank != 0) return;

    if (p.logits != nullptr)
        for (int e = threadIdx.x; e < p.E; e += blockDim.x) p.logits[(size_t)head * p.E + e] = s_logits[e];
    __syncthreads();
    if (warp == 0) {
        warp_softmax_topk(s_logits, p.E, p.K, lane, p.inds + (size_t)head * p.K, p.gates + (size_t)head * p.K);
        mirror_inds(p.mirror != nullptr ? p.mirror + (size_t)head * p.K : nullptr, p.inds + (size_t)head * p.K, p.K, lane);
    }
}

// Appendix A, sigmoid-group routing, one warp per row of given logits: sigma = sigmoid(l); a group's
// score is the sum of its two largest selection scores (sigma, plus a bias when one is given); the
// best `keep` of the `n` groups survive (ties to the lower group); top-K among the survivors by
// selection score (ties to the lower index); w = scale * sigma[inds] / (sum sigma[inds] + 1e-20):
// the weights use the raw sigmoid.  Winners are written in ascending index.
__global__ void __launch_bounds__(128) sigmoid_group_topk_rows_kernel(const float* logits, const float* bias, int T, int E, int K,
                                                                      int n, int keep, float scale, int32_t* inds, float* gates) {
    extern __shared__ float smem[];
    const unsigned full = 0xFFFFFFFFu;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int t = blockIdx.x * 4 + warp;
    if (t >= T) return;
    float* sig = smem + warp * 2 * E;          // [E] raw sigmoid
    float* sel = sig + E;                      // [E] selection score; NaN = not a candidate (any more)
    for (int e = lane; e < E; e += 32) {
        const float sg = 1.f / (1.f + expf(-logits[(size_t)t * E + e]));
        sig[e] = sg;
        sel[e] = bias != nullptr ? sg + bias[e] : sg;
    }
    __syncwarp();
    // group scores.  When the groups divide the warp, 32 / n lanes share a group: each scans its part,
    // the (largest, second largest) pairs are merged by a butterfly, and every lane of the group
    // ends up with the group's score; otherwise lane g scans group g alone.
    const int per = E / n;
    float gs = -CUDART_INF_F;
    const int lpg = 32 / n;                    // lanes per group (when n divides 32)
    const bool split = (32 % n) == 0 && (per % lpg) == 0;
    if (split || lane < n) {
        const int grp = split ? lane / lpg : lane, part = split ? lane % lpg : 0, cnt = split ? per / lpg : per;
        float m1 = -CUDART_INF_F, m2 = -CUDART_INF_F;
        for (int i = 0; i < cnt; ++i) {
            const float v = sel[grp * per + part * cnt + i];
            if (v > m1) { m2 = m1; m1 = v; } else if (v > m2) m2 = v;
        }
        if (split) {
            for (int o = 1; o < lpg; o <<= 1) {
                const float o1 = __shfl_xor_sync(full, m1, o), o2 = __shfl_xor_sync(full, m2, o);
                const float hi = fmaxf(m1, o1), lo = fminf(m1, o1);
                m2 = fmaxf(lo, fmaxf(m2, o2));
                m1 = hi;
            }
        }
        gs = m1 + m2;
    }
    int rank = 0;
    const int mygrp = split ? lane / lpg : lane;
    for (int j = 0; j < n; ++j) {
        const float gj = __shfl_sync(full, gs, split ? j * lpg : j);
        rank += (gj > gs || (gj == gs && j < mygrp)) ? 1 : 0;
    }
    const unsigned alive_l = __ballot_sync(full, (split || lane < n) && rank < keep);
    // (one bit per group)
    unsigned alive = 0u;
    for (int j = 0; j < n; ++j) alive |= ((alive_l >> (split ? j * lpg : j)) & 1u) << j;
    for (int e = lane; e < E; e += 32)
        if (!((alive >> (e / per)) & 1u)) sel[e] = __int_as_float(0x7fffffff);
    __syncwarp();
    // top-K among the survivors, ties to the lower index
    float myv = 0.f;
    int myi = 0x7FFFFFFF;
    if (E <= 256) {
        warp_topk_reg<8>(sel, E, K, lane, myv, myi);
        if (lane < K && myi != 0x7FFFFFFF) myv = sig[myi];
    } else {
        // every lane keeps its best remaining candidate, the owner of a round's winner rescans
        uint32_t key;
        int idx;
        lane_best(sel, E, lane, key, idx);
        for (int j = 0; j < K; ++j) {
            const uint32_t best = __reduce_max_sync(full, idx == 0x7FFFFFFF ? 0u : key);
            const int cand = (idx != 0x7FFFFFFF && key == best) ? idx : 0x7FFFFFFF;
            const int win = (int)__reduce_min_sync(full, (unsigned)cand);
            if (win == 0x7FFFFFFF) break;                   // fewer than K survivors
            if (lane == j) { myv = sig[win]; myi = win; }
            __syncwarp();
            if (idx == win) {
                sel[win] = __int_as_float(0x7fffffff);
                lane_best(sel, E, lane, key, idx);
            }
            __syncwarp();
        }
    }
    const float sum = warp_sum((lane < K && myi != 0x7FFFFFFF) ? myv : 0.f);
    int pos = 0;
    for (int i = 0; i < K; ++i) {
        const int oi = __shfl_sync(full, myi, i);
        pos += (oi < myi) ? 1 : 0;
    }
    if (lane < K && myi != 0x7FFFFFFF) {
        inds[(size_t)t * K + pos] = myi;
        gates[(size_t)t * K + pos] = scale * myv / (sum + 1e-20f);
    }
}

int32_t run_prerouter(const edg_layer_desc* d, const void* W_pre, const void* s, int32_t n_heads,
                      int32_t* inds, float* gates, float* logits_opt, cudaStream_t st, int shared_head,
                      int32_t* mirror) {
    int32_t rc = check_desc(d);
    if (rc != EDG_OK) return rc;
    if (!W_pre || !s || !inds || !gates || n_heads < 1 || n_heads > 65535) return EDG_E_INVAL;
    if (!aligned(W_pre, 16) || !aligned(s, 16)) return EDG_E_INVAL;
    PreParams p{W_pre, static_cast<const uint16_t*>(s), inds, gates, logits_opt, d->H, d->E, d->K, shared_head, mirror};

    const bool batched = shared_head != 0 && n_heads > 1;     // one head, several tokens: a cluster per block of tokens
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kPreCluster, batched ? (n_heads + kTokBlock - 1) / kTokBlock : n_heads, 1);
    cfg.blockDim = dim3(kPreWarps * 32, 1, 1);
    cfg.dynamicSmemBytes = (size_t)(d->E + d->H) * sizeof(float) * (batched ? kTokBlock : 1);
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = kPreCluster;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (batched) {
        static bool configured = false;
        if (!configured) {
            EDG_CUDA_TRY(cudaFuncSetAttribute(prerouter_tokens_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
            EDG_CUDA_TRY(cudaFuncSetAttribute(prerouter_tokens_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
            EDG_CUDA_TRY(cudaFuncSetAttribute(prerouter_tokens_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
            configured = true;
        }
        if (cfg.dynamicSmemBytes > 200 * 1024) return EDG_E_SHAPE;
        // an fp16 head whose rows and columns split into whole MMA tiles goes to the tensor cores
        if (d->pre_dtype == EDG_F16 && d->E % (16 * kPreCluster) == 0 && d->H % (32 * kPreWarps) == 0) {
            cfg.dynamicSmemBytes = (size_t)kTokBlock * d->E * 4 + kPreWarps * 256 * 4 + (size_t)kTokBlock * (d->H * 2 + 64);
            EDG_CUDA_TRY(cudaLaunchKernelEx(&cfg, prerouter_tokens_mma_kernel, p, (int)n_heads));
            return EDG_OK;
        }
        if (d->pre_dtype == EDG_F16) EDG_CUDA_TRY(cudaLaunchKernelEx(&cfg, prerouter_tokens_kernel<__half>, p, (int)n_heads));
        else EDG_CUDA_TRY(cudaLaunchKernelEx(&cfg, prerouter_tokens_kernel<float>, p, (int)n_heads));
        return EDG_OK;
    }
    if (d->pre_dtype == EDG_F16) EDG_CUDA_TRY(cudaLaunchKernelEx(&cfg, prerouter_kernel<__half>, p));
    else EDG_CUDA_TRY(cudaLaunchKernelEx(&cfg, prerouter_kernel<float>, p));
    return EDG_OK;
}

}  // namespace edg

extern "C" int32_t prerouter_topk(const edg_layer_desc* desc, const void* W_pre, const void* s, int32_t n_heads,
                                  int32_t* inds, float* gates, float* logits_opt, int32_t* inds_host_mirror_opt,
                                  void* stream) {
    return edg::run_prerouter(desc, W_pre, s, n_heads, inds, gates, logits_opt, static_cast<cudaStream_t>(stream), 0,
                              inds_host_mirror_opt);
}

extern "C" int32_t prerouter_topk_tokens(const edg_layer_desc* desc, const void* W_pre, const void* s, int32_t T,
                                         int32_t* inds, float* gates, float* logits_opt, void* stream) {
    return edg::run_prerouter(desc, W_pre, s, T, inds, gates, logits_opt, static_cast<cudaStream_t>(stream), 1);
}

extern "C" int32_t softmax_topk_rows(const edg_layer_desc* desc, const float* logits, int32_t T,
                                     int32_t* inds, float* gates, void* stream) {
    int32_t rc = edg::check_desc(desc);
    if (rc != EDG_OK) return rc;
    if (!logits || !inds || !gates || T < 1) return EDG_E_INVAL;
    const size_t sm = 4 * (size_t)desc->E * sizeof(float);
    edg::softmax_topk_rows_kernel<<<(T + 3) / 4, 128, sm, static_cast<cudaStream_t>(stream)>>>(
        logits, T, desc->E, desc->K, inds, gates);
    EDG_CUDA_TRY(cudaGetLastError());
    return EDG_OK;
}

extern "C" int32_t sigmoid_group_topk_rows(const float* logits, int32_t T, int32_t E, int32_t K, int32_t n_groups,
                                           int32_t keep_groups, float scale, const float* bias_opt,
                                           int32_t* inds, float* gates, void* stream) {
    if (!logits || !inds || !gates || T < 1) return EDG_E_INVAL;
    if (E < 2 || E > 1024 || n_groups < 1 || n_groups > 32 || E % n_groups != 0 || E / n_groups < 2) return EDG_E_SHAPE;
    if (keep_groups < 1 || keep_groups > n_groups || K < 1 || K > 32 || K > keep_groups * (E / n_groups)) return EDG_E_SHAPE;
    const size_t sm = 4 * 2 * (size_t)E * sizeof(float);
    edg::sigmoid_group_topk_rows_kernel<<<(T + 3) / 4, 128, sm, static_cast<cudaStream_t>(stream)>>>(
        logits, bias_opt, T, E, K, n_groups, keep_groups, scale, inds, gates);
    EDG_CUDA_TRY(cudaGetLastError());
    return EDG_OK;
}

extern "C" int32_t prerouter_mlp_topk(const edg_layer_desc* desc, const edg_mlp_head* head, const void* s,
                                      const int32_t* cur_inds, const int32_t* prev_inds, int32_t n_heads,
                                      int32_t* inds, float* gates, float* logits_opt, void* stream) {
    return edg::run_prerouter_mlp(desc, head, s, cur_inds, prev_inds, n_heads, inds, gates, logits_opt,
                                  static_cast<cudaStream_t>(stream), nullptr);
}

int32_t edg::run_prerouter_mlp(const edg_layer_desc* desc, const edg_mlp_head* head, const void* s,
                               const int32_t* cur_inds, const int32_t* prev_inds, int32_t n_heads,
                               int32_t* inds, float* gates, float* logits_opt, cudaStream_t stream, int32_t* mirror) {
    int32_t rc = edg::check_desc(desc);
    if (rc != EDG_OK) return rc;
    if (!head || !head->W1 || !head->W2 || !s || !cur_inds || !prev_inds || !inds || !gates || n_heads < 1 || n_heads > 65535)
        return EDG_E_INVAL;
    const int D = head->width;
    if (D < 8 || D > 4096 || D % 8 != 0 || desc->H % 8 != 0 || (desc->H + 2 * desc->E) % 8 != 0) return EDG_E_SHAPE;
    if (!edg::aligned(head->W1, 16) || !edg::aligned(head->W2, 16) || !edg::aligned(s, 16) ||
        (head->W_res && !edg::aligned(head->W_res, 16)))
        return EDG_E_INVAL;
    edg::MlpParams p{static_cast<const __half*>(head->W1), static_cast<const __half*>(head->b1),
                     static_cast<const __half*>(head->W2), static_cast<const __half*>(head->b2), head->W_res,
                     static_cast<const uint16_t*>(s), cur_inds, prev_inds, inds, gates, logits_opt,
                     desc->H, desc->E, desc->K, D, mirror};
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(edg::kPreCluster, n_heads, 1);
    cfg.blockDim = dim3(edg::kMlpWarps * 32, 1, 1);
    cfg.dynamicSmemBytes = (size_t)(desc->E + desc->H + D) * sizeof(float);
    cfg.stream = stream;
    if (cfg.dynamicSmemBytes > 48 * 1024) return EDG_E_SHAPE;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = edg::kPreCluster;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (desc->pre_dtype == EDG_F16) EDG_CUDA_TRY(cudaLaunchKernelEx(&cfg, edg::prerouter_mlp_kernel<__half>, p));
    else EDG_CUDA_TRY(cudaLaunchKernelEx(&cfg, edg::prerouter_mlp_kernel<float>, p));
    return EDG_OK;
}
