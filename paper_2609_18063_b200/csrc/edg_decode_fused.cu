// The batch-1 layer-step as ONE kernel (a1-a2 for the next step, a3 take, a4-a6 for this step).
//
// Work split.  Every routed expert k gets one thread-block cluster of kC = 16 CTAs; one more
// cluster evaluates the prerouter head.  Inside an expert's cluster:
//   * each CTA owns I/16 rows of gate and up and H/16 rows of down.  At kernel start one thread
//     issues bulk asynchronous copies (cp.async.bulk, completion on mbarriers) that bring the
//     CTA's whole slice of the record -- codes and (scale, zero) pairs -- into shared memory, so
//     all of the expert's bytes are in flight from the first microsecond and the down weights
//     arrive while gate/up is being computed;
//   * the rank-r LoRA projections A.x are split over the CTAs and all-gathered through
//     distributed shared memory; so is h = silu(gate) * up and the per-slice partial of A_down.h;
//   * two cluster barriers order the exchange (the first one is split into arrive / wait around
//     the gate/up GEMV so nobody waits on it).
// Across experts the reduce y = sum_k w_k o_k goes through a [K][H] fp32 scratch: each CTA writes
// its gate-weighted slice, and the last CTA to arrive for a slice (one atomic counter per slice)
// sums the K partials in ascending k, so the result does not depend on arrival order.
#include <cooperative_groups.h>

#include "edg_common.cuh"

namespace cg = cooperative_groups;

namespace edg {

constexpr int kC = 16;            // CTAs per cluster
constexpr int kFW = 8;            // warps per CTA
constexpr int kStages = 4;        // gate/up copy stages per CTA
constexpr int kMaxRank = 64;
constexpr uint32_t kSpinLimit = 1u << 22;   // bounded mbarrier polling

struct FusedParams {
    const uint8_t* pool;
    const int32_t* slots;         // [K] slots, or expert ids when table != null
    const int32_t* table;         // [E] or null
    const int32_t* experts;       // [K] or null
    const float* gates;           // [K]
    const uint16_t* x;            // [H] bf16
    edg_lora lora;
    void* y;                      // [H]
    int32_t* status;
    int32_t* counters;            // [kC], zero between launches
    float* partial;               // [K][H]
    const void* W_pre;            // [E][H] or null
    int32_t* inds_next;
    float* gates_next;
    float* logits_next;
    int H, I, E, K, group, rank, n_adapters, n_slots, pre_dtype, out_dtype;
    float sigma;
    RecordLayout L;
};

// ---------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls, raises the status word and lets the caller go on
// (the result is then wrong but flagged, and every barrier is still reached).
__device__ __forceinline__ void mbar_wait(uint64_t* bar, uint32_t parity, int32_t* status) {
    for (uint32_t i = 0; i < kSpinLimit; ++i)
        if (mbar_try_wait(bar, parity)) return;
    atomicExch(status, EDG_E_TIMEOUT);
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

__device__ __forceinline__ void store_y(void* y, int out_dtype, size_t i, float v) {
    if (out_dtype == EDG_F32) store_out<float>(static_cast<float*>(y), i, v);
    else if (out_dtype == EDG_F16) store_out<__half>(static_cast<__half*>(y), i, v);
    else store_out<bf16_t>(static_cast<bf16_t*>(y), i, v);
}

// dot of a bf16 row with the bf16 hidden state, both read from global (L2), one warp
__device__ __forceinline__ float warp_dot_bf16(const uint16_t* a, const uint16_t* b, int n, int lane) {
    float acc = 0.f;
    for (int c = lane * 8; c < n; c += 256) {
        const uint4 u = *reinterpret_cast<const uint4*>(a + c);
        const uint4 v = *reinterpret_cast<const uint4*>(b + c);
        acc = fmaf(bf16_lo(u.x), bf16_lo(v.x), acc); acc = fmaf(bf16_hi(u.x), bf16_hi(v.x), acc);
        acc = fmaf(bf16_lo(u.y), bf16_lo(v.y), acc); acc = fmaf(bf16_hi(u.y), bf16_hi(v.y), acc);
        acc = fmaf(bf16_lo(u.z), bf16_lo(v.z), acc); acc = fmaf(bf16_hi(u.z), bf16_hi(v.z), acc);
        acc = fmaf(bf16_lo(u.w), bf16_lo(v.w), acc); acc = fmaf(bf16_hi(u.w), bf16_hi(v.w), acc);
    }
    return warp_sum(acc);
}

// shared-memory carve-up of an expert CTA (byte offsets), identical on host and device
struct FusedSmem {
    uint32_t bars, s_u, s_h, s_ud_part, s_ud, s_gu, s_o, flag;
    uint32_t c_gate, c_up, z_gate, z_up, c_down, z_down, total;
};
__host__ __device__ inline FusedSmem fused_smem(int H, int I, int group) {
    FusedSmem S;
    const uint32_t rows_gu = I / kC, rows_d = H / kC;
    uint32_t o = 0;
    S.bars = o;       o += 8 * (kStages + 1);
    o = (o + 15) / 16 * 16;
    S.s_u = o;        o += 2 * kMaxRank * 4;
    S.s_h = o;        o += (uint32_t)I * 4;
    S.s_ud_part = o;  o += kC * kMaxRank * 4;
    S.s_ud = o;       o += kMaxRank * 4;
    S.s_gu = o;       o += 2 * rows_gu * 4;
    S.s_o = o;        o += rows_d * 4;
    S.flag = o;       o += 16;
    o = (o + 127) / 128 * 128;
    S.c_gate = o;     o += rows_gu * (uint32_t)H / 2;
    S.c_up = o;       o += rows_gu * (uint32_t)H / 2;
    S.z_gate = o;     o += rows_gu * (uint32_t)(H / group) * 4;
    S.z_up = o;       o += rows_gu * (uint32_t)(H / group) * 4;
    S.c_down = o;     o += rows_d * (uint32_t)I / 2;
    S.z_down = o;     o += rows_d * (uint32_t)(I / group) * 4;
    S.total = o;
    return S;
}

// ---------------------------------------------------------------- prerouter role (one cluster)

template <typename WT>
__device__ __forceinline__ float pre_row_dot(const void* W, size_t row, const float* sx, int H, int lane);
template <>
__device__ __forceinline__ float pre_row_dot<__half>(const void* W, size_t row, const float* sx, int H, int lane) {
    const uint4* wp = reinterpret_cast<const uint4*>(static_cast<const __half*>(W) + row * H);
    float acc = 0.f;
#pragma unroll 4
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
    return warp_sum(acc);
}
template <>
__device__ __forceinline__ float pre_row_dot<float>(const void* W, size_t row, const float* sx, int H, int lane) {
    const uint4* wp = reinterpret_cast<const uint4*>(static_cast<const float*>(W) + row * H);
    float acc = 0.f;
#pragma unroll 4
    for (int c = lane; c < H / 4; c += 32) {
        const uint4 w = ld_stream16(wp + c);
        const float* x = sx + c * 4;
        acc = fmaf(__uint_as_float(w.x), x[0], acc); acc = fmaf(__uint_as_float(w.y), x[1], acc);
        acc = fmaf(__uint_as_float(w.z), x[2], acc); acc = fmaf(__uint_as_float(w.w), x[3], acc);
    }
    return warp_sum(acc);
}

__device__ void prerouter_role(const FusedParams& p, uint8_t* smem, int crank) {
    cg::cluster_group cluster = cg::this_cluster();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float* s_logits = reinterpret_cast<float*>(smem);     // [E]
    float* s_x = s_logits + p.E;                          // [H]
    cluster_arrive();                                     // (#0) every CTA of the cluster is running ...
    for (int i = threadIdx.x; i < p.H; i += blockDim.x) s_x[i] = bf16_bits_to_float(p.x[i]);
    __syncthreads();
    cluster_wait();                                       // ... before anyone writes into a peer's shared memory
    float* leader = cluster.map_shared_rank(s_logits, 0);
    const int per = (p.E + kC - 1) / kC;
    const int e0 = crank * per, e1 = min(p.E, e0 + per);
    for (int e = e0 + warp; e < e1; e += kFW) {
        const float l = p.pre_dtype == EDG_F16 ? pre_row_dot<__half>(p.W_pre, e, s_x, p.H, lane)
                                               : pre_row_dot<float>(p.W_pre, e, s_x, p.H, lane);
        if (lane == 0) leader[e] = l;
    }
    cluster_arrive();
    cluster_wait();
    if (crank != 0) return;
    if (p.logits_next != nullptr)
        for (int e = threadIdx.x; e < p.E; e += blockDim.x) p.logits_next[e] = s_logits[e];
    __syncthreads();
    if (warp == 0) warp_softmax_topk(s_logits, p.E, p.K, lane, p.inds_next, p.gates_next);
}

// ---------------------------------------------------------------- the fused kernel
// NCH = H / 1024 (chunks of a gate/up row per lane), LPR_I = I / 32 (lanes per down row).

template <int NCH, int LPR_I>
__global__ void __launch_bounds__(kFW * 32, 1) fused_layer_kernel(FusedParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank();
    const int k = blockIdx.x / kC;                 // cluster index: expert position, or K = prerouter
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;

    if (k == p.K) { prerouter_role(p, smem, crank); return; }

    const FusedSmem S = fused_smem(p.H, p.I, p.group);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S.bars);
    float* s_u = reinterpret_cast<float*>(smem + S.s_u);            // [2][kMaxRank]
    float* s_h = reinterpret_cast<float*>(smem + S.s_h);            // [I]
    float* s_ud_part = reinterpret_cast<float*>(smem + S.s_ud_part);// [kC][kMaxRank]
    float* s_ud = reinterpret_cast<float*>(smem + S.s_ud);          // [kMaxRank]
    float* s_gu = reinterpret_cast<float*>(smem + S.s_gu);          // [2][rows_gu]
    float* s_o = reinterpret_cast<float*>(smem + S.s_o);            // [rows_d]
    int* s_flag = reinterpret_cast<int*>(smem + S.flag);

    const int rows_gu = p.I / kC, rows_d = p.H / kC;
    const int n0_gu = crank * rows_gu, n0_d = crank * rows_d;
    const int r = p.rank;

    // ---- a3: take.  The decision is the same in every CTA of the cluster.
    int slot = p.slots[k];
    int expert = p.table != nullptr ? slot : (p.experts != nullptr ? p.experts[k] : 0);
    if (p.table != nullptr) slot = (slot >= 0 && slot < p.E) ? p.table[slot] : -1;
    int ad = 0;
    if (r > 0 && p.n_adapters != 1) ad = (expert >= 0 && expert < p.E) ? expert : -1;
    const bool valid = slot >= 0 && slot < p.n_slots && ad >= 0;

    if (valid) {
        cluster_arrive();                 // (#0) a peer's shared memory may be written only once it runs
        const uint8_t* rec = p.pool + (size_t)slot * p.L.bytes;
        const int row_b = p.H / 2, grp_b = (p.H / p.group) * 4;
        const int rs = rows_gu / kStages;                            // gate/up rows per stage

        // ---- issue every copy of this CTA's slice
        if (tid == 0) {
            for (int s = 0; s <= kStages; ++s) mbar_init(&bars[s], 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            for (int s = 0; s < kStages; ++s) {
                const int lr = s * rs;                               // local row
                const size_t gr = (size_t)(n0_gu + lr);              // row in the expert
                mbar_expect_tx(&bars[s], 2u * rs * (row_b + grp_b));
                bulk_g2s(smem + S.c_gate + lr * row_b, rec + p.L.codes_gate + gr * row_b, rs * row_b, &bars[s]);
                bulk_g2s(smem + S.c_up + lr * row_b, rec + p.L.codes_up + gr * row_b, rs * row_b, &bars[s]);
                bulk_g2s(smem + S.z_gate + lr * grp_b, rec + p.L.sz_gate + gr * grp_b, rs * grp_b, &bars[s]);
                bulk_g2s(smem + S.z_up + lr * grp_b, rec + p.L.sz_up + gr * grp_b, rs * grp_b, &bars[s]);
            }
            const int drow_b = p.I / 2, dgrp_b = (p.I / p.group) * 4;
            mbar_expect_tx(&bars[kStages], (uint32_t)rows_d * (drow_b + dgrp_b));
            bulk_g2s(smem + S.c_down, rec + p.L.codes_down + (size_t)n0_d * drow_b, rows_d * drow_b, &bars[kStages]);
            bulk_g2s(smem + S.z_down, rec + p.L.sz_down + (size_t)n0_d * dgrp_b, rows_d * dgrp_b, &bars[kStages]);
        }

        // ---- hidden state -> pre-scaled registers (each lane owns NCH chunks of 32)
        float xs[NCH][32], xsum[NCH];
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const uint4* xp = reinterpret_cast<const uint4*>(p.x + (lane + 32 * i) * 32);
            float xv[32];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint4 v = xp[q];
                xv[q * 8 + 0] = bf16_lo(v.x); xv[q * 8 + 1] = bf16_hi(v.x);
                xv[q * 8 + 2] = bf16_lo(v.y); xv[q * 8 + 3] = bf16_hi(v.y);
                xv[q * 8 + 4] = bf16_lo(v.z); xv[q * 8 + 5] = bf16_hi(v.z);
                xv[q * 8 + 6] = bf16_lo(v.w); xv[q * 8 + 7] = bf16_hi(v.w);
            }
            xsum[i] = scale_chunk(xv, xs[i]);
        }

        cluster_wait();                   // (#0)
        // ---- LoRA: this CTA's share of the 2r rows of A_gate / A_up, broadcast to the cluster
        if (r > 0) {
            const int per = (2 * r + kC - 1) / kC;
            for (int q = crank * per + warp; q < min(2 * r, (crank + 1) * per); q += kFW) {
                const int proj = q / r, j = q % r;
                const uint16_t* A = reinterpret_cast<const uint16_t*>(proj ? p.lora.A_up : p.lora.A_gate) + ((size_t)ad * r + j) * p.H;
                const float v = warp_dot_bf16(A, p.x, p.H, lane);
                if (lane < kC) cluster.map_shared_rank(s_u, lane)[proj * kMaxRank + j] = v;
            }
        }
        __syncthreads();                  // barriers initialised before anyone polls them
        cluster_arrive();                 // (#1) my A.x values are out; wait for the others later

        // ---- gate/up GEMV over this CTA's rows, stage by stage as the copies land
        {
            const int groups = p.H / p.group;
            for (int lr = warp; lr < rows_gu; lr += kFW) {
                mbar_wait(&bars[lr / rs], 0, p.status);
                float ag = 0.f, au = 0.f;
#pragma unroll
                for (int i = 0; i < NCH; ++i) {
                    const int c = lane + 32 * i;
                    const uint4 wg = *reinterpret_cast<const uint4*>(smem + S.c_gate + lr * row_b + c * 16);
                    const uint4 wu = *reinterpret_cast<const uint4*>(smem + S.c_up + lr * row_b + c * 16);
                    const uint32_t zg = *reinterpret_cast<const uint32_t*>(smem + S.z_gate + (lr * groups + (c * 32) / p.group) * 4);
                    const uint32_t zu = *reinterpret_cast<const uint32_t*>(smem + S.z_up + (lr * groups + (c * 32) / p.group) * 4);
                    ag += chunk_affine(chunk_dot(wg, xs[i]), xsum[i], zg);
                    au += chunk_affine(chunk_dot(wu, xs[i]), xsum[i], zu);
                }
                ag = warp_sum(ag);
                au = warp_sum(au);
                if (lane == 0) { s_gu[lr] = ag * kUnscale; s_gu[rows_gu + lr] = au * kUnscale; }
            }
        }
        __syncthreads();
        cluster_wait();                   // (#1) every CTA's A.x has landed in s_u

        // ---- finish gate/up: LoRA B, SiLU, product; all-gather h and the partial of A_down . h
        if (warp == 0) {
            float hval = 0.f;
            if (lane < rows_gu) {
                float g = s_gu[lane], u = s_gu[rows_gu + lane];
                if (r > 0) {
                    const size_t bo = ((size_t)ad * p.I + n0_gu + lane) * r;
                    const uint16_t* Bg = reinterpret_cast<const uint16_t*>(p.lora.B_gate) + bo;
                    const uint16_t* Bu = reinterpret_cast<const uint16_t*>(p.lora.B_up) + bo;
                    float dg = 0.f, du = 0.f;
                    for (int j = 0; j < r; ++j) {
                        dg = fmaf(bf16_bits_to_float(Bg[j]), s_u[j], dg);
                        du = fmaf(bf16_bits_to_float(Bu[j]), s_u[kMaxRank + j], du);
                    }
                    g = fmaf(p.sigma, dg, g);
                    u = fmaf(p.sigma, du, u);
                }
                hval = silu_f(g) * u;
                for (int c = 0; c < kC; ++c) cluster.map_shared_rank(s_h, c)[n0_gu + lane] = hval;
            }
            for (int j = 0; j < r; ++j) {
                const uint16_t* Ad = reinterpret_cast<const uint16_t*>(p.lora.A_down) + ((size_t)ad * r + j) * p.I + n0_gu;
                float v = lane < rows_gu ? bf16_bits_to_float(Ad[lane]) * hval : 0.f;
                v = warp_sum(v);
                if (lane < kC) cluster.map_shared_rank(s_ud_part, lane)[crank * kMaxRank + j] = v;
            }
        }
        cluster_arrive();                 // (#2)
        cluster_wait();                   // h and the A_down partials of the whole expert are here

        // ---- down GEMV over this CTA's H/16 output rows
        if (tid < r) {
            float v = 0.f;
            for (int c = 0; c < kC; ++c) v += s_ud_part[c * kMaxRank + tid];
            s_ud[tid] = v;
        }
        constexpr int RPW = 32 / LPR_I;
        const int sub = lane % LPR_I, rsub = lane / LPR_I;
        float hs[32];
        float hsum;
        {
            float hv[32];
            const float4* hp = reinterpret_cast<const float4*>(s_h + sub * 32);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const float4 v = hp[q];
                hv[q * 4 + 0] = v.x; hv[q * 4 + 1] = v.y; hv[q * 4 + 2] = v.z; hv[q * 4 + 3] = v.w;
            }
            hsum = scale_chunk(hv, hs);
        }
        __syncthreads();                  // s_ud ready
        mbar_wait(&bars[kStages], 0, p.status);
        const float gate_k = p.gates[k];
        const int drow_b = p.I / 2, dgroups = p.I / p.group;
        for (int lr = warp * RPW + rsub; lr < rows_d; lr += kFW * RPW) {
            const uint4 wd = *reinterpret_cast<const uint4*>(smem + S.c_down + lr * drow_b + sub * 16);
            const uint32_t zd = *reinterpret_cast<const uint32_t*>(smem + S.z_down + (lr * dgroups + (sub * 32) / p.group) * 4);
            float acc = chunk_affine(chunk_dot(wd, hs), hsum, zd);
            acc = group_sum<LPR_I>(acc);
            if (sub == 0) {
                float o = acc * kUnscale;
                if (r > 0) {
                    const uint16_t* Bd = reinterpret_cast<const uint16_t*>(p.lora.B_down) + ((size_t)ad * p.H + n0_d + lr) * r;
                    float dd = 0.f;
                    for (int j = 0; j < r; ++j) dd = fmaf(bf16_bits_to_float(Bd[j]), s_ud[j], dd);
                    o = fmaf(p.sigma, dd, o);
                }
                s_o[lr] = gate_k * o;
            }
        }
        __syncthreads();
    } else {
        if (tid == 0) atomicExch(p.status, EDG_E_RANGE);
        for (int i = tid; i < rows_d; i += blockDim.x) s_o[i] = 0.f;     // a skipped expert contributes nothing
        __syncthreads();
    }

    // ---- a6: publish this expert's gate-weighted slice; the last arriver sums the K partials
    for (int i = tid; i < rows_d; i += blockDim.x) p.partial[(size_t)k * p.H + n0_d + i] = s_o[i];
    __threadfence();
    __syncthreads();
    if (tid == 0) s_flag[0] = (atomicAdd(&p.counters[crank], 1) == p.K - 1) ? 1 : 0;
    __syncthreads();
    if (s_flag[0]) {
        __threadfence();
        for (int i = tid; i < rows_d; i += blockDim.x) {
            float yv = 0.f;
            for (int kk = 0; kk < p.K; ++kk) yv += __ldcg(&p.partial[(size_t)kk * p.H + n0_d + i]);
            store_y(p.y, p.out_dtype, (size_t)n0_d + i, yv);
        }
        if (tid == 0) p.counters[crank] = 0;
    }
}

// ---------------------------------------------------------------- host side

bool fused_supported(const edg_layer_desc& d) {
    if (!((d.H == 1024 || d.H == 2048) && (d.I == 256 || d.I == 512))) return false;
    if ((d.I / kC) % kStages != 0 || d.I / kC > 32) return false;
    return fused_smem(d.H, d.I, d.group).total <= 200 * 1024;
}

template <int NCH, int LPR_I>
static cudaError_t launch_fused(const FusedParams& p, bool with_pre, size_t smem, cudaStream_t st) {
    auto kern = fused_layer_kernel<NCH, LPR_I>;
    static bool configured = false;       // per-process, per-instantiation one-time attributes
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((p.K + (with_pre ? 1 : 0)) * kC, 1, 1);
    cfg.blockDim = dim3(kFW * 32, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = kC;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, p);
}

// One fused launch for a batch-1 layer-step.  W_pre may be null (no prediction).
int32_t run_fused_layer(const edg_layer_desc* d, const void* slot_pool, const int32_t* slots, const int32_t* table,
                        const int32_t* experts, const float* gates, const void* x, const edg_lora* lora, void* y,
                        const void* W_pre, int32_t* inds_next, float* gates_next, float* logits_next,
                        void* workspace, cudaStream_t st) {
    const bool has_lora = lora != nullptr && d->rank > 0;
    FusedParams p{};
    p.pool = static_cast<const uint8_t*>(slot_pool);
    p.slots = slots; p.table = table; p.experts = experts; p.gates = gates;
    p.x = static_cast<const uint16_t*>(x);
    if (has_lora) p.lora = *lora;
    p.y = y;
    const WorkspaceLayout W = workspace_layout(*d, 1);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    p.status = reinterpret_cast<int32_t*>(ws + W.ctrl);
    p.counters = reinterpret_cast<int32_t*>(ws + W.ctrl + 64);
    p.partial = reinterpret_cast<float*>(ws + W.partial);
    p.W_pre = W_pre; p.inds_next = inds_next; p.gates_next = gates_next; p.logits_next = logits_next;
    p.H = d->H; p.I = d->I; p.E = d->E; p.K = d->K; p.group = d->group;
    p.rank = has_lora ? d->rank : 0;
    p.n_adapters = d->n_adapters; p.n_slots = d->n_slots;
    p.pre_dtype = d->pre_dtype; p.out_dtype = d->out_dtype;
    p.sigma = d->lora_scale;
    p.L = record_layout(d->H, d->I, d->group);
    size_t smem = fused_smem(d->H, d->I, d->group).total;
    const size_t pre_smem = (size_t)(d->E + d->H) * sizeof(float);
    if (W_pre != nullptr && pre_smem > smem) smem = pre_smem;
    const bool with_pre = W_pre != nullptr;
    cudaError_t e;
    if (d->H == 2048 && d->I == 512) e = launch_fused<2, 16>(p, with_pre, smem, st);
    else if (d->H == 2048 && d->I == 256) e = launch_fused<2, 8>(p, with_pre, smem, st);
    else if (d->H == 1024 && d->I == 512) e = launch_fused<1, 16>(p, with_pre, smem, st);
    else if (d->H == 1024 && d->I == 256) e = launch_fused<1, 8>(p, with_pre, smem, st);
    else return EDG_E_SHAPE;
    EDG_CUDA_TRY(e);
    return EDG_OK;
}

}  // namespace edg
