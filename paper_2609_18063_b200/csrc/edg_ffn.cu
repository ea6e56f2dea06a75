// a4-a6: int4 group-quantised SwiGLU expert FFN with the unmerged LoRA delta and the
// gate-weighted reduce (Sec. 3.1 "Math contract", Sec. 3.3, Appendix A weights).
//
// Batch-1 decode is bound by streaming the int4 codes from HBM once; the kernels are fused
// dequant GEMVs: 128-bit coalesced code loads, exact int4->fp32 by masking (see edg_common.cuh),
// fp32 accumulation, a warp-shuffle reduction per output row, gate*up*SiLU fused before down.
#include "edg_common.cuh"

namespace edg {

int32_t run_grouped(const edg_layer_desc* d, const void* slot_pool, int32_t T, const int32_t* slots, const int32_t* table,
                    const int32_t* experts, const float* gates, const void* x, const edg_lora* lora, void* y,
                    void* workspace, cudaStream_t st);

struct FfnParams {
    const uint8_t* pool;        // slot records of one layer
    const int32_t* slots;       // [T][K] slot per routed expert, or expert ids when `table` is set
    const int32_t* table;       // optional slot table [E] (take): slot = table[slots[.]]
    const int32_t* experts;     // [T][K] expert ids (per-expert adapters) or null
    const float* gates;         // [T][K]
    const uint16_t* x;          // [T][H] bf16
    edg_lora lora;
    void* y;                    // [T][H]
    int32_t* status;            // device status word
    float* u_gu;                // [T][n_sets][2][rank]
    float* h;                   // [T][K][I]
    float* u_d;                 // [T][K][rank]
    int H, I, E, K, group, rank, n_adapters, n_slots;
    float sigma;
    RecordLayout L;
};

__device__ __forceinline__ int resolve_slot(const FfnParams& p, int tk) {
    int s = p.slots[tk];
    if (p.table != nullptr) {
        if (s < 0 || s >= p.E) return -1;
        s = p.table[s];
    }
    return (s < 0 || s >= p.n_slots) ? -1 : s;
}

__device__ __forceinline__ int resolve_adapter(const FfnParams& p, int tk) {
    if (p.n_adapters == 1) return 0;
    const int e = p.table != nullptr ? p.slots[tk] : p.experts[tk];
    return (e < 0 || e >= p.E) ? -1 : e;
}

// ---------------------------------------------------------------- rank-r projections u = A . v
// One warp per 8 outputs of one token (or pair): the vector is loaded once per sweep and used for the
// 8 rows of A, whose loads are in flight together.
//   phase 0: v = x (bf16), outputs u_gu[t][set][proj][j];  phase 1: v = h[t][k] (float), outputs u_d[t][k][j].
__global__ void __launch_bounds__(256) lora_a_kernel(FfnParams p, int phase, int n_sets) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.y;
    const int r = p.rank;
    const int g8 = (r + 7) / 8;                                  // groups of 8 outputs per (set, proj) or per pair
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (phase == 0) {
        if (warp >= n_sets * 2 * g8) return;
        const int jg = warp % g8, proj = (warp / g8) & 1, set = warp / (2 * g8);
        const int ad = p.n_adapters == 1 ? 0 : resolve_adapter(p, t * p.K + set);
        if (ad < 0) { if (lane == 0) atomicExch(p.status, EDG_E_RANGE); return; }
        const uint16_t* A = reinterpret_cast<const uint16_t*>(proj ? p.lora.A_up : p.lora.A_gate) + ((size_t)ad * r + jg * 8) * p.H;
        const int nj = min(8, r - jg * 8);
        const uint16_t* xv = p.x + (size_t)t * p.H;
        for (int c = lane * 8; c < p.H; c += 256) {
            const uint4 b = *reinterpret_cast<const uint4*>(xv + c);
            uint4 a[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) a[u] = *reinterpret_cast<const uint4*>(A + (size_t)min(u, nj - 1) * p.H + c);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                acc[u] = fmaf(bf16_lo(a[u].x), bf16_lo(b.x), acc[u]); acc[u] = fmaf(bf16_hi(a[u].x), bf16_hi(b.x), acc[u]);
                acc[u] = fmaf(bf16_lo(a[u].y), bf16_lo(b.y), acc[u]); acc[u] = fmaf(bf16_hi(a[u].y), bf16_hi(b.y), acc[u]);
                acc[u] = fmaf(bf16_lo(a[u].z), bf16_lo(b.z), acc[u]); acc[u] = fmaf(bf16_hi(a[u].z), bf16_hi(b.z), acc[u]);
                acc[u] = fmaf(bf16_lo(a[u].w), bf16_lo(b.w), acc[u]); acc[u] = fmaf(bf16_hi(a[u].w), bf16_hi(b.w), acc[u]);
            }
        }
        float* out = p.u_gu + (((size_t)t * n_sets + set) * 2 + proj) * r + jg * 8;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float v = warp_sum(acc[u]);
            if (lane == 0 && u < nj) out[u] = v;
        }
    } else {
        if (warp >= p.K * g8) return;
        const int jg = warp % g8, k = warp / g8;
        const int ad = resolve_adapter(p, t * p.K + k);
        if (ad < 0) { if (lane == 0) atomicExch(p.status, EDG_E_RANGE); return; }
        const uint16_t* A = reinterpret_cast<const uint16_t*>(p.lora.A_down) + ((size_t)ad * r + jg * 8) * p.I;
        const int nj = min(8, r - jg * 8);
        const float* hv = p.h + ((size_t)t * p.K + k) * p.I;
        for (int c = lane * 8; c < p.I; c += 256) {
            const float4 h0 = *reinterpret_cast<const float4*>(hv + c);
            const float4 h1 = *reinterpret_cast<const float4*>(hv + c + 4);
            uint4 a[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) a[u] = *reinterpret_cast<const uint4*>(A + (size_t)min(u, nj - 1) * p.I + c);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                acc[u] = fmaf(bf16_lo(a[u].x), h0.x, acc[u]); acc[u] = fmaf(bf16_hi(a[u].x), h0.y, acc[u]);
                acc[u] = fmaf(bf16_lo(a[u].y), h0.z, acc[u]); acc[u] = fmaf(bf16_hi(a[u].y), h0.w, acc[u]);
                acc[u] = fmaf(bf16_lo(a[u].z), h1.x, acc[u]); acc[u] = fmaf(bf16_hi(a[u].z), h1.y, acc[u]);
                acc[u] = fmaf(bf16_lo(a[u].w), h1.z, acc[u]); acc[u] = fmaf(bf16_hi(a[u].w), h1.w, acc[u]);
            }
        }
        float* out = p.u_d + ((size_t)t * p.K + k) * r + jg * 8;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float v = warp_sum(acc[u]);
            if (lane == 0 && u < nj) out[u] = v;
        }
    }
}

// sum_j B[row][j] * u[j]  (B bf16 [.][rank]); 16-byte loads when the row allows it, so the
// loads of a row are independent of one another
__device__ __forceinline__ float lora_b_dot(const uint16_t* Brow, const float* u, int r) {
    float acc = 0.f;
    if ((r & 7) == 0) {
        for (int j = 0; j < r; j += 8) {
            const uint4 b = *reinterpret_cast<const uint4*>(Brow + j);
            acc = fmaf(bf16_lo(b.x), u[j + 0], acc); acc = fmaf(bf16_hi(b.x), u[j + 1], acc);
            acc = fmaf(bf16_lo(b.y), u[j + 2], acc); acc = fmaf(bf16_hi(b.y), u[j + 3], acc);
            acc = fmaf(bf16_lo(b.z), u[j + 4], acc); acc = fmaf(bf16_hi(b.z), u[j + 5], acc);
            acc = fmaf(bf16_lo(b.w), u[j + 6], acc); acc = fmaf(bf16_hi(b.w), u[j + 7], acc);
        }
    } else {
        for (int j = 0; j < r; ++j) acc = fmaf(bf16_bits_to_float(Brow[j]), u[j], acc);
    }
    return acc;
}

// ---------------------------------------------------------------- gate/up -> h
// A row of H codes is H/32 chunks of 16 bytes.  LPR lanes share a row (LPR = min(32, H/32));
// each lane owns NCH chunks of the row (NCH = H/32/LPR) and keeps their pre-scaled activations
// in registers for every row it visits.  A warp pass covers RPW = 32/LPR rows.
constexpr int kWarps = 8;
constexpr int kPasses = 2;

template <int LPR, int NCH>
__global__ void __launch_bounds__(kWarps * 32) gate_up_kernel(FfnParams p) {
    constexpr int RPW = 32 / LPR;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane % LPR, rsub = lane / LPR;
    const int k = blockIdx.y, t = blockIdx.z, tk = t * p.K + k;
    __shared__ float su[2][64];

    const int slot = resolve_slot(p, tk);
    const int ad = p.rank > 0 ? resolve_adapter(p, tk) : 0;
    if (slot < 0 || ad < 0) { if (threadIdx.x == 0) atomicExch(p.status, EDG_E_RANGE); return; }
    const uint8_t* rec = p.pool + (size_t)slot * p.L.bytes;

    if (p.rank > 0 && threadIdx.x < 2 * p.rank) {
        const int n_sets = p.n_adapters == 1 ? 1 : p.K;
        const int set = p.n_adapters == 1 ? 0 : k;
        const int proj = threadIdx.x / p.rank, j = threadIdx.x % p.rank;
        su[proj][j] = p.u_gu[(((size_t)t * n_sets + set) * 2 + proj) * p.rank + j];
    }

    float xs[NCH][32], xsum[NCH];
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int c = sub + LPR * i;
        const uint4* xp = reinterpret_cast<const uint4*>(p.x + (size_t)t * p.H + c * 32);
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
    __syncthreads();

    const int row0 = blockIdx.x * (kWarps * RPW * kPasses);
    uint4 cg[kPasses][NCH], cu[kPasses][NCH];
    uint32_t zg[kPasses][NCH], zu[kPasses][NCH];
#pragma unroll
    for (int ps = 0; ps < kPasses; ++ps) {
        const int n = row0 + (ps * kWarps + warp) * RPW + rsub;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int c = sub + LPR * i;
            const size_t co = code_off(p.H, n, c);
            const size_t so = sz_off(p.H, p.group, n, (c * 32) / p.group);
            cg[ps][i] = ld_stream16(rec + p.L.codes_gate + co);
            cu[ps][i] = ld_stream16(rec + p.L.codes_up + co);
            zg[ps][i] = ld_stream4(rec + p.L.sz_gate + so);
            zu[ps][i] = ld_stream4(rec + p.L.sz_up + so);
        }
    }
#pragma unroll
    for (int ps = 0; ps < kPasses; ++ps) {
        const int n = row0 + (ps * kWarps + warp) * RPW + rsub;
        float ag = 0.f, au = 0.f;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            ag += chunk_affine(chunk_dot(cg[ps][i], xs[i]), xsum[i], zg[ps][i]);
            au += chunk_affine(chunk_dot(cu[ps][i], xs[i]), xsum[i], zu[ps][i]);
        }
        ag = group_sum<LPR>(ag);
        au = group_sum<LPR>(au);
        if (sub == 0) {
            float g = ag * kUnscale, u = au * kUnscale;
            if (p.rank > 0) {
                const size_t bo = ((size_t)ad * p.I + n) * p.rank;
                g = fmaf(p.sigma, lora_b_dot(reinterpret_cast<const uint16_t*>(p.lora.B_gate) + bo, su[0], p.rank), g);
                u = fmaf(p.sigma, lora_b_dot(reinterpret_cast<const uint16_t*>(p.lora.B_up) + bo, su[1], p.rank), u);
            }
            p.h[(size_t)tk * p.I + n] = silu_f(g) * u;
        }
    }
}

// ---------------------------------------------------------------- down + gate-weighted reduce -> y
// Each CTA owns kWarps * RPW output rows and walks the K experts in the order given, so the
// reduce y = sum_k w_k o_k is a fixed-order fp32 sum with no atomics.
template <int LPR, int NCH, typename OutT>
__global__ void __launch_bounds__(kWarps * 32) down_kernel(FfnParams p) {
    constexpr int RPW = 32 / LPR;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane % LPR, rsub = lane / LPR;
    const int t = blockIdx.z;
    const int n = blockIdx.x * (kWarps * RPW) + warp * RPW + rsub;
    extern __shared__ float sud[];            // [K][rank]

    for (int i = threadIdx.x; i < p.K * p.rank; i += blockDim.x) sud[i] = p.u_d[(size_t)t * p.K * p.rank + i];
    __syncthreads();

    float yv = 0.f;
    for (int k = 0; k < p.K; ++k) {
        const int tk = t * p.K + k;
        const int slot = resolve_slot(p, tk);
        const int ad = p.rank > 0 ? resolve_adapter(p, tk) : 0;
        if (slot < 0 || ad < 0) { if (threadIdx.x == 0) atomicExch(p.status, EDG_E_RANGE); continue; }
        const uint8_t* rec = p.pool + (size_t)slot * p.L.bytes;
        uint4 cd[NCH];
        uint32_t zd[NCH];
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int c = sub + LPR * i;
            cd[i] = ld_stream16(rec + p.L.codes_down + down_code_off(p.H, p.I, n, c));
            zd[i] = ld_stream4(rec + p.L.sz_down + down_sz_off(p.H, p.I, p.group, n, (c * 32) / p.group));
        }
        float acc = 0.f;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            const int c = sub + LPR * i;
            const float4* hp = reinterpret_cast<const float4*>(p.h + (size_t)tk * p.I + c * 32);
            float hv[32], hs[32];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const float4 v = hp[q];
                hv[q * 4 + 0] = v.x; hv[q * 4 + 1] = v.y; hv[q * 4 + 2] = v.z; hv[q * 4 + 3] = v.w;
            }
            const float hsum = scale_chunk(hv, hs);
            acc += chunk_affine(chunk_dot(cd[i], hs), hsum, zd[i]);
        }
        acc = group_sum<LPR>(acc);
        if (sub == 0) {
            float o = acc * kUnscale;
            if (p.rank > 0)
                o = fmaf(p.sigma, lora_b_dot(reinterpret_cast<const uint16_t*>(p.lora.B_down) + ((size_t)ad * p.H + n) * p.rank,
                                             sud + k * p.rank, p.rank), o);
            yv = fmaf(p.gates[tk], o, yv);
        }
    }
    if (sub == 0) store_out<OutT>(reinterpret_cast<OutT*>(p.y), (size_t)t * p.H + n, yv);
}

// ---------------------------------------------------------------- host dispatch

template <int LPR, int NCH>
static void launch_gate_up(const FfnParams& p, int T, cudaStream_t st) {
    constexpr int rows = kWarps * (32 / LPR) * kPasses;
    dim3 grid(p.I / rows, p.K, T);
    gate_up_kernel<LPR, NCH><<<grid, kWarps * 32, 0, st>>>(p);
}

template <int LPR, int NCH>
static void launch_down(const FfnParams& p, int T, int out_dtype, cudaStream_t st) {
    constexpr int rows = kWarps * (32 / LPR);
    dim3 grid(p.H / rows, 1, T);
    const size_t sm = (size_t)p.K * (p.rank > 0 ? p.rank : 1) * sizeof(float);
    if (out_dtype == EDG_F32) down_kernel<LPR, NCH, float><<<grid, kWarps * 32, sm, st>>>(p);
    else if (out_dtype == EDG_F16) down_kernel<LPR, NCH, __half><<<grid, kWarps * 32, sm, st>>>(p);
    else down_kernel<LPR, NCH, bf16_t><<<grid, kWarps * 32, sm, st>>>(p);
}

#define EDG_DISPATCH_CHUNKS(chunks, FN, ...)                         \
    switch (chunks) {                                                \
        case 4:   FN<4, 1>(__VA_ARGS__); break;                      \
        case 8:   FN<8, 1>(__VA_ARGS__); break;                      \
        case 16:  FN<16, 1>(__VA_ARGS__); break;                     \
        case 32:  FN<32, 1>(__VA_ARGS__); break;                     \
        case 64:  FN<32, 2>(__VA_ARGS__); break;                     \
        case 128: FN<32, 4>(__VA_ARGS__); break;                     \
        default: return EDG_E_SHAPE;                                 \
    }

// Runs a4-a6 for T tokens.  `table` non-null: `slots` holds expert ids to be mapped (device take).
int32_t run_ffn(const edg_layer_desc* d, const void* slot_pool, int32_t T, const int32_t* slots,
                const int32_t* table, const int32_t* experts, const float* gates, const void* x,
                const edg_lora* lora, void* y, void* workspace, size_t workspace_bytes, cudaStream_t st) {
    int32_t rc = check_desc(d);
    if (rc != EDG_OK) return rc;
    if (!slot_pool || !slots || !gates || !x || !y || !workspace || T < 1 || T > 65535) return EDG_E_INVAL;
    if (!aligned(slot_pool, 256) || !aligned(x, 16) || !aligned(y, 16)) return EDG_E_INVAL;
    const WorkspaceLayout W = workspace_layout(*d, T);
    if (workspace_bytes < W.bytes || !aligned(workspace, 256)) return EDG_E_WORKSPACE;
    const bool has_lora = lora != nullptr && d->rank > 0;
    if (has_lora) {
        if (!lora->A_gate || !lora->B_gate || !lora->A_up || !lora->B_up || !lora->A_down || !lora->B_down) return EDG_E_INVAL;
        if (d->n_adapters != 1 && table == nullptr && experts == nullptr) return EDG_E_INVAL;
    }

    // batch-1 decode on the shapes the fused kernel covers: one launch for the whole FFN
    if (T == 1 && fused_supported(*d))
        return run_fused_layer(d, slot_pool, slots, table, experts, gates, x, has_lora ? lora : nullptr, y,
                               nullptr, nullptr, nullptr, nullptr, workspace, -1, -1, 0, -1, st);

    // several tokens: group the (token, choice) pairs per expert and run the tensor-core path
    if (T > 1) return run_grouped(d, slot_pool, T, slots, table, experts, gates, x, has_lora ? lora : nullptr, y, workspace, st);

    FfnParams p{};
    p.pool = static_cast<const uint8_t*>(slot_pool);
    p.slots = slots; p.table = table; p.experts = experts; p.gates = gates;
    p.x = static_cast<const uint16_t*>(x);
    if (has_lora) p.lora = *lora;
    p.y = y;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    p.status = reinterpret_cast<int32_t*>(ws + W.ctrl);
    p.u_gu = reinterpret_cast<float*>(ws + W.u_gu);
    p.h = reinterpret_cast<float*>(ws + W.h);
    p.u_d = reinterpret_cast<float*>(ws + W.u_d);
    p.H = d->H; p.I = d->I; p.E = d->E; p.K = d->K; p.group = d->group;
    p.rank = has_lora ? d->rank : 0;
    p.n_adapters = d->n_adapters; p.n_slots = d->n_slots;
    p.sigma = d->lora_scale;
    p.L = record_layout(d->H, d->I, d->group);

    const int n_sets = d->n_adapters == 1 ? 1 : d->K;
    if (has_lora) {
        const int warps = n_sets * 2 * p.rank;
        lora_a_kernel<<<dim3((warps + 7) / 8, T), 256, 0, st>>>(p, 0, n_sets);
    }
    EDG_DISPATCH_CHUNKS(d->H / 32, launch_gate_up, p, T, st);
    if (has_lora) {
        const int warps = p.K * p.rank;
        lora_a_kernel<<<dim3((warps + 7) / 8, T), 256, 0, st>>>(p, 1, n_sets);
    }
    EDG_DISPATCH_CHUNKS(d->I / 32, launch_down, p, T, d->out_dtype, st);
    EDG_CUDA_TRY(cudaGetLastError());
    return EDG_OK;
}

// rank-r projections for the grouped path: phase 0 = A_gate/A_up . x, phase 1 = A_down . h
void launch_lora_a(const edg_layer_desc* d, const void* slots, const void* table, const void* experts, const void* x,
                   const edg_lora* lora, float* u_gu, float* h, float* u_d, int32_t* status, int T, int phase, cudaStream_t st) {
    FfnParams p{};
    p.slots = static_cast<const int32_t*>(slots); p.table = static_cast<const int32_t*>(table);
    p.experts = static_cast<const int32_t*>(experts);
    p.x = static_cast<const uint16_t*>(x);
    p.lora = *lora;
    p.status = status; p.u_gu = u_gu; p.h = h; p.u_d = u_d;
    p.H = d->H; p.I = d->I; p.E = d->E; p.K = d->K; p.group = d->group; p.rank = d->rank;
    p.n_adapters = d->n_adapters; p.n_slots = d->n_slots;
    const int n_sets = d->n_adapters == 1 ? 1 : d->K;
    const int g8 = (p.rank + 7) / 8;
    const int warps = phase == 0 ? n_sets * 2 * g8 : p.K * g8;
    lora_a_kernel<<<dim3((warps + 7) / 8, T), 256, 0, st>>>(p, phase, n_sets);
}

}  // namespace edg

extern "C" int32_t edg_ffn_workspace_bytes(const edg_layer_desc* desc, int32_t T, size_t* bytes) {
    int32_t rc = edg::check_desc(desc);
    if (rc != EDG_OK) return rc;
    if (!bytes || T < 1) return EDG_E_INVAL;
    *bytes = edg::workspace_layout(*desc, T).bytes;
    return EDG_OK;
}

extern "C" int32_t edg_workspace_status(const void* workspace, void* stream, int32_t* status) {
    if (!workspace || !status) return EDG_E_INVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    EDG_CUDA_TRY(cudaMemcpyAsync(status, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    EDG_CUDA_TRY(cudaStreamSynchronize(st));
    return EDG_OK;
}

extern "C" int32_t moe_expert_ffn_int4_lora(const edg_layer_desc* desc, const void* slot_pool, const int32_t* slot_table,
                                            int32_t T, const int32_t* slots, const int32_t* experts, const float* gates,
                                            const void* x, const edg_lora* lora, void* y,
                                            void* workspace, size_t workspace_bytes, void* stream) {
    return edg::run_ffn(desc, slot_pool, T, slots, slot_table, experts, gates, x, lora, y, workspace,
                        workspace_bytes, static_cast<cudaStream_t>(stream));
}
