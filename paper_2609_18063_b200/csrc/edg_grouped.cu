// a4'-a6' grouped form: batched decode and prefill (T tokens, each with its own top-K routing).
//
// (token, choice) pairs are grouped per slot; each group is a small GEMM in which the expert's
// int4 weights are the 16-row operand of the tensor-core MMA and the group's tokens are its
// columns, so a weight tile is dequantised once and reused by every token of the tile:
//     gate/up:  [128 rows of I] x [64 tokens]  over K = H,   h = silu(g) * u fused in registers
//     down:     [256 rows of H] x [64 tokens]  over K = I
// int4 -> fp16 is done in registers: a 32-bit word holds 8 codes of one row; (w & 0x000F000F) |
// 0x64006400 is the half2 (1024 + q0, 1024 + q4) and so on; the offset and the zero point are
// removed in fp16, which is exact (integers below 16), so the MMA multiplies exact (q - z) with the
// activations and accumulates in fp32.  The group scale is applied to the fp32 partial sum of
// each 64-k block.  Activations are exact in fp16 for gate/up (bf16 inputs) and are fed as an
// fp16 (hi, lo) pair for down, where the input h is fp32.  The MMA's k slots are permuted to match
// the nibble order: the activation tile is written to shared memory in the same permutation, so a
// B fragment is one 16-byte read.
// The LoRA delta is one more MMA k-step with A = B_lora rows and B = sigma * (A_lora . x).
// Every pair's gate-weighted output goes to a [T*K][H] scratch and is reduced per token in the
// order of its K choices, so y does not depend on how the groups were scheduled.
#include "edg_grouped.cuh"

namespace edg {

constexpr int G_NTOK_MAX = 64;    // tokens per tile: 8 MMA column tiles for large groups, 1 (8 tokens) for small ones
constexpr int G_KC = 256;         // gate/up: k per staged chunk (8 super-steps of 32)
constexpr int G_KD = 128;         // down: k per staged chunk
constexpr int G_WARPS = 8;
constexpr int G_XS = G_KC * 2 + 64;   // bytes per token row of the staged activations (padded: conflict-free 16-byte reads)
constexpr int G_CS = G_KC / 2 + 16;   // bytes per weight row of the staged codes (padded: conflict-free 4-byte reads)
constexpr int G_XSD = G_KD * 2 + 64;
constexpr int G_CSD = G_KD / 2 + 16;

// The LoRA delta as one MMA k-step per 16 ranks: acc += Bl[rows][r] . (sigma * u[token][r]).
// Bl: bf16 [..][rank], row pointers for rows g and g+8 of the tile; u row pointers per column tile.
template <int G_NT>
__device__ __forceinline__ void lora_mma(float (&acc)[G_NT][4], const uint16_t* b_row_g, const uint16_t* b_row_g8,
                                         const float* const (&u_tok)[G_NT], int rank, float sigma, int t4) {
    for (int kr = 0; kr < rank; kr += 16) {
        auto ld2 = [&](const uint16_t* row, int c) -> uint32_t {
            const float a = (kr + c) < rank ? bf16_bits_to_float(row[kr + c]) : 0.f;
            const float b = (kr + c + 1) < rank ? bf16_bits_to_float(row[kr + c + 1]) : 0.f;
            return h2_as_u32(__floats2half2_rn(a, b));
        };
        const uint32_t a0 = ld2(b_row_g, 2 * t4), a1 = ld2(b_row_g8, 2 * t4);
        const uint32_t a2 = ld2(b_row_g, 2 * t4 + 8), a3 = ld2(b_row_g8, 2 * t4 + 8);
#pragma unroll
        for (int nt = 0; nt < G_NT; ++nt) {
            const float* u = u_tok[nt];
            auto ldu = [&](int c) -> uint32_t {
                const float a = (u != nullptr && (kr + c) < rank) ? sigma * u[kr + c] : 0.f;
                const float b = (u != nullptr && (kr + c + 1) < rank) ? sigma * u[kr + c + 1] : 0.f;
                return h2_as_u32(__floats2half2_rn(a, b));
            };
            mma16816(acc[nt], a0, a1, a2, a3, ldu(2 * t4), ldu(2 * t4 + 8));
        }
    }
}

// ---------------------------------------------------------------- grouping

__global__ void resolve_pairs_kernel(GroupedParams p) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= p.T * p.K) return;
    int s = p.slots[i];
    const int e = p.table != nullptr ? s : (p.experts != nullptr ? p.experts[i] : 0);
    if (p.table != nullptr) s = (s >= 0 && s < p.E) ? p.table[s] : -1;
    int ad = 0;
    if (p.rank > 0 && p.n_adapters != 1) ad = (e >= 0 && e < p.E) ? e : -1;
    if (s < 0 || s >= p.n_slots || ad < 0) { s = -1; atomicExch(p.status, EDG_E_RANGE); }
    p.pair_slot[i] = s;
    p.pair_ad[i] = ad;
}

// One CTA per slot: the slot's pairs in ascending pair index (deterministic, no atomics).  Each
// warp owns a contiguous range of pairs; a first pass counts, a second pass writes at the offsets.
constexpr int kListWarps = 16;
__global__ void __launch_bounds__(kListWarps * 32) build_lists_kernel(GroupedParams p) {
    const int s = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __shared__ int s_cnt[kListWarps];
    const int P = p.T * p.K;
    const int per = ((P + kListWarps - 1) / kListWarps + 31) / 32 * 32;      // pairs per warp, a multiple of 32
    const int lo = warp * per, hi = min(P, lo + per);
    int cnt = 0;
    for (int base = lo; base < hi; base += 32) {
        const int i = base + lane;
        cnt += __popc(__ballot_sync(0xFFFFFFFFu, i < hi && p.pair_slot[i] == s));
    }
    if (lane == 0) s_cnt[warp] = cnt;
    __syncthreads();
    int off = 0, total = 0;
    for (int w = 0; w < kListWarps; ++w) { if (w < warp) off += s_cnt[w]; total += s_cnt[w]; }
    for (int base = lo; base < hi; base += 32) {
        const int i = base + lane;
        const bool m = i < hi && p.pair_slot[i] == s;
        const unsigned bal = __ballot_sync(0xFFFFFFFFu, m);
        if (m) p.lists[(size_t)s * p.T + off + __popc(bal & ((1u << lane) - 1))] = i;
        off += __popc(bal);
    }
    if (threadIdx.x == 0) p.counts[s] = total;
}

// Tile table: slot s contributes ceil(count / ntok) tiles; an exclusive scan over the slots gives
// each its first tile.  One CTA, slots strided over the threads, scan through shared memory.
__global__ void __launch_bounds__(1024) build_tiles_kernel(GroupedParams p) {
    __shared__ int s_n[1024];
    const int tid = threadIdx.x;
    // n_slots can exceed the block: each thread owns a contiguous run of slots
    const int per = (p.n_slots + 1023) / 1024;
    const int s0 = tid * per, s1 = min(p.n_slots, s0 + per);
    int mine = 0;
    for (int s = s0; s < s1; ++s) mine += (p.counts[s] + p.ntok - 1) / p.ntok;
    s_n[tid] = mine;
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {          // inclusive scan
        const int v = tid >= o ? s_n[tid - o] : 0;
        __syncthreads();
        s_n[tid] += v;
        __syncthreads();
    }
    int n = s_n[tid] - mine;                       // exclusive prefix
    for (int s = s0; s < s1; ++s)
        for (int first = 0; first < p.counts[s]; first += p.ntok) { p.tiles[2 * n] = s; p.tiles[2 * n + 1] = first; ++n; }
    if (tid == 1023) *p.n_tiles = s_n[1023];
}

// ---------------------------------------------------------------- gate/up
// CTA = (tile of up to 64 pairs of one slot) x (128 rows of I).  Warp w owns rows 16w..16w+15 of
// both gate and up, so silu(g) * u is formed in registers.

template <int G_NT>
__global__ void __launch_bounds__(G_WARPS * 32, G_NT == 1 ? 4 : 2) grouped_gate_up_kernel(GroupedParams p) {
    constexpr int G_NTOK = G_NT * 8;
    const int tile = blockIdx.x;
    if (tile >= *p.n_tiles) return;
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* s_x = smem;                                          // [64][G_XS]
    uint8_t* s_cg = s_x + G_NTOK * G_XS;                          // [128][G_CS]
    uint8_t* s_cu = s_cg + 128 * G_CS;
    const int ng = G_KC / p.group;                                // groups per chunk
    uint32_t* s_zg = reinterpret_cast<uint32_t*>(s_cu + 128 * G_CS);   // [128][ng] (scale, zero) pairs
    uint32_t* s_zu = s_zg + 128 * ng;
    int* s_pair = reinterpret_cast<int*>(s_zu + 128 * ng);        // [64]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t4 = lane & 3;
    const int slot = p.tiles[2 * tile], first = p.tiles[2 * tile + 1];
    const int cnt = min(G_NTOK, p.counts[slot] - first);
    const int row0 = blockIdx.y * 128;
    const uint8_t* rec = p.pool + (size_t)slot * p.L.bytes;
    if (tid < G_NTOK) s_pair[tid] = tid < cnt ? p.lists[(size_t)slot * p.T + first + tid] : -1;
    __syncthreads();

    float ag[G_NT][4], au[G_NT][4];
#pragma unroll
    for (int nt = 0; nt < G_NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) { ag[nt][i] = 0.f; au[nt][i] = 0.f; }

    for (int kc = 0; kc < p.H / G_KC; ++kc) {
        __syncthreads();
        for (int idx = tid; idx < G_NTOK * 4; idx += G_WARPS * 32) {   // activations: token idx/4, 64 k starting at (idx%4)*64
            const int i = idx >> 2, q = idx & 3;
            const int pair = s_pair[i];
            const uint16_t* src = pair >= 0 ? p.x + (size_t)(pair / p.K) * p.H + kc * G_KC + q * 64 : nullptr;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                uint4 out = make_uint4(0, 0, 0, 0);
                if (src != nullptr) {
                    const uint4 v = *reinterpret_cast<const uint4*>(src + j * 8);
                    const float f[8] = {bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y),
                                        bf16_lo(v.z), bf16_hi(v.z), bf16_lo(v.w), bf16_hi(v.w)};
                    out = permute8(f);
                }
                *reinterpret_cast<uint4*>(s_x + i * G_XS + (q * 8 + j) * 16) = out;
            }
        }
#pragma unroll
        for (int m = 0; m < 4; ++m) {   // codes: 128 rows x 128 bytes per matrix
            const int idx = tid + 256 * m, row = idx >> 3, seg = idx & 7;
            const size_t off = code_off(p.H, row0 + row, kc * (G_KC / 32) + seg);
            *reinterpret_cast<uint4*>(s_cg + row * G_CS + seg * 16) = ld_stream16(rec + p.L.codes_gate + off);
            *reinterpret_cast<uint4*>(s_cu + row * G_CS + seg * 16) = ld_stream16(rec + p.L.codes_up + off);
        }
        for (int idx = tid; idx < 128 * ng; idx += 256) {
            const int row = idx / ng, gi = idx % ng;
            const size_t off = sz_off(p.H, p.group, row0 + row, kc * ng + gi);
            s_zg[idx] = ld_stream4(rec + p.L.sz_gate + off);
            s_zu[idx] = ld_stream4(rec + p.L.sz_up + off);
        }
        __syncthreads();

        const int r_lo = 16 * warp + g, r_hi = r_lo + 8;
        const int sb = p.group >= 64 ? 2 : 1;                    // super-steps (32 k) per scaled block
        for (int ss0 = 0; ss0 < G_KC / 32; ss0 += sb) {
            const int gi = (ss0 * 32) / p.group;
            const __half2 zg0 = u32_as_h2(s_zg[r_lo * ng + gi]), zg1 = u32_as_h2(s_zg[r_hi * ng + gi]);
            const __half2 zu0 = u32_as_h2(s_zu[r_lo * ng + gi]), zu1 = u32_as_h2(s_zu[r_hi * ng + gi]);
            const float sg0 = __low2float(zg0), sg1 = __low2float(zg1), su0 = __low2float(zu0), su1 = __low2float(zu1);
            uint32_t Ag[2][2][4], Au[2][2][4];     // [super-step][row g / g+8][(k0,k4) (k1,k5) (k2,k6) (k3,k7)]
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                if (u < sb) {
                    const int ss = ss0 + u;
                    dequant_word(*reinterpret_cast<const uint32_t*>(s_cg + r_lo * G_CS + ss * 16 + t4 * 4), __high2half2(zg0), Ag[u][0]);
                    dequant_word(*reinterpret_cast<const uint32_t*>(s_cg + r_hi * G_CS + ss * 16 + t4 * 4), __high2half2(zg1), Ag[u][1]);
                    dequant_word(*reinterpret_cast<const uint32_t*>(s_cu + r_lo * G_CS + ss * 16 + t4 * 4), __high2half2(zu0), Au[u][0]);
                    dequant_word(*reinterpret_cast<const uint32_t*>(s_cu + r_hi * G_CS + ss * 16 + t4 * 4), __high2half2(zu1), Au[u][1]);
                }
            }
#pragma unroll
            for (int nt = 0; nt < G_NT; ++nt) {
                float cg[4], cu[4];
                const uint4 b = *reinterpret_cast<const uint4*>(s_x + (8 * nt + g) * G_XS + (4 * ss0 + t4) * 16);
                mma16816_zero(cg, Ag[0][0][0], Ag[0][1][0], Ag[0][0][1], Ag[0][1][1], b.x, b.y);
                mma16816(cg, Ag[0][0][2], Ag[0][1][2], Ag[0][0][3], Ag[0][1][3], b.z, b.w);
                mma16816_zero(cu, Au[0][0][0], Au[0][1][0], Au[0][0][1], Au[0][1][1], b.x, b.y);
                mma16816(cu, Au[0][0][2], Au[0][1][2], Au[0][0][3], Au[0][1][3], b.z, b.w);
                if (sb == 2) {
                    const uint4 c = *reinterpret_cast<const uint4*>(s_x + (8 * nt + g) * G_XS + (4 * (ss0 + 1) + t4) * 16);
                    mma16816(cg, Ag[1][0][0], Ag[1][1][0], Ag[1][0][1], Ag[1][1][1], c.x, c.y);
                    mma16816(cg, Ag[1][0][2], Ag[1][1][2], Ag[1][0][3], Ag[1][1][3], c.z, c.w);
                    mma16816(cu, Au[1][0][0], Au[1][1][0], Au[1][0][1], Au[1][1][1], c.x, c.y);
                    mma16816(cu, Au[1][0][2], Au[1][1][2], Au[1][0][3], Au[1][1][3], c.z, c.w);
                }
                ag[nt][0] = fmaf(sg0, cg[0], ag[nt][0]); ag[nt][1] = fmaf(sg0, cg[1], ag[nt][1]);
                ag[nt][2] = fmaf(sg1, cg[2], ag[nt][2]); ag[nt][3] = fmaf(sg1, cg[3], ag[nt][3]);
                au[nt][0] = fmaf(su0, cu[0], au[nt][0]); au[nt][1] = fmaf(su0, cu[1], au[nt][1]);
                au[nt][2] = fmaf(su1, cu[2], au[nt][2]); au[nt][3] = fmaf(su1, cu[3], au[nt][3]);
            }
        }
    }

    // ---- LoRA delta, SiLU, product; h[pair][row]
    const int r_lo = row0 + 16 * warp + g, r_hi = r_lo + 8;
    if (p.rank > 0) {
        const int first_pair = s_pair[0];
        const int ad = first_pair >= 0 ? p.pair_ad[first_pair] : 0;      // one slot = one expert = one adapter
        const int n_sets = p.n_adapters == 1 ? 1 : p.K;
        const float* ug[G_NT];
        const float* uu[G_NT];
#pragma unroll
        for (int nt = 0; nt < G_NT; ++nt) {
            const int pair = s_pair[8 * nt + g];
            if (pair >= 0) {
                const int tok = pair / p.K, set = p.n_adapters == 1 ? 0 : pair % p.K;
                ug[nt] = p.u_gu + (((size_t)tok * n_sets + set) * 2 + 0) * p.rank;
                uu[nt] = ug[nt] + p.rank;
            } else { ug[nt] = nullptr; uu[nt] = nullptr; }
        }
        const uint16_t* Bg = reinterpret_cast<const uint16_t*>(p.lora.B_gate) + (size_t)ad * p.I * p.rank;
        const uint16_t* Bu = reinterpret_cast<const uint16_t*>(p.lora.B_up) + (size_t)ad * p.I * p.rank;
        lora_mma<G_NT>(ag, Bg + (size_t)r_lo * p.rank, Bg + (size_t)r_hi * p.rank, ug, p.rank, p.sigma, t4);
        lora_mma<G_NT>(au, Bu + (size_t)r_lo * p.rank, Bu + (size_t)r_hi * p.rank, uu, p.rank, p.sigma, t4);
    }
#pragma unroll
    for (int nt = 0; nt < G_NT; ++nt) {
        const int p0 = s_pair[8 * nt + 2 * t4], p1 = s_pair[8 * nt + 2 * t4 + 1];
        if (p0 >= 0) {
            p.h[(size_t)p0 * p.I + r_lo] = silu_f(ag[nt][0]) * au[nt][0];
            p.h[(size_t)p0 * p.I + r_hi] = silu_f(ag[nt][2]) * au[nt][2];
        }
        if (p1 >= 0) {
            p.h[(size_t)p1 * p.I + r_lo] = silu_f(ag[nt][1]) * au[nt][1];
            p.h[(size_t)p1 * p.I + r_hi] = silu_f(ag[nt][3]) * au[nt][3];
        }
    }
}

// ---------------------------------------------------------------- down
// CTA = (tile of up to 64 pairs of one slot) x (256 rows of H).  Warp w owns rows 32w..32w+31.

template <int G_NT>
__global__ void __launch_bounds__(G_WARPS * 32, G_NT == 1 ? 4 : 2) grouped_down_kernel(GroupedParams p) {
    constexpr int G_NTOK = G_NT * 8;
    const int tile = blockIdx.x;
    if (tile >= *p.n_tiles) return;
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t* s_x = smem;                                          // [64][G_XSD]  h, fp16 high part
    uint8_t* s_xl = s_x + G_NTOK * G_XSD;                         // [64][G_XSD]  h, fp16 residual
    uint8_t* s_c = s_xl + G_NTOK * G_XSD;                         // [256][G_CSD]
    const int ng = G_KD / p.group > 0 ? G_KD / p.group : 1;       // groups per chunk (a 128-group spans the chunk)
    uint32_t* s_z = reinterpret_cast<uint32_t*>(s_c + 256 * G_CSD);    // [256][ng]
    int* s_pair = reinterpret_cast<int*>(s_z + 256 * ng);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t4 = lane & 3;
    const int slot = p.tiles[2 * tile], first = p.tiles[2 * tile + 1];
    const int cnt = min(G_NTOK, p.counts[slot] - first);
    const int row0 = blockIdx.y * 256;
    const uint8_t* rec = p.pool + (size_t)slot * p.L.bytes;
    if (tid < G_NTOK) s_pair[tid] = tid < cnt ? p.lists[(size_t)slot * p.T + first + tid] : -1;
    __syncthreads();

    float acc[2][G_NT][4];
#pragma unroll
    for (int m = 0; m < 2; ++m)
#pragma unroll
        for (int nt = 0; nt < G_NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[m][nt][i] = 0.f;

    for (int kc = 0; kc < p.I / G_KD; ++kc) {
        __syncthreads();
        for (int idx = tid; idx < G_NTOK * 4; idx += G_WARPS * 32) {   // h: token idx/4, 32 k starting at (idx%4)*32, fp32 -> fp16 (hi, lo)
            const int i = idx >> 2, q = idx & 3;
            const int pair = s_pair[i];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint4 hi = make_uint4(0, 0, 0, 0), lo = make_uint4(0, 0, 0, 0);
                if (pair >= 0) {
                    const float* src = p.h + (size_t)pair * p.I + kc * G_KD + q * 32 + j * 8;
                    const float4 a = *reinterpret_cast<const float4*>(src);
                    const float4 b = *reinterpret_cast<const float4*>(src + 4);
                    const float f[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
                    hi = permute8(f);
                    lo = permute8_lo(f);
                }
                *reinterpret_cast<uint4*>(s_x + i * G_XSD + (q * 4 + j) * 16) = hi;
                *reinterpret_cast<uint4*>(s_xl + i * G_XSD + (q * 4 + j) * 16) = lo;
            }
        }
#pragma unroll
        for (int m = 0; m < 4; ++m) {   // codes: 256 rows x 64 bytes, from the sliced layout
            const int idx = tid + 256 * m, row = idx >> 2, seg = idx & 3;
            *reinterpret_cast<uint4*>(s_c + row * G_CSD + seg * 16) =
                ld_stream16(rec + p.L.codes_down + down_code_off(p.H, p.I, row0 + row, kc * (G_KD / 32) + seg));
        }
        for (int idx = tid; idx < 256 * ng; idx += 256) {
            const int row = idx / ng, gi = idx % ng;
            s_z[idx] = ld_stream4(rec + p.L.sz_down + down_sz_off(p.H, p.I, p.group, row0 + row, (kc * G_KD) / p.group + gi));
        }
        __syncthreads();

        const int sb = p.group >= 64 ? 2 : 1;
        for (int ss0 = 0; ss0 < G_KD / 32; ss0 += sb) {
            const int gi = p.group >= G_KD ? 0 : (ss0 * 32) / p.group;
#pragma unroll
            for (int m = 0; m < 2; ++m) {
                const int r_lo = 32 * warp + 16 * m + g, r_hi = r_lo + 8;
                const __half2 z0 = u32_as_h2(s_z[r_lo * ng + gi]), z1 = u32_as_h2(s_z[r_hi * ng + gi]);
                const float s0 = __low2float(z0), s1 = __low2float(z1);
                uint32_t A[2][2][4];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    if (u < sb) {
                        const int ss = ss0 + u;
                        dequant_word(*reinterpret_cast<const uint32_t*>(s_c + r_lo * G_CSD + ss * 16 + t4 * 4), __high2half2(z0), A[u][0]);
                        dequant_word(*reinterpret_cast<const uint32_t*>(s_c + r_hi * G_CSD + ss * 16 + t4 * 4), __high2half2(z1), A[u][1]);
                    }
                }
#pragma unroll
                for (int nt = 0; nt < G_NT; ++nt) {
                    float c[4];
                    const int xo = (8 * nt + g) * G_XSD + (4 * ss0 + t4) * 16;
                    const uint4 bh = *reinterpret_cast<const uint4*>(s_x + xo), bl = *reinterpret_cast<const uint4*>(s_xl + xo);
                    mma16816_zero(c, A[0][0][0], A[0][1][0], A[0][0][1], A[0][1][1], bl.x, bl.y);
                    mma16816(c, A[0][0][2], A[0][1][2], A[0][0][3], A[0][1][3], bl.z, bl.w);
                    mma16816(c, A[0][0][0], A[0][1][0], A[0][0][1], A[0][1][1], bh.x, bh.y);
                    mma16816(c, A[0][0][2], A[0][1][2], A[0][0][3], A[0][1][3], bh.z, bh.w);
                    if (sb == 2) {
                        const uint4 ch = *reinterpret_cast<const uint4*>(s_x + xo + 64), cl = *reinterpret_cast<const uint4*>(s_xl + xo + 64);
                        mma16816(c, A[1][0][0], A[1][1][0], A[1][0][1], A[1][1][1], cl.x, cl.y);
                        mma16816(c, A[1][0][2], A[1][1][2], A[1][0][3], A[1][1][3], cl.z, cl.w);
                        mma16816(c, A[1][0][0], A[1][1][0], A[1][0][1], A[1][1][1], ch.x, ch.y);
                        mma16816(c, A[1][0][2], A[1][1][2], A[1][0][3], A[1][1][3], ch.z, ch.w);
                    }
                    acc[m][nt][0] = fmaf(s0, c[0], acc[m][nt][0]); acc[m][nt][1] = fmaf(s0, c[1], acc[m][nt][1]);
                    acc[m][nt][2] = fmaf(s1, c[2], acc[m][nt][2]); acc[m][nt][3] = fmaf(s1, c[3], acc[m][nt][3]);
                }
            }
        }
    }

    // ---- LoRA delta, gate weight; o[pair][row]
    const int first_pair = s_pair[0];
    const int ad = (p.rank > 0 && first_pair >= 0) ? p.pair_ad[first_pair] : 0;
    const float* ud[G_NT];
#pragma unroll
    for (int nt = 0; nt < G_NT; ++nt) {
        const int pair = s_pair[8 * nt + g];
        ud[nt] = (p.rank > 0 && pair >= 0) ? p.u_d + (size_t)pair * p.rank : nullptr;
    }
#pragma unroll
    for (int m = 0; m < 2; ++m) {
        const int r_lo = row0 + 32 * warp + 16 * m + g, r_hi = r_lo + 8;
        if (p.rank > 0) {
            const uint16_t* Bd = reinterpret_cast<const uint16_t*>(p.lora.B_down) + (size_t)ad * p.H * p.rank;
            lora_mma<G_NT>(acc[m], Bd + (size_t)r_lo * p.rank, Bd + (size_t)r_hi * p.rank, ud, p.rank, p.sigma, t4);
        }
#pragma unroll
        for (int nt = 0; nt < G_NT; ++nt) {
            const int p0 = s_pair[8 * nt + 2 * t4], p1 = s_pair[8 * nt + 2 * t4 + 1];
            if (p0 >= 0) {
                const float w = p.gates[p0];
                p.o[(size_t)p0 * p.H + r_lo] = w * acc[m][nt][0];
                p.o[(size_t)p0 * p.H + r_hi] = w * acc[m][nt][2];
            }
            if (p1 >= 0) {
                const float w = p.gates[p1];
                p.o[(size_t)p1 * p.H + r_lo] = w * acc[m][nt][1];
                p.o[(size_t)p1 * p.H + r_hi] = w * acc[m][nt][3];
            }
        }
    }
}

// y[t] = sum_k o[t*K + k], in the order of the token's choices
template <typename OutT>
__global__ void __launch_bounds__(256) reduce_pairs_kernel(GroupedParams p) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)p.T * p.H) return;
    const int t = (int)(i / p.H), n = (int)(i % p.H);
    float v = 0.f;
    for (int k = 0; k < p.K; ++k) {
        const int pair = t * p.K + k;
        if (p.pair_slot[pair] >= 0) v += p.o[(size_t)pair * p.H + n];
    }
    store_out<OutT>(reinterpret_cast<OutT*>(p.y), i, v);
}

// ---------------------------------------------------------------- host

struct FfnParams;   // generic-path parameters (edg_ffn.cu)
void launch_lora_a(const edg_layer_desc* d, const void* slots, const void* table, const void* experts, const void* x,
                   const edg_lora* lora, float* u_gu, float* h, float* u_d, int32_t* status, int T, int phase, cudaStream_t st);

int32_t run_grouped(const edg_layer_desc* d, const void* slot_pool, int32_t T, const int32_t* slots, const int32_t* table,
                    const int32_t* experts, const float* gates, const void* x, const edg_lora* lora, void* y,
                    void* workspace, cudaStream_t st) {
    if (d->I % 128 != 0 || d->H % 256 != 0 || G_KC % d->group != 0 || d->group > G_KD) return EDG_E_SHAPE;
    const bool has_lora = lora != nullptr && d->rank > 0;
    const WorkspaceLayout W = workspace_layout(*d, T);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    GroupedParams p{};
    p.pool = static_cast<const uint8_t*>(slot_pool);
    p.slots = slots; p.table = table; p.experts = experts; p.gates = gates;
    p.x = static_cast<const uint16_t*>(x);
    if (has_lora) p.lora = *lora;
    p.y = y;
    p.status = reinterpret_cast<int32_t*>(ws + W.ctrl);
    p.u_gu = reinterpret_cast<float*>(ws + W.u_gu);
    p.h = reinterpret_cast<float*>(ws + W.h);
    p.u_d = reinterpret_cast<float*>(ws + W.u_d);
    p.o = reinterpret_cast<float*>(ws + W.o);
    p.pair_slot = reinterpret_cast<int32_t*>(ws + W.pair_slot);
    p.pair_ad = reinterpret_cast<int32_t*>(ws + W.pair_ad);
    p.counts = reinterpret_cast<int32_t*>(ws + W.counts);
    p.n_tiles = reinterpret_cast<int32_t*>(ws + W.n_tiles);
    p.tiles = reinterpret_cast<int32_t*>(ws + W.tiles);
    p.lists = reinterpret_cast<int32_t*>(ws + W.lists);
    p.hq = ws + W.hq;
    p.xq = ws + W.xq;
    p.T = T; p.H = d->H; p.I = d->I; p.E = d->E; p.K = d->K; p.group = d->group;
    p.rank = has_lora ? d->rank : 0;
    p.n_adapters = d->n_adapters; p.n_slots = d->n_slots; p.out_dtype = d->out_dtype;
    p.sigma = d->lora_scale;
    p.L = record_layout(d->H, d->I, d->group);

    const int P = T * d->K;
    // few tokens per expert (batched decode): tiles of 8 tokens, the kernels are then bound by streaming
    // the weights; many (prefill): tiles of 64 so a dequantised weight tile is reused 8 times more
    const bool small = P <= 8 * d->n_slots;
    // large groups: tiles of 128 tokens on the tcgen05 path
    const bool umma = !small && umma_grouped_supported(*d);
    p.ntok = small ? 8 : (umma ? kUmmaTokens : 64);
    const int max_tiles = (P + p.ntok - 1) / p.ntok + d->n_slots;
    resolve_pairs_kernel<<<(P + 255) / 256, 256, 0, st>>>(p);
    build_lists_kernel<<<d->n_slots, kListWarps * 32, 0, st>>>(p);
    build_tiles_kernel<<<1, 1024, 0, st>>>(p);
    if (has_lora && !launch_lora_ax_tokens(d, x, lora, p.u_gu, T, st))
        launch_lora_a(d, slots, table, experts, x, lora, p.u_gu, p.h, p.u_d, p.status, T, 0, st);

    // small groups on the shapes the batch-1 kernel covers: one streaming kernel for the whole FFN
    if (small && grouped_stream_supported(*d))
        return run_grouped_stream(d, p, reinterpret_cast<float*>(ws + W.o_part), ws + W.xt, max_tiles, st);

    const int ng = G_KC / d->group, ngd = G_KD / d->group;
    const size_t sm_gu = (size_t)p.ntok * G_XS + 2 * 128 * G_CS + 2 * 128 * ng * 4 + p.ntok * 4;
    const size_t sm_d = (size_t)2 * p.ntok * G_XSD + 256 * G_CSD + 256 * ngd * 4 + p.ntok * 4;
    static bool configured = false;
    if (!configured) {
        EDG_CUDA_TRY(cudaFuncSetAttribute(grouped_gate_up_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024));
        EDG_CUDA_TRY(cudaFuncSetAttribute(grouped_down_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024));
        EDG_CUDA_TRY(cudaFuncSetAttribute(grouped_gate_up_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024));
        EDG_CUDA_TRY(cudaFuncSetAttribute(grouped_down_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024));
        configured = true;
    }
    if (umma) EDG_CUDA_TRY(launch_umma_gate_up(p, max_tiles, st));
    else if (small) grouped_gate_up_kernel<1><<<dim3(max_tiles, d->I / 128), G_WARPS * 32, sm_gu, st>>>(p);
    else grouped_gate_up_kernel<8><<<dim3(max_tiles, d->I / 128), G_WARPS * 32, sm_gu, st>>>(p);
    if (has_lora && !launch_lora_adh_pairs(d, lora, p.h, p.u_d, P, st))
        launch_lora_a(d, slots, table, experts, x, lora, p.u_gu, p.h, p.u_d, p.status, T, 1, st);
    if (umma) EDG_CUDA_TRY(launch_umma_down(p, max_tiles, st));
    else if (small) grouped_down_kernel<1><<<dim3(max_tiles, d->H / 256), G_WARPS * 32, sm_d, st>>>(p);
    else grouped_down_kernel<8><<<dim3(max_tiles, d->H / 256), G_WARPS * 32, sm_d, st>>>(p);
    const size_t n_out = (size_t)T * d->H;
    const int rb = (int)((n_out + 255) / 256);
    if (d->out_dtype == EDG_F32) reduce_pairs_kernel<float><<<rb, 256, 0, st>>>(p);
    else if (d->out_dtype == EDG_F16) reduce_pairs_kernel<__half><<<rb, 256, 0, st>>>(p);
    else reduce_pairs_kernel<bf16_t><<<rb, 256, 0, st>>>(p);
    EDG_CUDA_TRY(cudaGetLastError());
    return EDG_OK;
}

}  // namespace edg
