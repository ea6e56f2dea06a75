// a4'-a6' for small groups (batched decode: a few tokens per routed expert): the streaming pipeline of
// the batch-1 layer kernel with the eight columns of the MMA carrying the tokens of a tile.
//
// Batched decode is bound by streaming the union of the routed experts from HBM once.  The tiles
// built by the grouping kernels hold up to 8 (token, choice) pairs of one slot.  A work item is one
// quarter of the intermediate dimension of one tile; persistent thread-block clusters of 4 CTAs
// (2 CTAs per SM) take the items round-robin.  For an item a CTA streams the same bytes as in the
// batch-1 kernel -- its 2 x I/16 gate/up rows over all of K through two stage buffers (first half
// of K, second half), then its H/4 rows of the quarter's down block -- by bulk asynchronous
// copies on mbarriers, the next item's first half being issued as soon as the down block has been
// consumed, so a CTA always has a load in flight.  The codes go to the tensor cores as biased
// fp16 (five instructions per eight codes, edg_mma.cuh); the B operand holds the tile's 8 tokens
// (fp16 of the bf16 states for gate/up; value and residual of the fp32 h as two MMAs for down);
// bias, zero point and scale are applied in fp32 per 64-code block and per token.  h is exchanged
// inside the cluster by remote stores that count on the receiver's mbarrier.  The rank-r
// projections A.x come from the grouped path's pre-pass; B rows and A_down columns are staged
// per item; B_down (A_down h) is added per quarter (it is linear in h).  Every item writes its
// gate-weighted partial rows to [pair][quarter][H]; the reduce sums a token's K x 4 partials in a
// fixed order.
#include "edg_grouped.cuh"
#include "edg_ptx.cuh"

namespace edg {

constexpr int SC = 4;              // CTAs per cluster
constexpr int SW_ = 4;             // warps per CTA
constexpr int ST = 8;              // tokens per tile = MMA columns
constexpr int SMaxRank = 64;

struct StreamSmem {
    uint32_t stage0, stage_bytes, mat_codes, mat_sz, sz0, d_codes, d_sz;
    uint32_t lora0, lora_bytes;
    uint32_t bars, part, gu, hloc, h, hb, hsum, hbias, u, udp, ud, info, total;
    // the tile record in global memory (pre-pass): x fragments, block sums, then what an item copies in: projections, pair table
    uint32_t g_xsum, g_xbias, g_u, g_small, g_bytes;
};

// byte offsets, identical on host and device (rows_gu = I/16 gate/up rows per CTA and matrix, rows_d = H/4, sw = I/4)
__host__ __device__ inline StreamSmem stream_smem(int H, int I, int group, int rank) {
    StreamSmem S;
    const uint32_t rows_gu = I / 16, rows_d = H / SC, sw = I / 4, tg = rows_gu / 16;
    S.mat_codes = (uint32_t)(H / 128) * 256;
    S.mat_sz = (uint32_t)((H / 4) / group) * 64;
    S.sz0 = 2 * tg * S.mat_codes;
    S.stage_bytes = 2 * tg * (S.mat_codes + S.mat_sz);
    uint32_t o = 0;
    S.stage0 = o;  o += 2 * S.stage_bytes;
    S.d_codes = S.stage0;
    S.d_sz = S.stage0 + rows_d * sw / 2;
    S.lora_bytes = 3 * rows_gu * (uint32_t)rank * 2;
    S.lora0 = o;   o += 2 * S.lora_bytes;
    o = (o + 15) / 16 * 16;
    S.bars = o;    o += 8 * 8;
    // The tile record as the pre-pass writes it: [token][H/8] uint4 x as fp16 B words in k-slot order, [block][token]
    // sums (plain, and as the biased codes weigh them) -- these are read by the MMA loops straight from the L2 -- then
    // [token][2][rank] projections and the pair table, which an item copies into shared memory.
    const uint32_t rr = rank > 0 ? (uint32_t)rank : 8u;
    S.g_xsum = ST * (uint32_t)H * 2;
    S.g_xbias = S.g_xsum + ST * (uint32_t)(H / 32) * 4;
    S.g_u = S.g_xbias + ST * (uint32_t)(H / 32) * 4;
    S.g_small = ST * 2 * rr * 4 + 128;                        // projections + pair table
    S.g_bytes = S.g_u + S.g_small;
    S.u = o;       o += 2 * S.g_small;                        // two buffers of ([token][2][rank] projections, [8] pair, [8] gate, [8] adapter, [8] token)
    S.info = S.u + ST * 2 * rr * 4;
    S.part = o;    o += SW_ * 2 * rows_gu * ST * 4;           // [warp][2 rows_gu][token]
    S.gu = o;      o += 2 * rows_gu * ST * 4;                 // [2 rows_gu][token]
    S.hloc = o;    o += rows_gu * ST * 4;                     // [rows_gu][token]
    S.h = o;       o += 2 * sw * ST * 4;                      // [2][sw][token]
    S.hb = o;      o += (sw / 32) * 2 * ST * 4 * 16;          // [chunk][hi/lo][token][4] uint4
    S.hsum = o;    o += ST * (sw / 32) * 4;
    S.hbias = o;   o += ST * (sw / 32) * 4;
    S.udp = o;     o += 2 * SC * ST * rr * 4;                 // [2][cta][token][rank]: partials of A_down h
    S.ud = o;      o += ST * rr * 4;                          // [token][rank]
    S.total = (o + 15) / 16 * 16;
    return S;
}

struct StreamParams {
    GroupedParams g;
    float* o_part;                // [T*K][4][H]
    uint8_t* xt;                  // [tiles][rec_bytes + 128]: per tile, what an item needs besides the weights (written by the pre-pass)
    int gshift;
    StreamSmem S;
};

enum { SB_DOWN = 2, SB_LORA = 3, SB_H = 5, SB_X = 7, SNumBars = 8 };

// two bf16 (one 32-bit word, low half first) as an fp16 pair
__device__ __forceinline__ uint32_t bf16x2_to_h2(uint32_t w) {
    return h2_as_u32(__floats2half2_rn(bf16_lo(w), bf16_hi(w)));
}
// One LoRA k-step on the tensor cores: c += Bl[rows g, g+8][kr .. kr+15] . v[kr .. kr+15][token g8], Bl rows bf16
// (row pointers for rows g and g + 8 of the tile; rank a multiple of 8, entries beyond it are zero), v given per lane
// as the two fp16 pairs of its token column: k = kr + 2 t4, +1 and kr + 2 t4 + 8, +9.
__device__ __forceinline__ void lora_step(float (&c)[4], const uint16_t* row_g, const uint16_t* row_g8, int kr, int rank, int t4,
                                          uint32_t b0, uint32_t b1) {
    const int k0 = kr + 2 * t4, k1 = k0 + 8;
    const uint32_t a0 = k0 < rank ? bf16x2_to_h2(*reinterpret_cast<const uint32_t*>(row_g + k0)) : 0u;
    const uint32_t a1 = k0 < rank ? bf16x2_to_h2(*reinterpret_cast<const uint32_t*>(row_g8 + k0)) : 0u;
    const uint32_t a2 = k1 < rank ? bf16x2_to_h2(*reinterpret_cast<const uint32_t*>(row_g + k1)) : 0u;
    const uint32_t a3 = k1 < rank ? bf16x2_to_h2(*reinterpret_cast<const uint32_t*>(row_g8 + k1)) : 0u;
    mma16816(c, a0, a1, a2, a3, b0, b1);
}
// the B words of lora_step from an fp32 vector v[rank] of the lane's token, scaled by sigma
__device__ __forceinline__ void lora_bwords(const float* v, int kr, int rank, int t4, float sigma, uint32_t& b0, uint32_t& b1) {
    const int k0 = kr + 2 * t4, k1 = k0 + 8;
    b0 = k0 < rank ? h2_as_u32(__floats2half2_rn(sigma * v[k0], sigma * v[k0 + 1])) : 0u;
    b1 = k1 < rank ? h2_as_u32(__floats2half2_rn(sigma * v[k1], sigma * v[k1 + 1])) : 0u;
}

template <int NCW, int DCH, int TG, int TD, int CPB>
__global__ void __launch_bounds__(SW_ * 32, 3) grouped_stream_kernel(const __grid_constant__ StreamParams sp) {
    extern __shared__ __align__(128) uint8_t smem[];
    const GroupedParams& p = sp.g;
    const StreamSmem& S = sp.S;
    const int cl = blockIdx.x / SC, n_cl = gridDim.x / SC, crank = blockIdx.x % SC;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, tid = threadIdx.x;
    const int g8 = lane >> 2, t4 = lane & 3;
    constexpr int rows_gu = 16 * TG, rows_d = 128 * TD, sw = 32 * DCH, NT = 2 * TG;
    const int r = p.rank, n0_d = crank * rows_d;
    const int cps = p.H / 128, gpst = (p.H / 4) >> sp.gshift, gps = sw >> sp.gshift;

    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S.bars);
    float* s_part = reinterpret_cast<float*>(smem + S.part);         // [warp][2 rows_gu][ST]
    float* s_gu = reinterpret_cast<float*>(smem + S.gu);             // [2 rows_gu][ST]
    float* s_hloc = reinterpret_cast<float*>(smem + S.hloc);         // [rows_gu][ST]
    float* s_h = reinterpret_cast<float*>(smem + S.h);               // [2][sw][ST]
    uint4* s_hb = reinterpret_cast<uint4*>(smem + S.hb);             // [chunk][2][ST][4]
    float* s_hsum = reinterpret_cast<float*>(smem + S.hsum);         // [block][ST]
    float* s_hbias = reinterpret_cast<float*>(smem + S.hbias);
    float* s_udp = reinterpret_cast<float*>(smem + S.udp);           // [2][SC][ST][r]
    float* s_ud = reinterpret_cast<float*>(smem + S.ud);             // [ST][r]
    const size_t xt_stride = S.g_bytes;

    const int n_items = 4 * *p.n_tiles;
    const int my_items = cl < n_items ? (n_items - cl + n_cl - 1) / n_cl : 0;
    const uint32_t h_bytes = (uint32_t)(sw * ST + SC * ST * r) * 4u;
    if (tid == 0) {
        for (int b = 0; b < SNumBars; ++b) mbar_init(&bars[b], b < 2 ? 2 : 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (my_items > 0) mbar_expect_tx(&bars[SB_H], h_bytes);
        if (my_items > 1) mbar_expect_tx(&bars[SB_H + 1], h_bytes);
    }
    cluster_arrive();
    cluster_wait();                        // every CTA's barriers exist before anyone sends
    if (my_items == 0) return;             // (the same for all CTAs of a cluster)

    auto item_slot = [&](int j) { return p.tiles[2 * ((cl + j * n_cl) >> 2)]; };
    auto item_quarter = [&](int j) { return (cl + j * n_cl) & 3; };
    auto item_rec = [&](int j) { return p.pool + (size_t)item_slot(j) * p.L.bytes; };
    // K quarters 2 pair, 2 pair + 1 of item j's gate/up rows into stages 0 and 1: warp v issues runs 4 (v & 1) .. + 3 of stage v / 2
    auto issue_gu = [&](int j, int pair) {
        const int c = item_quarter(j);
        const uint8_t* rec = item_rec(j);
        const uint64_t pol = policy_evict_first();
        const int s = warp >> 1, run = (warp & 1) * 4 + lane, kq = pair * 2 + s;
        const int n_runs = min(4, max(0, 4 * TG - (warp & 1) * 4));
        if (lane == 0) mbar_expect_tx(&bars[s], (uint32_t)(n_runs / 2) * (S.mat_codes + S.mat_sz));
        __syncwarp();
        if (lane < n_runs) {
            uint8_t* st = smem + S.stage0 + s * S.stage_bytes;
            const int mt = run >> 1, is_sz = run & 1, m = mt / TG, ti = mt % TG;
            const int n = c * sw + crank * rows_gu + 16 * ti;
            if (!is_sz) bulk_g2s_hint(st + mt * S.mat_codes, rec + (m ? p.L.codes_up : p.L.codes_gate) + code_off(p.H, n, kq * cps),
                                      S.mat_codes, &bars[s], pol);
            else bulk_g2s_hint(st + S.sz0 + mt * S.mat_sz, rec + (m ? p.L.sz_up : p.L.sz_gate) + sz_off(p.H, p.group, n, kq * gpst),
                               S.mat_sz, &bars[s], pol);
        }
    };
    // the adapter slices of item j (the adapter of the tile's first pair; tiles of one slot share it) into buffer j & 1
    auto issue_lora = [&](int j, int ad) {
        const int c = item_quarter(j);
        const uint32_t bgu = rows_gu * r * 2, ad_row = rows_gu * 2;
        uint8_t* buf = smem + S.lora0 + (j & 1) * S.lora_bytes;
        const int n0 = c * sw + crank * rows_gu;
        if (lane == 0) mbar_expect_tx(&bars[SB_LORA + (j & 1)], 2 * bgu + r * ad_row);
        __syncwarp();
        const size_t bo = ((size_t)ad * p.I + n0) * r * 2;
        if (lane == 0) bulk_g2s(buf, static_cast<const uint8_t*>(p.lora.B_gate) + bo, bgu, &bars[SB_LORA + (j & 1)]);
        if (lane == 1) bulk_g2s(buf + bgu, static_cast<const uint8_t*>(p.lora.B_up) + bo, bgu, &bars[SB_LORA + (j & 1)]);
        for (int q = lane; q < r; q += 32)
            bulk_g2s(buf + 2 * bgu + q * ad_row, static_cast<const uint8_t*>(p.lora.A_down) + (((size_t)ad * r + q) * p.I + n0) * 2,
                     ad_row, &bars[SB_LORA + (j & 1)]);
    };
    // adapter of a tile: that of its first pair (a slot holds one expert, so all its pairs agree)
    auto tile_adapter = [&](int j) {
        const int tile = (cl + j * n_cl) >> 2;
        const int pr = p.lists[(size_t)p.tiles[2 * tile] * p.T + p.tiles[2 * tile + 1]];
        return r > 0 ? p.pair_ad[pr] : 0;
    };

    // the tile record of item j: x fragments, sums and projections into the one buffer, the pair table into buffer j & 1
    auto issue_x = [&](int j) {
        if (warp == SW_ - 2 && lane == 2) {
            const uint8_t* src = sp.xt + (size_t)((cl + j * n_cl) >> 2) * xt_stride;
            mbar_expect_tx(&bars[SB_X], S.g_small);
            bulk_g2s(smem + S.u + (j & 1) * S.g_small, src + S.g_u, S.g_small, &bars[SB_X]);
        }
    };
    issue_gu(0, 0);
    issue_x(0);
    if (r > 0 && warp == SW_ - 1) issue_lora(0, tile_adapter(0));

#pragma unroll 1
    for (int j = 0; j < my_items; ++j) {
        const int it = cl + j * n_cl, tile = it >> 2, c = it & 3;
        const int slot = p.tiles[2 * tile], first = p.tiles[2 * tile + 1];
        const uint8_t* rec = p.pool + (size_t)slot * p.L.bytes;
        const uint32_t par = j & 1, par2 = (j >> 1) & 1;

        // ---- the tile's pairs, their tokens' states as the B operand (fp16, k-slot order), block sums
        // ---- the tile's record (pairs, their tokens' states as the B operand, block sums, projections) has been on its way
        mbar_wait(&bars[SB_X], par, p.status);
        const float* s_u = reinterpret_cast<const float*>(smem + S.u + par * S.g_small);                // [ST][2][r]
        const int* s_pair = reinterpret_cast<const int*>(smem + S.info + par * S.g_small);   // [8] pair, [8] gate bits, [8] adapter, [8] token
        const uint8_t* trec = sp.xt + (size_t)tile * xt_stride;                               // the tile's x fragments and sums, in the L2
        const int* s_gate = s_pair + 8;
        const int ad = s_pair[16];
        // ---- gate/up: warp w owns K slice w of each half for every (matrix, row tile); 8 token columns
        {
            const int s = warp / 2;
            const uint8_t* st = smem + S.stage0 + s * S.stage_bytes;
            const int ch0 = (warp & 1) * NCW;
            float a[NT][4];
#pragma unroll
            for (int mt = 0; mt < NT; ++mt) { a[mt][0] = 0.f; a[mt][1] = 0.f; a[mt][2] = 0.f; a[mt][3] = 0.f; }
            const uint8_t* cbase = st + ch0 * 256 + g8 * 16 + t4 * 4;
#pragma unroll 1
            for (int half = 0; half < 2; ++half) {
                const int vw = warp + SW_ * half;
                // this warp's B words of the half (token g8) and the block sums of its two tokens: asked for before the
                // wait for the weights, so both trips overlap
                uint4 xbw[NCW];
                float2 xsw[NCW / CPB], xbw2[NCW / CPB];
                {
                    const uint4* xbp = reinterpret_cast<const uint4*>(trec) + g8 * (p.H / 8) + (vw * NCW) * 4 + t4;
#pragma unroll
                    for (int i = 0; i < NCW; ++i) xbw[i] = __ldg(xbp + i * 4);
                    const float* xsp = reinterpret_cast<const float*>(trec + S.g_xsum) + ((vw * NCW) / CPB) * ST + 2 * t4;
                    const float* xbp2 = reinterpret_cast<const float*>(trec + S.g_xbias) + ((vw * NCW) / CPB) * ST + 2 * t4;
#pragma unroll
                    for (int i = 0; i < NCW / CPB; ++i) {
                        xsw[i] = __ldg(reinterpret_cast<const float2*>(xsp + i * ST));
                        xbw2[i] = __ldg(reinterpret_cast<const float2*>(xbp2 + i * ST));
                    }
                }
                mbar_wait(&bars[s], half, p.status);
#pragma unroll
                for (int ib = 0; ib < NCW / CPB; ++ib) {
                    float cfr[NT][4];
#pragma unroll
                    for (int u = 0; u < CPB; ++u) {
                        const int i = ib * CPB + u;
                        const uint4 xb = xbw[i];
#pragma unroll
                        for (int mt = 0; mt < NT; ++mt) {
                            const uint8_t* cw = cbase + mt * S.mat_codes + i * 256;
                            uint32_t alo[4], ahi[4];
                            dequant_word_b(*reinterpret_cast<const uint32_t*>(cw), alo);
                            dequant_word_b(*reinterpret_cast<const uint32_t*>(cw + 128), ahi);
                            if (u == 0) mma16816_zero(cfr[mt], alo[0], ahi[0], alo[1], ahi[1], xb.x, xb.y);
                            else mma16816(cfr[mt], alo[0], ahi[0], alo[1], ahi[1], xb.x, xb.y);
                            mma16816(cfr[mt], alo[2], ahi[2], alo[3], ahi[3], xb.z, xb.w);
                        }
                    }
                    const int gi = ((ch0 + ib * CPB) * 32) >> sp.gshift;
                    const float2 xs = xsw[ib], xbi = xbw2[ib];
#pragma unroll
                    for (int mt = 0; mt < NT; ++mt) {
                        const uint8_t* zw = st + S.sz0 + mt * S.mat_sz + gi * 64 + g8 * 4;
                        const __half2 z0 = u32_as_h2(*reinterpret_cast<const uint32_t*>(zw));
                        const __half2 z1 = u32_as_h2(*reinterpret_cast<const uint32_t*>(zw + 32));
                        const float s0 = __low2float(z0), q0 = __high2float(z0), s1 = __low2float(z1), q1 = __high2float(z1);
                        a[mt][0] = fmaf(s0, fmaf(-q0, xs.x, cfr[mt][0] - xbi.x), a[mt][0]);
                        a[mt][1] = fmaf(s0, fmaf(-q0, xs.y, cfr[mt][1] - xbi.y), a[mt][1]);
                        a[mt][2] = fmaf(s1, fmaf(-q1, xs.x, cfr[mt][2] - xbi.x), a[mt][2]);
                        a[mt][3] = fmaf(s1, fmaf(-q1, xs.y, cfr[mt][3] - xbi.y), a[mt][3]);
                    }
                }
                if (half == 0) {
                    __syncthreads();
                    issue_gu(j, 1);
                }
            }
            // the adapter's B rows as one more k-step per 16 ranks, by one warp: a += B[rows][r] . (sigma A x)[r][token]
            if (r > 0 && warp == 0) {
                mbar_wait(&bars[SB_LORA + par], par2, p.status);
                const uint16_t* lb = reinterpret_cast<const uint16_t*>(smem + S.lora0 + par * S.lora_bytes);
                for (int kr = 0; kr < r; kr += 16) {
#pragma unroll
                    for (int mt = 0; mt < NT; ++mt) {
                        uint32_t b0, b1;
                        lora_bwords(s_u + (g8 * 2 + mt / TG) * r, kr, r, t4, p.sigma, b0, b1);
                        lora_step(a[mt], lb + (size_t)(mt * 16 + g8) * r, lb + (size_t)(mt * 16 + 8 + g8) * r, kr, r, t4, b0, b1);
                    }
                }
            }
#pragma unroll
            for (int mt = 0; mt < NT; ++mt) {
                float* pr = s_part + ((size_t)warp * 2 * rows_gu + mt * 16 + g8) * ST + 2 * t4;
                *reinterpret_cast<float2*>(pr) = make_float2(a[mt][0], a[mt][1]);
                *reinterpret_cast<float2*>(pr + 8 * ST) = make_float2(a[mt][2], a[mt][3]);
            }
        }
        __syncthreads();
        // both stages are free: the quarter's down block follows; so is the x buffer: the next item's tile record
        if (j + 1 < my_items) issue_x(j + 1);
        if (warp == SW_ - 2 && lane < 2) {
            const uint64_t pol = policy_evict_first();
            const uint32_t dcb = (uint32_t)rows_d * sw / 2, dzb = (uint32_t)rows_d * gps * 4;
            if (lane == 0) mbar_expect_tx(&bars[SB_DOWN], dcb + dzb);
            __syncwarp(0x3u);
            if (lane == 0) bulk_g2s_hint(smem + S.d_codes, rec + p.L.codes_down + down_code_off(p.H, p.I, n0_d, c * (sw / 32)), dcb, &bars[SB_DOWN], pol);
            else bulk_g2s_hint(smem + S.d_sz, rec + p.L.sz_down + down_sz_off(p.H, p.I, p.group, n0_d, c * gps), dzb, &bars[SB_DOWN], pol);
        }
        // sum the K slices
        for (int i = tid * 4; i < 2 * rows_gu * ST; i += SW_ * 32 * 4) {
            float4 v = *reinterpret_cast<const float4*>(&s_part[i]);
#pragma unroll
            for (int w = 1; w < SW_; ++w) {
                const float4 t = *reinterpret_cast<const float4*>(&s_part[(size_t)w * 2 * rows_gu * ST + i]);
                v.x += t.x; v.y += t.y; v.z += t.z; v.w += t.w;
            }
            *reinterpret_cast<float4*>(&s_gu[i]) = v;
        }
        __syncthreads();

        // ---- SiLU, product
        const uint8_t* lbuf = smem + S.lora0 + par * S.lora_bytes;
        if (r > 0) mbar_wait(&bars[SB_LORA + par], par2, p.status);      // (every thread reads the staged slices below)
        for (int i = tid; i < rows_gu * ST; i += SW_ * 32) s_hloc[i] = silu_f(s_gu[i]) * s_gu[rows_gu * ST + i];
        __syncthreads();
        // all-gather h inside the cluster: this CTA's rows_gu x 8 values go to every CTA, 16 bytes at a time
        float* hq = s_h + par * sw * ST;
        {
            constexpr int vecs = rows_gu * ST / 4;
            for (int i = tid; i < vecs * SC; i += SW_ * 32) {
                const int v = i % vecs, dst = i / vecs;
                st_async_f32x4(map_to_cta(&hq[crank * rows_gu * ST + 4 * v], dst), *reinterpret_cast<const float4*>(&s_hloc[4 * v]),
                               map_to_cta(&bars[SB_H + par], dst));
            }
        }
        // partial of A_down . h over this CTA's rows of h on the tensor cores (one warp): [r x rows_gu] . [rows_gu x 8 tokens],
        // sent to every CTA of the cluster
        float* udp = s_udp + par * SC * ST * r;
        if (r > 0 && warp == 1) {
            const uint16_t* Ad = reinterpret_cast<const uint16_t*>(lbuf + 2 * rows_gu * r * 2);     // [r][rows_gu]
            for (int jr = 0; jr < r; jr += 16) {
                float cc[4] = {0.f, 0.f, 0.f, 0.f};
                for (int kk = 0; kk < rows_gu; kk += 16) {
                    const int k0 = kk + 2 * t4, k1 = k0 + 8;
                    const uint32_t b0 = h2_as_u32(__floats2half2_rn(s_hloc[k0 * ST + g8], s_hloc[(k0 + 1) * ST + g8]));
                    const uint32_t b1 = h2_as_u32(__floats2half2_rn(s_hloc[k1 * ST + g8], s_hloc[(k1 + 1) * ST + g8]));
                    const bool lo_ok = jr + g8 < r, hi_ok = jr + 8 + g8 < r;
                    const uint16_t* rg = Ad + (size_t)(jr + g8) * rows_gu;
                    const uint16_t* rg8 = Ad + (size_t)(jr + 8 + g8) * rows_gu;
                    const uint32_t a0 = lo_ok ? bf16x2_to_h2(*reinterpret_cast<const uint32_t*>(rg + k0)) : 0u;
                    const uint32_t a1 = hi_ok ? bf16x2_to_h2(*reinterpret_cast<const uint32_t*>(rg8 + k0)) : 0u;
                    const uint32_t a2 = lo_ok ? bf16x2_to_h2(*reinterpret_cast<const uint32_t*>(rg + k1)) : 0u;
                    const uint32_t a3 = hi_ok ? bf16x2_to_h2(*reinterpret_cast<const uint32_t*>(rg8 + k1)) : 0u;
                    mma16816(cc, a0, a1, a2, a3, b0, b1);
                }
                // cc: (rank jr + g8, tokens 2 t4, 2 t4 + 1), (rank jr + 8 + g8, the same tokens)
                for (int dst = 0; dst < SC; ++dst) {
                    const uint32_t rb = map_to_cta(&bars[SB_H + par], dst);
                    if (jr + g8 < r) {
                        st_async_f32(map_to_cta(&udp[(crank * ST + 2 * t4) * r + jr + g8], dst), cc[0], rb);
                        st_async_f32(map_to_cta(&udp[(crank * ST + 2 * t4 + 1) * r + jr + g8], dst), cc[1], rb);
                    }
                    if (jr + 8 + g8 < r) {
                        st_async_f32(map_to_cta(&udp[(crank * ST + 2 * t4) * r + jr + 8 + g8], dst), cc[2], rb);
                        st_async_f32(map_to_cta(&udp[(crank * ST + 2 * t4 + 1) * r + jr + 8 + g8], dst), cc[3], rb);
                    }
                }
            }
        }
        mbar_wait(&bars[SB_H + par], par2, p.status);

        // ---- h as the B operand of down (fp16 value and residual per token), block sums, A_down h
        for (int i = tid; i < ST * r; i += SW_ * 32) {
            float v = 0.f;
            for (int cc = 0; cc < SC; ++cc) v += udp[cc * ST * r + i];
            s_ud[i] = v;
        }
        for (int i = tid; i < DCH * 2 * ST * 4; i += SW_ * 32) {
            const int q = i & 3, tk = (i >> 2) % ST, lo = ((i >> 2) / ST) & 1, ch = (i >> 2) / (2 * ST);
            float f[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] = hq[(ch * 32 + q * 8 + e) * ST + tk];
            s_hb[i] = lo ? permute8_lo(f) : permute8(f);
        }
        for (int base = 0; base < (DCH / CPB) * ST; base += SW_ * 4) {
            // (block, token) sums over 32 CPB values: 8 threads each, 16 sums per round
            const int bt = base + (tid >> 3), sub = tid & 7;
            float v = 0.f, vo = 0.f;
            if (bt < (DCH / CPB) * ST) {
                const int blk = bt / ST, tk = bt % ST;
                for (int e = sub * 4 * CPB; e < (sub + 1) * 4 * CPB; e += 2) {
                    v += hq[(blk * 32 * CPB + e) * ST + tk];
                    vo += hq[(blk * 32 * CPB + e + 1) * ST + tk];
                }
            }
            v = group_sum<8>(v);
            vo = group_sum<8>(vo);
            if (bt < (DCH / CPB) * ST && sub == 0) {
                s_hsum[bt] = v + vo;
                s_hbias[bt] = fmaf(1024.f, v, 64.f * vo);
            }
        }
        __syncthreads();
        if (tid == 0 && j + 2 < my_items) mbar_expect_tx(&bars[SB_H + par], h_bytes);
        mbar_wait(&bars[SB_DOWN], par, p.status);

        // ---- down: this quarter's columns for this CTA's H/4 output rows; two MMAs per k-step (h value, h residual)
        {
            const uint8_t* dbase = smem + S.d_codes + g8 * 16 + t4 * 4;
            const uint8_t* dsz = smem + S.d_sz;
            const int pa = s_pair[2 * t4], pb = s_pair[2 * t4 + 1];
            const float ga = __int_as_float(s_gate[2 * t4]), gb = __int_as_float(s_gate[2 * t4 + 1]);
            const uint16_t* Bd = static_cast<const uint16_t*>(p.lora.B_down) + ((size_t)ad * p.H + n0_d) * r;
#pragma unroll 1
            for (int ps = 0; ps < 2; ++ps) {
                float acc[TD][4];
#pragma unroll
                for (int tt = 0; tt < TD; ++tt) { acc[tt][0] = 0.f; acc[tt][1] = 0.f; acc[tt][2] = 0.f; acc[tt][3] = 0.f; }
                // the B_down words of this pass's row tiles (first 16 ranks) are asked for now and used in the epilogue
                uint32_t bd[TD][4];
                if (r > 0) {
#pragma unroll
                    for (int tt = 0; tt < TD; ++tt) {
                        const int ti = warp + SW_ * (ps * TD + tt);
                        const uint16_t* rg = Bd + (size_t)(ti * 16 + g8) * r;
                        const uint16_t* rg8 = rg + (size_t)8 * r;
                        const int k0 = 2 * t4, k1 = k0 + 8;
                        bd[tt][0] = __ldg(reinterpret_cast<const uint32_t*>(rg + k0));
                        bd[tt][1] = __ldg(reinterpret_cast<const uint32_t*>(rg8 + k0));
                        bd[tt][2] = k1 < r ? __ldg(reinterpret_cast<const uint32_t*>(rg + k1)) : 0u;
                        bd[tt][3] = k1 < r ? __ldg(reinterpret_cast<const uint32_t*>(rg8 + k1)) : 0u;
                    }
                }
#pragma unroll 1
                for (int ib = 0; ib < DCH / CPB; ++ib) {
                    float cfr[TD][4];
#pragma unroll
                    for (int u = 0; u < CPB; ++u) {
                        const int i = ib * CPB + u;
                        const uint4 hv = s_hb[((i * 2 + 0) * ST + g8) * 4 + t4];
                        const uint4 hl = s_hb[((i * 2 + 1) * ST + g8) * 4 + t4];
#pragma unroll
                        for (int tt = 0; tt < TD; ++tt) {
                            const int ti = warp + SW_ * (ps * TD + tt);
                            const uint8_t* cw = dbase + (ti * DCH + i) * 256;
                            uint32_t alo[4], ahi[4];
                            dequant_word_b(*reinterpret_cast<const uint32_t*>(cw), alo);
                            dequant_word_b(*reinterpret_cast<const uint32_t*>(cw + 128), ahi);
                            if (u == 0) mma16816_zero(cfr[tt], alo[0], ahi[0], alo[1], ahi[1], hv.x, hv.y);
                            else mma16816(cfr[tt], alo[0], ahi[0], alo[1], ahi[1], hv.x, hv.y);
                            mma16816(cfr[tt], alo[2], ahi[2], alo[3], ahi[3], hv.z, hv.w);
                            mma16816(cfr[tt], alo[0], ahi[0], alo[1], ahi[1], hl.x, hl.y);
                            mma16816(cfr[tt], alo[2], ahi[2], alo[3], ahi[3], hl.z, hl.w);
                        }
                    }
                    const int gi = (ib * CPB * 32) >> sp.gshift;
                    const float2 hs = *reinterpret_cast<const float2*>(&s_hsum[ib * ST + 2 * t4]);
                    const float2 hbi = *reinterpret_cast<const float2*>(&s_hbias[ib * ST + 2 * t4]);
#pragma unroll
                    for (int tt = 0; tt < TD; ++tt) {
                        const int ti = warp + SW_ * (ps * TD + tt);
                        const uint8_t* zw = dsz + (ti * gps + gi) * 64 + g8 * 4;
                        const __half2 z0 = u32_as_h2(*reinterpret_cast<const uint32_t*>(zw));
                        const __half2 z1 = u32_as_h2(*reinterpret_cast<const uint32_t*>(zw + 32));
                        const float s0 = __low2float(z0), q0 = __high2float(z0), s1 = __low2float(z1), q1 = __high2float(z1);
                        acc[tt][0] = fmaf(s0, fmaf(-q0, hs.x, cfr[tt][0] - hbi.x), acc[tt][0]);
                        acc[tt][1] = fmaf(s0, fmaf(-q0, hs.y, cfr[tt][1] - hbi.y), acc[tt][1]);
                        acc[tt][2] = fmaf(s1, fmaf(-q1, hs.x, cfr[tt][2] - hbi.x), acc[tt][2]);
                        acc[tt][3] = fmaf(s1, fmaf(-q1, hs.y, cfr[tt][3] - hbi.y), acc[tt][3]);
                    }
                }
                // epilogue: + sigma B_down (A_down h), gate weight, the pair's partial rows of this quarter
#pragma unroll
                for (int tt = 0; tt < TD; ++tt) {
                    const int ti = warp + SW_ * (ps * TD + tt);
                    const int r_lo = ti * 16 + g8, r_hi = r_lo + 8;
                    // B_down rows as one more k-step per 16 ranks: acc += B_down[rows][r] . (sigma A_down h)[r][token]
                    if (r > 0) {
                        uint32_t b0, b1;
                        lora_bwords(s_ud + g8 * r, 0, r, t4, p.sigma, b0, b1);
                        mma16816(acc[tt], bf16x2_to_h2(bd[tt][0]), bf16x2_to_h2(bd[tt][1]), bf16x2_to_h2(bd[tt][2]), bf16x2_to_h2(bd[tt][3]), b0, b1);
                    }
                    for (int kr = 16; kr < r; kr += 16) {
                        uint32_t b0, b1;
                        lora_bwords(s_ud + g8 * r, kr, r, t4, p.sigma, b0, b1);
                        lora_step(acc[tt], Bd + (size_t)r_lo * r, Bd + (size_t)r_hi * r, kr, r, t4, b0, b1);
                    }
                    if (pa >= 0) {
                        float* o = sp.o_part + ((size_t)pa * 4 + c) * p.H + n0_d;
                        o[r_lo] = ga * acc[tt][0];
                        o[r_hi] = ga * acc[tt][2];
                    }
                    if (pb >= 0) {
                        float* o = sp.o_part + ((size_t)pb * 4 + c) * p.H + n0_d;
                        o[r_lo] = gb * acc[tt][1];
                        o[r_hi] = gb * acc[tt][3];
                    }
                }
            }
        }
        // the next item's first half of K once every warp is done with the down block
        if (j + 1 < my_items) {
            __syncthreads();
            issue_gu(j + 1, 0);
            if (r > 0 && warp == SW_ - 1) issue_lora(j + 1, tile_adapter(j + 1));
        }
    }
}

// Pre-pass, one CTA per tile: everything an item of the tile needs besides the weights, in the order the streaming
// kernel keeps it in shared memory -- the tokens' states as fp16 B words in k-slot order, their per-block sums (plain
// and as the biased codes weigh them), the rank-r projections A_gate x / A_up x, and the pair table.
template <int CPB>
__global__ void __launch_bounds__(256) stream_tile_kernel(StreamParams sp) {
    const GroupedParams& p = sp.g;
    const StreamSmem& S = sp.S;
    const int tile = blockIdx.x;
    if (tile >= *p.n_tiles) return;
    const int slot = p.tiles[2 * tile], first = p.tiles[2 * tile + 1];
    const int cnt = min(ST, p.counts[slot] - first);
    uint8_t* rec = sp.xt + (size_t)tile * S.g_bytes;
    uint4* xb = reinterpret_cast<uint4*>(rec);
    float* xsum = reinterpret_cast<float*>(rec + S.g_xsum);
    float* xbias = reinterpret_cast<float*>(rec + S.g_xbias);
    float* u = reinterpret_cast<float*>(rec + S.g_u);
    int* info = reinterpret_cast<int*>(rec + S.g_u + S.g_small - 128);
    __shared__ int s_pr[ST];
    const int tid = threadIdx.x;
    if (tid < ST) {
        const int pr = tid < cnt ? p.lists[(size_t)slot * p.T + first + tid] : -1;
        s_pr[tid] = pr;
        info[tid] = pr;
        info[8 + tid] = pr >= 0 ? __float_as_int(p.gates[pr]) : 0;
        info[16 + tid] = pr >= 0 ? p.pair_ad[pr] : 0;
        info[24 + tid] = pr >= 0 ? pr / p.K : -1;
    }
    __syncthreads();
    for (int tk = 0; tk < ST; ++tk) {
        const int tok = s_pr[tk] >= 0 ? s_pr[tk] / p.K : -1;
        for (int t0 = 0; t0 * 8 < p.H; t0 += 256) {
            const int t = t0 + tid;
            float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            if (tok >= 0 && t * 8 < p.H) {
                const uint4 v = *reinterpret_cast<const uint4*>(p.x + (size_t)tok * p.H + t * 8);
                f[0] = bf16_lo(v.x); f[1] = bf16_hi(v.x); f[2] = bf16_lo(v.y); f[3] = bf16_hi(v.y);
                f[4] = bf16_lo(v.z); f[5] = bf16_hi(v.z); f[6] = bf16_lo(v.w); f[7] = bf16_hi(v.w);
            }
            float sum = 0.f, sodd = 0.f;
#pragma unroll
            for (int e = 0; e < 8; e += 2) {
                sum += __half2float(__float2half_rn(f[e]));
                sodd += __half2float(__float2half_rn(f[e + 1]));
            }
            sum = group_sum<4 * CPB>(sum);
            sodd = group_sum<4 * CPB>(sodd);
            if (t * 8 < p.H) {
                xb[tk * (p.H / 8) + t] = permute8(f);
                if ((t % (4 * CPB)) == 0) {
                    xsum[(t / (4 * CPB)) * ST + tk] = sum + sodd;
                    xbias[(t / (4 * CPB)) * ST + tk] = fmaf(1024.f, sum, 64.f * sodd);
                }
            }
        }
    }
    if (p.rank > 0) {
        const int r = p.rank, n_sets = p.n_adapters == 1 ? 1 : p.K;
        for (int i = tid; i < ST * 2 * r; i += 256) {
            const int tk = i / (2 * r), q = i % (2 * r), pr = s_pr[tk];
            u[i] = pr >= 0 ? p.u_gu[(((size_t)(pr / p.K) * n_sets + (p.n_adapters == 1 ? 0 : pr % p.K)) * 2) * r + q] : 0.f;
        }
    }
}

// y[t] = sum over the token's K choices and the four quarters of each, in a fixed order
template <typename OutT>
__global__ void __launch_bounds__(256) reduce_parts_kernel(StreamParams sp) {
    const GroupedParams& p = sp.g;
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)p.T * p.H) return;
    const int t = (int)(i / p.H), n = (int)(i % p.H);
    float v = 0.f;
    for (int k = 0; k < p.K; ++k) {
        const int pair = t * p.K + k;
        if (p.pair_slot[pair] < 0) continue;
        const float* o = sp.o_part + (size_t)pair * 4 * p.H + n;
        v += (o[0] + o[p.H]) + (o[2 * (size_t)p.H] + o[3 * (size_t)p.H]);
    }
    store_out<OutT>(reinterpret_cast<OutT*>(p.y), i, v);
}

constexpr size_t kStreamSmemLimit = 113 * 1024;    // two CTAs per SM at the largest ranks, three up to rank 16

bool grouped_stream_supported(const edg_layer_desc& d) {
    if (!((d.H == 1024 || d.H == 2048) && (d.I == 256 || d.I == 512))) return false;
    if (d.group > 128 || (d.group & (d.group - 1)) != 0) return false;
    if (d.rank % 8 != 0 || d.rank > SMaxRank) return false;
    return stream_smem(d.H, d.I, d.group, d.rank).total <= kStreamSmemLimit;
}

template <int NCW, int DCH, int TG, int TD, int CPB>
static cudaError_t launch_stream(const StreamParams& sp, cudaStream_t st) {
    auto kern = grouped_stream_kernel<NCW, DCH, TG, TD, CPB>;
    static bool configured = false;
    static int n_clusters = 0;          // clusters the device holds at once: the persistent grid
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStreamSmemLimit);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(SC, 1, 1);
    cfg.blockDim = dim3(SW_ * 32, 1, 1);
    cfg.dynamicSmemBytes = sp.S.total;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = SC;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (!configured) {
        // (fewer than two clusters' worth per four SMs where a GPC has an odd number of SMs: ask)
        cudaError_t e = cudaOccupancyMaxActiveClusters(&n_clusters, kern, &cfg);
        if (e != cudaSuccess) return e;
        if (n_clusters < 1) return cudaErrorLaunchOutOfResources;
        configured = true;
    }
    cfg.gridDim = dim3(n_clusters * SC, 1, 1);          // persistent: every cluster resident from the start
    return cudaLaunchKernelEx(&cfg, kern, sp);
}

// the two tile kernels and the reduce of the small-group path in one streaming kernel + reduce
int32_t run_grouped_stream(const edg_layer_desc* d, const GroupedParams& g, float* o_part, uint8_t* xt, int max_tiles, cudaStream_t st) {
    StreamParams sp{};
    sp.g = g;
    sp.o_part = o_part;
    sp.xt = xt;
    sp.S = stream_smem(d->H, d->I, d->group, g.rank);
    sp.gshift = 0;
    while ((1 << sp.gshift) < d->group) ++sp.gshift;
    cudaError_t e;
    const bool wide = d->group >= 64;
    if (wide) stream_tile_kernel<2><<<max_tiles, 256, 0, st>>>(sp);
    else stream_tile_kernel<1><<<max_tiles, 256, 0, st>>>(sp);
    if (d->H == 2048 && d->I == 512) e = wide ? launch_stream<8, 4, 2, 4, 2>(sp, st) : launch_stream<8, 4, 2, 4, 1>(sp, st);
    else if (d->H == 2048 && d->I == 256) e = wide ? launch_stream<8, 2, 1, 4, 2>(sp, st) : launch_stream<8, 2, 1, 4, 1>(sp, st);
    else if (d->H == 1024 && d->I == 512) e = wide ? launch_stream<4, 4, 2, 2, 2>(sp, st) : launch_stream<4, 4, 2, 2, 1>(sp, st);
    else if (d->H == 1024 && d->I == 256) e = wide ? launch_stream<4, 2, 1, 2, 2>(sp, st) : launch_stream<4, 2, 1, 2, 1>(sp, st);
    else return EDG_E_SHAPE;
    EDG_CUDA_TRY(e);
    const size_t n_out = (size_t)g.T * d->H;
    const int rb = (int)((n_out + 255) / 256);
    if (d->out_dtype == EDG_F32) reduce_parts_kernel<float><<<rb, 256, 0, st>>>(sp);
    else if (d->out_dtype == EDG_F16) reduce_parts_kernel<__half><<<rb, 256, 0, st>>>(sp);
    else reduce_parts_kernel<bf16_t><<<rb, 256, 0, st>>>(sp);
    EDG_CUDA_TRY(cudaGetLastError());
    return EDG_OK;
}

}  // namespace edg

namespace edg {
size_t grouped_stream_tile_bytes(const edg_layer_desc& d) {
    return stream_smem(d.H, d.I, d.group, d.rank).g_bytes;
}
}  // namespace edg
