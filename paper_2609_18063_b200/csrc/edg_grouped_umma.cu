// a4'-a6' grouped form for large token groups (prefill) on the 5th-generation tensor cores.
//
// A CTA computes a tile [128 weight rows] x [up to 128 tokens of one expert]: the expert's weights are
// the A operand (M = 128), the gathered token states the B operand (N = tokens), both K-major in shared
// memory; tcgen05.mma accumulates in tensor memory (fp32), one elected thread issues, completion is
// tracked by tcgen05.commit on mbarriers, and the epilogue reads the accumulators with tcgen05.ld.
//
// Exact weights from fp16 operands.  w = s * (q - z) has up to 16 significant bits (11 of the fp16
// scale, 5 of the integer), one fp16 cannot hold it, and rounding it costs more than the parity bar
// allows.  So every weight is fed as two fp16 values: hi = fp16(s (q - z)) and the residual
// lo = s (q - z) - hi, which is exact (an fma computes it without rounding); the tile is multiplied
// twice into the same accumulator.  The bf16 activations convert to fp16 exactly; the fp32 h of the
// down projection is fed as an fp16 value plus an fp16 residual (hi.hi + lo.hi + hi.lo).
//
// Operand layout in shared memory (no swizzle): core matrices of 8 rows x 16 bytes, a [128 x 32] fp16
// tile being [k core 0..3][row group 0..15][8 rows][16 B]; the descriptor's leading byte offset is the
// distance between k cores (2048), its stride byte offset the distance between row groups (128).
// The 8 k values of a core row are kept in the order (k0,k4,k1,k5,k2,k6,k3,k7) in which the int4 codes
// come out of a 32-bit word -- for A and B alike, so the dot product is unchanged.
//
// Warps 0-7 (two threads per weight row and per token, each covering half of a stage's k) dequantise /
// convert into a ring of two (gate/up) or three (down) stages, with the loads of the next chunk in flight while the current one is
// processed, and later run the epilogue (each warp its 32 lanes of tensor memory, half of the token
// columns); warp 8 allocates the tensor memory and its lane 0 issues the MMAs.
// Every wait is bounded: a wait that gives up raises the status word and the kernel still frees its
// tensor memory and returns.
#include "edg_grouped.cuh"

namespace edg {
namespace {

constexpr int U_TN = kUmmaTokens;            // token columns per tile
constexpr int U_KC = 32;                     // k per stage
constexpr int U_STAGES_MAX = 3;
constexpr uint32_t U_TILE = 128 * U_KC * 2;  // bytes of a [128 x 32] fp16 operand tile
constexpr uint32_t U_LBO = 16 * 128;         // between k cores
constexpr uint32_t U_SBO = 128;              // between row groups
constexpr uint32_t U_SPIN = 1u << 22;
constexpr int U_PROD_WARPS = 8;
constexpr int U_THREADS = (U_PROD_WARPS + 1) * 32;

__device__ __forceinline__ uint32_t s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(uint64_t* b, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_arrive(uint64_t* b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s32(b)) : "memory");
}
__device__ __forceinline__ void bar_wait(uint64_t* b, uint32_t parity, int32_t* status) {
    uint32_t ok = 0, it = 0;
    while (!ok && ++it < U_SPIN)
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                     : "=r"(ok) : "r"(s32(b)), "r"(parity) : "memory");
    if (!ok) atomicExch(status, EDG_E_TIMEOUT);
}
// shared-memory matrix descriptor: K-major, no swizzle
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)((U_LBO >> 4) & 0x3FFF) << 16) |
           ((uint64_t)((U_SBO >> 4) & 0x3FFF) << 32) | ((uint64_t)1 << 46);
}
// instruction descriptor: fp32 accumulator, fp16 A and B, both K-major, M = 128, N = n
__device__ __forceinline__ uint32_t umma_idesc(int n) {
    return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, bool accumulate) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate ? 1u : 0u) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* b) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(s32(b)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr));
}

// offset of (row r, k core kc) inside an operand tile
__device__ __forceinline__ uint32_t core_off(int r, int kc) { return (uint32_t)(((kc * 16 + (r >> 3)) * 8 + (r & 7)) * 16); }

// One 32-bit word = 8 codes of a row -> the core row of s (q - z): fp16 value and exact fp16 residual.
__device__ __forceinline__ void dequant_hi_lo(uint32_t w, __half2 s2, __half2 z2, uint4& hi, uint4& lo) {
    uint32_t q[4];
    dequant_word(w, z2, q);                              // (q - z): (k0,k4) (k1,k5) (k2,k6) (k3,k7)
    uint32_t h[4], l[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __half2 qz = u32_as_h2(q[i]);
        const __half2 a = __hmul2(s2, qz);
        h[i] = h2_as_u32(a);
        l[i] = h2_as_u32(__hfma2(s2, qz, __hneg2(a)));
    }
    hi = make_uint4(h[0], h[1], h[2], h[3]);
    lo = make_uint4(l[0], l[1], l[2], l[3]);
}

// 8 bf16 -> 8 fp16 in natural order (adapter matrices)
__device__ __forceinline__ uint4 bf16x8_to_f16(uint4 v) {
    uint4 o;
    o.x = h2_as_u32(__floats2half2_rn(bf16_lo(v.x), bf16_hi(v.x)));
    o.y = h2_as_u32(__floats2half2_rn(bf16_lo(v.y), bf16_hi(v.y)));
    o.z = h2_as_u32(__floats2half2_rn(bf16_lo(v.z), bf16_hi(v.z)));
    o.w = h2_as_u32(__floats2half2_rn(bf16_lo(v.w), bf16_hi(v.w)));
    return o;
}
// 8 fp32 * sigma -> 8 fp16 in natural order; missing entries (j >= n) are zero
__device__ __forceinline__ uint4 f32x8_to_f16(const float* src, int n, float sigma) {
    float f[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) f[j] = (src != nullptr && j < n) ? sigma * src[j] : 0.f;
    uint4 o;
    o.x = h2_as_u32(__floats2half2_rn(f[0], f[1]));
    o.y = h2_as_u32(__floats2half2_rn(f[2], f[3]));
    o.z = h2_as_u32(__floats2half2_rn(f[4], f[5]));
    o.w = h2_as_u32(__floats2half2_rn(f[6], f[7]));
    return o;
}

struct UmmaSmem {
    uint8_t* stage[U_STAGES_MAX];
    uint64_t* full;     // [stages] operands written (one arrival per producer warp)
    uint64_t* empty;    // [stages] MMAs that read the stage have completed
    uint64_t* done;     // all MMAs of the tile have completed
    uint32_t* tptr;
    int* pair;          // [U_TN]
};
__device__ __forceinline__ UmmaSmem carve(uint8_t* smem, int tiles_per_stage, int stages) {
    UmmaSmem S;
    for (int s = 0; s < U_STAGES_MAX; ++s) S.stage[s] = smem + (size_t)(s < stages ? s : 0) * tiles_per_stage * U_TILE;
    uint8_t* o = smem + (size_t)stages * tiles_per_stage * U_TILE;
    S.full = reinterpret_cast<uint64_t*>(o);
    S.empty = S.full + U_STAGES_MAX;
    S.done = S.empty + U_STAGES_MAX;
    S.tptr = reinterpret_cast<uint32_t*>(S.done + 1);
    S.pair = reinterpret_cast<int*>(S.tptr + 2);
    return S;
}
constexpr size_t umma_smem_bytes(int tiles_per_stage, int stages) { return (size_t)stages * tiles_per_stage * U_TILE + 128 + U_TN * 4; }
constexpr int U_STAGES_GU = 2, U_STAGES_D = 2;

// common prologue: pair list, barriers, tensor memory
__device__ __forceinline__ uint32_t umma_begin(const GroupedParams& p, const UmmaSmem& S, int slot, int first, int cnt, int cols, int full_count) {
    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid < U_TN) S.pair[tid] = tid < cnt ? p.lists[(size_t)slot * p.T + first + tid] : -1;
    if (tid == 0) {
        for (int s = 0; s < U_STAGES_MAX; ++s) { bar_init(&S.full[s], full_count); bar_init(&S.empty[s], 1); }
        bar_init(S.done, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == U_PROD_WARPS) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s32(S.tptr)), "r"(cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    return *S.tptr;
}
__device__ __forceinline__ void umma_end(uint32_t tmem, int cols) {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if ((threadIdx.x >> 5) == U_PROD_WARPS)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(cols) : "memory");
}
// a producer warp has written its part of a stage
__device__ __forceinline__ void stage_written(uint64_t* full) {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // generic-proxy writes -> visible to the tensor core
    __syncwarp();
    if ((threadIdx.x & 31) == 0) bar_arrive(full);
}

// ---------------------------------------------------------------- token states as operand tiles
// xq[tile][chunk of 32 k][128 tokens x 32 k]: thread = (token of the tile, k core); the four row blocks
// of a tile then fetch every chunk with one bulk copy instead of gathering it again.
__global__ void __launch_bounds__(256) umma_gather_x_kernel(GroupedParams p) {
    const int tile = blockIdx.y;
    if (tile >= *p.n_tiles) return;
    const int slot = p.tiles[2 * tile], first = p.tiles[2 * tile + 1];
    const int cnt = min(U_TN, p.counts[slot] - first);
    const int cores = p.H / 8;                                   // 16-byte pieces per token
    uint8_t* out = p.xq + (size_t)tile * (p.H / 32) * U_TILE;
    // consecutive threads take consecutive tokens of one k core: their 16-byte pieces are adjacent
    // in the operand tile (coalesced writes); the reads are 16 bytes from 128 different rows
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < U_TN * cores; i += gridDim.x * blockDim.x) {
        const int tok = i % U_TN, kcg = i / U_TN;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (tok < cnt) {
            const int pair = p.lists[(size_t)slot * p.T + first + tok];
            const uint4 raw = *reinterpret_cast<const uint4*>(p.x + (size_t)(pair / p.K) * p.H + kcg * 8);
            const float f[8] = {bf16_lo(raw.x), bf16_hi(raw.x), bf16_lo(raw.y), bf16_hi(raw.y),
                                bf16_lo(raw.z), bf16_hi(raw.z), bf16_lo(raw.w), bf16_hi(raw.w)};
            v = permute8(f);
        }
        *reinterpret_cast<uint4*>(out + (size_t)(kcg >> 2) * U_TILE + core_off(tok, kcg & 3)) = v;
    }
}

// ---------------------------------------------------------------- gate/up
// stage = [gate hi][gate lo][up hi][up lo][x] (x by one bulk copy per chunk); tensor memory: gate in
// columns 0..127, up in 128..255.  Thread t dequantises row t % 128 of gate (t < 128) or up.
__global__ void __launch_bounds__(U_THREADS, 2) umma_gate_up_kernel(GroupedParams p) {
    const int tile = blockIdx.y;             // row blocks of a tile are neighbours in the grid: they share its activations in L2
    if (tile >= *p.n_tiles) return;
    extern __shared__ __align__(128) uint8_t smem[];
    const UmmaSmem S = carve(smem, 5, U_STAGES_GU);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = p.tiles[2 * tile], first = p.tiles[2 * tile + 1];
    const int cnt = min(U_TN, p.counts[slot] - first);
    const int row0 = blockIdx.x * 128;
    const uint8_t* rec = p.pool + (size_t)slot * p.L.bytes;
    const uint32_t tmem = umma_begin(p, S, slot, first, cnt, 2 * U_TN, U_PROD_WARPS + 1);
    const int n_chunks = p.H / U_KC;
    const int r_chunks = p.rank > 0 ? (p.rank + 31) / 32 : 0;          // adapter: chunks of up to 32 ranks
    const int gshift = 31 - __clz(p.group);

    if (warp < U_PROD_WARPS) {
        const int r = tid & 127, half = tid >> 7;                    // weight row; matrix (0 gate, 1 up) and, in the epilogue, half of the columns
        const int pair = S.pair[r];
        const uint8_t* xq = p.xq + (size_t)tile * (p.H / 32) * U_TILE;
        const uint8_t* cp = rec + (half ? p.L.codes_up : p.L.codes_gate);
        const uint8_t* zp = rec + (half ? p.L.sz_up : p.L.sz_gate);
        uint4 cw = ld_stream16(cp + code_off(p.H, row0 + r, 0));
        const int n_groups = p.H >> gshift;
        uint32_t nsz = ld_stream4(zp + sz_off(p.H, p.group, row0 + r, 0));      // (scale, zero) one group ahead
        __half2 sc = __float2half2_rn(0.f), zr = sc;
        for (int c = 0; c < n_chunks; ++c) {
            const int st = c % U_STAGES_GU;
            const uint32_t use = (uint32_t)(c / U_STAGES_GU);
            uint4 nw = cw;
            if (c + 1 < n_chunks) nw = ld_stream16(cp + code_off(p.H, row0 + r, c + 1));   // in flight during this chunk
            if (((c * U_KC) & (p.group - 1)) == 0) {                 // a new group: its (scale, zero), and the load of the next
                const __half2 a = u32_as_h2(nsz);
                sc = __low2half2(a); zr = __high2half2(a);
                nsz = ld_stream4(zp + sz_off(p.H, p.group, row0 + r, min(((c * U_KC) >> gshift) + 1, n_groups - 1)));
            }
            bar_wait(&S.empty[st], (use & 1) ^ 1, p.status);          // the MMAs that read this stage are done
            uint8_t* sb = S.stage[st];
            if (tid == 0) {
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s32(&S.full[st])), "r"(U_TILE) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(s32(sb + 4 * U_TILE)), "l"(xq + (size_t)c * U_TILE), "r"(U_TILE), "r"(s32(&S.full[st])) : "memory");
            }
            const uint32_t w[4] = {cw.x, cw.y, cw.z, cw.w};
#pragma unroll
            for (int kc = 0; kc < 4; ++kc) {
                uint4 hi, lo;
                dequant_hi_lo(w[kc], sc, zr, hi, lo);
                *reinterpret_cast<uint4*>(sb + (2 * half) * U_TILE + core_off(r, kc)) = hi;
                *reinterpret_cast<uint4*>(sb + (2 * half + 1) * U_TILE + core_off(r, kc)) = lo;
            }
            stage_written(&S.full[st]);
            cw = nw;
        }
        // the adapter as extra k: A = B_gate / B_up rows (fp16 of bf16), B = sigma * (A_gate x) / sigma * (A_up x);
        // the threads of matrix m write its A rows and its B rows (gate's B in slot 4, up's in slot 1)
        if (r_chunks > 0) {
            const int first_pair = S.pair[0];
            const int ad = first_pair >= 0 ? p.pair_ad[first_pair] : 0;
            const int n_sets = p.n_adapters == 1 ? 1 : p.K;
            const float* um = nullptr;
            if (pair >= 0) um = p.u_gu + (((size_t)(pair / p.K) * n_sets + (p.n_adapters == 1 ? 0 : pair % p.K)) * 2 + half) * p.rank;
            const uint16_t* Bm = reinterpret_cast<const uint16_t*>(half ? p.lora.B_up : p.lora.B_gate) + ((size_t)ad * p.I + row0 + r) * p.rank;
            for (int rc = 0; rc < r_chunks; ++rc) {
                const int c = n_chunks + rc, st = c % U_STAGES_GU;
                const uint32_t use = (uint32_t)(c / U_STAGES_GU);
                bar_wait(&S.empty[st], (use & 1) ^ 1, p.status);
                uint8_t* sb = S.stage[st];
#pragma unroll
                for (int kc = 0; kc < 4; ++kc) {
                    const int j0 = rc * 32 + kc * 8, n = p.rank - j0;          // rank is a multiple of 8
                    uint4 a = make_uint4(0, 0, 0, 0);
                    if (n > 0) a = bf16x8_to_f16(*reinterpret_cast<const uint4*>(Bm + j0));
                    *reinterpret_cast<uint4*>(sb + (2 * half) * U_TILE + core_off(r, kc)) = a;
                    *reinterpret_cast<uint4*>(sb + (half ? 1 : 4) * U_TILE + core_off(r, kc)) = f32x8_to_f16(um != nullptr ? um + j0 : nullptr, n, p.sigma);
                }
                if (tid == 0) bar_arrive(&S.full[st]);               // stands in for the bulk copy's arrival
                stage_written(&S.full[st]);
            }
        }
        // ---- epilogue: h = silu(gate) * up, thread = weight row, 32 token columns at a time
        bar_wait(S.done, 0, p.status);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        for (int c0 = half * (U_TN / 2); c0 < min(cnt, (half + 1) * (U_TN / 2)); c0 += 32) {
            uint32_t g[32], u[32];
            tmem_ld32(lane_addr + c0, g);
            tmem_ld32(lane_addr + U_TN + c0, u);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            // h goes out twice: fp32 per pair (for the down adapter's projection), and as the down
            // kernel's B operand: fp16 value and fp16 residual in operand-tile order, this row being k
            // index i = row0 + r of the tile's chunk i / 32 (k core (i % 32) / 8, slot of i % 8 in the
            // (k0,k4,k1,k5,k2,k6,k3,k7) order)
            const int i = row0 + r, e = i & 7;
            uint8_t* hq = p.hq + ((size_t)tile * (p.I / 32) + (i >> 5)) * 2 * U_TILE + (size_t)((e < 4 ? 2 * e : 2 * (e - 4) + 1) * 2);
            const int kc = (i & 31) >> 3;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const int pr = (c0 + j) < cnt ? S.pair[c0 + j] : -1;
                if (pr >= 0) {
                    const float hv = silu_f(__uint_as_float(g[j])) * __uint_as_float(u[j]);
                    p.h[(size_t)pr * p.I + i] = hv;
                    const __half hh = __float2half_rn(hv);
                    const __half hl = __float2half_rn(hv - __half2float(hh));
                    *reinterpret_cast<__half*>(hq + core_off(c0 + j, kc)) = hh;
                    *reinterpret_cast<__half*>(hq + U_TILE + core_off(c0 + j, kc)) = hl;
                }
            }
        }
    } else if (lane == 0) {
        // ---- the MMA issuer.  Descriptors differ only in their address field: base + offset >> 4.
        const uint32_t idesc = umma_idesc((cnt + 15) & ~15);
        const uint64_t d0 = umma_desc(s32(S.stage[0]));
        constexpr uint64_t kTile = U_TILE >> 4, kStep = (2 * U_LBO) >> 4, kStage = (5 * U_TILE) >> 4;
        const uint32_t tg = tmem, tu = tmem + U_TN;
        for (int c = 0; c < n_chunks; ++c) {
            const int st = c % U_STAGES_GU;
            bar_wait(&S.full[st], (uint32_t)(c / U_STAGES_GU) & 1, p.status);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t ds = d0 + st * kStage;
#pragma unroll
            for (int ks = 0; ks < U_KC / 16; ++ks) {
                const uint64_t dk = ds + ks * kStep, db = dk + 4 * kTile;
                umma(tg, dk, db, idesc, c > 0 || ks > 0);
                umma(tg, dk + kTile, db, idesc, true);
                umma(tu, dk + 2 * kTile, db, idesc, c > 0 || ks > 0);
                umma(tu, dk + 3 * kTile, db, idesc, true);
            }
            umma_commit(&S.empty[st]);
        }
        for (int rc = 0; rc < r_chunks; ++rc) {
            const int c = n_chunks + rc, st = c % U_STAGES_GU;
            bar_wait(&S.full[st], (uint32_t)(c / U_STAGES_GU) & 1, p.status);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t ds = d0 + st * kStage;
            const int ksteps = min(2, (p.rank - rc * 32 + 15) / 16);
            for (int ks = 0; ks < ksteps; ++ks) {
                const uint64_t dk = ds + ks * kStep;
                umma(tg, dk, dk + 4 * kTile, idesc, true);
                umma(tu, dk + 2 * kTile, dk + kTile, idesc, true);
            }
            umma_commit(&S.empty[st]);
        }
        umma_commit(S.done);
    }
    umma_end(tmem, 2 * U_TN);
}

// ---------------------------------------------------------------- down
// A CTA covers 256 output rows (two accumulators of 128 columns in tensor memory) for the tile's tokens:
// stage = [W0 hi][W0 lo][W1 hi][W1 lo][h hi][h lo], the h tiles arriving by one bulk copy per chunk
// (written in operand order by the gate/up kernel), thread t dequantising row t of the 256.
// o = gate weight * (W h + sigma B (A h))
__global__ void __launch_bounds__(U_THREADS, 2) umma_down_kernel(GroupedParams p) {
    const int tile = blockIdx.y;             // row blocks of a tile are neighbours in the grid: they share its activations in L2
    if (tile >= *p.n_tiles) return;
    extern __shared__ __align__(128) uint8_t smem[];
    const UmmaSmem S = carve(smem, 6, U_STAGES_D);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int slot = p.tiles[2 * tile], first = p.tiles[2 * tile + 1];
    const int cnt = min(U_TN, p.counts[slot] - first);
    const int row0 = blockIdx.x * 256;
    const uint8_t* rec = p.pool + (size_t)slot * p.L.bytes;
    const uint32_t tmem = umma_begin(p, S, slot, first, cnt, 2 * U_TN, U_PROD_WARPS + 1);
    const int n_chunks = p.I / U_KC;
    const int r_chunks = p.rank > 0 ? (p.rank + 31) / 32 : 0;
    const int gshift = 31 - __clz(p.group);

    if (warp < U_PROD_WARPS) {
        const int r = tid & 127, m = tid >> 7;                       // row r of half m: output row row0 + tid
        const uint8_t* hq = p.hq + (size_t)tile * (p.I / 32) * 2 * U_TILE;
        const uint8_t* cdp = rec + p.L.codes_down;
        uint4 cd = ld_stream16(cdp + down_code_off(p.H, p.I, row0 + tid, 0));
        const int n_groups = p.I >> gshift;
        uint32_t nsz = ld_stream4(rec + p.L.sz_down + down_sz_off(p.H, p.I, p.group, row0 + tid, 0));
        __half2 sd = __float2half2_rn(0.f), zd = sd;
        for (int c = 0; c < n_chunks; ++c) {
            const int st = c % U_STAGES_D;
            const uint32_t use = (uint32_t)(c / U_STAGES_D);
            uint4 nd = cd;
            if (c + 1 < n_chunks) nd = ld_stream16(cdp + down_code_off(p.H, p.I, row0 + tid, c + 1));
            if (((c * U_KC) & (p.group - 1)) == 0) {
                const __half2 a = u32_as_h2(nsz);
                sd = __low2half2(a); zd = __high2half2(a);
                nsz = ld_stream4(rec + p.L.sz_down + down_sz_off(p.H, p.I, p.group, row0 + tid, min(((c * U_KC) >> gshift) + 1, n_groups - 1)));
            }
            bar_wait(&S.empty[st], (use & 1) ^ 1, p.status);
            uint8_t* sb = S.stage[st];
            if (tid == 0) {
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s32(&S.full[st])), "r"(2 * U_TILE) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(s32(sb + 4 * U_TILE)), "l"(hq + (size_t)c * 2 * U_TILE), "r"(2 * U_TILE), "r"(s32(&S.full[st])) : "memory");
            }
            const uint32_t wd[4] = {cd.x, cd.y, cd.z, cd.w};
#pragma unroll
            for (int kc = 0; kc < 4; ++kc) {
                uint4 hi, lo;
                dequant_hi_lo(wd[kc], sd, zd, hi, lo);
                *reinterpret_cast<uint4*>(sb + (2 * m) * U_TILE + core_off(r, kc)) = hi;
                *reinterpret_cast<uint4*>(sb + (2 * m + 1) * U_TILE + core_off(r, kc)) = lo;
            }
            stage_written(&S.full[st]);
            cd = nd;
        }
        if (r_chunks > 0) {
            const int first_pair = S.pair[0];
            const int ad = first_pair >= 0 ? p.pair_ad[first_pair] : 0;
            const int pair = S.pair[r];
            const float* ud = (m == 0 && pair >= 0) ? p.u_d + (size_t)pair * p.rank : nullptr;
            const uint16_t* Bd = reinterpret_cast<const uint16_t*>(p.lora.B_down) + ((size_t)ad * p.H + row0 + tid) * p.rank;
            for (int rc = 0; rc < r_chunks; ++rc) {
                const int c = n_chunks + rc, st = c % U_STAGES_D;
                const uint32_t use = (uint32_t)(c / U_STAGES_D);
                bar_wait(&S.empty[st], (use & 1) ^ 1, p.status);
                uint8_t* sb = S.stage[st];
#pragma unroll
                for (int kc = 0; kc < 4; ++kc) {
                    const int j0 = rc * 32 + kc * 8, n = p.rank - j0;
                    uint4 a = make_uint4(0, 0, 0, 0);
                    if (n > 0) a = bf16x8_to_f16(*reinterpret_cast<const uint4*>(Bd + j0));
                    *reinterpret_cast<uint4*>(sb + (2 * m) * U_TILE + core_off(r, kc)) = a;
                    if (m == 0) *reinterpret_cast<uint4*>(sb + 4 * U_TILE + core_off(r, kc)) = f32x8_to_f16(ud != nullptr ? ud + j0 : nullptr, n, p.sigma);
                }
                if (tid == 0) bar_arrive(&S.full[st]);               // stands in for the bulk copy's arrival
                stage_written(&S.full[st]);
            }
        }
        // ---- epilogue: o[pair][row] = gate weight * acc; thread t = row t, accumulator t / 128
        bar_wait(S.done, 0, p.status);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + m * U_TN;
        for (int c0 = 0; c0 < cnt; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(lane_addr + c0, v);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const int pr = (c0 + j) < cnt ? S.pair[c0 + j] : -1;
                if (pr >= 0) p.o[(size_t)pr * p.H + row0 + tid] = p.gates[pr] * __uint_as_float(v[j]);
            }
        }
    } else if (lane == 0) {
        const uint32_t idesc = umma_idesc((cnt + 15) & ~15);
        const uint64_t d0 = umma_desc(s32(S.stage[0]));
        constexpr uint64_t kTile = U_TILE >> 4, kStep = (2 * U_LBO) >> 4, kStage = (6 * U_TILE) >> 4;
        for (int c = 0; c < n_chunks; ++c) {
            const int st = c % U_STAGES_D;
            bar_wait(&S.full[st], (uint32_t)(c / U_STAGES_D) & 1, p.status);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t ds = d0 + st * kStage;
#pragma unroll
            for (int ks = 0; ks < U_KC / 16; ++ks) {
                const uint64_t w0 = ds + ks * kStep, hhi = w0 + 4 * kTile;
#pragma unroll
                for (int m = 0; m < 2; ++m) {
                    const uint64_t whi = w0 + 2 * m * kTile;
                    umma(tmem + m * U_TN, whi, hhi, idesc, c > 0 || ks > 0);
                    umma(tmem + m * U_TN, whi + kTile, hhi, idesc, true);
                    umma(tmem + m * U_TN, whi, hhi + kTile, idesc, true);
                }
            }
            umma_commit(&S.empty[st]);
        }
        for (int rc = 0; rc < r_chunks; ++rc) {
            const int c = n_chunks + rc, st = c % U_STAGES_D;
            bar_wait(&S.full[st], (uint32_t)(c / U_STAGES_D) & 1, p.status);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t ds = d0 + st * kStage;
            const int ksteps = min(2, (p.rank - rc * 32 + 15) / 16);
            for (int ks = 0; ks < ksteps; ++ks) {
                const uint64_t w0 = ds + ks * kStep;
                umma(tmem, w0, w0 + 4 * kTile, idesc, true);
                umma(tmem + U_TN, w0 + 2 * kTile, w0 + 4 * kTile, idesc, true);
            }
            umma_commit(&S.empty[st]);
        }
        umma_commit(S.done);
    }
    umma_end(tmem, 2 * U_TN);
}

}  // namespace

bool umma_grouped_supported(const edg_layer_desc& d) {
    return d.H % 256 == 0 && d.I % 128 == 0 && (d.group & (d.group - 1)) == 0 && d.group >= 32 && d.rank % 8 == 0;
}

cudaError_t launch_umma_gate_up(const GroupedParams& p, int max_tiles, cudaStream_t st) {
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(umma_gate_up_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)umma_smem_bytes(5, U_STAGES_GU));
        if (e != cudaSuccess) return e;
        configured = true;
    }
    umma_gather_x_kernel<<<dim3(8, max_tiles), 256, 0, st>>>(p);
    umma_gate_up_kernel<<<dim3(p.I / 128, max_tiles), U_THREADS, umma_smem_bytes(5, U_STAGES_GU), st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_umma_down(const GroupedParams& p, int max_tiles, cudaStream_t st) {
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(umma_down_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)umma_smem_bytes(6, U_STAGES_D));
        if (e != cudaSuccess) return e;
        configured = true;
    }
    umma_down_kernel<<<dim3(p.H / 256, max_tiles), U_THREADS, umma_smem_bytes(6, U_STAGES_D), st>>>(p);
    return cudaGetLastError();
}

}  // namespace edg
