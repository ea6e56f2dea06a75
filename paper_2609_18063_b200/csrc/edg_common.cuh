// Shared host/device helpers of the streaming-MoE decode library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/edg_moe.h"

namespace edg {

// ---------------------------------------------------------------- host: errors

void set_cuda_error(cudaError_t e);            // records the error for edg_last_cuda_error
#define EDG_CUDA_TRY(expr)                                                   \
    do {                                                                     \
        cudaError_t _e = (expr);                                             \
        if (_e != cudaSuccess) { ::edg::set_cuda_error(_e); return EDG_E_CUDA; } \
    } while (0)

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// ---------------------------------------------------------------- record layout
// One expert record: [gate codes][up codes][down codes][gate sz][up sz][down sz].
// Codes are int4, low nibble first inside every 32-bit word (code k of a word in bits 4k..4k+3);
// sz is one (scale, zero) fp16 pair per group.  Every [N][Kd] matrix is stored tile-major:
//     codes: [N/16 row tiles][Kd/32 chunks][16 rows][16 bytes]     (a chunk = 32 consecutive codes of a row)
//     sz:    [N/16 row tiles][Kd/group groups][16 rows][4 bytes]
// so the 16 rows x 32 codes that one tensor-core k-step touches are 256 contiguous bytes (read
// without shared-memory bank conflicts), and any block of whole row tiles is one contiguous run
// for a bulk copy.  gate and up are [I][H].  down is stored as kDownSlices column slices, each a
// tile-major [H][I/kDownSlices] matrix: the batch-1 kernel splits the down projection over the
// intermediate dimension.  All section offsets are multiples of 256 bytes for the shapes
// edg_check_desc admits.
struct RecordLayout {
    uint32_t codes_gate, codes_up, codes_down;   // byte offsets
    uint32_t sz_gate, sz_up, sz_down;
    uint32_t bytes;
};

constexpr int kDownSlices = 4;

// byte offset, inside a tile-major code section of a [.][Kd] matrix, of chunk c (codes 32c..32c+31) of row n
__host__ __device__ inline size_t code_off(int Kd, int n, int c) {
    return ((((size_t)(n >> 4) * (Kd / 32) + c) * 16) + (n & 15)) * 16;
}
// byte offset, inside a tile-major sz section, of the (scale, zero) pair of group gi of row n
__host__ __device__ inline size_t sz_off(int Kd, int group, int n, int gi) {
    return ((((size_t)(n >> 4) * (Kd / group) + gi) * 16) + (n & 15)) * 4;
}
// the same for the sliced down matrix [H][I]
__host__ __device__ inline size_t down_code_off(int H, int I, int n, int c) {
    const int sw = I / kDownSlices, cps = sw / 32;            // slice width in codes, chunks per row-slice
    return (size_t)(c / cps) * ((size_t)H * sw / 2) + code_off(sw, n, c % cps);
}
__host__ __device__ inline size_t down_sz_off(int H, int I, int group, int n, int gi) {
    const int sw = I / kDownSlices, gps = sw / group;         // groups per row-slice
    return (size_t)(gi / gps) * ((size_t)H * gps * 4) + sz_off(sw, group, n, gi % gps);
}

__host__ __device__ inline RecordLayout record_layout(int H, int I, int group) {
    RecordLayout L;
    const uint32_t c = (uint32_t)H * (uint32_t)I / 2u;
    const uint32_t s = (uint32_t)H * (uint32_t)I / (uint32_t)group * 4u;
    L.codes_gate = 0;
    L.codes_up = c;
    L.codes_down = 2 * c;
    L.sz_gate = 3 * c;
    L.sz_up = 3 * c + s;
    L.sz_down = 3 * c + 2 * s;
    L.bytes = 3 * c + 3 * s;
    return L;
}

// Workspace layout for T tokens (floats unless noted).  The first kCtrlBytes bytes are a control
// block that must start out zero: its first int32 is the device-side status word, the rest are the
// counters of the ring that chained batch-1 layer-steps share (arrivals of the reduce, head rows
// delivered, reducers finished -- one set per ring slot).
constexpr int kPairWords = 64;         // words behind the logits of a ring slot: 32 (expert, gate) pairs, the routing itself
constexpr int kHandoffRing = 128;      // ring slots shared by chained batch-1 layer-steps in flight
constexpr int kDepWords = 16;           // words per ring slot of the dependent chain: 4 sums of squares, 4 "rows written" flags, a counter
constexpr size_t kCtrlBytes = 4096;    // control block: status word at 0, then the ring's counters
constexpr size_t kCtrlCounters = 64;                               // [ring][4] arrivals per block of output rows
constexpr size_t kCtrlHead = kCtrlCounters + kHandoffRing * 16;    // [ring] head rows delivered
constexpr size_t kCtrlDone = kCtrlHead + kHandoffRing * 4;         // [ring] reducers finished
constexpr size_t kCtrlNorm = kCtrlDone + kHandoffRing * 4;         // [ring] reducers that have delivered their sum of squares (dependent chain)
static_assert(kCtrlNorm + kHandoffRing * 4 <= kCtrlBytes, "control block too small");

struct WorkspaceLayout {
    size_t ctrl;      // kCtrlBytes control block
    size_t u_gu;      // [T][n_sets][2][rank] float : A_gate x and A_up x
    size_t h;         // [T][K][I] float            : silu(gate) * up
    size_t u_d;       // [T][K][rank] float         : A_down h
    size_t logits;    // [ring][E + 64] float     : next-step head logits, then the (expert, gate) pairs chosen from them, handed to the chained next step; one set per ring slot
    size_t partial;   // [ring][4(K+1)][H] float  : gate-weighted partial expert outputs of the fused batch-1 kernel, one set per ring slot
    size_t dep;       // [ring][8] float          : dependent chain: kC partial sums of squares of x + y, then the "next state written" flag
    size_t lone_bytes;// what a batch-1 call that never chains needs: everything up to the first set of partials
    // grouped path (T > 1) only:
    size_t o;         // [T*K][H] float             : gate-weighted output of every (token, choice) pair
    size_t o_part;    // [T*K][4][H] float          : the same per quarter of the intermediate dimension (small groups only)
    size_t xt;        // [T*K/8 + n_slots] tile records of the streaming small-group kernel: x fragments, block sums, projections, pair table
    size_t pair_slot; // [T*K] int32                : resolved slot of every pair (-1: skipped)
    size_t pair_ad;   // [T*K] int32                : adapter of every pair
    size_t counts;    // [n_slots] int32            : pairs per slot
    size_t n_tiles;   // int32
    size_t tiles;     // [T*K/8 + n_slots][2] int32 : (slot, first position) of every tile of 8 or 64 pairs
    size_t lists;     // [n_slots][T] int32         : pairs of every slot, ascending
    size_t hq;        // [T*K/128 + n_slots][I/32][2][128 x 32] fp16: h of every 128-token tile as tensor-core operand tiles (value, residual)
    size_t xq;        // [T*K/128 + n_slots][H/32][128 x 32] fp16: the gathered token states of every tile as operand tiles
    size_t bytes;
};

__host__ __device__ inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline WorkspaceLayout workspace_layout(const edg_layer_desc& d, int T) {
    WorkspaceLayout W;
    const size_t n_sets = d.n_adapters == 1 ? 1 : (size_t)d.K;
    const size_t r = d.rank > 0 ? (size_t)d.rank : 1;
    W.ctrl = 0;
    W.u_gu = kCtrlBytes;
    W.h = round_up(W.u_gu + (size_t)T * n_sets * 2 * r * sizeof(float), 256);
    W.u_d = round_up(W.h + (size_t)T * d.K * d.I * sizeof(float), 256);
    W.logits = round_up(W.u_d + (size_t)T * d.K * r * sizeof(float), 256);
    W.dep = round_up(W.logits + (size_t)kHandoffRing * (d.E + kPairWords) * sizeof(float), 256);
    W.partial = round_up(W.dep + (size_t)kHandoffRing * kDepWords * sizeof(float), 256);
    const size_t one_set = (size_t)kDownSlices * (d.K + 1) * d.H * sizeof(float);   // K routed experts and the shared expert
    W.lone_bytes = W.partial + one_set;
    size_t end = round_up(W.partial + (size_t)kHandoffRing * one_set, 256);
    W.o_part = W.xt = end;
    W.o = W.pair_slot = W.pair_ad = W.counts = W.n_tiles = W.tiles = W.lists = W.hq = W.xq = end;
    if (T > 1) {
        const size_t P = (size_t)T * d.K;
        W.o = end;                 end = round_up(W.o + P * d.H * sizeof(float), 256);
        const bool small = P <= 8 * (size_t)d.n_slots;
        W.o_part = end;            end = round_up(W.o_part + (small ? P * 4 * d.H * sizeof(float) : 0), 256);
        // a tile record: 8 tokens of fp16 state, two sums per 32 activations and token, 2 x rank projections per token, pair table
        const size_t rr = d.rank > 0 ? (size_t)d.rank : 8;
        const size_t tile_rec = (size_t)8 * d.H * 2 + 2 * 8 * (size_t)(d.H / 32) * 4 + 8 * 2 * rr * 4 + 128;
        W.xt = end;                end = round_up(W.xt + (small ? (P / 8 + 1 + d.n_slots) * tile_rec : 0), 256);
        W.pair_slot = end;         end = round_up(W.pair_slot + P * 4, 256);
        W.pair_ad = end;           end = round_up(W.pair_ad + P * 4, 256);
        W.counts = end;            end = round_up(W.counts + (size_t)d.n_slots * 4, 256);
        W.n_tiles = end;           end += 256;
        W.tiles = end;             end = round_up(W.tiles + (P / 8 + 1 + d.n_slots) * 8, 256);
        W.lists = end;             end = round_up(W.lists + (size_t)d.n_slots * T * 4, 256);
        W.hq = end;                end = round_up(W.hq + ((P + 127) / 128 + d.n_slots) * (size_t)(d.I / 32) * 2 * 8192, 256);
        W.xq = end;                end = round_up(W.xq + ((P + 127) / 128 + d.n_slots) * (size_t)(d.H / 32) * 8192, 256);
    }
    W.bytes = end;
    return W;
}

int32_t check_desc(const edg_layer_desc* d);   // EDG_OK or EDG_E_INVAL / EDG_E_SHAPE

// ---------------------------------------------------------------- host entry points shared by the translation units

// What the batch-1 layer kernel can do beyond the plain layer-step; all optional.
struct FusedExtras {
    int32_t* inds_mirror = nullptr;        // [K] copy of inds_next in mapped pinned host memory
    void* x_next = nullptr;                // [H] bf16: bf16(rmsnorm(x + y)) written by the kernel's last reducer
    float eps = 1e-6f;
    int dep_wait = -1;                     // ring slot whose flag announces this step's x (chained dependent steps)
    const void* shared_rec = nullptr;      // device record of the layer's shared expert: runs as one more expert with gate 1
    const edg_lora* shared_lora = nullptr; // its adapter (leading dimension 1), or null
};

bool fused_supported(const edg_layer_desc& d);
// One fused launch for a batch-1 layer-step (edg_decode_fused.cu).  W_pre may be null (no prediction).
int32_t run_fused_layer(const edg_layer_desc* d, const void* slot_pool, const int32_t* slots, const int32_t* table,
                        const int32_t* experts, const float* gates, const void* x, const edg_lora* lora, void* y,
                        const void* W_pre, int32_t* inds_next, float* gates_next, float* logits_next,
                        void* workspace, int flag_in, int flag_out, int ring, int stale, cudaStream_t st,
                        const FusedExtras* extras = nullptr);
// a4-a6 for T tokens on whatever kernels fit the shape (edg_ffn.cu)
int32_t run_ffn(const edg_layer_desc* d, const void* slot_pool, int32_t T, const int32_t* slots,
                const int32_t* table, const int32_t* experts, const float* gates, const void* x,
                const edg_lora* lora, void* y, void* workspace, size_t workspace_bytes, cudaStream_t st);
// a1-a2 for n_heads (head, state) pairs, or for n_heads states of one head (edg_prerouter.cu)
int32_t run_prerouter(const edg_layer_desc* d, const void* W_pre, const void* s, int32_t n_heads,
                      int32_t* inds, float* gates, float* logits_opt, cudaStream_t st, int shared_head = 0,
                      int32_t* mirror = nullptr);
// the full head (fc1 -> gelu -> fc2 + residual path) for n_heads (head, state) pairs
int32_t run_prerouter_mlp(const edg_layer_desc* desc, const edg_mlp_head* head, const void* s,
                          const int32_t* cur_inds, const int32_t* prev_inds, int32_t n_heads,
                          int32_t* inds, float* gates, float* logits_opt, cudaStream_t stream, int32_t* mirror);

// ---------------------------------------------------------------- device helpers
#ifdef __CUDACC__

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

// bf16 pair packed in one 32-bit word (low half = first element)
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Sum over aligned groups of LPR lanes (LPR a power of two <= 32).
template <int LPR>
__device__ __forceinline__ float group_sum(float v) {
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// ---- int4 -> fp32 without conversion instructions.
//
// A float whose exponent field is 0 or 1 has the value (bit pattern) * 2^-149, so masking one
// nibble of a packed word in place gives q * 2^(4p - 149) exactly for nibble positions p = 0..5
// (bits 0..23).  Nibbles 6 and 7 are brought to positions 4 and 5 by one shift.  The matching
// activation is pre-multiplied by 2^(XS - 4p), so every product is q * x * 2^(XS - 149) and the
// running sum is an ordinary fp32 dot product of exact integer codes with x, scaled by a power
// of two.  The zero point and the scale are applied per 32-code chunk on the fp32 partial sum:
//     sum_k s (q_k - z) x_k = s * (sum_k q_k x_k - z * sum_k x_k).
// Requires subnormal inputs to be honoured (no -ftz, no --use_fast_math).
constexpr int XS = 100;                                  // activation pre-scale exponent
__device__ __forceinline__ float pow2f(int e) { return __uint_as_float((uint32_t)(e + 127) << 23); }

// position of nibble j (0..7) after the masks below, and the exponent its activation carries
__device__ __forceinline__ int nibble_pos(int j) { return j < 6 ? j : j - 2; }

// xs[j] for a 32-code chunk: x_j * 2^(XS - 4 pos(j % 8)).  Returns sum_j x_j * 2^(XS - 149).
__device__ __forceinline__ float scale_chunk(const float (&x)[32], float (&xs)[32]) {
    float sum = 0.f;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        xs[j] = x[j] * pow2f(XS - 4 * nibble_pos(j & 7));
        sum += x[j];
    }
    return sum * pow2f(XS - 149);
}

__device__ __forceinline__ void word_fma(uint32_t w, const float* xs, float& a, float& b, float& c, float& d) {
    const uint32_t w2 = w >> 8;
    a = fmaf(__uint_as_float(w & 0x0000000Fu), xs[0], a);
    b = fmaf(__uint_as_float(w & 0x000000F0u), xs[1], b);
    c = fmaf(__uint_as_float(w & 0x00000F00u), xs[2], c);
    d = fmaf(__uint_as_float(w & 0x0000F000u), xs[3], d);
    a = fmaf(__uint_as_float(w & 0x000F0000u), xs[4], a);
    b = fmaf(__uint_as_float(w & 0x00F00000u), xs[5], b);
    c = fmaf(__uint_as_float(w2 & 0x000F0000u), xs[6], c);
    d = fmaf(__uint_as_float(w2 & 0x00F00000u), xs[7], d);
}

// 2^(XS-149) * sum_{j<32} q_j x_j for one 16-byte chunk of codes (four independent chains).
__device__ __forceinline__ float chunk_dot(const uint4& q, const float (&xs)[32]) {
    float a = 0.f, b = 0.f, c = 0.f, d = 0.f;
    word_fma(q.x, xs + 0, a, b, c, d);
    word_fma(q.y, xs + 8, a, b, c, d);
    word_fma(q.z, xs + 16, a, b, c, d);
    word_fma(q.w, xs + 24, a, b, c, d);
    return (a + b) + (c + d);
}

// s * (qx - z * xsum): one chunk's contribution, still scaled by 2^(XS-149).  sz = (scale, zero) fp16 pair.
__device__ __forceinline__ float chunk_affine(float qx, float xsum, uint32_t sz) {
    const __half2 h = *reinterpret_cast<const __half2*>(&sz);
    const float2 f = __half22float2(h);
    return f.x * fmaf(-f.y, xsum, qx);
}

constexpr float kUnscale = 562949953421312.0f;           // 2^(149 - XS) = 2^49

__device__ __forceinline__ float silu_f(float v) { return v / (1.f + __expf(-v)); }

// read-only 16-byte / 4-byte loads that do not pollute L1 (weights are streamed once)
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint32_t ld_stream4(const void* p) {
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

// Order-preserving map float -> uint32 (larger float <=> larger key; -0 < +0 is harmless here).
__device__ __forceinline__ uint32_t float_key(float v) {
    const uint32_t u = __float_as_uint(v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Best remaining candidate of a lane: entries lane, lane+32, ... of work[]; taken entries hold NaN.
__device__ __forceinline__ void lane_best(const float* work, int E, int lane, uint32_t& key, int& idx) {
    key = 0u;
    idx = 0x7FFFFFFF;
    for (int e = lane; e < E; e += 32) {
        const float v = work[e];
        if (v == v) {                                   // not taken (and not a NaN logit)
            const uint32_t kk = float_key(v);
            if (idx == 0x7FFFFFFF || kk > key) { key = kk; idx = e; }   // ascending e: the lowest index wins ties
        }
    }
}

// Inverse of float_key.
__device__ __forceinline__ float key_float(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// Shared tail of the two top-k variants: lane j < K holds winner j (value myv, index myi, or
// myi == INT_MAX when there were fewer than K finite logits), lane 0 the largest.  Writes the
// winners in ascending index with gates exp(l - max) / sum over the winners.
__device__ __forceinline__ void topk_emit(float myv, int myi, int K, int lane, int32_t* inds, float* gates) {
    const unsigned full = 0xFFFFFFFFu;
    const float m = __shfl_sync(full, myv, 0);
    const float ex = (lane < K && myi != 0x7FFFFFFF) ? expf(myv - m) : 0.f;
    const float sum = warp_sum(ex);
    int rank = 0;
#pragma unroll 1
    for (int i = 0; i < K; ++i) {
        const int oi = __shfl_sync(full, myi, i);
        rank += (oi < myi) ? 1 : 0;
    }
    if (lane < K && myi != 0x7FFFFFFF) {
        inds[rank] = myi;
        gates[rank] = ex / sum;
    }
}

// Top-k with the candidates in registers: lane l holds entries l, l+32, ... (V = 8 per lane,
// E <= 256) as sortable keys, 0 meaning absent / NaN.  Every lane first sorts its own candidates
// (descending key, ascending index among equals) with a fixed network; a round is then one
// warp-wide max on the lanes' best keys, the owner popping its list.  Only when several lanes hold
// the same best key does a second reduction (min over their indices) decide.
__device__ __forceinline__ void topk_cex(uint32_t& ka, int& ia, uint32_t& kb, int& ib) {
    // (ka, ia) is the earlier position: swap when b must come first
    const bool sw = kb > ka || (kb == ka && ib < ia);
    const uint32_t tk = sw ? kb : ka, uk = sw ? ka : kb;
    const int ti = sw ? ib : ia, ui = sw ? ia : ib;
    ka = tk; kb = uk; ia = ti; ib = ui;
}

// (the selection alone: lane j < K ends up with winner j -- value myv, index myi, or myi == INT_MAX
// when there were fewer than K candidates; entries of work[] that are NaN are not candidates)
template <int V>
__device__ __forceinline__ void warp_topk_reg(const float* work, int E, int K, int lane, float& myv, int& myi) {
    static_assert(V == 8, "the sorting network below is for 8 candidates per lane");
    const unsigned full = 0xFFFFFFFFu;
    uint32_t key[V];
    int idx[V];
#pragma unroll
    for (int u = 0; u < V; ++u) {
        const int e = u * 32 + lane;
        const float v = e < E ? work[e] : __int_as_float(0x7fffffff);
        key[u] = (v == v) ? float_key(v) : 0u;
        idx[u] = e;
    }
    // 19-comparator network for 8 inputs
#define EDG_CEX(a, b) topk_cex(key[a], idx[a], key[b], idx[b])
    EDG_CEX(0, 1); EDG_CEX(2, 3); EDG_CEX(4, 5); EDG_CEX(6, 7);
    EDG_CEX(0, 2); EDG_CEX(1, 3); EDG_CEX(4, 6); EDG_CEX(5, 7);
    EDG_CEX(1, 2); EDG_CEX(5, 6); EDG_CEX(0, 4); EDG_CEX(3, 7);
    EDG_CEX(1, 5); EDG_CEX(2, 6);
    EDG_CEX(1, 4); EDG_CEX(3, 6);
    EDG_CEX(2, 4); EDG_CEX(3, 5);
    EDG_CEX(3, 4);
#undef EDG_CEX
    myv = 0.f;
    myi = 0x7FFFFFFF;
#pragma unroll 1
    for (int j = 0; j < K; ++j) {
        const uint32_t best = __reduce_max_sync(full, key[0]);
        if (best == 0u) break;                                   // fewer than K finite logits
        const unsigned who = __ballot_sync(full, key[0] == best);
        int win;
        if ((who & (who - 1)) == 0u) win = __shfl_sync(full, idx[0], __ffs(who) - 1);
        else win = (int)__reduce_min_sync(full, key[0] == best ? (unsigned)idx[0] : 0x7FFFFFFFu);
        if (lane == j) { myv = key_float(best); myi = win; }
        if (key[0] == best && idx[0] == win) {                   // the owner pops its list
#pragma unroll
            for (int u = 0; u + 1 < V; ++u) { key[u] = key[u + 1]; idx[u] = idx[u + 1]; }
            key[V - 1] = 0u;
        }
    }
}

template <int V>
__device__ __forceinline__ void warp_softmax_topk_reg(const float* work, int E, int K, int lane, int32_t* inds, float* gates) {
    float myv;
    int myi;
    warp_topk_reg<V>(work, E, K, lane, myv, myi);
    topk_emit(myv, myi, K, lane, inds, gates);
}

// Top-k of work[0..E) by one warp, ties to the lower index; the K winners are written in
// ascending index with gate weights exp(l - max) / sum over the winners (which equals
// softmax(l)[inds] / sum softmax(l)[inds]: the full-softmax denominator cancels).
// Up to 256 candidates are kept in registers; beyond that every lane caches its best remaining
// candidate in `work` (which is then overwritten) and only the winning lane rescans its entries.
__device__ __forceinline__ void warp_softmax_topk(float* work, int E, int K, int lane, int32_t* inds, float* gates) {
    if (E <= 256) {
        warp_softmax_topk_reg<8>(work, E, K, lane, inds, gates);
        return;
    }
    const unsigned full = 0xFFFFFFFFu;
    float myv = 0.f;
    int myi = 0x7FFFFFFF;
    uint32_t key;
    int idx;
    lane_best(work, E, lane, key, idx);
    for (int j = 0; j < K; ++j) {
        const uint32_t best = __reduce_max_sync(full, idx == 0x7FFFFFFF ? 0u : key);
        const int cand = (idx != 0x7FFFFFFF && key == best) ? idx : 0x7FFFFFFF;
        const int win = (int)__reduce_min_sync(full, (unsigned)cand);
        if (win == 0x7FFFFFFF) break;                   // fewer than K finite logits
        const float wv = work[win];
        if (lane == j) { myv = wv; myi = win; }
        __syncwarp();
        if (idx == win) {                               // the owner retires it and looks for its next best
            work[win] = __int_as_float(0x7fffffff);
            lane_best(work, E, lane, key, idx);
        }
        __syncwarp();
    }
    topk_emit(myv, myi, K, lane, inds, gates);
}

// A warp's K freshly written indices, copied to a mirror in mapped pinned host memory with
// system-scope stores.  Each entry is final by itself: a host that has filled the mirror with -1
// beforehand may poll it and take the prediction as complete once all K entries are >= 0.
__device__ __forceinline__ void mirror_inds(int32_t* mirror, const int32_t* inds, int K, int lane) {
    __syncwarp();
    if (mirror != nullptr && lane < K) {
        const int v = inds[lane];
        asm volatile("st.relaxed.sys.global.s32 [%0], %1;" ::"l"(mirror + lane), "r"(v) : "memory");
    }
}

template <typename T> __device__ __forceinline__ void store_out(T* y, size_t i, float v);
template <> __device__ __forceinline__ void store_out<float>(float* y, size_t i, float v) { y[i] = v; }
template <> __device__ __forceinline__ void store_out<__half>(__half* y, size_t i, float v) { y[i] = __float2half_rn(v); }
struct bf16_t { uint16_t bits; };
template <> __device__ __forceinline__ void store_out<bf16_t>(bf16_t* y, size_t i, float v) {
    uint32_t u = __float_as_uint(v);
    u += 0x7FFFu + ((u >> 16) & 1u);                      // round to nearest even (finite inputs)
    y[i].bits = (uint16_t)(u >> 16);
}

#endif  // __CUDACC__

}  // namespace edg
