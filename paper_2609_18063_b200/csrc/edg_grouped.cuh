// Parameters shared by the grouped (T > 1) kernels: the mma.sync tiles for small groups and the
// tcgen05 tiles for large ones.
#pragma once

#include "edg_mma.cuh"

namespace edg {

struct GroupedParams {
    const uint8_t* pool;
    const int32_t* slots;     // [T][K] slots, or expert ids when table != null
    const int32_t* table;
    const int32_t* experts;
    const float* gates;       // [T][K]
    const uint16_t* x;        // [T][H] bf16
    edg_lora lora;
    void* y;
    int32_t* status;
    float* u_gu;              // [T][n_sets][2][rank]
    float* h;                 // [T*K][I]
    float* u_d;               // [T*K][rank]
    float* o;                 // [T*K][H]
    int32_t* pair_slot;       // [T*K]
    int32_t* pair_ad;         // [T*K]
    int32_t* counts;          // [n_slots]
    int32_t* lists;           // [n_slots][T]
    int32_t* tiles;           // [max tiles][2] = (slot, first position in the slot's list)
    int32_t* n_tiles;
    uint8_t* hq;              // h of every 128-token tile as fp16 operand tiles (tcgen05 path)
    uint8_t* xq;              // the gathered token states of every tile as fp16 operand tiles (tcgen05 path)
    int T, H, I, E, K, group, rank, n_adapters, n_slots, out_dtype;
    int ntok;                 // tokens per tile of this call (8, 64 or 128)
    float sigma;
    RecordLayout L;
};

// tcgen05 path for large groups (prefill): tiles of 128 tokens
constexpr int kUmmaTokens = 128;
bool umma_grouped_supported(const edg_layer_desc& d);
cudaError_t launch_umma_gate_up(const GroupedParams& p, int max_tiles, cudaStream_t st);
cudaError_t launch_umma_down(const GroupedParams& p, int max_tiles, cudaStream_t st);

// streaming path for small groups (batched decode): tiles of 8 tokens through the batch-1 kernel's pipeline
bool grouped_stream_supported(const edg_layer_desc& d);
int32_t run_grouped_stream(const edg_layer_desc* d, const GroupedParams& g, float* o_part, uint8_t* xt, int max_tiles, cudaStream_t st);

// adapter projections for many tokens / pairs on the tensor cores (one shared adapter); false = shape not covered
bool launch_lora_ax_tokens(const edg_layer_desc* d, const void* x, const edg_lora* lora, float* u_gu, int T, cudaStream_t st);
bool launch_lora_adh_pairs(const edg_layer_desc* d, const edg_lora* lora, const float* h, float* u_d, int P, cudaStream_t st);

}  // namespace edg
