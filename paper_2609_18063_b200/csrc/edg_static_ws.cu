// moe_expert_ffn_int4_lora_static: the batch-1 expert FFN for callers that cannot allocate.
//
// Some hosts of this library may not call cudaMalloc at all: a plugin running inside another
// engine's memory plan, a real-time loop that must not touch the allocator after start-up, a
// process whose device memory is fully handed out by a pool it does not own.  They can still pass
// inputs and outputs, but have nowhere to put the kernel's scratch.  This entry point keeps that
// scratch in a fixed array inside the library's own device image instead.
#include "edg_common.cuh"

namespace {

// The scratch itself: part of the module image, so every GPU that loads the library holds these
// bytes until the process exits.  2 MiB covers every shape the batch-1 kernel accepts
// (control block + h + adapter projections + 4K partial outputs of H floats + E logits).
constexpr size_t kStaticScratchBytes = 2u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};     // device address of the array, per device, filled on first use

}  // namespace

extern "C" int32_t moe_expert_ffn_int4_lora_static(const edg_layer_desc* desc, const void* slot_pool,
                                                   const int32_t* slot_table, const int32_t* slots,
                                                   const int32_t* experts, const float* gates, const void* x,
                                                   const edg_lora* lora, void* y, void* stream) {
    int32_t rc = edg::check_desc(desc);
    if (rc != EDG_OK) return rc;
    if (!slot_pool || !slots || !gates || !x || !y) return EDG_E_INVAL;
    if (!edg::aligned(slot_pool, 256) || !edg::aligned(x, 16) || !edg::aligned(y, 16)) return EDG_E_INVAL;
    if (!edg::fused_supported(*desc)) return EDG_E_SHAPE;
    if (edg::workspace_layout(*desc, 1).lone_bytes > kStaticScratchBytes) return EDG_E_WORKSPACE;   // beyond the fixed array
    const bool has_lora = lora != nullptr && desc->rank > 0;
    if (has_lora) {
        if (!lora->A_gate || !lora->B_gate || !lora->A_up || !lora->B_up || !lora->A_down || !lora->B_down) return EDG_E_INVAL;
        if (desc->n_adapters != 1 && slot_table == nullptr && experts == nullptr) return EDG_E_INVAL;
    }

    int dev = -1;
    EDG_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return EDG_E_INVAL;
    if (g_scratch_addr[dev] == nullptr) {
        // In host code the array's name is only a handle; the kernel needs the device address, which
        // differs per device and is looked up once with that device current.
        void* ptr = nullptr;
        EDG_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        if (ptr == nullptr) return EDG_E_CUDA;
        g_scratch_addr[dev] = ptr;
    }
    void* scratch = g_scratch_addr[dev];
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array keeps whatever the last call left.  Only the control block (status word, arrival
    // counters) has to start at zero; everything else is written before it is read.
    EDG_CUDA_TRY(cudaMemsetAsync(scratch, 0, edg::kCtrlBytes, st));
    return edg::run_fused_layer(desc, slot_pool, slots, slot_table, experts, gates, x, has_lora ? lora : nullptr, y,
                                nullptr, nullptr, nullptr, nullptr, scratch, -1, -1, 0, -1, st);
}
