// The hidden state a decoder would hand to the next layer-step, x_next = bf16(rmsnorm(x + y)) with
// unit gain: residual connection plus the next block's input norm.  Not part of the paper's method --
// its engine has attention and a shared expert between two MoE blocks -- but the smallest stand-in
// that makes consecutive layer-steps data-dependent the way a real decoder's are: step t+1 cannot
// start its arithmetic before step t's output exists.  Used by the dependent-chain benchmark and
// its step-local parity test.
#include "edg_common.cuh"

namespace edg {

constexpr int kNormThreads = 256;

template <typename YT> __device__ __forceinline__ float load_y(const void* y, int i);
template <> __device__ __forceinline__ float load_y<float>(const void* y, int i) { return static_cast<const float*>(y)[i]; }
template <> __device__ __forceinline__ float load_y<__half>(const void* y, int i) { return __half2float(static_cast<const __half*>(y)[i]); }
template <> __device__ __forceinline__ float load_y<bf16_t>(const void* y, int i) {
    return bf16_bits_to_float(static_cast<const uint16_t*>(y)[i]);
}

// One CTA: H <= 4096 elements, up to 16 per thread, kept in registers between the two passes.
template <typename YT>
__global__ void __launch_bounds__(kNormThreads) next_state_kernel(const uint16_t* x, const void* y, uint16_t* x_next, int H, float eps) {
    __shared__ float s_part[kNormThreads / 32];
    float v[16];
    float ss = 0.f;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const int i = j * kNormThreads + threadIdx.x;
        v[j] = i < H ? bf16_bits_to_float(x[i]) + load_y<YT>(y, i) : 0.f;
        ss = fmaf(v[j], v[j], ss);
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kNormThreads / 32; ++w) tot += s_part[w];
    const float inv = rsqrtf(tot / (float)H + eps);
    bf16_t* out = reinterpret_cast<bf16_t*>(x_next);
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const int i = j * kNormThreads + threadIdx.x;
        if (i < H) store_out<bf16_t>(out, i, v[j] * inv);
    }
}

}  // namespace edg

extern "C" int32_t edg_next_hidden_state(const edg_layer_desc* desc, const void* x, const void* y, void* x_next,
                                         float eps, void* stream) {
    int32_t rc = edg::check_desc(desc);
    if (rc != EDG_OK) return rc;
    if (!x || !y || !x_next) return EDG_E_INVAL;
    if (desc->H > 16 * edg::kNormThreads) return EDG_E_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint16_t* xb = static_cast<const uint16_t*>(x);
    uint16_t* xn = static_cast<uint16_t*>(x_next);
    if (desc->out_dtype == EDG_F32) edg::next_state_kernel<float><<<1, edg::kNormThreads, 0, st>>>(xb, y, xn, desc->H, eps);
    else if (desc->out_dtype == EDG_F16) edg::next_state_kernel<__half><<<1, edg::kNormThreads, 0, st>>>(xb, y, xn, desc->H, eps);
    else edg::next_state_kernel<edg::bf16_t><<<1, edg::kNormThreads, 0, st>>>(xb, y, xn, desc->H, eps);
    EDG_CUDA_TRY(cudaGetLastError());
    return EDG_OK;
}
