// Harness glue of the layer-stack workload, not part of the paper's method: the residual connection and a
// parameter-free RMS norm between two MoE layers, y = v * rsqrt(mean(v^2) + eps) with v = x + moe_out in fp32,
// rounded once to bf16. One CTA per token; the row stays in registers between the two passes.
#include "mira_internal.cuh"

namespace mira {
namespace {

constexpr int kNormThreads = 256;
constexpr int kNormMaxPerThread = 16384 / (kNormThreads * 2);     // bf16 pairs per thread at the largest hidden size

__global__ void __launch_bounds__(kNormThreads) k_residual_rmsnorm(const __nv_bfloat162* __restrict__ x,
                                                                   const __nv_bfloat162* __restrict__ y, int C2, float eps,
                                                                   __nv_bfloat162* __restrict__ out) {
    __shared__ float s_red[kNormThreads / 32];
    pdl_wait();            // the layer's combine kernel; launched into the same programmatic chain as the layer's kernels,
    pdl_launch();          // so the next layer's routing kernel is resident when this one ends
    const size_t row = (size_t)blockIdx.x * C2;
    float2 v[kNormMaxPerThread];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < kNormMaxPerThread; ++i) {
        const int c = threadIdx.x + i * kNormThreads;
        if (c < C2) {
            const float2 a = __bfloat1622float2(x[row + c]), b = __bfloat1622float2(y[row + c]);
            v[i] = make_float2(a.x + b.x, a.y + b.y);
            ss = fmaf(v[i].x, v[i].x, ss); ss = fmaf(v[i].y, v[i].y, ss);
        }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < kNormThreads / 32; ++i) tot += s_red[i];
    const float r = rsqrtf(tot / (float)(2 * C2) + eps);
#pragma unroll
    for (int i = 0; i < kNormMaxPerThread; ++i) {
        const int c = threadIdx.x + i * kNormThreads;
        if (c < C2) out[row + c] = __floats2bfloat162_rn(v[i].x * r, v[i].y * r);
    }
}

}  // namespace
}  // namespace mira

extern "C" mira_status mira_residual_rmsnorm(const void* x, const void* moe_out, int32_t T, int32_t hidden, float eps,
                                             void* out, void* stream) {
    using namespace mira;
    if (!x || !moe_out || !out || T < 0 || hidden < 2 || (hidden & 1) || hidden > 16384) return MIRA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(moe_out) | reinterpret_cast<uintptr_t>(out)) & 3u) return MIRA_ERR_ALIGN;
    if (T == 0) return MIRA_OK;
    MIRA_CUDA_OK(launch_pdl(k_residual_rmsnorm, dim3(T), dim3(kNormThreads), 0, static_cast<cudaStream_t>(stream),
                            static_cast<const __nv_bfloat162*>(x), static_cast<const __nv_bfloat162*>(moe_out), hidden / 2, eps,
                            static_cast<__nv_bfloat162*>(out)));
    MIRA_CUDA_OK(cudaGetLastError());
    return MIRA_OK;
}
