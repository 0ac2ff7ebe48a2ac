// Activation math for the epilogues.  Two flavours: "precise" for the fp32 path
// (CUDA math library accuracy) and "fast" for the bf16 paths, where one
// tanh.approx (relative error about 2^-11) is far below the bf16 output rounding.
#pragma once
#include <cuda_runtime.h>

namespace pike {

enum : int { ACT_NONE = 0, ACT_GELU_ERF = 1, ACT_GELU_TANH = 2, ACT_SILU = 3 };

__device__ __forceinline__ float tanh_approx(float x)
{
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int ACT>
__device__ __forceinline__ float act_precise(float y)
{
    if constexpr (ACT == ACT_GELU_ERF) {
        return 0.5f * y * (1.0f + erff(y * 0.70710678118654752f));
    } else if constexpr (ACT == ACT_GELU_TANH) {
        const float u = 0.79788456080286536f * (y + 0.044715f * y * y * y);
        return 0.5f * y * (1.0f + tanhf(u));
    } else if constexpr (ACT == ACT_SILU) {
        return y / (1.0f + expf(-y));
    } else {
        return y;
    }
}

template <int ACT>
__device__ __forceinline__ float act_fast(float y)
{
    if constexpr (ACT == ACT_GELU_ERF) {
        return 0.5f * y * (1.0f + erff(y * 0.70710678118654752f));
    } else if constexpr (ACT == ACT_GELU_TANH) {
        const float y2 = y * y;
        const float u = y * fmaf(0.044715f * 0.79788456080286536f, y2, 0.79788456080286536f);
        const float h = 0.5f * y;
        return fmaf(h, tanh_approx(u), h);
    } else if constexpr (ACT == ACT_SILU) {
        // sigmoid(y) = 0.5 + 0.5 tanh(y/2)
        const float h = 0.5f * y;
        return fmaf(h, tanh_approx(h), h);
    } else {
        return y;
    }
}

}  // namespace pike
