// fp32 Linear + bias + activation + scale + residual + row reduction in ONE kernel
// on the CUDA cores (true fp32 FMA; TF32 would miss the 1e-4 bound once LayerNorm
// divides by a standard deviation below one).
//
// One CTA owns R complete output rows, so the LayerNorm / softmax reduction over
// N never leaves the CTA: thread (tx, ty) accumulates column tx over the k-slice
// ty, the slices are summed through shared memory, and the threads with ty == 0
// apply the epilogue and take part in warp-shuffle + shared-memory row reductions.
#include "../device/act.cuh"
#include "kernels.h"

namespace pike {
namespace {

constexpr int KCHUNK = 1024;  // x is staged through shared memory in chunks of K

template <int R, bool MAX>
__device__ __forceinline__ void block_reduce(float (&v)[R], float *red /*[R][32]*/, int tid, int nwarps_active,
                                             bool active)
{
    // all threads of the CTA call this (it synchronises); only `active` threads contribute
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        float x = active ? v[r] : (MAX ? -INFINITY : 0.0f);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float y = __shfl_xor_sync(0xffffffffu, x, o);
            x = MAX ? fmaxf(x, y) : x + y;
        }
        if (lane == 0 && warp < nwarps_active) red[r * 32 + warp] = x;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < R; ++r) {
        float x = (lane < nwarps_active) ? red[r * 32 + lane] : (MAX ? -INFINITY : 0.0f);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float y = __shfl_xor_sync(0xffffffffu, x, o);
            x = MAX ? fmaxf(x, y) : x + y;
        }
        v[r] = x;
    }
    __syncthreads();
}

template <int R, int ACT>
__global__ void __launch_bounds__(1024, 1) fp32_chain_kernel(Fp32ChainArgs a, int npad, int kslices)
{
    extern __shared__ float smem[];
    float *x_s = smem;                         // [R][KCHUNK]
    float *part = x_s + R * KCHUNK;            // [kslices][R][npad]
    float *red = part + kslices * R * npad;    // [R][32]

    const int tid = threadIdx.x;
    const int tx = tid % npad, ty = tid / npad;
    const int row0 = blockIdx.x * R;
    const bool col_ok = tx < a.N;

    float acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = 0.0f;

    for (int k0 = 0; k0 < a.K; k0 += KCHUNK) {
        const int kc = min(KCHUNK, a.K - k0);
        __syncthreads();
        for (int i = tid; i < R * kc; i += blockDim.x) {
            const int r = i / kc, k = i - r * kc;
            const int row = row0 + r;
            x_s[r * KCHUNK + k] = (row < a.M) ? a.x[(long long)row * a.ldx + k0 + k] : 0.0f;
        }
        __syncthreads();
        if (col_ok) {
            if (!a.w_is_nk) {
                const float *wp = a.w + (long long)k0 * a.ldw + tx;
#pragma unroll 8
                for (int k = ty; k < kc; k += kslices) {
                    const float wv = __ldg(wp + (long long)k * a.ldw);
#pragma unroll
                    for (int r = 0; r < R; ++r) acc[r] = fmaf(x_s[r * KCHUNK + k], wv, acc[r]);
                }
            } else {
                const float *wp = a.w + (long long)tx * a.ldw + k0;
#pragma unroll 8
                for (int k = ty; k < kc; k += kslices) {
                    const float wv = __ldg(wp + k);
#pragma unroll
                    for (int r = 0; r < R; ++r) acc[r] = fmaf(x_s[r * KCHUNK + k], wv, acc[r]);
                }
            }
        }
    }

    // sum the k-slices
    if (kslices > 1) {
#pragma unroll
        for (int r = 0; r < R; ++r) part[(ty * R + r) * npad + tx] = acc[r];
        __syncthreads();
        if (ty == 0) {
            for (int s = 1; s < kslices; ++s)
#pragma unroll
                for (int r = 0; r < R; ++r) acc[r] += part[(s * R + r) * npad + tx];
        }
    }

    const bool active = (ty == 0) && col_ok;
    const int nwarps_active = npad / 32;
    float v[R];
    if (active) {
        const float b = a.bias ? a.bias[tx] : 0.0f;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int row = row0 + r;
            float y = a.scale * act_precise<ACT>(acc[r] + b);
            if (a.residual && row < a.M) y += a.residual[(long long)row * a.ldr + tx];
            v[r] = y;
        }
    } else {
#pragma unroll
        for (int r = 0; r < R; ++r) v[r] = 0.0f;
    }

    if (a.reduce == 1) {  // LayerNorm: two passes over the register-resident row
        float s[R];
#pragma unroll
        for (int r = 0; r < R; ++r) s[r] = v[r];
        block_reduce<R, false>(s, red, tid, nwarps_active, active);
        float mean[R], d2[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            mean[r] = s[r] / (float)a.N;
            const float d = v[r] - mean[r];
            d2[r] = d * d;
        }
        block_reduce<R, false>(d2, red, tid, nwarps_active, active);
        if (active) {
            const float g = a.gamma ? a.gamma[tx] : 1.0f;
            const float be = a.beta ? a.beta[tx] : 0.0f;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const float rstd = rsqrtf(d2[r] / (float)a.N + a.eps);
                v[r] = (v[r] - mean[r]) * rstd * g + be;
            }
        }
    } else if (a.reduce == 2) {  // softmax
        float mx[R];
#pragma unroll
        for (int r = 0; r < R; ++r) mx[r] = v[r];
        block_reduce<R, true>(mx, red, tid, nwarps_active, active);
        float e[R], s[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            e[r] = expf(v[r] - mx[r]);
            s[r] = e[r];
        }
        block_reduce<R, false>(s, red, tid, nwarps_active, active);
#pragma unroll
        for (int r = 0; r < R; ++r) v[r] = e[r] / s[r];
    }

    if (active) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int row = row0 + r;
            if (row < a.M) a.out[(long long)row * a.ldo + tx] = v[r];
        }
    }
}

template <int R>
cudaError_t launch_r(const Fp32ChainArgs &a, int npad, int kslices, size_t smem, cudaStream_t stream)
{
    const dim3 grid((a.M + R - 1) / R), block(npad * kslices);
    auto go = [&](auto kern) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<grid, block, smem, stream>>>(a, npad, kslices);
        return cudaGetLastError();
    };
    switch (a.act) {
    case ACT_GELU_ERF:  return go(fp32_chain_kernel<R, ACT_GELU_ERF>);
    case ACT_GELU_TANH: return go(fp32_chain_kernel<R, ACT_GELU_TANH>);
    case ACT_SILU:      return go(fp32_chain_kernel<R, ACT_SILU>);
    default:            return go(fp32_chain_kernel<R, ACT_NONE>);
    }
}

}  // namespace

cudaError_t launch_fp32_chain(const Fp32ChainArgs &a, cudaStream_t stream)
{
    const int npad = ((a.N + 31) / 32) * 32;            // N <= 1024 checked by the caller
    int kslices = 1024 / npad;
    if (kslices > 4) kslices = 4;
    if (kslices < 1) kslices = 1;
    // rows per CTA: keep the grid near two CTAs per SM for large M, one row per CTA for small M
    int R = 1;
    while (R < 8 && (a.M + R - 1) / R > 296) R *= 2;
    auto smem_for = [&](int r) { return sizeof(float) * (size_t)(r * KCHUNK + kslices * r * npad + r * 32); };
    switch (R) {
    case 1:  return launch_r<1>(a, npad, kslices, smem_for(1), stream);
    case 2:  return launch_r<2>(a, npad, kslices, smem_for(2), stream);
    case 4:  return launch_r<4>(a, npad, kslices, smem_for(4), stream);
    default: return launch_r<8>(a, npad, kslices, smem_for(8), stream);
    }
}

}  // namespace pike
