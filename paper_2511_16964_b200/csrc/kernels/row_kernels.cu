// Bandwidth-bound row kernels: bf16 LayerNorm (the MLP block's prologue) and the
// second half of the split-row softmax (combine per-tile partials, normalise in place).
#include "../device/ptx.cuh"
#include "kernels.h"

namespace pike {
namespace {

constexpr int LN_THREADS = 256;
constexpr int LN_MAX_CHUNKS = 8;  // 16-byte chunks per thread held in registers: D <= 256*8*8 = 16384

__device__ __forceinline__ float block_sum(float x, float *red, int tid)
{
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    if (lane == 0) red[warp] = x;
    __syncthreads();
    x = (lane < LN_THREADS / 32) ? red[lane] : 0.0f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    __syncthreads();
    return x;
}

__device__ __forceinline__ float load_param(const void *p, int is_f32, int i, float dflt)
{
    if (p == nullptr) return dflt;
    return is_f32 ? static_cast<const float *>(p)[i] : __bfloat162float(static_cast<const __nv_bfloat16 *>(p)[i]);
}

// One CTA per row; the row stays in registers between the mean pass, the
// variance pass (sum of squared deviations, not E[x^2]-E[x]^2) and the store, so
// HBM sees one read and one write per element.
__global__ void __launch_bounds__(LN_THREADS)
layernorm_bf16_kernel(const __nv_bfloat16 *__restrict__ x, long long ldx, __nv_bfloat16 *__restrict__ z,
                      long long ldz, const void *gamma, int gamma_f32, const void *beta, int beta_f32, float eps,
                      int D)
{
    __shared__ float red[32];
    const int tid = threadIdx.x;
    const long long row = blockIdx.x;
    const uint4 *xr = reinterpret_cast<const uint4 *>(x + row * ldx);
    const int nchunks = D / 8;  // D % 8 == 0

    uint4 c[LN_MAX_CHUNKS];
    float sum = 0.0f;
#pragma unroll
    for (int i = 0; i < LN_MAX_CHUNKS; ++i) {
        const int ci = tid + i * LN_THREADS;
        if (ci < nchunks) {
            c[i] = xr[ci];
            const uint32_t w[4] = {c[i].x, c[i].y, c[i].z, c[i].w};
#pragma unroll
            for (int h = 0; h < 4; ++h) sum += bf16_lo(w[h]) + bf16_hi(w[h]);
        }
    }
    const float mean = block_sum(sum, red, tid) / (float)D;
    float ss = 0.0f;
#pragma unroll
    for (int i = 0; i < LN_MAX_CHUNKS; ++i) {
        const int ci = tid + i * LN_THREADS;
        if (ci < nchunks) {
            const uint32_t w[4] = {c[i].x, c[i].y, c[i].z, c[i].w};
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const float a = bf16_lo(w[h]) - mean, b = bf16_hi(w[h]) - mean;
                ss += a * a + b * b;
            }
        }
    }
    const float rstd = rsqrtf(block_sum(ss, red, tid) / (float)D + eps);
    uint4 *zr = reinterpret_cast<uint4 *>(z + row * ldz);
#pragma unroll
    for (int i = 0; i < LN_MAX_CHUNKS; ++i) {
        const int ci = tid + i * LN_THREADS;
        if (ci < nchunks) {
            const uint32_t w[4] = {c[i].x, c[i].y, c[i].z, c[i].w};
            uint32_t o[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const int e = ci * 8 + 2 * h;
                const float a = (bf16_lo(w[h]) - mean) * rstd * load_param(gamma, gamma_f32, e, 1.0f) +
                                load_param(beta, beta_f32, e, 0.0f);
                const float b = (bf16_hi(w[h]) - mean) * rstd * load_param(gamma, gamma_f32, e + 1, 1.0f) +
                                load_param(beta, beta_f32, e + 1, 0.0f);
                o[h] = pack_bf16x2(a, b);
            }
            zr[ci] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

constexpr int SM_THREADS = 256;

// One CTA per row: combine the per-tile (max, sum exp) pairs
//   m = max_t m_t,  l = sum_t l_t * exp(m_t - m)
// then p = exp(v - m) / l in place (one read and one write of the row).
__global__ void __launch_bounds__(SM_THREADS)
softmax_finish_kernel(float *__restrict__ v, long long ldv, const float2 *__restrict__ partials, int num_n_tiles,
                      int N)
{
    __shared__ float red[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long row = blockIdx.x;
    const float2 *pr = partials + row * num_n_tiles;

    float m = -INFINITY;
    for (int t = tid; t < num_n_tiles; t += SM_THREADS) m = fmaxf(m, pr[t].x);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) red[warp] = m;
    __syncthreads();
    m = (lane < SM_THREADS / 32) ? red[lane] : -INFINITY;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    __syncthreads();

    float l = 0.0f;
    for (int t = tid; t < num_n_tiles; t += SM_THREADS) {
        const float2 pt = pr[t];
        l += pt.y * expf(pt.x - m);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    if (lane == 0) red[warp] = l;
    __syncthreads();
    l = (lane < SM_THREADS / 32) ? red[lane] : 0.0f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    const float inv = 1.0f / l;

    float4 *vr = reinterpret_cast<float4 *>(v + row * ldv);  // N % 4 == 0, ldv % 4 == 0
    for (int i = tid; i < N / 4; i += SM_THREADS) {
        float4 a = vr[i];
        a.x = expf(a.x - m) * inv;
        a.y = expf(a.y - m) * inv;
        a.z = expf(a.z - m) * inv;
        a.w = expf(a.w - m) * inv;
        vr[i] = a;
    }
}

}  // namespace

cudaError_t launch_layernorm_bf16(const void *x, long long ldx, void *z, long long ldz, const void *gamma,
                                  int gamma_f32, const void *beta, int beta_f32, float eps, int M, int D,
                                  cudaStream_t stream)
{
    if (M <= 0) return cudaSuccess;
    if (D % 8 != 0 || D > LN_THREADS * LN_MAX_CHUNKS * 8) return cudaErrorInvalidValue;
    layernorm_bf16_kernel<<<M, LN_THREADS, 0, stream>>>(static_cast<const __nv_bfloat16 *>(x), ldx,
                                                         static_cast<__nv_bfloat16 *>(z), ldz, gamma, gamma_f32, beta,
                                                         beta_f32, eps, D);
    return cudaGetLastError();
}

cudaError_t launch_softmax_finish(float *v, long long ldv, const float2 *partials, int num_n_tiles, int M, int N,
                                  cudaStream_t stream)
{
    if (M <= 0) return cudaSuccess;
    softmax_finish_kernel<<<M, SM_THREADS, 0, stream>>>(v, ldv, partials, num_n_tiles, N);
    return cudaGetLastError();
}

}  // namespace pike
