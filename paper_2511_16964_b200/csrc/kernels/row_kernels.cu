// Bandwidth-bound row kernels: 16-bit (bf16 or f16) LayerNorm (the MLP block's prologue) and the
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

__device__ __forceinline__ float load_param(const void *p, int is_f32, int i, float dflt, bool f16)
{
    if (p == nullptr) return dflt;
    return is_f32 ? static_cast<const float *>(p)[i] : h16_at(p, i, f16);
}

// One CTA per row; the row stays in registers between the mean pass, the
// variance pass (sum of squared deviations, not E[x^2]-E[x]^2) and the store, so
// HBM sees one read and one write per element.
__global__ void __launch_bounds__(LN_THREADS)
layernorm_bf16_kernel(const uint16_t *__restrict__ x, long long ldx, uint16_t *__restrict__ z,
                      long long ldz, const void *gamma, int gamma_f32, const void *beta, int beta_f32, float eps,
                      int D, int f16_flag)
{
    const bool f16 = f16_flag != 0;
    __shared__ float red[32];
    const int tid = threadIdx.x;
    const long long row = blockIdx.x;
    pdl_wait();
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
            for (int h = 0; h < 4; ++h) sum += h16_lo(w[h], f16) + h16_hi(w[h], f16);
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
                const float a = h16_lo(w[h], f16) - mean, b = h16_hi(w[h], f16) - mean;
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
                const float a = (h16_lo(w[h], f16) - mean) * rstd * load_param(gamma, gamma_f32, e, 1.0f, f16) +
                                load_param(beta, beta_f32, e, 0.0f, f16);
                const float b = (h16_hi(w[h], f16) - mean) * rstd * load_param(gamma, gamma_f32, e + 1, 1.0f, f16) +
                                load_param(beta, beta_f32, e + 1, 0.0f, f16);
                o[h] = pack_h16x2(a, b, f16);
            }
            zr[ci] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

// One WARP per row for rows of at most 4096 elements, in a persistent grid (one CTA per SM, twelve warps).
// Each warp streams its rows through a private two-stage ring in shared memory filled by bulk copies
// (one elected lane issues them, an mbarrier per stage counts the bytes): while a row is being reduced and
// normalised in registers, the next two are already in flight, so loads, arithmetic and stores of different
// rows overlap inside every warp instead of all warps of an SM loading, computing and storing in phase.
// The row sits in 16 x 16-byte registers per lane and both reductions are pure shuffles.  gamma and beta are
// copied to shared memory once per CTA (every warp needs all of them for every row).
constexpr int LNW_WARPS = 12;
constexpr int LNW_STAGES = 2;
constexpr int LNW_MAX_CHUNKS = 16;  // D <= 32 * 16 * 8 = 4096
constexpr int LNW_STAGE_BYTES = LNW_MAX_CHUNKS * 32 * 16;   // 8 KiB: one row of 4096 16-bit elements
constexpr int LNW_PARAM_BYTES = LNW_MAX_CHUNKS * 32 * 8 * 4;   // 16 KiB: 4096 fp32 values (or 16-bit ones in half of it)
constexpr size_t LNW_SMEM_BYTES = 128 + (size_t)LNW_WARPS * LNW_STAGES * LNW_STAGE_BYTES + 2 * LNW_PARAM_BYTES;

// eight consecutive parameters starting at element e (e % 8 == 0) as fp32, from the CTA's copy in shared memory;
// KIND 0 = absent, 1 = 16-bit (the type of x), 2 = f32
template <int KIND, bool F16>
__device__ __forceinline__ void smem_param8(const uint8_t *p, int e, float dflt, float (&out)[8])
{
    if constexpr (KIND == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) out[i] = dflt;
    } else if constexpr (KIND == 2) {
        const float4 a = *reinterpret_cast<const float4 *>(p + (size_t)e * 4);
        const float4 b = *reinterpret_cast<const float4 *>(p + (size_t)e * 4 + 16);
        out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
        out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
    } else {
        const uint4 v = *reinterpret_cast<const uint4 *>(p + (size_t)e * 2);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int h = 0; h < 4; ++h) { out[2 * h] = h16_lo(w[h], F16); out[2 * h + 1] = h16_hi(w[h], F16); }
    }
}

template <int GK, int BK, bool F16>
__global__ void __launch_bounds__(LNW_WARPS * 32, 1)
layernorm_bf16_warp_kernel(const uint16_t *__restrict__ x, long long ldx, uint16_t *__restrict__ z,
                           long long ldz, const void *gamma, const void *beta, float eps, int M, int D,
                           unsigned int *status, unsigned long long limit_ns)
{
    extern __shared__ uint8_t lnw_smem[];
    __shared__ uint64_t full[LNW_WARPS][LNW_STAGES];
    __shared__ uint32_t abort_word;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    pdl_wait();
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(lnw_smem) + 127) & ~uintptr_t(127));
    uint8_t *ring = base + (size_t)warp * LNW_STAGES * LNW_STAGE_BYTES;
    uint8_t *gamma_s = base + (size_t)LNW_WARPS * LNW_STAGES * LNW_STAGE_BYTES, *beta_s = gamma_s + LNW_PARAM_BYTES;
    const int nchunks = D / 8;
    const uint32_t row_bytes = (uint32_t)D * 2;
    const long long stride = (long long)gridDim.x * LNW_WARPS;
    const long long first = (long long)blockIdx.x * LNW_WARPS + warp;
    if (threadIdx.x == 0) abort_word = 0;
    // each warp owns its barriers: it initialises them and puts its first rows in flight at once, before the
    // CTA stages the parameters
    if (lane == 0) {
        for (int k = 0; k < LNW_STAGES; ++k) mbar_init(&full[warp][k], 1);
        fence_barrier_init();
        for (int k = 0; k < LNW_STAGES; ++k) {
            const long long r = first + k * stride;
            if (r < M) {
                mbar_arrive_expect_tx(&full[warp][k], row_bytes);
                bulk_load_1d(ring + k * LNW_STAGE_BYTES, x + r * ldx, row_bytes, &full[warp][k]);
            }
        }
    }
    // gamma / beta -> shared memory, 16 bytes per thread and turn (D is a multiple of 8, so both sizes are of 16)
    if constexpr (GK != 0)
        for (int o = threadIdx.x * 16; o < D * (GK == 2 ? 4 : 2); o += LNW_WARPS * 32 * 16)
            *reinterpret_cast<uint4 *>(gamma_s + o) = __ldg(reinterpret_cast<const uint4 *>(static_cast<const uint8_t *>(gamma) + o));
    if constexpr (BK != 0)
        for (int o = threadIdx.x * 16; o < D * (BK == 2 ? 4 : 2); o += LNW_WARPS * 32 * 16)
            *reinterpret_cast<uint4 *>(beta_s + o) = __ldg(reinterpret_cast<const uint4 *>(static_cast<const uint8_t *>(beta) + o));
    __syncthreads();
    const WaitCtx ctx{status, &abort_word, limit_ns, KID_LAYERNORM};
    int it = 0;
    for (long long row = first; row < M; row += stride, ++it) {
    const int stage = it % LNW_STAGES;
    mbar_wait(&full[warp][stage], (uint32_t)(it / LNW_STAGES) & 1u, ctx, 1u);
    const uint4 *xr = reinterpret_cast<const uint4 *>(ring + stage * LNW_STAGE_BYTES);

    uint4 c[LNW_MAX_CHUNKS];
#pragma unroll
    for (int i = 0; i < LNW_MAX_CHUNKS; ++i) {
        const int ci = lane + i * 32;
        c[i] = ci < nchunks ? xr[ci] : make_uint4(0u, 0u, 0u, 0u);
    }
    // every lane has taken its chunks out of the stage: refill it with the row two turns ahead
    __syncwarp();
    if (lane == 0) {
        const long long rn = row + LNW_STAGES * stride;
        if (rn < M) {
            mbar_arrive_expect_tx(&full[warp][stage], row_bytes);
            bulk_load_1d(ring + stage * LNW_STAGE_BYTES, x + rn * ldx, row_bytes, &full[warp][stage]);
        }
    }
    // all arithmetic on fp32 pairs (one 16-bit word = two elements): the kernel moves 4 bytes per element and is
    // otherwise bound by how many instructions per element the warp has to issue.  Mean and variance come from ONE
    // pass over values shifted by the row's first element (sums of d and d^2 with d = v - v0; the shift removes the
    // cancellation a plain sum of squares would suffer when the mean dwarfs the spread).
    const float v0 = __shfl_sync(0xffffffffu, h16_lo(c[0].x, F16), 0);
    const uint64_t neg_v0 = pack_f32x2(-v0, -v0);
    uint64_t s1[2] = {0ull, 0ull}, s2[2] = {0ull, 0ull};
#pragma unroll
    for (int i = 0; i < LNW_MAX_CHUNKS; ++i) {
        if (lane + i * 32 < nchunks) {              // padding chunks hold no elements
            const uint32_t w[4] = {c[i].x, c[i].y, c[i].z, c[i].w};
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const uint64_t d2 = add_f32x2(h16x2_to_f32x2(w[h], F16), neg_v0);
                s1[h & 1] = add_f32x2(s1[h & 1], d2);
                s2[h & 1] = fma_f32x2(d2, d2, s2[h & 1]);
            }
        }
    }
    float a0, a1, b0, b1;
    unpack_f32x2(add_f32x2(s1[0], s1[1]), a0, a1);
    unpack_f32x2(add_f32x2(s2[0], s2[1]), b0, b1);
    float sd = a0 + a1, sq = b0 + b1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {              // the two reductions interleaved
        sd += __shfl_xor_sync(0xffffffffu, sd, o);
        sq += __shfl_xor_sync(0xffffffffu, sq, o);
    }
    const float inv_d = 1.0f / (float)D;
    const float md = sd * inv_d;                    // mean of d
    const float rstd = rsqrtf(fmaxf(sq * inv_d - md * md, 0.0f) + eps);
    const float mean = v0 + md;
    const uint64_t rstd2 = pack_f32x2(rstd, rstd), shift2 = pack_f32x2(-mean * rstd, -mean * rstd);
    uint4 *zr = reinterpret_cast<uint4 *>(z + row * ldz);
#pragma unroll
    for (int i = 0; i < LNW_MAX_CHUNKS; ++i) {
        const int ci = lane + i * 32;
        if (ci < nchunks) {
            const uint32_t w[4] = {c[i].x, c[i].y, c[i].z, c[i].w};
            float g[8], be[8];
            smem_param8<GK, F16>(gamma_s, ci * 8, 1.0f, g);
            smem_param8<BK, F16>(beta_s, ci * 8, 0.0f, be);
            uint32_t o[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                // ((v - mean) * rstd) * g + be as two fused multiply-adds: v * rstd + (-mean * rstd), then * g + be
                const uint64_t n2 = fma_f32x2(h16x2_to_f32x2(w[h], F16), rstd2, shift2);
                float y0, y1;
                unpack_f32x2(fma_f32x2(n2, pack_f32x2(g[2 * h], g[2 * h + 1]), pack_f32x2(be[2 * h], be[2 * h + 1])), y0, y1);
                o[h] = pack_h16x2(y0, y1, F16);
            }
            zr[ci] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
    }   // rows of this warp
}

constexpr int SM_THREADS = 256;

// One CTA per row: combine the per-tile (max, sum exp) pairs
//   m = max_t m_t,  l = sum_t l_t * exp(m_t - m)
// then p = exp(v - m) / l in place (one read and one write of the row).
__global__ void __launch_bounds__(SM_THREADS)
softmax_finish_kernel(float *__restrict__ v, long long ldv, const float2 *__restrict__ partials, int num_n_tiles,
                      long long pair_row_stride, long long pair_tile_stride, int N)
{
    __shared__ float red[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long row = blockIdx.x;
    pdl_wait();
    // pair t of this row; [row][tile] for one GEMM's tiles, [shard][row] for pairs gathered from other GPUs
    const float2 *pr = partials + row * pair_row_stride;

    float m = -INFINITY;
    for (int t = tid; t < num_n_tiles; t += SM_THREADS) m = fmaxf(m, pr[t * pair_tile_stride].x);
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
        const float2 pt = pr[t * pair_tile_stride];
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

constexpr int STATS_THREADS = 256;

// One warp per row: fold the row's per-tile (max, sum exp) pairs into one pair for the whole row,
//   m = max_t m_t,  l = sum_t l_t * exp(m_t - m),
// the statistics a GPU publishes for its slice of the columns when a softmax is split over several GPUs.
__global__ void __launch_bounds__(STATS_THREADS)
softmax_row_stats_kernel(const float2 *__restrict__ partials, int num_n_tiles, float2 *__restrict__ stats, int M)
{
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * (STATS_THREADS / 32) + (threadIdx.x >> 5);
    pdl_wait();
    if (row >= M) return;
    const float2 *pr = partials + row * num_n_tiles;
    float m = -INFINITY;
    for (int t = lane; t < num_n_tiles; t += 32) m = fmaxf(m, pr[t].x);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float l = 0.0f;
    for (int t = lane; t < num_n_tiles; t += 32) {
        const float2 pt = pr[t];
        l += pt.y * expf(pt.x - m);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
    if (lane == 0) stats[row] = make_float2(m, l);
}

// Second half of a LayerNorm split across GEMM tiles.  One CTA per row: combine the per-tile
// (mean_t, M2_t) pairs (tile t holds n_t = min(tile_n, N - t*tile_n) columns)
//   mean = sum_t n_t mean_t / N,   M2 = sum_t M2_t + sum_t n_t (mean_t - mean)^2,   var = M2 / N
// then out = (v - mean) / sqrt(var + eps) * gamma + beta in place (one read and one write of the row).
template <bool OUT_F32>
__global__ void __launch_bounds__(SM_THREADS)
layernorm_finish_kernel(void *__restrict__ vout, long long ldv, const float2 *__restrict__ partials, int num_n_tiles,
                        int tile_n, int N, const void *gamma, int gamma_f32, const void *beta, int beta_f32, float eps,
                        int f16_flag)
{
    __shared__ float red[32];
    const bool f16 = f16_flag != 0;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long row = blockIdx.x;
    pdl_wait();
    const float2 *pr = partials + row * num_n_tiles;
    auto block_sum256 = [&](float x) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        if (lane == 0) red[warp] = x;
        __syncthreads();
        x = (lane < SM_THREADS / 32) ? red[lane] : 0.0f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        __syncthreads();
        return x;
    };
    float a = 0.0f;
    for (int t = tid; t < num_n_tiles; t += SM_THREADS) a += (float)min(tile_n, N - t * tile_n) * pr[t].x;
    const float mean = block_sum256(a) / (float)N;
    float b = 0.0f;
    for (int t = tid; t < num_n_tiles; t += SM_THREADS) {
        const float2 pt = pr[t];
        const float d = pt.x - mean;
        b += pt.y + (float)min(tile_n, N - t * tile_n) * d * d;
    }
    const float rstd = rsqrtf(block_sum256(b) / (float)N + eps);

    if (OUT_F32) {
        float4 *vr = reinterpret_cast<float4 *>(static_cast<float *>(vout) + row * ldv);
        for (int i = tid; i < N / 4; i += SM_THREADS) {
            float4 x = vr[i];
            const int e = i * 4;
            x.x = (x.x - mean) * rstd * load_param(gamma, gamma_f32, e, 1.0f, f16) +
                  load_param(beta, beta_f32, e, 0.0f, f16);
            x.y = (x.y - mean) * rstd * load_param(gamma, gamma_f32, e + 1, 1.0f, f16) +
                  load_param(beta, beta_f32, e + 1, 0.0f, f16);
            x.z = (x.z - mean) * rstd * load_param(gamma, gamma_f32, e + 2, 1.0f, f16) +
                  load_param(beta, beta_f32, e + 2, 0.0f, f16);
            x.w = (x.w - mean) * rstd * load_param(gamma, gamma_f32, e + 3, 1.0f, f16) +
                  load_param(beta, beta_f32, e + 3, 0.0f, f16);
            vr[i] = x;
        }
    } else {
        uint4 *vr = reinterpret_cast<uint4 *>(static_cast<uint16_t *>(vout) + row * ldv);
        for (int i = tid; i < N / 8; i += SM_THREADS) {
            const uint4 x = vr[i];
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
            uint32_t o[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const int e = i * 8 + 2 * h;
                const float lo = (h16_lo(w[h], f16) - mean) * rstd * load_param(gamma, gamma_f32, e, 1.0f, f16) +
                                 load_param(beta, beta_f32, e, 0.0f, f16);
                const float hi = (h16_hi(w[h], f16) - mean) * rstd * load_param(gamma, gamma_f32, e + 1, 1.0f, f16) +
                                 load_param(beta, beta_f32, e + 1, 0.0f, f16);
                o[h] = pack_h16x2(lo, hi, f16);
            }
            vr[i] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

}  // namespace

cudaError_t launch_layernorm_finish(void *v, int out_f32, long long ldv, const float2 *partials, int num_n_tiles,
                                    int tile_n, int M, int N, const void *gamma, int gamma_f32, const void *beta,
                                    int beta_f32, float eps, int f16, cudaStream_t stream, bool pdl)
{
    if (M <= 0) return cudaSuccess;
    auto kern = out_f32 ? layernorm_finish_kernel<true> : layernorm_finish_kernel<false>;
    return launch_kernel(kern, dim3(M), dim3(SM_THREADS), 0, stream, pdl, v, ldv, partials, num_n_tiles, tile_n, N, gamma,
                         gamma_f32, beta, beta_f32, eps, f16);
}

cudaError_t setup_row_kernels()
{
#define PIKE_LN_SETUP(G, B)                                                                                         \
    {                                                                                                               \
        cudaError_t e = cudaFuncSetAttribute(layernorm_bf16_warp_kernel<G, B, true>,                                \
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LNW_SMEM_BYTES);     \
        if (e != cudaSuccess) return e;                                                                             \
        e = cudaFuncSetAttribute(layernorm_bf16_warp_kernel<G, B, false>,                                           \
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)LNW_SMEM_BYTES);                 \
        if (e != cudaSuccess) return e;                                                                             \
    }
    PIKE_LN_SETUP(0, 0) PIKE_LN_SETUP(0, 1) PIKE_LN_SETUP(0, 2) PIKE_LN_SETUP(1, 0) PIKE_LN_SETUP(1, 1)
    PIKE_LN_SETUP(1, 2) PIKE_LN_SETUP(2, 0) PIKE_LN_SETUP(2, 1) PIKE_LN_SETUP(2, 2)
#undef PIKE_LN_SETUP
    return cudaSuccess;
}

cudaError_t launch_layernorm_bf16(const void *x, long long ldx, void *z, long long ldz, const void *gamma,
                                  int gamma_f32, const void *beta, int beta_f32, float eps, int M, int D, int f16,
                                  unsigned int *status, unsigned long long limit_ns, int num_sms, cudaStream_t stream,
                                  bool pdl)
{
    if (M <= 0) return cudaSuccess;
    if (D % 8 != 0 || D > LN_THREADS * LN_MAX_CHUNKS * 8) return cudaErrorInvalidValue;
    if (D <= 32 * LNW_MAX_CHUNKS * 8) {
        const int gk = gamma == nullptr ? 0 : (gamma_f32 ? 2 : 1), bk = beta == nullptr ? 0 : (beta_f32 ? 2 : 1);
        // persistent: one CTA per SM (the ring takes most of its shared memory), fewer if there are few rows
        if (num_sms < 1) num_sms = 1;
        const int want = (M + LNW_WARPS - 1) / LNW_WARPS;
        const dim3 grid(want < num_sms ? want : num_sms), block(LNW_WARPS * 32);
        const uint16_t *xp = static_cast<const uint16_t *>(x);
        uint16_t *zp = static_cast<uint16_t *>(z);
#define PIKE_LN_CASE(G, B)                                                                                          \
    if (gk == G && bk == B) {                                                                                       \
        auto kern = f16 ? layernorm_bf16_warp_kernel<G, B, true> : layernorm_bf16_warp_kernel<G, B, false>;        \
        return launch_kernel(kern, grid, block, LNW_SMEM_BYTES, stream, pdl, xp, ldx, zp, ldz, gamma, beta, eps, M, D, \
                             status, limit_ns);                                                                     \
    }
        PIKE_LN_CASE(0, 0) PIKE_LN_CASE(0, 1) PIKE_LN_CASE(0, 2) PIKE_LN_CASE(1, 0) PIKE_LN_CASE(1, 1)
        PIKE_LN_CASE(1, 2) PIKE_LN_CASE(2, 0) PIKE_LN_CASE(2, 1) PIKE_LN_CASE(2, 2)
#undef PIKE_LN_CASE
        return cudaErrorInvalidValue;   // not reached: every (gk, bk) has a case
    }
    return launch_kernel(layernorm_bf16_kernel, dim3(M), dim3(LN_THREADS), 0, stream, pdl,
                         static_cast<const uint16_t *>(x), ldx, static_cast<uint16_t *>(z), ldz, gamma, gamma_f32, beta,
                         beta_f32, eps, D, f16);
}

cudaError_t launch_softmax_finish(float *v, long long ldv, const float2 *partials, int num_n_tiles, int M, int N,
                                  cudaStream_t stream, long long pair_row_stride, long long pair_tile_stride, bool pdl)
{
    if (M <= 0) return cudaSuccess;
    if (pair_row_stride == 0) pair_row_stride = num_n_tiles;
    return launch_kernel(softmax_finish_kernel, dim3(M), dim3(SM_THREADS), 0, stream, pdl, v, ldv, partials, num_n_tiles,
                         pair_row_stride, pair_tile_stride, N);
}

cudaError_t launch_softmax_row_stats(const float2 *partials, int num_n_tiles, float2 *stats, int M, cudaStream_t stream,
                                     bool pdl)
{
    if (M <= 0) return cudaSuccess;
    const int rows_per_block = STATS_THREADS / 32;
    return launch_kernel(softmax_row_stats_kernel, dim3((M + rows_per_block - 1) / rows_per_block), dim3(STATS_THREADS), 0,
                         stream, pdl, partials, num_n_tiles, stats, M);
}

}  // namespace pike
