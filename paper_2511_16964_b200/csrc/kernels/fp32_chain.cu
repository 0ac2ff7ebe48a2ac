// fp32 Linear + bias + activation + scale + residual + row reduction in ONE kernel
// on the CUDA cores (true fp32 FMA; TF32 would miss the 1e-4 bound once LayerNorm
// divides by a standard deviation below one).
//
// A thread-block CLUSTER owns a block of BM complete output rows; its CTAs split the N columns
// (BN = 32, 64 or 128 columns each, at most 8 CTAs for N <= 1024).  Each CTA stages only its own
// column slice of W (K x BN) and the BM rows of x in shared memory, so W crosses the L2 once per
// row block instead of once per CTA-row as a one-CTA-per-row layout would have it, and the
// whole problem spreads over many SMs even when M is small.  Thread (lane, warp) accumulates
// columns lane + 32c of rows warp + 8i; k runs in ascending order per output (plain fp32 FMA).
// The LayerNorm / softmax reduction over N never leaves the cluster: every warp reduces its rows
// over the CTA's columns with shuffles, the CTAs publish one pair per row - (mean, sum of squared
// deviations) or (max, sum exp) - in their shared memory, and after one cluster barrier every CTA
// merges the pairs of all ranks through distributed shared memory.
#include "../device/act.cuh"
#include "../device/ptx.cuh"
#include "kernels.h"

namespace pike {
namespace {

constexpr int FT = 256;                    // 8 warps: warp = row lane, lane = column lane
constexpr int SMEM_FLOATS_MAX = 24576;     // 96 KiB of operand tiles per CTA
constexpr int MAX_BM = 32;

__device__ __forceinline__ float act_by_id(int act, float y)
{
    switch (act) {
    case ACT_GELU_ERF:  return act_precise<ACT_GELU_ERF>(y);
    case ACT_GELU_TANH: return act_precise<ACT_GELU_TANH>(y);
    case ACT_SILU:      return act_precise<ACT_SILU>(y);
    default:            return y;
    }
}

__device__ __forceinline__ float warp_sum_f(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}
__device__ __forceinline__ float warp_max_f(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}

// RPT rows and CW columns per thread: the CTA tile is (8 RPT) x (32 CW).  NK: w is [N,K].
template <int RPT, int CW, bool NK>
__global__ void __launch_bounds__(FT) fp32_chain_kernel(const Fp32ChainArgs a, const int kc)
{
    constexpr int BM = 8 * RPT, BN = 32 * CW;
    extern __shared__ __align__(16) float smem[];
    __shared__ float2 stat[MAX_BM];        // this CTA's per-row pair, read by the whole cluster
    float *x_s = smem;                     // [BM][kc]
    float *w_s = x_s + BM * kc;            // [kc][BN], or [BN][kc + 1] for NK (odd pitch: no bank conflicts)

    const int tid = threadIdx.x, lane = tid & 31, rg = tid >> 5;
    const int cn = (int)cluster_nctas(), rank = (int)cluster_ctarank();
    const long long row0 = (long long)((int)blockIdx.x / cn) * BM;
    const int n0 = rank * BN;
    const int n_loc = min(max(a.N - n0, 0), BN);      // columns this CTA owns (0 for a padding rank)
    pdl_wait();

    float acc[RPT][CW][4];
#pragma unroll
    for (int i = 0; i < RPT; ++i)
#pragma unroll
        for (int c = 0; c < CW; ++c)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][c][j] = 0.0f;
    // the per-column parameters are fetched now, so their latency hides under the main loop
    float bias_r[CW], gamma_r[CW], beta_r[CW];
#pragma unroll
    for (int c = 0; c < CW; ++c) {
        const int col = n0 + lane + 32 * c;
        const bool col_ok = col < a.N;
        bias_r[c] = (a.bias != nullptr && col_ok) ? __ldg(a.bias + col) : 0.0f;
        gamma_r[c] = (a.reduce == 1 && a.gamma != nullptr && col_ok) ? __ldg(a.gamma + col) : 1.0f;
        beta_r[c] = (a.reduce == 1 && a.beta != nullptr && col_ok) ? __ldg(a.beta + col) : 0.0f;
    }

    const bool x_vec = (a.ldx & 3) == 0;                         // rows of x start on 16-byte boundaries
    const bool w_vec = (a.ldw & 3) == 0 && (n_loc & 3) == 0;
    for (int k0 = 0; k0 < a.K; k0 += kc) {
        const int kn = min(kc, a.K - k0);
        const int kn4 = kn & ~3;
        __syncthreads();                                         // the previous chunk has been consumed
        // Everything is fetched with asynchronous copies, so all of a thread's loads are in flight together (the
        // problem is small: its time is a few memory latencies, which must not add up).  16-byte copies where
        // the rows are 16-byte aligned, 4-byte copies otherwise; elements outside the tensors are written as zeros.
        // ---- x rows [row0, row0 + BM) x k [k0, k0 + kn)
        const int kr = (kn + 3) & ~3;          // the FMA loop reads k in quads: positions kn .. kr-1 must hold zeros
        if (x_vec) {
            for (int idx = tid; idx < BM * (kr >> 2); idx += FT) {
                const int r = idx / (kr >> 2), k = (idx - r * (kr >> 2)) << 2;
                const long long row = row0 + r;
                const float *src = a.x + (row < a.M ? row * a.ldx + k0 + k : 0);
                if (k < kn4) {
                    cp_async_16(x_s + r * kc + k, src, row < a.M);
                } else {                        // the quad that holds the end of the row, element by element
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const bool ok = row < a.M && k + j < kn;
                        cp_async_4(x_s + r * kc + k + j, ok ? src + j : a.x, ok);
                    }
                }
            }
        } else {
            for (int idx = tid; idx < BM * kr; idx += FT) {
                const int r = idx / kr, k = idx - r * kr;
                const long long row = row0 + r;
                const bool ok = row < a.M && k < kn;
                cp_async_4(x_s + r * kc + k, ok ? a.x + row * a.ldx + k0 + k : a.x, ok);
            }
        }
        // ---- this CTA's column slice of W
        if (n_loc > 0) {
            if constexpr (!NK) {
                if (w_vec) {
                    for (int idx = tid; idx < kr * (BN >> 2); idx += FT) {
                        const int k = idx / (BN >> 2), c = (idx - k * (BN >> 2)) << 2;
                        const bool ok = c < n_loc && k < kn;
                        cp_async_16(w_s + k * BN + c, ok ? a.w + (long long)(k0 + k) * a.ldw + n0 + c : a.w, ok);
                    }
                } else {
                    for (int idx = tid; idx < kr * BN; idx += FT) {
                        const int k = idx / BN, c = idx - k * BN;
                        const bool ok = c < n_loc && k < kn;
                        cp_async_4(w_s + k * BN + c, ok ? a.w + (long long)(k0 + k) * a.ldw + n0 + c : a.w, ok);
                    }
                }
            } else {
                // [N,K] weights land transposed, one element per copy: the odd pitch that keeps the FMA loop free of
                // bank conflicts leaves no 16-byte aligned rows
                const int pitch = kc + 1;
                for (int idx = tid; idx < BN * kr; idx += FT) {
                    const int c = idx / kr, k = idx - c * kr;
                    const bool ok = c < n_loc && k < kn;
                    cp_async_4(w_s + c * pitch + k, ok ? a.w + (long long)(n0 + c) * a.ldw + k0 + k : a.w, ok);
                }
            }
        }
        cp_async_wait_all();
        __syncthreads();
        if (n_loc > 0) {
            // four k at a time: one 16-byte broadcast load of x per row, four column loads of w, and four
            // independent accumulators per output (k = 0, 1, 2, 3 mod 4) so that consecutive FMAs do not wait
            // for one another; the tail of a chunk that is not a multiple of four reads the zeros staged above
#pragma unroll 2
            for (int k = 0; k < kn; k += 4) {
                float4 xv[RPT];
                float wv[CW][4];
#pragma unroll
                for (int i = 0; i < RPT; ++i) xv[i] = *reinterpret_cast<const float4 *>(x_s + (rg + 8 * i) * kc + k);
#pragma unroll
                for (int c = 0; c < CW; ++c)
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        wv[c][j] = NK ? w_s[(lane + 32 * c) * (kc + 1) + k + j] : w_s[(k + j) * BN + lane + 32 * c];
#pragma unroll
                for (int i = 0; i < RPT; ++i)
#pragma unroll
                    for (int c = 0; c < CW; ++c) {
                        acc[i][c][0] = fmaf(xv[i].x, wv[c][0], acc[i][c][0]);
                        acc[i][c][1] = fmaf(xv[i].y, wv[c][1], acc[i][c][1]);
                        acc[i][c][2] = fmaf(xv[i].z, wv[c][2], acc[i][c][2]);
                        acc[i][c][3] = fmaf(xv[i].w, wv[c][3], acc[i][c][3]);
                    }
            }
        }
    }

    // ---- epilogue in registers: bias -> activation -> scale -> residual
    float v[RPT][CW];
#pragma unroll
    for (int c = 0; c < CW; ++c) {
        const int col = n0 + lane + 32 * c;
        const bool col_ok = col < a.N;
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
            const long long row = row0 + rg + 8 * i;
            const float dot = (acc[i][c][0] + acc[i][c][1]) + (acc[i][c][2] + acc[i][c][3]);
            float y = a.scale * act_by_id(a.act, dot + bias_r[c]);
            if (a.residual != nullptr && col_ok && row < a.M) y += __ldg(a.residual + row * a.ldr + col);
            v[i][c] = y;
        }
    }

    if (a.reduce != 0) {
        // ---- this CTA's pair per row (warp = row, lanes = this CTA's columns)
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
            float s0, s1;
            if (a.reduce == 1) {                       // LayerNorm: (mean, sum of squared deviations) of n_loc values
                float s = 0.0f;
#pragma unroll
                for (int c = 0; c < CW; ++c) s += (lane + 32 * c < n_loc) ? v[i][c] : 0.0f;
                const float mean = n_loc > 0 ? warp_sum_f(s) / (float)n_loc : 0.0f;
                float d2 = 0.0f;
#pragma unroll
                for (int c = 0; c < CW; ++c) {
                    const float d = v[i][c] - mean;
                    d2 += (lane + 32 * c < n_loc) ? d * d : 0.0f;
                }
                s0 = mean;
                s1 = warp_sum_f(d2);
            } else {                                   // softmax: (max, sum exp(v - max))
                float m = -INFINITY;
#pragma unroll
                for (int c = 0; c < CW; ++c) m = fmaxf(m, (lane + 32 * c < n_loc) ? v[i][c] : -INFINITY);
                m = warp_max_f(m);
                float s = 0.0f;
#pragma unroll
                for (int c = 0; c < CW; ++c) s += (lane + 32 * c < n_loc) ? expf(v[i][c] - m) : 0.0f;
                s0 = m;
                s1 = warp_sum_f(s);
            }
            if (lane == 0) stat[rg + 8 * i] = make_float2(s0, s1);
        }
        cluster_sync_all();                            // every rank's pairs are visible cluster-wide
        // ---- merge the ranks' pairs (lane r fetches rank r's pair; merged in rank order, so every CTA
        //      of the cluster computes bit-identical statistics)
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
            float2 mine = make_float2(0.0f, 0.0f);
            if (lane < cn) mine = ld_shared_cluster_f32x2(mapa_shared(smem_u32(&stat[rg + 8 * i]), (uint32_t)lane));
            if (a.reduce == 1) {
                float n_run = 0.0f, mean = 0.0f, m2 = 0.0f;
                for (int r = 0; r < cn; ++r) {
                    const float mr = __shfl_sync(0xffffffffu, mine.x, r), qr = __shfl_sync(0xffffffffu, mine.y, r);
                    const float nr = (float)min(max(a.N - r * BN, 0), BN);
                    if (nr > 0.0f) {                   // pairwise (Chan) update: no E[x^2] - E[x]^2 cancellation
                        const float n_new = n_run + nr, delta = mr - mean;
                        mean += delta * (nr / n_new);
                        m2 += qr + delta * delta * (n_run * nr / n_new);
                        n_run = n_new;
                    }
                }
                const float rstd = rsqrtf(m2 / (float)a.N + a.eps);
#pragma unroll
                for (int c = 0; c < CW; ++c) v[i][c] = (v[i][c] - mean) * rstd * gamma_r[c] + beta_r[c];
            } else {
                float m = -INFINITY;
                for (int r = 0; r < cn; ++r) m = fmaxf(m, __shfl_sync(0xffffffffu, mine.x, r));
                float l = 0.0f;
                for (int r = 0; r < cn; ++r) {
                    const float mr = __shfl_sync(0xffffffffu, mine.x, r), lr = __shfl_sync(0xffffffffu, mine.y, r);
                    if (lr > 0.0f) l += lr * expf(mr - m);
                }
                const float inv = 1.0f / l;
#pragma unroll
                for (int c = 0; c < CW; ++c) v[i][c] = expf(v[i][c] - m) * inv;
            }
        }
        // Every read of the peers' pairs is done.  No CTA may leave while a peer still reads ITS pairs, so the
        // cluster meets once more before exit; the arrival is posted here (it orders nothing, hence relaxed) and
        // only waited for after the output stores, which therefore overlap the rendezvous.
        cluster_arrive_relaxed();
    }

#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const long long row = row0 + rg + 8 * i;
#pragma unroll
        for (int c = 0; c < CW; ++c) {
            const int col = n0 + lane + 32 * c;
            if (row < a.M && col < a.N) a.out[row * a.ldo + col] = v[i][c];
        }
    }
    if (a.reduce != 0) cluster_wait();
}

template <int RPT, int CW, bool NK>
cudaError_t launch_one(const Fp32ChainArgs &a, int cn, cudaStream_t stream)
{
    constexpr int BM = 8 * RPT, BN = 32 * CW;
    int kc = (SMEM_FLOATS_MAX / (BM + BN + 1)) & ~3;
    const int k4 = (a.K + 3) & ~3;
    if (kc > k4) kc = k4;
    const size_t smem = sizeof(float) * ((size_t)BM * kc + (NK ? (size_t)BN * (kc + 1) : (size_t)kc * BN));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(cn * ((a.M + BM - 1) / BM)));
    cfg.blockDim = dim3(FT);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cn; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see launch_kernel
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.pdl != 0 ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, fp32_chain_kernel<RPT, CW, NK>, a, kc);
}

template <int RPT, int CW>
cudaError_t launch_nk(const Fp32ChainArgs &a, int cn, cudaStream_t stream)
{
    return a.w_is_nk ? launch_one<RPT, CW, true>(a, cn, stream) : launch_one<RPT, CW, false>(a, cn, stream);
}

template <int RPT>
cudaError_t launch_cw(const Fp32ChainArgs &a, int cw, int cn, cudaStream_t stream)
{
    switch (cw) {
    case 1:  return launch_nk<RPT, 1>(a, cn, stream);
    case 2:  return launch_nk<RPT, 2>(a, cn, stream);
    default: return launch_nk<RPT, 4>(a, cn, stream);
    }
}

template <int RPT, int CW, bool NK>
cudaError_t setup_one()
{
    return cudaFuncSetAttribute(fp32_chain_kernel<RPT, CW, NK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)(sizeof(float) * (SMEM_FLOATS_MAX + 8 * 32 * 4)));
}

}  // namespace

cudaError_t setup_fp32_chain()
{
    cudaError_t e = cudaSuccess;
#define PIKE_FP32_SETUP(R, C)                                                      \
    if (e == cudaSuccess) e = setup_one<R, C, false>();                            \
    if (e == cudaSuccess) e = setup_one<R, C, true>();
    PIKE_FP32_SETUP(1, 1) PIKE_FP32_SETUP(1, 2) PIKE_FP32_SETUP(1, 4)
    PIKE_FP32_SETUP(2, 1) PIKE_FP32_SETUP(2, 2) PIKE_FP32_SETUP(2, 4)
    PIKE_FP32_SETUP(4, 1) PIKE_FP32_SETUP(4, 2) PIKE_FP32_SETUP(4, 4)
#undef PIKE_FP32_SETUP
    return e;
}

cudaError_t launch_fp32_chain(const Fp32ChainArgs &a, int num_sms, cudaStream_t stream)
{
    if (a.M <= 0) return cudaSuccess;
    // columns per CTA: the narrowest slice that keeps the cluster within 8 CTAs (N <= 1024 checked by the caller)
    const int cw = a.N <= 256 ? 1 : (a.N <= 512 ? 2 : 4);
    const int need = (a.N + 32 * cw - 1) / (32 * cw);
    int cn = 1;
    while (cn < need) cn *= 2;                          // power of two; ranks past N own no columns
    // rows per CTA: small problems spread over as many SMs as they can fill, large ones amortise W over more rows
    if ((long long)cn * ((a.M + 7) / 8) <= 2ll * num_sms) return launch_cw<1>(a, cw, cn, stream);
    if ((long long)cn * ((a.M + 15) / 16) <= 4ll * num_sms) return launch_cw<2>(a, cw, cn, stream);
    return launch_cw<4>(a, cw, cn, stream);
}

}  // namespace pike
