// fp32 Linear + bias + activation + scale + residual + row reduction in ONE kernel
// on the CUDA cores (true fp32 FMA; TF32 would miss the 1e-4 bound once LayerNorm
// divides by a standard deviation below one).
//
// A thread-block CLUSTER owns a block of BM complete output rows; its CTAs split the N columns
// (BN = 32, 64 or 128 columns each, at most 8 CTAs for N <= 1024).  Each CTA stages only its own
// column slice of W (K x BN) and the BM rows of x in shared memory, so W crosses the L2 once per
// row block instead of once per CTA-row as a one-CTA-per-row layout would have it, and the
// whole problem spreads over many SMs even when M is small.
// Two kernels share the staging, the epilogue and the reduction:
//  - fp32_chain_splitk_kernel (BM = 8; small problems, whose time is a chain of latencies): groups of
//    threads split k, every thread accumulates a 4 x 4 register tile over its k slice (16 FMAs per 16-byte
//    shared-memory load of either operand: the shared-memory pipe, not the FMA pipe, bounds a tile this small),
//    and the slices' partial sums meet in shared memory.  Operands arrive as two tiled copies on one mbarrier
//    where the tensors allow a tensor map.
//  - fp32_chain_kernel (BM = 16, 32 or 64, 128 columns per CTA; problems that fill the chip): warp = rows
//    warp + 8i, lane = four adjacent columns, over all of k.
// The LayerNorm / softmax reduction over N never leaves the cluster: every warp reduces its rows
// over the CTA's columns with shuffles, the CTAs publish one pair per row - (mean, sum of squared
// deviations) or (max, sum exp) - in their shared memory, and after one cluster barrier every CTA
// merges the pairs of all ranks through distributed shared memory.
#include "../device/act.cuh"
#include "../device/ptx.cuh"
#include "kernels.h"

#include <string.h>

namespace pike {
namespace {

constexpr int FT = 256;                    // 8 warps
constexpr int SMEM_FLOATS_MAX = 24576;     // 96 KiB of shared memory per CTA
constexpr int MAX_BM = 64;
constexpr int SPLITK_BM = 8;

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

// A thread's c-th column inside the CTA's slice: strided over the warp (lane + 32c), or, ADJ, CW adjacent
// columns per lane (one 16-byte shared-memory load of W feeds four of them).
template <int CW, bool ADJ>
__device__ __forceinline__ int col_in_cta(int lane, int c) { return ADJ ? CW * lane + c : lane + 32 * c; }

// The per-column parameters of a thread's columns; fetched before the main loop so that their latency hides
// under it.
template <int CW>
struct ColParams {
    float bias[CW], gamma[CW], beta[CW];
};
template <int CW, bool ADJ = false>
__device__ __forceinline__ void load_col_params(const Fp32ChainArgs &a, int n0, int lane, ColParams<CW> &p)
{
#pragma unroll
    for (int c = 0; c < CW; ++c) {
        const int col = n0 + col_in_cta<CW, ADJ>(lane, c);
        const bool col_ok = col < a.N;
        p.bias[c] = (a.bias != nullptr && col_ok) ? __ldg(a.bias + col) : 0.0f;
        p.gamma[c] = (a.reduce == 1 && a.gamma != nullptr && col_ok) ? __ldg(a.gamma + col) : 1.0f;
        p.beta[c] = (a.reduce == 1 && a.beta != nullptr && col_ok) ? __ldg(a.beta + col) : 0.0f;
    }
}

// ---- staging with per-thread asynchronous copies: any alignment, any tail.  16-byte copies where the rows
// are 16-byte aligned, 4-byte copies otherwise; elements outside the tensors are written as zeros.  All of a
// thread's copies are in flight together; the caller waits for them (cp_async_wait_all + __syncthreads).
// x rows [row0, row0 + BM) x k [k0, k0 + kn) -> x_s [BM][kc]; positions kn .. kr-1 (kr = kn rounded up to four:
// the FMA loops read k in quads) are zeroed.
template <int BM>
__device__ __forceinline__ void stage_x_cp_async(const Fp32ChainArgs &a, float *x_s, int kc, int k0, int kn,
                                                 long long row0, int tid)
{
    const int kn4 = kn & ~3, kr = (kn + 3) & ~3;
    if ((a.ldx & 3) == 0) {
        const int qpr = kr >> 2;               // quads per row
        for (int idx = tid; idx < BM * qpr; idx += FT) {
            const int r = idx / qpr, k = (idx - r * qpr) << 2;
            const long long row = row0 + r;
            const float *src = a.x + (row < a.M ? row * a.ldx + k0 + k : 0);
            if (k < kn4) {
                cp_async_16(x_s + r * kc + k, src, row < a.M);
            } else {                            // the quad that holds the end of the row, element by element
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
}
// This CTA's column slice of W: [kc][BN], or for [N,K] weights transposed as [BN][kc + 1], one element per
// copy (the odd pitch that keeps the FMA loop free of bank conflicts leaves no 16-byte aligned rows).
template <int BN, bool NK>
__device__ __forceinline__ void stage_w_cp_async(const Fp32ChainArgs &a, float *w_s, int kc, int k0, int kn, int n0,
                                                 int n_loc, int tid)
{
    const int kr = (kn + 3) & ~3;
    if constexpr (!NK) {
        if ((a.ldw & 3) == 0 && (n_loc & 3) == 0) {
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
        const int pitch = kc + 1;
        for (int idx = tid; idx < BN * kr; idx += FT) {
            const int c = idx / kr, k = idx - c * kr;
            const bool ok = c < n_loc && k < kn;
            cp_async_4(w_s + c * pitch + k, ok ? a.w + (long long)(n0 + c) * a.ldw + k0 + k : a.w, ok);
        }
    }
}

// ---- from the dot products to the stored output: bias -> activation -> scale -> residual in registers, then
// the row reduction.  Warp rg owns rows rg + 8i of the block, lane the columns n0 + col_in_cta(lane, c).
template <int RPT, int CW, bool ADJ = false>
__device__ __forceinline__ void epilogue_reduce_store(const Fp32ChainArgs &a, float (&v)[RPT][CW],
                                                      const ColParams<CW> &p, float2 *stat, long long row0, int n0,
                                                      int n_loc, int lane, int rg, int cn)
{
    constexpr int BN = 32 * CW;
#pragma unroll
    for (int c = 0; c < CW; ++c) {
        const int col = n0 + col_in_cta<CW, ADJ>(lane, c);
        const bool col_ok = col < a.N;
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
            const long long row = row0 + rg + 8 * i;
            float y = a.scale * act_by_id(a.act, v[i][c] + p.bias[c]);
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
                // one pass over values shifted by the CTA's first column (the shift keeps sum d^2 - (sum d)^2 / n
                // free of the cancellation a plain sum of squares suffers when the mean dwarfs the spread); the two
                // sums travel through the shuffles side by side
                const float v0 = __shfl_sync(0xffffffffu, v[i][0], 0);
                float sd = 0.0f, sq = 0.0f;
#pragma unroll
                for (int c = 0; c < CW; ++c) {
                    const float d = (col_in_cta<CW, ADJ>(lane, c) < n_loc) ? v[i][c] - v0 : 0.0f;
                    sd += d;
                    sq = fmaf(d, d, sq);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    sd += __shfl_xor_sync(0xffffffffu, sd, o);
                    sq += __shfl_xor_sync(0xffffffffu, sq, o);
                }
                const float inv = n_loc > 0 ? 1.0f / (float)n_loc : 0.0f;
                s0 = n_loc > 0 ? v0 + sd * inv : 0.0f;
                s1 = fmaxf(sq - sd * sd * inv, 0.0f);
            } else {                                   // softmax: (max, sum exp(v - max))
                float m = -INFINITY;
#pragma unroll
                for (int c = 0; c < CW; ++c) m = fmaxf(m, (col_in_cta<CW, ADJ>(lane, c) < n_loc) ? v[i][c] : -INFINITY);
                m = warp_max_f(m);
                float s = 0.0f;
#pragma unroll
                for (int c = 0; c < CW; ++c) s += (col_in_cta<CW, ADJ>(lane, c) < n_loc) ? expf(v[i][c] - m) : 0.0f;
                s0 = m;
                s1 = warp_sum_f(s);
            }
            if (lane == 0) stat[rg + 8 * i] = make_float2(s0, s1);
        }
        cluster_sync_all();                            // every rank's pairs are visible cluster-wide
        // ---- merge the ranks' pairs: lane l fetches the pair of rank l mod 8, so every group of eight lanes holds
        //      all ranks and three shuffle steps give every lane the merged value (the same tree in every CTA, so
        //      the whole cluster computes bit-identical statistics).  LayerNorm pools the ranks' moments about
        //      rank 0's mean (deviations of means: no E[x^2] - E[x]^2 cancellation), three sums side by side.
        const int rk = lane & 7;
        const float nr = rk < cn ? (float)min(max(a.N - rk * BN, 0), BN) : 0.0f;       // columns of rank rk
        const float inv_n = 1.0f / (float)a.N;
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
            float2 mine = make_float2(0.0f, 0.0f);
            if (rk < cn) mine = ld_shared_cluster_f32x2(mapa_shared(smem_u32(&stat[rg + 8 * i]), (uint32_t)rk));
            if (a.reduce == 1) {
                const float mean0 = __shfl_sync(0xffffffffu, mine.x, 0);       // every lane takes part in the shuffle
                const float e = nr > 0.0f ? mine.x - mean0 : 0.0f;
                float sa = nr * e, sb = nr * e * e, sc = mine.y;
#pragma unroll
                for (int o = 4; o > 0; o >>= 1) {
                    sa += __shfl_xor_sync(0xffffffffu, sa, o);
                    sb += __shfl_xor_sync(0xffffffffu, sb, o);
                    sc += __shfl_xor_sync(0xffffffffu, sc, o);
                }
                const float mean = mean0 + sa * inv_n;
                const float m2 = fmaxf(sc + sb - sa * sa * inv_n, 0.0f);
                const float rstd = rsqrtf(m2 * inv_n + a.eps);
#pragma unroll
                for (int c = 0; c < CW; ++c) v[i][c] = (v[i][c] - mean) * rstd * p.gamma[c] + p.beta[c];
            } else {
                const bool has = nr > 0.0f && mine.y > 0.0f;
                float m = has ? mine.x : -INFINITY;
#pragma unroll
                for (int o = 4; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
                float l = has ? mine.y * expf(mine.x - m) : 0.0f;
#pragma unroll
                for (int o = 4; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
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
            const int col = n0 + col_in_cta<CW, ADJ>(lane, c);
            if (row < a.M && col < a.N) a.out[row * a.ldo + col] = v[i][c];
        }
    }
    if (a.reduce != 0) cluster_wait();
}

// ---- small problems: the warps split k ------------------------------------------------------------
// CTA tile 8 x (32 CW).  A thread accumulates 4 rows x 4 adjacent columns over one of 16 / CW slices of every
// staged k chunk (k ascending): per four k it issues four 16-byte loads of x and four of W for 64 FMAs (one
// column and 8 rows per thread, measured first, spent 3,000 cycles in this loop at 128 x 256 x 256 against 2,000
// for everything else: a 16-byte load whose lanes all read one address still costs the pipe as much as one that
// reads 512 bytes).  The slices' partial sums meet in shared memory and are added in a fixed tree.
// Staging: where the tensors allow a tensor map (16-byte aligned base and row pitch; W as [K,N]) ONE thread
// fetches the chunk's x rows and W slice as two tiled copies completing on one mbarrier (bounded wait); rows,
// columns and k past the tensors arrive as zeros.  Otherwise the per-thread asynchronous copies above.
// (Row-wise untiled bulk copies were measured too: 264 small copies per CTA queue up for about 11 cycles each.)
// NK: w is [N,K].
template <int CW, bool NK>
__global__ void __launch_bounds__(FT) fp32_chain_splitk_kernel(const Fp32ChainArgs a, const int kc, const int tma_x,
                                                               const int tma_w,
                                                               const __grid_constant__ CUtensorMap tm_x,
                                                               const __grid_constant__ CUtensorMap tm_w)
{
    constexpr int BM = SPLITK_BM, BN = 32 * CW;
    extern __shared__ uint8_t smem_raw[];
    __shared__ float2 stat[BM];            // this CTA's per-row pair, read by the whole cluster
    __shared__ uint64_t full;              // the tiled copies of a chunk complete here
    __shared__ uint32_t abort_word;
    // tiled copies want 128-byte aligned destinations: x_s is, and w_s follows it by 32 kc bytes (kc a multiple of 4)
    float *x_s = reinterpret_cast<float *>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));   // [BM][kc]
    float *w_s = x_s + BM * kc;                            // [kc][BN], or [BN][kc + 1] for NK
    float *red = w_s + (((NK ? BN * (kc + 1) : kc * BN) + 3) & ~3);   // [16 / CW k slices][BM][BN], 16-byte aligned

    const int tid = threadIdx.x, lane = tid & 31, wp = tid >> 5;
    const int cn = (int)cluster_nctas(), rank = (int)cluster_ctarank();
    const long long row0 = (long long)((int)blockIdx.x / cn) * BM;
    const int n0 = rank * BN;
    const int n_loc = min(max(a.N - n0, 0), BN);          // columns this CTA owns (0 for a padding rank)
    const bool x_tiled = tma_x != 0, w_tiled = !NK && tma_w != 0 && n_loc > 0;
    const uint32_t chunk_bytes = (x_tiled ? (uint32_t)(BM * kc * 4) : 0u) + (w_tiled ? (uint32_t)(kc * BN * 4) : 0u);
    if (tid == 0) {
        abort_word = 0;
        mbar_init(&full, 1);
        fence_barrier_init();
        if (x_tiled) tma_prefetch_desc(&tm_x);
        if (w_tiled) tma_prefetch_desc(&tm_w);
    }
    __syncthreads();
    pdl_wait();
    const WaitCtx ctx{a.status, &abort_word, a.limit_ns, KID_FP32_CHAIN};

    // thread tile: 4 rows x 4 adjacent columns; 8 CW column groups x 2 row groups cover the CTA tile, and
    // NS = 16 / CW groups of such threads split k.  Lanes: column group, then the low part of the k slice; warps:
    // row group, then the high part (so a warp's x loads touch one row group and distinct banks).
    constexpr int CG = 8 * CW, NS = 16 / CW, S_LO = 32 / CG;
    const int cg = lane % CG, rgp = wp & 1, slice = (wp >> 1) * S_LO + lane / CG;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[i][c] = 0.0f;
    ColParams<CW> prm;

    uint32_t phase = 0;
    for (int k0 = 0; k0 < a.K; k0 += kc) {
        const int kn = min(kc, a.K - k0);
        const int kr = (kn + 3) & ~3;
        if (k0 > 0) __syncthreads();       // the previous chunk has been consumed
        if (tid == 0 && chunk_bytes != 0) {
            mbar_arrive_expect_tx(&full, chunk_bytes);     // whole boxes: what lies outside the tensors is zero-filled
            if (a.test_withhold_loads == 0) {
                if (x_tiled) tma_load_2d(x_s, &tm_x, &full, k0, (int)row0);
                if (w_tiled) tma_load_2d(w_s, &tm_w, &full, n0, k0);
            }
        }
        if (!x_tiled) stage_x_cp_async<BM>(a, x_s, kc, k0, kn, row0, tid);
        if (!w_tiled && n_loc > 0) stage_w_cp_async<BN, NK>(a, w_s, kc, k0, kn, n0, n_loc, tid);
        if (k0 == 0) load_col_params<CW>(a, n0, lane, prm);   // in flight beside the operands
        cp_async_wait_all();
        if (chunk_bytes != 0) {
            if (!mbar_wait(&full, phase, ctx, 1u)) abort_drain();   // ran out: let the copies land, finish with what is there
            phase ^= 1u;
        }
        __syncthreads();
        if (n_loc > 0) {
            const int ks = (((kr + NS - 1) / NS) + 3) & ~3;          // k per slice, a multiple of four
            const int kb = slice * ks, ke = min(kb + ks, kr);
            const float *xp = x_s + (rgp * 4) * kc;
#pragma unroll 2
            for (int k = kb; k < ke; k += 4) {
                float4 xv[4];
                float wv[4][4];                                        // [k offset][column]
#pragma unroll
                for (int i = 0; i < 4; ++i) xv[i] = *reinterpret_cast<const float4 *>(xp + i * kc + k);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if constexpr (NK) {
#pragma unroll
                        for (int c = 0; c < 4; ++c) wv[j][c] = w_s[(4 * cg + c) * (kc + 1) + k + j];
                    } else {
                        const float4 t = *reinterpret_cast<const float4 *>(w_s + (k + j) * BN + 4 * cg);
                        wv[j][0] = t.x; wv[j][1] = t.y; wv[j][2] = t.z; wv[j][3] = t.w;
                    }
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        float t = acc[i][c];
                        t = fmaf(xv[i].x, wv[0][c], t);
                        t = fmaf(xv[i].y, wv[1][c], t);
                        t = fmaf(xv[i].z, wv[2][c], t);
                        t = fmaf(xv[i].w, wv[3][c], t);
                        acc[i][c] = t;
                    }
            }
        }
    }

    // ---- the slices' partial sums -> thread (warp = row, lane = column), added in a fixed tree
#pragma unroll
    for (int i = 0; i < 4; ++i)
        *reinterpret_cast<float4 *>(red + (slice * BM + rgp * 4 + i) * BN + 4 * cg) =
            make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    __syncthreads();
    float v[1][CW];
#pragma unroll
    for (int c = 0; c < CW; ++c) {
        float part[NS];
#pragma unroll
        for (int w = 0; w < NS; ++w) part[w] = red[(w * BM + wp) * BN + lane + 32 * c];
#pragma unroll
        for (int step = 1; step < NS; step *= 2)
#pragma unroll
            for (int w = 0; w + step < NS; w += 2 * step) part[w] += part[w + step];
        v[0][c] = part[0];
    }
    epilogue_reduce_store<1, CW>(a, v, prm, stat, row0, n0, n_loc, lane, wp, cn);
}

// ---- problems that fill the chip: every thread walks all of k ---------------------------------------
// CTA tile (8 RPT) x 128: warp rg owns rows rg + 8i, a lane FOUR ADJACENT columns ([K,N] weights: one 16-byte
// load of W per k feeds 4 RPT FMAs and a 16-byte broadcast of x per row feeds 16, so the FMA pipe rather than
// the shared-memory pipe sets the pace at RPT = 8) or, for [N,K] weights (staged transposed with an odd pitch),
// columns lane + 32c.  k ascending per output.  Two CTAs fit an SM and cover each other's staging.
template <int RPT, bool NK>
__global__ void __launch_bounds__(FT, 2) fp32_chain_kernel(const Fp32ChainArgs a, const int kc)
{
    constexpr int CW = 4, BM = 8 * RPT, BN = 32 * CW;
    constexpr bool ADJ = !NK;
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

    float acc[RPT][CW];
#pragma unroll
    for (int i = 0; i < RPT; ++i)
#pragma unroll
        for (int c = 0; c < CW; ++c) acc[i][c] = 0.0f;
    ColParams<CW> prm;
    load_col_params<CW, ADJ>(a, n0, lane, prm);

    for (int k0 = 0; k0 < a.K; k0 += kc) {
        const int kn = min(kc, a.K - k0);
        __syncthreads();                                         // the previous chunk has been consumed
        stage_x_cp_async<BM>(a, x_s, kc, k0, kn, row0, tid);
        if (n_loc > 0) stage_w_cp_async<BN, NK>(a, w_s, kc, k0, kn, n0, n_loc, tid);
        cp_async_wait_all();
        __syncthreads();
        if (n_loc > 0) {
            // four k at a time (the tail of a chunk that is not a multiple of four reads the zeros staged above)
#pragma unroll 2
            for (int k = 0; k < kn; k += 4) {
                float4 xv[RPT];
                float wv[4][CW];                                 // [k offset][column]
#pragma unroll
                for (int i = 0; i < RPT; ++i) xv[i] = *reinterpret_cast<const float4 *>(x_s + (rg + 8 * i) * kc + k);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if constexpr (NK) {
#pragma unroll
                        for (int c = 0; c < CW; ++c) wv[j][c] = w_s[(lane + 32 * c) * (kc + 1) + k + j];
                    } else {
                        const float4 t = *reinterpret_cast<const float4 *>(w_s + (k + j) * BN + 4 * lane);
                        wv[j][0] = t.x; wv[j][1] = t.y; wv[j][2] = t.z; wv[j][3] = t.w;
                    }
                }
#pragma unroll
                for (int i = 0; i < RPT; ++i)
#pragma unroll
                    for (int c = 0; c < CW; ++c) {
                        float t = acc[i][c];
                        t = fmaf(xv[i].x, wv[0][c], t);
                        t = fmaf(xv[i].y, wv[1][c], t);
                        t = fmaf(xv[i].z, wv[2][c], t);
                        t = fmaf(xv[i].w, wv[3][c], t);
                        acc[i][c] = t;
                    }
            }
        }
    }
    epilogue_reduce_store<RPT, CW, ADJ>(a, acc, prm, stat, row0, n0, n_loc, lane, rg, cn);
}

template <typename Kernel, typename... Extra>
cudaError_t launch_clusters(Kernel kern, const Fp32ChainArgs &a, int bm, int cn, size_t smem, int kc, cudaStream_t stream,
                            Extra... extra)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(cn * ((a.M + bm - 1) / bm)));
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
    return cudaLaunchKernelEx(&cfg, kern, a, kc, extra...);
}

// chunk length along k: what fits the shared memory beside the other operand, a multiple of four
int chunk_k(int K, int rpt, int cw, bool tiled)
{
    const int bm = 8 * rpt, bn = 32 * cw;                   // (cw = 4 whenever rpt > 1)
    int kc = rpt == 1 ? ((SMEM_FLOATS_MAX - 16 * SPLITK_BM * 32 - bn - 4) / (bm + bn)) & ~3
                      : (SMEM_FLOATS_MAX / (bm + bn + 1)) & ~3;
    if (tiled && kc > 256) kc = 256;                       // a tensor-map box has at most 256 elements per dimension
    const int k4 = (K + 3) & ~3;
    return kc > k4 ? k4 : kc;
}

template <int RPT, bool NK>
cudaError_t launch_one(const Fp32ChainArgs &a, const Fp32ChainPlan &p, cudaStream_t stream)
{
    constexpr int BM = 8 * RPT, BN = 128;
    const size_t smem = sizeof(float) * ((size_t)BM * p.kc + (NK ? (size_t)BN * (p.kc + 1) : (size_t)p.kc * BN));
    return launch_clusters(fp32_chain_kernel<RPT, NK>, a, BM, p.cn, smem, p.kc, stream);
}

template <int CW, bool NK>
cudaError_t launch_splitk(const Fp32ChainArgs &a, const Fp32ChainPlan &p, const CUtensorMap &tm_x, const CUtensorMap &tm_w,
                          cudaStream_t stream)
{
    constexpr int BM = SPLITK_BM, BN = 32 * CW;
    const size_t smem = 128 + sizeof(float) * ((size_t)BM * p.kc + (NK ? (size_t)BN * (p.kc + 1) + 3 : (size_t)p.kc * BN) +
                                               (size_t)16 * BM * 32);
    return launch_clusters(fp32_chain_splitk_kernel<CW, NK>, a, BM, p.cn, smem, p.kc, stream, p.tma_x, p.tma_w, tm_x, tm_w);
}

cudaError_t launch_splitk_cw(const Fp32ChainArgs &a, const Fp32ChainPlan &p, const CUtensorMap &tm_x, const CUtensorMap &tm_w,
                             cudaStream_t stream)
{
    switch (p.cw * 2 + (a.w_is_nk ? 1 : 0)) {
    case 2:  return launch_splitk<1, false>(a, p, tm_x, tm_w, stream);
    case 3:  return launch_splitk<1, true>(a, p, tm_x, tm_w, stream);
    case 4:  return launch_splitk<2, false>(a, p, tm_x, tm_w, stream);
    case 5:  return launch_splitk<2, true>(a, p, tm_x, tm_w, stream);
    case 8:  return launch_splitk<4, false>(a, p, tm_x, tm_w, stream);
    default: return launch_splitk<4, true>(a, p, tm_x, tm_w, stream);
    }
}

template <int RPT>
cudaError_t launch_rows(const Fp32ChainArgs &a, const Fp32ChainPlan &p, cudaStream_t stream)
{
    return a.w_is_nk ? launch_one<RPT, true>(a, p, stream) : launch_one<RPT, false>(a, p, stream);
}

template <typename Kernel>
cudaError_t raise_smem_limit(Kernel kern)
{
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)(sizeof(float) * (SMEM_FLOATS_MAX + 8 * 32 * 4)));
}

}  // namespace

cudaError_t setup_fp32_chain()
{
    cudaError_t e = cudaSuccess;
#define PIKE_FP32_SETUP(R)                                                                        \
    if (e == cudaSuccess) e = raise_smem_limit(fp32_chain_kernel<R, false>);                     \
    if (e == cudaSuccess) e = raise_smem_limit(fp32_chain_kernel<R, true>);
    PIKE_FP32_SETUP(2) PIKE_FP32_SETUP(4) PIKE_FP32_SETUP(8)
#undef PIKE_FP32_SETUP
#define PIKE_FP32_SETUP(C)                                                                        \
    if (e == cudaSuccess) e = raise_smem_limit(fp32_chain_splitk_kernel<C, false>);              \
    if (e == cudaSuccess) e = raise_smem_limit(fp32_chain_splitk_kernel<C, true>);
    PIKE_FP32_SETUP(1) PIKE_FP32_SETUP(2) PIKE_FP32_SETUP(4)
#undef PIKE_FP32_SETUP
    return e;
}

Fp32ChainPlan plan_fp32_chain(const Fp32ChainArgs &a, int num_sms)
{
    Fp32ChainPlan p = {};
    // columns per CTA: the narrowest slice that keeps the cluster within 8 CTAs (N <= 1024 checked by the caller)
    p.cw = a.N <= 256 ? 1 : (a.N <= 512 ? 2 : 4);
    const int need = (a.N + 32 * p.cw - 1) / (32 * p.cw);
    p.cn = 1;
    while (p.cn < need) p.cn *= 2;                      // power of two; ranks past N own no columns
    // small problems (at most two CTAs of 8 rows per SM) spread over as many SMs as they can with narrow column
    // slices and split k inside the CTA; everything else takes 128 columns per CTA and as many rows per CTA (64,
    // 32, 16) as still leave every SM two CTAs
    if ((long long)p.cn * ((a.M + 7) / 8) <= 2ll * num_sms) {
        p.rpt = 1;
    } else {
        p.cw = 4;
        const int need128 = (a.N + 127) / 128;
        p.cn = 1;
        while (p.cn < need128) p.cn *= 2;
        if ((long long)p.cn * ((a.M + 63) / 64) >= 2ll * num_sms) p.rpt = 8;
        else if ((long long)p.cn * ((a.M + 31) / 32) >= 2ll * num_sms) p.rpt = 4;
        else p.rpt = 2;
    }
    if (p.rpt == 1) {   // tensor maps want 16-byte aligned bases and row pitches
        p.tma_x = (a.ldx & 3) == 0 && (reinterpret_cast<uintptr_t>(a.x) & 15) == 0;
        p.tma_w = !a.w_is_nk && (a.ldw & 3) == 0 && (reinterpret_cast<uintptr_t>(a.w) & 15) == 0;
    }
    p.kc = chunk_k(a.K, p.rpt, p.cw, p.tma_x || p.tma_w);
    p.x_box[0] = (uint32_t)p.kc;      p.x_box[1] = SPLITK_BM;
    p.w_box[0] = (uint32_t)(32 * p.cw); p.w_box[1] = (uint32_t)p.kc;
    return p;
}

cudaError_t launch_fp32_chain(const Fp32ChainArgs &a, const Fp32ChainPlan &p, const CUtensorMap *tm_x, const CUtensorMap *tm_w,
                              cudaStream_t stream)
{
    if (a.M <= 0) return cudaSuccess;
    CUtensorMap none;
    memset(&none, 0, sizeof(none));
    const CUtensorMap &mx = (p.tma_x && tm_x != nullptr) ? *tm_x : none, &mw = (p.tma_w && tm_w != nullptr) ? *tm_w : none;
    switch (p.rpt) {
    case 1:  return launch_splitk_cw(a, p, mx, mw, stream);
    case 2:  return launch_rows<2>(a, p, stream);
    case 4:  return launch_rows<4>(a, p, stream);
    default: return launch_rows<8>(a, p, stream);
    }
}

}  // namespace pike
