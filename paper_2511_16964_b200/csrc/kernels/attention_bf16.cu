// GEMM -> online softmax -> GEMM attention chain on tcgen05 / tensor memory.
// The score tile lives in tensor memory and registers only; nothing but Q, K, V
// and O touches HBM.
//
// One CTA per (batch*head, 128-query tile), 192 threads:
//   warp 0      TMA producer: Q once, then K_j / V_j tiles (128 keys x 128 d) into
//               two-stage 128-byte-swizzled rings
//   warp 1      MMA issuer: S_j = Q K_j^T (K-major operands) into TMEM columns
//               [0,128); PV_j = P_j V_j (V is the MN-major B operand) into [128,256)
//   warps 2..5  softmax: thread = query row.  Pass 1 reads S_j for the row maximum,
//               pass 2 recomputes p = 2^(s*c - m), rounds to bf16 and writes P_j to
//               shared memory in the K-major swizzled operand layout.  The running
//               output O lives in registers: O = O*alpha + PV_j is folded in one tile
//               late, so PV_j overlaps the next tile's S MMA and softmax.
// Causal masking is computed from indices on the diagonal tile only; tiles above the
// diagonal are never loaded.  CTAs are ordered longest-first.
#include "../device/ptx.cuh"
#include "kernels.h"

namespace pike {
namespace {

constexpr int D = 128;
constexpr int BQ = 128, BKV = 128;
constexpr int KV_STAGES = 2;
constexpr int SUB_BYTES = 128 * 64 * 2;       // one 128-row x 64-element swizzled sub-tile: 16 KiB
constexpr int TILE_BYTES = 2 * SUB_BYTES;     // 128 x 128 bf16: 32 KiB
constexpr int THREADS = 192;
constexpr int SOFTMAX_THREADS = 128;
constexpr int TMEM_COLS = 256;
constexpr uint32_t COL_S = 0, COL_PV = 128;

struct __align__(8) Ctrl {
    uint64_t q_full;
    uint64_t k_full[KV_STAGES], k_empty[KV_STAGES];
    uint64_t v_full[KV_STAGES], v_empty[KV_STAGES];
    uint64_t s_full, p_full, o_full;
    uint32_t tmem_base;
    uint32_t abort;
};
constexpr size_t SMEM_BYTES = 1024 + (size_t)TILE_BYTES * (1 + 2 * KV_STAGES + 1) + sizeof(Ctrl);

enum : uint32_t { BAR_Q = 1, BAR_K_EMPTY, BAR_V_EMPTY, BAR_K_FULL, BAR_V_FULL, BAR_S_FULL, BAR_P_FULL, BAR_O_FULL };

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(THREADS, 1)
attention_bf16_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      const __grid_constant__ CUtensorMap tmV, const AttnArgs p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *q_s = base;
    uint8_t *k_s = q_s + TILE_BYTES;                  // [KV_STAGES]
    uint8_t *v_s = k_s + KV_STAGES * TILE_BYTES;      // [KV_STAGES]
    uint8_t *p_s = v_s + KV_STAGES * TILE_BYTES;
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(p_s + TILE_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_q_tiles = (p.S + BQ - 1) / BQ;
    const int qt = num_q_tiles - 1 - (int)(blockIdx.x / (unsigned)p.BH);   // longest first
    const int bh = (int)(blockIdx.x % (unsigned)p.BH);
    const int num_kv = p.causal ? qt + 1 : (p.S + BKV - 1) / BKV;

    if (threadIdx.x == 0) {
        mbar_init(&ctrl->q_full, 1);
        for (int s = 0; s < KV_STAGES; ++s) {
            mbar_init(&ctrl->k_full[s], 1); mbar_init(&ctrl->k_empty[s], 1);
            mbar_init(&ctrl->v_full[s], 1); mbar_init(&ctrl->v_empty[s], 1);
        }
        mbar_init(&ctrl->s_full, 1);
        mbar_init(&ctrl->p_full, SOFTMAX_THREADS);
        mbar_init(&ctrl->o_full, 1);
        ctrl->abort = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
    }
    if (warp == 1) {
        tmem_alloc(&ctrl->tmem_base, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    const WaitCtx ctx{p.status, &ctrl->abort, p.limit_ns, KID_ATTN};

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_arrive_expect_tx(&ctrl->q_full, TILE_BYTES);
            tma_load_3d(q_s, &tmQ, &ctrl->q_full, 0, qt * BQ, bh);
            tma_load_3d(q_s + SUB_BYTES, &tmQ, &ctrl->q_full, 64, qt * BQ, bh);
            for (int j = 0; j < num_kv; ++j) {
                const int s = j % KV_STAGES;
                const uint32_t ph = (j / KV_STAGES) & 1;
                mbar_wait(&ctrl->k_empty[s], ph ^ 1, ctx, BAR_K_EMPTY);
                mbar_arrive_expect_tx(&ctrl->k_full[s], TILE_BYTES);
                tma_load_3d(k_s + s * TILE_BYTES, &tmK, &ctrl->k_full[s], 0, j * BKV, bh);
                tma_load_3d(k_s + s * TILE_BYTES + SUB_BYTES, &tmK, &ctrl->k_full[s], 64, j * BKV, bh);
                mbar_wait(&ctrl->v_empty[s], ph ^ 1, ctx, BAR_V_EMPTY);
                mbar_arrive_expect_tx(&ctrl->v_full[s], TILE_BYTES);
                tma_load_3d(v_s + s * TILE_BYTES, &tmV, &ctrl->v_full[s], 0, j * BKV, bh);
                tma_load_3d(v_s + s * TILE_BYTES + SUB_BYTES, &tmV, &ctrl->v_full[s], 64, j * BKV, bh);
            }
        }
    } else if (warp == 1) {
        // -------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc_s = make_idesc_bf16(BQ, BKV, false, false);   // Q, K both K-major (d contiguous)
            const uint32_t idesc_o = make_idesc_bf16(BQ, D, false, true);      // P K-major, V MN-major (d contiguous)
            const uint32_t q_addr = smem_u32(q_s), p_addr = smem_u32(p_s);
            auto issue_s = [&](int j) {
                const int s = j % KV_STAGES;
                const uint32_t ph = (j / KV_STAGES) & 1;
                mbar_wait(&ctrl->k_full[s], ph, ctx, BAR_K_FULL);
                tc_fence_after();
                const uint32_t k_addr = smem_u32(k_s + s * TILE_BYTES);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (ks >> 2) * SUB_BYTES + (ks & 3) * 32;
                    umma_ss(tmem_base + COL_S, make_smem_desc_sw128(q_addr + off, 0, 1024),
                            make_smem_desc_sw128(k_addr + off, 0, 1024), idesc_s, ks != 0 ? 1u : 0u);
                }
                umma_commit(&ctrl->s_full);
                umma_commit(&ctrl->k_empty[s]);
            };
            mbar_wait(&ctrl->q_full, 0, ctx, BAR_Q);
            issue_s(0);
            for (int j = 0; j < num_kv; ++j) {
                const int s = j % KV_STAGES;
                const uint32_t ph = (j / KV_STAGES) & 1;
                mbar_wait(&ctrl->p_full, j & 1, ctx, BAR_P_FULL);   // P_j in smem, S_j and PV_{j-1} consumed
                tc_fence_after();
                if (j + 1 < num_kv) issue_s(j + 1);
                mbar_wait(&ctrl->v_full[s], ph, ctx, BAR_V_FULL);
                tc_fence_after();
                const uint32_t v_addr = smem_u32(v_s + s * TILE_BYTES);
#pragma unroll
                for (int ks = 0; ks < BKV / 16; ++ks) {
                    const uint32_t a_off = (ks >> 2) * SUB_BYTES + (ks & 3) * 32;
                    umma_ss(tmem_base + COL_PV, make_smem_desc_sw128(p_addr + a_off, 0, 1024),
                            make_smem_desc_sw128(v_addr + ks * 2048, SUB_BYTES, 1024), idesc_o, ks != 0 ? 1u : 0u);
                }
                umma_commit(&ctrl->o_full);
                umma_commit(&ctrl->v_empty[s]);
            }
        }
    } else {
        // ----------------------------------------------------------------- softmax
        const int q = warp & 3;
        const int r_in_tile = q * 32 + lane;
        const int qidx = qt * BQ + r_in_tile;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const float c = p.scale * 1.4426950408889634f;   // scores are kept in the log2 domain
        float o[D];
#pragma unroll
        for (int i = 0; i < D; ++i) o[i] = 0.0f;
        float m_run = -INFINITY, l_run = 0.0f, alpha_prev = 0.0f;

        for (int j = 0; j < num_kv; ++j) {
            const bool edge = (j == num_kv - 1);
            const int k0 = j * BKV;
            mbar_wait(&ctrl->s_full, j & 1, ctx, BAR_S_FULL);
            tc_fence_after();

            // pass 1: row maximum of the scaled, masked scores
            float tmax = -INFINITY;
#pragma unroll 1
            for (int cc = 0; cc < BKV / 32; ++cc) {
                uint32_t r[32];
                tmem_ld32(tmem_base + lane_addr + COL_S + cc * 32, r);
                tmem_ld_wait();
                if (edge) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int kidx = k0 + cc * 32 + i;
                        const bool ok = kidx < p.S && (!p.causal || kidx <= qidx);
                        if (ok) tmax = fmaxf(tmax, __uint_as_float(r[i]));
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) tmax = fmaxf(tmax, __uint_as_float(r[i]));
                }
            }
            // the scale is positive, so max(s)*c == max(s*c); rows past S keep -inf and are never stored
            float m_new = fmaxf(m_run, tmax * c);
            if (m_new == -INFINITY) m_new = 0.0f;
            const float alpha = ex2(m_run - m_new);

            // fold the previous tile's PV into the register accumulator
            if (j > 0) {
                mbar_wait(&ctrl->o_full, (j - 1) & 1, ctx, BAR_O_FULL);
                tc_fence_after();
#pragma unroll
                for (int cc = 0; cc < D / 32; ++cc) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + lane_addr + COL_PV + cc * 32, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[cc * 32 + i] = fmaf(o[cc * 32 + i], alpha_prev, __uint_as_float(r[i]));
                }
            }

            // pass 2: probabilities -> bf16 -> shared memory (K-major, 128-byte swizzle)
            float lsum = 0.0f;
            const float neg_m = -m_new;
#pragma unroll 1
            for (int cc = 0; cc < BKV / 32; ++cc) {
                uint32_t r[32];
                tmem_ld32(tmem_base + lane_addr + COL_S + cc * 32, r);
                tmem_ld_wait();
                float pr[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float e = ex2(fmaf(__uint_as_float(r[i]), c, neg_m));
                    if (edge) {
                        const int kidx = k0 + cc * 32 + i;
                        const bool ok = kidx < p.S && (!p.causal || kidx <= qidx);
                        e = ok ? e : 0.0f;
                    }
                    pr[i] = e;
                    lsum += e;
                }
                uint8_t *prow = p_s + (cc >> 1) * SUB_BYTES + r_in_tile * 128;
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const int chunk = ((cc & 1) * 4 + g) ^ (r_in_tile & 7);
                    *reinterpret_cast<uint4 *>(prow + chunk * 16) =
                        make_uint4(pack_bf16x2(pr[g * 8 + 0], pr[g * 8 + 1]), pack_bf16x2(pr[g * 8 + 2], pr[g * 8 + 3]),
                                   pack_bf16x2(pr[g * 8 + 4], pr[g * 8 + 5]), pack_bf16x2(pr[g * 8 + 6], pr[g * 8 + 7]));
                }
            }
            l_run = fmaf(l_run, alpha, lsum);
            m_run = m_new;
            alpha_prev = alpha;
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(&ctrl->p_full);
        }

        // last PV, normalise, store
        mbar_wait(&ctrl->o_full, (num_kv - 1) & 1, ctx, BAR_O_FULL);
        tc_fence_after();
        const float inv_l = 1.0f / l_run;
        __nv_bfloat16 *orow = static_cast<__nv_bfloat16 *>(p.out) + ((long long)bh * p.S + qidx) * D;
#pragma unroll
        for (int cc = 0; cc < D / 32; ++cc) {
            uint32_t r[32];
            tmem_ld32(tmem_base + lane_addr + COL_PV + cc * 32, r);
            tmem_ld_wait();
            if (qidx < p.S) {
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    float f[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        f[i] = fmaf(o[cc * 32 + g * 8 + i], alpha_prev, __uint_as_float(r[g * 8 + i])) * inv_l;
                    *reinterpret_cast<uint4 *>(orow + cc * 32 + g * 8) =
                        make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]),
                                   pack_bf16x2(f[6], f[7]));
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (ctrl->abort) abort_drain();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace

cudaError_t launch_attention_bf16(const CUtensorMap &tmQ, const CUtensorMap &tmK, const CUtensorMap &tmV,
                                  const AttnArgs &a, cudaStream_t stream)
{
    if (a.BH <= 0 || a.S <= 0) return cudaSuccess;
    const int num_q_tiles = (a.S + BQ - 1) / BQ;
    cudaError_t e = cudaFuncSetAttribute(attention_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)SMEM_BYTES);
    if (e != cudaSuccess) return e;
    attention_bf16_kernel<<<dim3((unsigned)num_q_tiles * (unsigned)a.BH), THREADS, SMEM_BYTES, stream>>>(tmQ, tmK, tmV, a);
    return cudaGetLastError();
}

}  // namespace pike
