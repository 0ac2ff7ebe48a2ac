// GEMM -> online softmax -> GEMM attention chain on tcgen05 / tensor memory.
// Scores and probabilities live in tensor memory and registers only; nothing but
// Q, K, V and O touches HBM.
//
// Persistent CTAs (one per SM) walk over work items = (batch*head, PAIR of 128-query tiles), longest
// items first, round-robin; barriers, rings and tensor memory carry over from item to item, so the next
// item's Q/K/V loads and first MMAs overlap the previous item's last softmax and output store.
// 384 threads = 3 warpgroups:
//   WG0  warp 0: TMA producer (both Q tiles once, then K_j / V_j tiles of 128 keys into
//        two-stage 128-byte-swizzled rings); warp 1: MMA issuer (one thread)
//   WG1  softmax for query tile 0        WG2  softmax for query tile 1   (thread = row)
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each.
//   S_t(j) = Q_t K_j^T      both operands K-major from shared memory
//   P_t(j) = 16-bit probabilities (the type of Q/K/V: bf16 or f16), written by the softmax threads over the first 64
//            columns of S_t (two per 32-bit column) and read by the second MMA as its
//            A operand straight from tensor memory
//   O_t   += P_t(j) V_j     V is the MN-major B operand; accumulates in tensor memory
// The MMA warp interleaves the two tiles (PV0, S0', PV1, S1', ...) so one tile's softmax
// runs under the other tile's MMAs.  P_t(j) is handed over in two parts, keys 0..95 (p_full) and keys
// 96..127 (p_half2): six of the eight PV MMAs run while the last chunk's exponentials are still being
// computed, and only two are left once it arrives.  (Three or four parts cost more in waits of the MMA
// warp than they gain.)
// The running maximum is only raised when it grows by more than 2^8 (probabilities stay bounded by
// 256 in between), so rescaling O in tensor memory is rare; it is done by the softmax threads
// themselves between two PV MMAs.
// Causal masking comes from indices on the diagonal tile only; tiles above the diagonal
// are never loaded.  Register budgets are re-partitioned
// with setmaxnreg (104 for WG0, 200 for the softmax warpgroups; 384 x 168 at launch).
#include "../device/ptx.cuh"
#include "kernels.h"

namespace pike {
namespace {

constexpr int BQ = 128, BKV = 128;
constexpr int KV_STAGES = 2;
constexpr int SUB_BYTES = 128 * 64 * 2;       // one 128-row x 64-element swizzled sub-tile: 16 KiB
constexpr int TILE_BYTES = 2 * SUB_BYTES;     // 128 x 128 bf16: 32 KiB
constexpr int THREADS = 384;
constexpr int SOFTMAX_THREADS = 128;          // per query tile
constexpr int TMEM_COLS = 512;
constexpr int REGS_AT_LAUNCH = 168, REGS_WG0 = 104, REGS_SOFTMAX = 200;
static_assert(128 * REGS_WG0 + 256 * REGS_SOFTMAX <= THREADS * REGS_AT_LAUNCH, "setmaxnreg split exceeds the pool");
constexpr float RESCALE_THRESHOLD = 8.0f;     // log2 domain

struct __align__(8) Ctrl {
    uint64_t q_full;
    uint64_t k_full[KV_STAGES], k_empty[KV_STAGES];
    uint64_t v_full[KV_STAGES], v_empty[KV_STAGES];
    uint64_t q_empty;
    uint64_t s_full[2], p_full[2], p_half2[2];   // p_full: keys 0..95 of P_t written, p_half2: keys 96..127
    uint64_t o_final[2], o_free[2];
    uint32_t tmem_base;
    uint32_t abort;
};
constexpr size_t SMEM_BYTES = 1024 + (size_t)TILE_BYTES * (2 + 2 * KV_STAGES) + sizeof(Ctrl);

enum : uint32_t { BAR_Q = 1, BAR_K_EMPTY, BAR_V_EMPTY, BAR_K_FULL, BAR_V_FULL, BAR_S_FULL, BAR_P_FULL, BAR_O_FINAL, BAR_Q_EMPTY, BAR_O_FREE, BAR_P_HALF2 };

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// F16 = the tensors are IEEE half instead of bf16 (operand format of both MMAs, P and the output).
// D = head dimension (64 or 128): one or two 64-wide swizzled sub-tiles per operand tile
template <int D, bool F16>
__global__ void __launch_bounds__(THREADS, 1)
attention_bf16_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      const __grid_constant__ CUtensorMap tmV, const AttnArgs p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *q_s = base;                               // [2] query tiles
    uint8_t *k_s = q_s + 2 * TILE_BYTES;               // [KV_STAGES]
    uint8_t *v_s = k_s + KV_STAGES * TILE_BYTES;       // [KV_STAGES]
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(v_s + KV_STAGES * TILE_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_q_tiles = (p.S + BQ - 1) / BQ;
    const int num_pairs = (num_q_tiles + 1) / 2;
    const int num_kv_all = (p.Sk + BKV - 1) / BKV;          // Sk == S unless this is cross attention
    constexpr int OPERAND_BYTES = (D / 64) * SUB_BYTES;     // bytes of one Q / K / V tile
    // Work order.  A "slot" is one head's longest remaining pair of query tiles together with its shortest
    // (under the causal mask pair u costs 4u+3 tile-MMAs, so every slot of a head costs the same); slots
    // are dealt round-robin to the persistent CTAs.  All CTAs get equal work, CTAs running at the same
    // time sit on neighbouring heads (their K/V tiles are shared through L2), and a CTA's second item
    // re-reads the K/V tiles its first item just used.  i counts this CTA's items: 2 per slot.
    const int slots_per_head = (num_pairs + 1) / 2;
    const int num_slots = slots_per_head * p.BH;
    // returns 0 = past the end, 1 = nothing to do for this i, 2 = item decoded; J[t] = KV tiles query
    // tile t walks over (0 if the second tile of the pair does not exist)
    auto decode = [&](int i, int &pair, int &bh, int (&J)[2]) -> int {
        const int v = (int)blockIdx.x + (i >> 1) * (int)gridDim.x;
        if (v >= num_slots) return 0;
        bh = v / slots_per_head;
        const int combo = v % slots_per_head;
        const int hi = num_pairs - 1 - combo, lo = combo;
        if ((i & 1) && lo >= hi) return 1;     // odd pair count: the middle pair is a slot by itself
        pair = (i & 1) ? lo : hi;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int qt = 2 * pair + t;
            J[t] = qt >= num_q_tiles ? 0 : (p.causal ? qt + 1 : num_kv_all);
        }
        return 2;
    };

    if (threadIdx.x == 0) {
        mbar_init(&ctrl->q_full, 1);
        for (int s = 0; s < KV_STAGES; ++s) {
            mbar_init(&ctrl->k_full[s], 1); mbar_init(&ctrl->k_empty[s], 1);
            mbar_init(&ctrl->v_full[s], 1); mbar_init(&ctrl->v_empty[s], 1);
        }
        mbar_init(&ctrl->q_empty, 1);
        for (int t = 0; t < 2; ++t) {
            mbar_init(&ctrl->s_full[t], 1); mbar_init(&ctrl->p_full[t], SOFTMAX_THREADS); mbar_init(&ctrl->p_half2[t], SOFTMAX_THREADS);
            mbar_init(&ctrl->o_final[t], 1); mbar_init(&ctrl->o_free[t], SOFTMAX_THREADS);
        }
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
    pdl_wait();                 // nothing above touched a global tensor
    const uint32_t tmem_base = ctrl->tmem_base;
    const WaitCtx ctx{p.status, &ctrl->abort, p.limit_ns, KID_ATTN};

    if (warp < 4) {
        setmaxnreg_dec<REGS_WG0>();
        if (warp == 0) {
            // -------------------------------------------------------- TMA producer (warp-uniform loop, one elected lane issues)
            const bool leader = elect_one();
            int g = 0, it = 0;      // KV tiles and items issued so far
            for (int i = 0;; ++i) {
                int pair, bh, J[2];
                const int st = decode(i, pair, bh, J);
                if (st == 0) break;
                if (st == 1) continue;
                const int Jmax = J[0] > J[1] ? J[0] : J[1];
                mbar_wait(&ctrl->q_empty, (it & 1) ^ 1, ctx, BAR_Q_EMPTY);   // the previous item's S MMAs are done
                if (leader) {
                    mbar_arrive_expect_tx(&ctrl->q_full, 2 * OPERAND_BYTES);
#pragma unroll
                    for (int t = 0; t < 2; ++t)
#pragma unroll
                        for (int h2 = 0; h2 < D / 64; ++h2)
                            tma_load_4d(q_s + t * TILE_BYTES + h2 * SUB_BYTES, &tmQ, &ctrl->q_full, h2 * 64,
                                        (2 * pair + t) * BQ, bh % p.H, bh / p.H);
                }
                __syncwarp();
                for (int j = 0; j < Jmax; ++j, ++g) {
                    const int s = g % KV_STAGES;
                    const uint32_t ph = (g / KV_STAGES) & 1;
                    mbar_wait(&ctrl->k_empty[s], ph ^ 1, ctx, BAR_K_EMPTY);
                    if (leader) {
                        mbar_arrive_expect_tx(&ctrl->k_full[s], OPERAND_BYTES);
#pragma unroll
                        for (int h2 = 0; h2 < D / 64; ++h2)
                            tma_load_4d(k_s + s * TILE_BYTES + h2 * SUB_BYTES, &tmK, &ctrl->k_full[s], h2 * 64, j * BKV,
                                        bh % p.H, bh / p.H);
                    }
                    __syncwarp();
                    mbar_wait(&ctrl->v_empty[s], ph ^ 1, ctx, BAR_V_EMPTY);
                    if (leader) {
                        mbar_arrive_expect_tx(&ctrl->v_full[s], OPERAND_BYTES);
#pragma unroll
                        for (int h2 = 0; h2 < D / 64; ++h2)
                            tma_load_4d(v_s + s * TILE_BYTES + h2 * SUB_BYTES, &tmV, &ctrl->v_full[s], h2 * 64, j * BKV,
                                        bh % p.H, bh / p.H);
                    }
                    __syncwarp();
                }
                ++it;
            }
        } else if (warp == 1) {
            // ---------------------------------------------------------- MMA issuer
            // The whole warp runs this loop (uniform control flow keeps descriptors and counters in
            // uniform registers); one elected lane issues the MMAs and commits.
            const bool leader = elect_one();
            const uint32_t idesc_s = make_idesc_bf16(BQ, BKV, false, false, F16);   // Q, K both K-major (d contiguous)
            const uint32_t idesc_o = make_idesc_bf16(BQ, D, false, true, F16);     // P K-major (TMEM), V MN-major
            // Descriptors are built once; the issue loops only add constants to them (this single thread's
            // instruction stream is on the critical path of every hand-off).
            const uint64_t q_desc0 = make_smem_desc_sw128(smem_u32(q_s), 0, 1024);
            const uint64_t q_desc1 = make_smem_desc_sw128(smem_u32(q_s + TILE_BYTES), 0, 1024);
            const uint64_t k_desc0 = make_smem_desc_sw128(smem_u32(k_s), 0, 1024);
            const uint64_t k_desc1 = make_smem_desc_sw128(smem_u32(k_s + TILE_BYTES), 0, 1024);
            const uint64_t v_desc0 = make_smem_desc_sw128(smem_u32(v_s), SUB_BYTES, 1024);
            const uint64_t v_desc1 = make_smem_desc_sw128(smem_u32(v_s + TILE_BYTES), SUB_BYTES, 1024);
            static_assert(KV_STAGES == 2, "descriptor selection below assumes two K/V stages");
            // S_t = Q_t K^T (K tile in ring stage ks) into columns [t*128, t*128+128)
            auto issue_s = [&](int t, int ks) {
                const uint64_t qd = t ? q_desc1 : q_desc0;
                const uint64_t kd = ks ? k_desc1 : k_desc0;
                const uint32_t d_tmem = tmem_base + t * 128;
                if (leader) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = (kk >> 2) * SUB_BYTES + (kk & 3) * 32;
                        umma_ss(d_tmem, desc_advance(qd, off), desc_advance(kd, off), idesc_s, kk != 0 ? 1u : 0u);
                    }
                    umma_commit(&ctrl->s_full[t]);
                }
                __syncwarp();
            };
            // O_t (+)= P_t V for one part of the keys of the V tile in ring stage vs: A = 16-bit P in TMEM (8 columns per 16 keys)
            auto issue_pv = [&](int t, int vs, bool first, int half) {
                const uint64_t vd = vs ? v_desc1 : v_desc0;
                const uint32_t d_tmem = tmem_base + 256 + t * 128, a_tmem = tmem_base + t * 128;
                if (leader) {
#pragma unroll
                    for (int kk = 0; kk < BKV / 16; ++kk) {
                        // first part: keys 0..95 (six MMAs), second part: keys 96..127 (two)
                        if ((kk < 6) == (half == 0))
                            umma_ts(d_tmem, a_tmem + kk * 8, desc_advance(vd, kk * 2048), idesc_o,
                                    (first && kk == 0) ? 0u : 1u);
                    }
                }
                __syncwarp();
            };
            auto commit = [&](uint64_t *bar) {
                if (leader) umma_commit(bar);
                __syncwarp();
            };
            int g = 0, it = 0;                 // KV tiles / items consumed so far
            uint32_t n_s[2] = {0, 0};          // softmax hand-offs per query tile so far
            uint32_t n_o[2] = {0, 0};          // items finished per query tile so far
            for (int i = 0;; ++i) {
                int pair, bh, J[2];
                const int st = decode(i, pair, bh, J);
                if (st == 0) break;
                if (st == 1) continue;
                const int Jmax = J[0] > J[1] ? J[0] : J[1];
                mbar_wait(&ctrl->q_full, it & 1, ctx, BAR_Q);
                mbar_wait(&ctrl->k_full[g % KV_STAGES], (g / KV_STAGES) & 1, ctx, BAR_K_FULL);
                tc_fence_after();
                if (J[0] > 0) issue_s(0, g % KV_STAGES);
                if (J[1] > 0) issue_s(1, g % KV_STAGES);
                commit(&ctrl->k_empty[g % KV_STAGES]);
                if (Jmax == 1) commit(&ctrl->q_empty);
                for (int j = 0; j < Jmax; ++j) {
                    const int gv = g + j, gk = g + j + 1;
                    const int sv = gv % KV_STAGES, sk = gk % KV_STAGES;
                    const bool nxt0 = j + 1 < J[0], nxt1 = j + 1 < J[1];
                    mbar_wait(&ctrl->v_full[sv], (gv / KV_STAGES) & 1, ctx, BAR_V_FULL);
                    if (nxt0 || nxt1) mbar_wait(&ctrl->k_full[sk], (gk / KV_STAGES) & 1, ctx, BAR_K_FULL);
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        if (j < J[t]) {
                            // the first PV of an item overwrites O_t: the previous item's O_t must have been read out
                            if (j == 0 && n_o[t] > 0) mbar_wait(&ctrl->o_free[t], (n_o[t] - 1) & 1, ctx, BAR_O_FREE);
                            mbar_wait(&ctrl->p_full[t], n_s[t] & 1, ctx, BAR_P_FULL);
                            tc_fence_after();
                            issue_pv(t, sv, j == 0, 0);
                            mbar_wait(&ctrl->p_half2[t], n_s[t] & 1, ctx, BAR_P_HALF2);
                            ++n_s[t];
                            tc_fence_after();
                            issue_pv(t, sv, j == 0, 1);
                            if (j == J[t] - 1) commit(&ctrl->o_final[t]);
                        }
                        if (t == 1) commit(&ctrl->v_empty[sv]);
                        if (j + 1 < J[t]) issue_s(t, sk);
                    }
                    if (nxt0 || nxt1) {
                        commit(&ctrl->k_empty[sk]);
                        if (j + 1 == Jmax - 1) commit(&ctrl->q_empty);   // the item's last S MMAs are issued
                    }
                }
                g += Jmax;
                n_o[0] += J[0] > 0;
                n_o[1] += J[1] > 0;
                ++it;
            }
        }
    } else {
        setmaxnreg_inc<REGS_SOFTMAX>();
        // --------------------------------------------------------------- softmax
        const int t = (warp >> 2) - 1;
        const int q = warp & 3;
        const int r_in_tile = q * 32 + lane;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const uint32_t s_addr = tmem_base + lane_addr + t * 128;
        const uint32_t o_addr = tmem_base + lane_addr + 256 + t * 128;
        const float c = p.scale * 1.4426950408889634f;   // scores are kept in the log2 domain
        uint32_t n_s = 0, n_o = 0;                       // hand-offs / items done by this query tile so far
        for (int i = 0;; ++i) {
            int pair, bh, J[2];
            const int st = decode(i, pair, bh, J);
            if (st == 0) break;
            if (st == 1) continue;
            const int Jt = J[t];
            if (Jt == 0) continue;
            const int qidx = (2 * pair + t) * BQ + r_in_tile;
            float m_used = -INFINITY, l_run = 0.0f;

            for (int j = 0; j < Jt; ++j, ++n_s) {
                const bool edge = (j == Jt - 1);
                const int k0 = j * BKV;
                mbar_wait(&ctrl->s_full[t], n_s & 1, ctx, BAR_S_FULL);
                tc_fence_after();

                uint32_t s[BKV];
#pragma unroll
                for (int cc = 0; cc < BKV / 32; ++cc)
                    tmem_ld32(s_addr + cc * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[cc * 32]));
                tmem_ld_wait();

                // eight independent partial maxima keep the dependency chains short
                float pm[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) pm[i] = -INFINITY;
                // chunks of 32 keys that hold a valid key for at least one row of this warp (the same in every lane)
                uint32_t live = 0xFu;
                if (edge) {
                    // A row's valid keys of this tile are its first n_valid: the tile ends at Sk and, under the
                    // causal mask, at the row's own index.  Masking is decided per 32-key chunk with bounds that
                    // hold for the whole warp (its rows are consecutive): chunks valid for every row take the plain
                    // path, chunks valid for none are skipped altogether (their probabilities are zero), and only
                    // the chunk the diagonal crosses pays for per-element compares.
                    const int kv_left = p.Sk - k0;
                    const int warp_row0 = (2 * pair + t) * BQ + q * 32;
                    const int n_valid = min(kv_left, p.causal ? qidx - k0 + 1 : BKV);
                    const int nv_min = min(kv_left, p.causal ? warp_row0 - k0 + 1 : BKV);
                    const int nv_max = min(kv_left, p.causal ? warp_row0 - k0 + 32 : BKV);
#pragma unroll
                    for (int cc = 0; cc < BKV / 32; ++cc) {
                        if (cc * 32 >= nv_max) {
                            live &= ~(1u << cc);
                        } else if ((cc + 1) * 32 > nv_min) {
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (cc * 32 + i >= n_valid) s[cc * 32 + i] = __float_as_uint(-INFINITY);
                        }
                    }
                }
                // (skipped chunks still hold scores: harmless in the maximum only if they are excluded)
#pragma unroll
                for (int cc = 0; cc < BKV / 32; ++cc) {
                    if (live & (1u << cc)) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) pm[i & 7] = fmaxf(pm[i & 7], __uint_as_float(s[cc * 32 + i]));
                    }
                }
                const float tmax = fmaxf(fmaxf(fmaxf(pm[0], pm[1]), fmaxf(pm[2], pm[3])),
                                         fmaxf(fmaxf(pm[4], pm[5]), fmaxf(pm[6], pm[7])));
                // the scale is positive, so max(s)*c == max(s*c)
                float m_new = tmax * c;
                if (m_new == -INFINITY) m_new = 0.0f;          // rows past S: nothing valid, never stored
                const bool grow = m_new > m_used + RESCALE_THRESHOLD;
                float alpha = 1.0f;
                if (grow) {
                    alpha = ex2(m_used - m_new);                // 0 on the first tile
                    m_used = m_new;
                }
                l_run *= alpha;
                // S_t(j) complete implies PV_t(j-1) complete: O_t is quiescent until we signal P_t(j)
                if (j > 0 && __any_sync(0xffffffffu, grow)) {
#pragma unroll 1
                    for (int cc = 0; cc < D / 32; ++cc) {
                        uint32_t o[32];
                        tmem_ld32(o_addr + cc * 32, o);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st32(o_addr + cc * 32, o);
                    }
                }

                const uint64_t c2 = pack_f32x2(c, c), neg_m2 = pack_f32x2(-m_used, -m_used);
                uint64_t ls2[4] = {0ull, 0ull, 0ull, 0ull};      // (0.0f, 0.0f) pairs
                // 32 keys at a time: their 16 packed probability columns overwrite score columns that are already
                // in registers; the MMA warp is told after the third chunk (keys 0..95) and after the last
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint32_t pk[16];
                    if (live & (1u << ch)) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            float x0, x1;
                            unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(s[ch * 32 + 2 * i]),
                                                              __uint_as_float(s[ch * 32 + 2 * i + 1])), c2, neg_m2),
                                         x0, x1);
                            const float e0 = ex2(x0), e1 = ex2(x1);
                            ls2[i & 3] = add_f32x2(ls2[i & 3], pack_f32x2(e0, e1));
                            pk[i] = pack_h16x2(e0, e1, F16);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) pk[i] = 0u;
                    }
                    tmem_st16(s_addr + ch * 16, pk);
                    if (ch >= 2) {
                        tmem_st_wait();
                        tc_fence_before();
                        mbar_arrive(ch == 2 ? &ctrl->p_full[t] : &ctrl->p_half2[t]);
                    }
                }
                {
                    float a0, a1;
                    unpack_f32x2(add_f32x2(add_f32x2(ls2[0], ls2[1]), add_f32x2(ls2[2], ls2[3])), a0, a1);
                    l_run += a0 + a1;
                }
            }

            // this tile's last PV is done: normalise and store, then hand O_t back to the MMA warp
            mbar_wait(&ctrl->o_final[t], n_o & 1, ctx, BAR_O_FINAL);
            ++n_o;
            tc_fence_after();
            const float inv_l = 1.0f / l_run;
            uint16_t *orow = static_cast<uint16_t *>(p.out) + (long long)(bh / p.H) * p.out_b +
                                  (long long)(bh % p.H) * p.out_h + (long long)qidx * p.out_s;
            const bool wide_ok = (reinterpret_cast<uintptr_t>(orow) & 31) == 0;   // rows are only known to be 16-byte aligned
#pragma unroll 1
            for (int cc = 0; cc < D / 32; ++cc) {
                uint32_t r[32];
                tmem_ld32(o_addr + cc * 32, r);
                tmem_ld_wait();
                if (qidx < p.S) {
                    uint32_t w[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        w[i] = pack_h16x2(__uint_as_float(r[2 * i]) * inv_l, __uint_as_float(r[2 * i + 1]) * inv_l, F16);
                    if (wide_ok) {
                        // thread = row, so a warp's store touches 32 different rows: 32-byte stores write whole
                        // sectors and halve the number of store instructions
#pragma unroll
                        for (int g = 0; g < 2; ++g)
                            st_global_32B(orow + cc * 32 + g * 16, &w[g * 8]);
                    } else {
#pragma unroll
                        for (int g = 0; g < 4; ++g)
                            *reinterpret_cast<uint4 *>(orow + cc * 32 + g * 8) =
                                make_uint4(w[g * 4], w[g * 4 + 1], w[g * 4 + 2], w[g * 4 + 3]);
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(&ctrl->o_free[t]);
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

template <int D, bool F16>
static cudaError_t launch_attention_d(const CUtensorMap &tmQ, const CUtensorMap &tmK, const CUtensorMap &tmV,
                                      const AttnArgs &a, int num_sms, cudaStream_t stream)
{
    const int num_q_tiles = (a.S + BQ - 1) / BQ;
    const int num_pairs = (num_q_tiles + 1) / 2;
    const long long num_items = (long long)((num_pairs + 1) / 2) * a.BH;   // slots: two items each
    const unsigned grid = (unsigned)(num_items < num_sms ? num_items : num_sms);   // persistent: one CTA per SM
    return launch_kernel(attention_bf16_kernel<D, F16>, dim3(grid), dim3(THREADS), SMEM_BYTES, stream, a.pdl != 0, tmQ, tmK,
                         tmV, a);
}

// shared-memory limit of one instantiation; regs_ok is cleared if it was compiled with fewer registers than
// the in-kernel setmaxnreg split draws on (threads x registers-at-launch)
template <int D, bool F16>
static cudaError_t setup_attention_d(bool *regs_ok)
{
    cudaFuncAttributes attr;
    cudaError_t e = cudaFuncGetAttributes(&attr, attention_bf16_kernel<D, F16>);
    if (e != cudaSuccess) return e;
    if (attr.numRegs * THREADS < 128 * REGS_WG0 + 256 * REGS_SOFTMAX) *regs_ok = false;
    return cudaFuncSetAttribute(attention_bf16_kernel<D, F16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)SMEM_BYTES);
}

}  // namespace

cudaError_t setup_attention_bf16(bool *regs_ok)
{
    *regs_ok = true;
    cudaError_t e;
    if ((e = setup_attention_d<64, false>(regs_ok)) != cudaSuccess) return e;
    if ((e = setup_attention_d<64, true>(regs_ok)) != cudaSuccess) return e;
    if ((e = setup_attention_d<128, false>(regs_ok)) != cudaSuccess) return e;
    return setup_attention_d<128, true>(regs_ok);
}

cudaError_t launch_attention_bf16(const CUtensorMap &tmQ, const CUtensorMap &tmK, const CUtensorMap &tmV,
                                  const AttnArgs &a, int num_sms, bool regs_ok, cudaStream_t stream)
{
    if (a.BH <= 0 || a.S <= 0 || a.Sk <= 0) return cudaSuccess;
    // refuse to launch (rather than wait forever inside the kernel) if the register split cannot be satisfied
    if (!regs_ok) return cudaErrorLaunchOutOfResources;
    if (a.D == 64)
        return a.f16 ? launch_attention_d<64, true>(tmQ, tmK, tmV, a, num_sms, stream)
                     : launch_attention_d<64, false>(tmQ, tmK, tmV, a, num_sms, stream);
    if (a.D == 128)
        return a.f16 ? launch_attention_d<128, true>(tmQ, tmK, tmV, a, num_sms, stream)
                     : launch_attention_d<128, false>(tmQ, tmK, tmV, a, num_sms, stream);
    return cudaErrorInvalidValue;
}

}  // namespace pike
