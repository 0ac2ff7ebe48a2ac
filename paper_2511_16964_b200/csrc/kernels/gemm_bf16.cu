// bf16 x bf16 -> fp32 GEMM on the 5th-generation tensor cores with the whole
// pointwise epilogue applied in registers before one store.
//
//   out[m,n] = scale * act( sum_k A[m,k] * W[k,n] + bias[n] ) + residual[m,n]
//
// Persistent clusters of two CTAs (cta_group::2), one cluster per SM pair, each cluster
// walking over 256 x 256 output tiles.  Per CTA (192 threads):
//   warp 0      TMA producer: this CTA's 128 rows of A and its 128 of the tile's 256 W
//               columns, 64 k at a time, into a 6-stage 128-byte-swizzled ring (32 KiB per
//               stage).  Both CTAs' loads complete on the LEADER's "full" barrier.
//   warp 1      allocates 512 tensor-memory columns (two 128x256 fp32 accumulator stages
//               per CTA); in the leader CTA one thread issues tcgen05.mma.cta_group::2
//               (256x256x16) for the pair and commits to mbarriers in both CTAs
//   warps 2..5  epilogue: tcgen05.ld this CTA's accumulator rows (thread = row, 32
//               columns at a time), bias/activation/scale/residual in registers, 16-byte
//               stores; optionally per-row partials - (max, sum exp) or (mean, sum of squared
//               deviations) - for a softmax / LayerNorm split across N tiles.  Runs under the
//               next tile's K loop.
// The pair halves the W traffic each SM's shared memory sees compared with a 128x256
// single-CTA tile, which was shared-memory-bandwidth bound.  No TMA multicast is used.
// Every mbarrier wait is bounded (see mbar_wait).
#include "../device/act.cuh"
#include "../device/ptx.cuh"
#include "kernels.h"

namespace pike {
namespace {

constexpr int BM = GEMM_BM;                     // rows per CTA (the pair covers 2*BM)
constexpr int BN = GEMM_BN, BK = GEMM_BK;
constexpr int BN_HALF = BN / 2;                 // W columns staged by each CTA
constexpr int STAGES = 6;
constexpr int A_BYTES = BM * BK * 2;            // 16 KiB
constexpr int B_BYTES = BN_HALF * BK * 2;       // 16 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;  // 32 KiB per CTA
constexpr int NUM_ACC = 2;
constexpr int TMEM_COLS = NUM_ACC * BN;         // 512
constexpr int THREADS = 192;
constexpr int EPI_THREADS = 128;
constexpr int EPI_WARPS = 4;

struct __align__(8) Ctrl {
    uint64_t full[STAGES];        // used in the leader: both CTAs' TMA bytes land here
    uint64_t empty[STAGES];       // in each CTA: stage consumed (multicast commit)
    uint64_t tmem_full[NUM_ACC];  // in each CTA: accumulator ready (multicast commit)
    uint64_t tmem_empty[NUM_ACC]; // used in the leader: 4 epilogue warps x 2 CTAs drained it
    uint32_t tmem_base;
    uint32_t abort;
    float bias[BN];
};
constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)STAGES * STAGE_BYTES + sizeof(Ctrl);

enum : uint32_t { BAR_EMPTY = 1, BAR_FULL = 2, BAR_TMEM_EMPTY = 3, BAR_TMEM_FULL = 4 };

// Rasterisation: tiles are walked in groups of `group` blocks of one dimension (the PANEL dimension), all blocks
// of the other dimension before the next group, panel block fastest.  The clusters that run together therefore
// share a few row blocks and a few column blocks (their k-slices meet in L2), and the group's panel - group x 256
// rows of A, or group x 256 columns of W - stays in L2 for the whole sweep while the other operand streams through
// once per group.  along_n == 0: the panel is a group of row blocks of A; 1: a group of column blocks of W.
__device__ __forceinline__ void tile_coords(int t, int num_m, int num_n, int group, int along_n, int &m_blk, int &n_blk)
{
    const int num_p = along_n ? num_n : num_m, num_s = along_n ? num_m : num_n;
    const int per_group = group * num_s;
    const int g = t / per_group;
    const int first_p = g * group;
    const int gsz = min(group, num_p - first_p);
    const int r = t - g * per_group;
    const int p_blk = first_p + r % gsz, s_blk = r / gsz;
    m_blk = along_n ? s_blk : p_blk;
    n_blk = along_n ? p_blk : s_blk;
}

// Work items.  The tiles are dealt round-robin to the persistent clusters, so the last, partial round leaves
// most clusters idle when only a few tiles remain.  If that remainder is at most half the cluster count, each
// of its tiles is split into two 256 x 128 halves (an MMA with N = 128 into the first half of the accumulator
// columns), which halves the length of the last round: 4096^2 outputs on 74 clusters are 256 tiles = 3 rounds
// + 34 tiles -> 3 rounds + 68 half tiles (3.5 instead of 4 rounds).  Not used when the epilogue emits one
// row-reduction pair per 256-column tile.
struct Work { int tile, col_off, ncols; };
struct WorkPlan { int full, items; };     // tiles in whole rounds; total work items
__device__ __forceinline__ WorkPlan work_plan(int num_tiles, int num_clusters, bool may_split)
{
    const int full = (num_tiles / num_clusters) * num_clusters;
    const int tail = num_tiles - full;
    const bool split = may_split && tail > 0 && 2 * tail <= num_clusters;
    return WorkPlan{split ? full : num_tiles, split ? full + 2 * tail : num_tiles};
}
__device__ __forceinline__ Work work_item(const WorkPlan &wp, int w)
{
    if (w < wp.full) return Work{w, 0, BN};
    const int sub = w - wp.full;
    return Work{wp.full + (sub >> 1), (sub & 1) * (BN / 2), BN / 2};
}

// Rows covered by the pair-row-tile with linear index m_lin.  Plain mode: 256 consecutive rows of A.
// Grouped mode: group e (rows off[e] .. off[e+1]) owns the row-tile indices starting at
//   T(e) = off[e] / 256 + e.
// T grows by at least ceil(len_e / 256) from one group to the next, so the groups' index ranges never
// overlap, the owner of an index is found by bisection over the offsets (O(log G) loads per tile, no
// scratch memory, no pass over all groups) and off[G] / 256 + G indices cover everything.  An index whose
// tile would start at or past its group's end is EMPTY: row0 == row_end, and every warp role skips the
// item.  A tile's rows stop at the end of its group; `group` selects the weight matrix and bias row.
// Offsets come from device memory the host cannot check, so each one is clamped to [0, M] (and an end
// to at least its start): whatever a router wrote there, no row outside the tensors is touched.
struct RowTile { int row0, row_end, group; };
__device__ __forceinline__ int clamp_offset(const int *offsets, int i, int lo, int hi)
{
    return min(max(__ldg(offsets + i), lo), hi);
}
__device__ __forceinline__ RowTile row_tile(const GemmArgs &p, int m_lin)
{
    if (p.group_offsets == nullptr) return RowTile{m_lin * 2 * BM, p.M, 0};
    int lo = 0, hi = p.num_groups - 1;      // the owner is the last group with T(e) <= m_lin
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (clamp_offset(p.group_offsets, mid, 0, p.M) / (2 * BM) + mid <= m_lin) lo = mid; else hi = mid - 1;
    }
    const int first = clamp_offset(p.group_offsets, lo, 0, p.M);
    const int end = clamp_offset(p.group_offsets, lo + 1, first, p.M);
    const long long local = (long long)m_lin - (first / (2 * BM) + lo);
    const long long row0 = first + local * (2 * BM);
    if (local < 0 || row0 >= end) return RowTile{p.M, p.M, 0};
    return RowTile{(int)row0, end, lo};
}
__device__ __forceinline__ int count_row_tiles(const GemmArgs &p)
{
    if (p.group_offsets == nullptr) return (p.M + 2 * BM - 1) / (2 * BM);
    return clamp_offset(p.group_offsets, p.num_groups, 0, p.M) / (2 * BM) + p.num_groups;
}

template <int ACT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmArgs p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(tiles + (size_t)STAGES * STAGE_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();           // 0 = leader
    const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
    const int num_m = count_row_tiles(p), num_n = (p.N + BN - 1) / BN;
    const int num_tiles = num_m * num_n;
    const int num_kb = (p.K + BK - 1) / BK;
    const WorkPlan plan = work_plan(num_tiles, num_clusters, p.row_partials == 0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&ctrl->full[s], 1); mbar_init(&ctrl->empty[s], 1); }
        for (int a = 0; a < NUM_ACC; ++a) { mbar_init(&ctrl->tmem_full[a], 1); mbar_init(&ctrl->tmem_empty[a], 2 * EPI_WARPS); }
        ctrl->abort = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) {
        tmem_alloc_pair(&ctrl->tmem_base, TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();          // the peer's barriers are initialised before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = ctrl->tmem_base;
    const WaitCtx ctx{p.status, &ctrl->abort, p.limit_ns, KID_GEMM};

    if (warp == 0) {
        // -------------------- TMA producer (warp-uniform loop, one elected lane issues)
        {
            const bool leader = elect_one();
            int s = 0;
            uint32_t ph = 0;
            for (int w = cluster_id; w < plan.items && !p.test_withhold_loads; w += num_clusters) {
                const Work wk = work_item(plan, w);
                int m_blk, n_blk;
                tile_coords(wk.tile, num_m, num_n, p.group_m, p.group_along_n, m_blk, n_blk);
                const RowTile rt = row_tile(p, m_blk);
                if (rt.row0 >= rt.row_end) continue;        // empty row tile (grouped mode): every role skips it
                const int row0 = rt.row0 + (int)rank * BM;
                // this CTA stages its half of the item's W columns; for a half tile the boxes keep their size
                // (the bytes a stage waits for stay the same) and only their first 64 columns are used
                const int col0 = n_blk * BN + wk.col_off + (int)rank * (wk.ncols / 2);
                for (int kb = 0; kb < num_kb; ++kb) {
                    mbar_wait(&ctrl->empty[s], ph ^ 1, ctx, BAR_EMPTY);
                    uint8_t *a_s = tiles + (size_t)s * STAGE_BYTES;
                    uint8_t *b_s = a_s + A_BYTES;
                    const uint32_t full_leader = mapa_shared(smem_u32(&ctrl->full[s]), 0);
                    if (leader) {
                        if (rank == 0) mbar_arrive_expect_tx(&ctrl->full[s], 2 * STAGE_BYTES);
                        tma_load_2d_pair(a_s, &tmA, full_leader, kb * BK, row0);
                        if (p.w_is_nk) {
                            tma_load_3d_pair(b_s, &tmB, full_leader, kb * BK, col0, rt.group);
                        } else {
#pragma unroll
                            for (int i = 0; i < BN_HALF / 64; ++i)
                                tma_load_3d_pair(b_s + i * (64 * BK * 2), &tmB, full_leader, col0 + i * 64, kb * BK, rt.group);
                        }
                    }
                    __syncwarp();
                    if (++s == STAGES) { s = 0; ph ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------- MMA issuer (leader CTA only; warp-uniform loop, one elected lane issues)
        if (rank == 0) {
            const bool leader = elect_one();
            const uint32_t idesc_full = make_idesc_bf16(2 * BM, BN, false, !p.w_is_nk, p.f16 != 0);
            const uint32_t idesc_half = make_idesc_bf16(2 * BM, BN / 2, false, !p.w_is_nk, p.f16 != 0);
            const uint32_t a_addr0 = smem_u32(tiles), b_addr0 = a_addr0 + A_BYTES;
            const uint64_t adesc0 = make_smem_desc_sw128(a_addr0, 0, 1024);
            const uint64_t bdesc0 = p.w_is_nk ? make_smem_desc_sw128(b_addr0, 0, 1024)
                                              : make_smem_desc_sw128(b_addr0, 64 * BK * 2, 1024);
            const uint32_t b_kstep = p.w_is_nk ? 32u : 2048u;     // bytes per 16-k step inside a stage
            int s = 0;
            uint32_t ph = 0;
            int it = 0;
            for (int w = cluster_id; w < plan.items; w += num_clusters) {
                const Work wk = work_item(plan, w);
                if (p.group_offsets != nullptr) {
                    int m_blk, n_blk;
                    tile_coords(wk.tile, num_m, num_n, p.group_m, p.group_along_n, m_blk, n_blk);
                    const RowTile rt = row_tile(p, m_blk);
                    if (rt.row0 >= rt.row_end) continue;
                }
                const uint32_t idesc = wk.ncols == BN ? idesc_full : idesc_half;
                const int acc = it & 1;
                const uint32_t aph = (it >> 1) & 1;
                mbar_wait_cluster(&ctrl->tmem_empty[acc], aph ^ 1, ctx, BAR_TMEM_EMPTY);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    mbar_wait_cluster(&ctrl->full[s], ph, ctx, BAR_FULL);
                    tc_fence_after();
                    // stage 0's descriptors were built once; a stage is a constant number of bytes further
                    const uint64_t adesc = desc_advance(adesc0, (uint32_t)s * STAGE_BYTES);
                    const uint64_t bdesc = desc_advance(bdesc0, (uint32_t)s * STAGE_BYTES);
                    if (leader) {
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)
                            umma_ss_pair(d_tmem, desc_advance(adesc, k * 32), desc_advance(bdesc, k * b_kstep), idesc,
                                         (kb | k) != 0 ? 1u : 0u);
                        umma_commit_pair(&ctrl->empty[s], 0x3);
                    }
                    __syncwarp();
                    if (++s == STAGES) { s = 0; ph ^= 1; }
                }
                if (leader) umma_commit_pair(&ctrl->tmem_full[acc], 0x3);
                __syncwarp();
                ++it;
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        const int et = threadIdx.x - 64;        // 0..127
        const bool f16 = p.f16 != 0;            // 16-bit tensors are IEEE half instead of bf16
        int it = 0;
        for (int w = cluster_id; w < plan.items; w += num_clusters) {
            const Work wk = work_item(plan, w);
            int m_blk, n_blk;
            tile_coords(wk.tile, num_m, num_n, p.group_m, p.group_along_n, m_blk, n_blk);
            const RowTile rt = row_tile(p, m_blk);
            if (rt.row0 >= rt.row_end) continue;
            const int acc = it & 1;
            const uint32_t aph = (it >> 1) & 1;
            const int n0 = n_blk * BN + wk.col_off;      // first output column of this item
            const int row = rt.row0 + (int)rank * BM + q * 32 + lane;
            const bool row_ok = row < rt.row_end;
            const long long bias0 = (long long)rt.group * p.N + n0;    // bias is [num_groups, N] in grouped mode

            // stage the tile's bias as fp32
            named_bar_sync(1, EPI_THREADS);
            for (int i = et; i < BN; i += EPI_THREADS) {
                float b = 0.0f;
                if (p.bias != nullptr && n0 + i < p.N)
                    b = p.bias_f32 ? static_cast<const float *>(p.bias)[bias0 + i]
                                   : h16_at(p.bias, bias0 + i, p.f16 != 0);
                ctrl->bias[i] = b;
            }
            named_bar_sync(1, EPI_THREADS);

            mbar_wait(&ctrl->tmem_full[acc], aph, ctx, BAR_TMEM_FULL);
            tc_fence_after();

            // softmax: running (max, sum exp); LayerNorm: running (mean, sum of squared deviations)
            float run_m = p.row_partials == 2 ? 0.0f : -INFINITY, run_l = 0.0f;
#pragma unroll 1
            for (int c = 0; c < wk.ncols / 32; ++c) {
                const int nc = n0 + c * 32;
                if (nc >= p.N) break;
                uint32_t r[32];
                tmem_ld32(tmem_base + acc * BN + c * 32 + (static_cast<uint32_t>(q * 32) << 16), r);

                // residual prefetch (thread = row, 32 consecutive columns)
                uint4 res16[4];
                float4 res32[8];
                const bool has_res = p.residual != nullptr && row_ok;
                if (has_res) {
                    if (p.residual_f32) {
                        const float *rp = static_cast<const float *>(p.residual) + (long long)row * p.ldr + nc;
#pragma unroll
                        for (int g = 0; g < 8; ++g)
                            res32[g] = (nc + g * 4 < p.N) ? *reinterpret_cast<const float4 *>(rp + g * 4)
                                                          : make_float4(0.f, 0.f, 0.f, 0.f);
                    } else {
                        const uint16_t *rp = static_cast<const uint16_t *>(p.residual) + (long long)row * p.ldr + nc;
                        if (nc + 32 <= p.N && (reinterpret_cast<uintptr_t>(rp) & 31) == 0) {
                            // whole, 32-byte aligned chunk: two 32-byte loads (thread = row: one sector per row each)
                            ld_global_32B(rp, reinterpret_cast<uint32_t *>(&res16[0]));
                            ld_global_32B(rp + 16, reinterpret_cast<uint32_t *>(&res16[2]));
                        } else {
#pragma unroll
                            for (int g = 0; g < 4; ++g)
                                res16[g] = (nc + g * 8 < p.N) ? *reinterpret_cast<const uint4 *>(rp + g * 8)
                                                              : make_uint4(0u, 0u, 0u, 0u);
                        }
                    }
                }
                tmem_ld_wait();

                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    v[j] = p.scale * act_fast<ACT>(__uint_as_float(r[j]) + ctrl->bias[c * 32 + j]);
                if (has_res) {
                    if (p.residual_f32) {
#pragma unroll
                        for (int g = 0; g < 8; ++g) {
                            v[g * 4 + 0] += res32[g].x; v[g * 4 + 1] += res32[g].y;
                            v[g * 4 + 2] += res32[g].z; v[g * 4 + 3] += res32[g].w;
                        }
                    } else {
#pragma unroll
                        for (int g = 0; g < 4; ++g) {
                            const uint32_t w4[4] = {res16[g].x, res16[g].y, res16[g].z, res16[g].w};
#pragma unroll
                            for (int h = 0; h < 4; ++h) {
                                v[g * 8 + 2 * h] += h16_lo(w4[h], f16);
                                v[g * 8 + 2 * h + 1] += h16_hi(w4[h], f16);
                            }
                        }
                    }
                }

                if (p.row_partials == 2) {
                    // LayerNorm partials: this chunk's (count, mean, sum of squared deviations), merged into
                    // the running triple of the tile row with the pairwise update (no E[x^2]-E[x]^2 cancellation)
                    const int cnt = min(32, p.N - nc);
                    float cs = 0.0f;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j < cnt) cs += v[j];
                    const float cmean = cs / (float)cnt;
                    float cm2 = 0.0f;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (j < cnt) cm2 += (v[j] - cmean) * (v[j] - cmean);
                    const float n_old = (float)(nc - n0), n_new = n_old + (float)cnt;
                    const float delta = cmean - run_m;
                    run_m += delta * ((float)cnt / n_new);             // run_m: running mean
                    run_l += cm2 + delta * delta * (n_old * (float)cnt / n_new);   // run_l: running M2
                } else if (p.row_partials) {
                    float cm = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (nc + j < p.N) cm = fmaxf(cm, v[j]);
                    const float nm = fmaxf(run_m, cm);
                    float s = 0.0f;
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (nc + j < p.N) s += __expf(v[j] - nm);
                    run_l = run_l * __expf(run_m - nm) + s;
                    run_m = nm;
                }

                // Thread = row, so one store instruction of a warp touches 32 different rows: where the chunk
                // lies fully inside N and starts on a 32-byte boundary it is written with 32-byte stores (whole
                // sectors, half as many instructions), else with 16-byte ones.
                if (row_ok) {
                    const bool whole = nc + 32 <= p.N;
                    if (p.out_f32) {
                        float *op = static_cast<float *>(p.out) + (long long)row * p.ldo + nc;
                        if (whole && (reinterpret_cast<uintptr_t>(op) & 31) == 0) {
#pragma unroll
                            for (int g = 0; g < 4; ++g)
                                st_global_32B(op + g * 8, reinterpret_cast<const uint32_t *>(&v[g * 8]));
                        } else {
#pragma unroll
                            for (int g = 0; g < 8; ++g)
                                if (nc + g * 4 < p.N)
                                    *reinterpret_cast<float4 *>(op + g * 4) =
                                        make_float4(v[g * 4], v[g * 4 + 1], v[g * 4 + 2], v[g * 4 + 3]);
                        }
                    } else {
                        uint16_t *op = static_cast<uint16_t *>(p.out) + (long long)row * p.ldo + nc;
                        uint32_t w[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) w[i] = pack_h16x2(v[2 * i], v[2 * i + 1], f16);
                        if (whole && (reinterpret_cast<uintptr_t>(op) & 31) == 0) {
                            st_global_32B(op, &w[0]);
                            st_global_32B(op + 16, &w[8]);
                        } else {
#pragma unroll
                            for (int g = 0; g < 4; ++g)
                                if (nc + g * 8 < p.N)
                                    *reinterpret_cast<uint4 *>(op + g * 8) =
                                        make_uint4(w[g * 4], w[g * 4 + 1], w[g * 4 + 2], w[g * 4 + 3]);
                        }
                    }
                }
            }
            // accumulator drained: one arrival per epilogue warp on the LEADER's barrier
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&ctrl->tmem_empty[acc]), 0));

            if (p.row_partials && row_ok) p.partials[(long long)row * num_n + n_blk] = make_float2(run_m, run_l);
            ++it;
        }
    }

    // ------------------------------------------------------------------ teardown
    tc_fence_before();
    __syncthreads();
    if (ctrl->abort) abort_drain();
    cluster_sync_all();          // neither CTA frees tensor memory while the pair may still use it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

}  // namespace

template <typename Kern>
static cudaError_t setup_one(Kern kern, int num_sms, int *max_clusters)
{
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
    if (e != cudaSuccess) return e;
    // how many CTA pairs the device can hold at once (one CTA per SM at this shared-memory size)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (num_sms / 2));
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        n = num_sms / 2;
    }
    if (n < *max_clusters) *max_clusters = n;
    return cudaSuccess;
}

cudaError_t setup_gemm_bf16(int num_sms, int *max_clusters)
{
    *max_clusters = num_sms / 2;
    cudaError_t e;
    if ((e = setup_one(gemm_bf16_kernel<ACT_NONE>, num_sms, max_clusters)) != cudaSuccess) return e;
    if ((e = setup_one(gemm_bf16_kernel<ACT_GELU_ERF>, num_sms, max_clusters)) != cudaSuccess) return e;
    if ((e = setup_one(gemm_bf16_kernel<ACT_GELU_TANH>, num_sms, max_clusters)) != cudaSuccess) return e;
    return setup_one(gemm_bf16_kernel<ACT_SILU>, num_sms, max_clusters);
}

cudaError_t launch_gemm_bf16(const CUtensorMap &tmA, const CUtensorMap &tmB, const GemmArgs &a, int max_clusters,
                             cudaStream_t stream)
{
    // grouped mode: the device derives the row tiles from the offsets itself; this is the host's upper bound
    const int num_m = a.group_offsets != nullptr ? a.M / (2 * BM) + a.num_groups : (a.M + 2 * BM - 1) / (2 * BM);
    const int num_n = (a.N + BN - 1) / BN;
    const long long num_tiles = (long long)num_m * num_n;
    if (num_tiles <= 0 || a.M <= 0 || max_clusters <= 0) return cudaSuccess;
    // Rasterisation.  Both operands come in slabs of 256 x K 16-bit values (a pair-row-block of A, a column block
    // of W).  One of them is the PANEL: a group of its slabs is walked against all slabs of the other operand, so
    // the panel is fetched once and the other operand once per group:
    //   traffic(panel = A) = bytes(A) + bytes(W) * groups_of_A,   traffic(panel = W) = bytes(W) + bytes(A) * groups_of_W
    // and the cheaper one is taken (the MLP's second GEMM, K = 16384, reads 11 % less with W as the panel).  A group
    // holds as many slabs as fit in PANEL_BYTES, at least 8 (with fewer the clusters that run together - 74 = about
    // 8 x 9 tiles - span too many slabs of the streaming operand).  Measured on B200 (DRAM bytes of the two MLP
    // GEMMs): a panel is only kept below about 32 MB - a quarter of the 126 MB L2, which is split over two dies and
    // shared with the streaming operand and the output: 1169 -> 402 MB for 8192x4096x16384.  L2 eviction priorities
    // on the loads (evict_last for the panel, evict_first or normal for the stream) were measured too and made the
    // reads worse by 40 to 110 %: a streamed slab is shared by the eight or nine clusters that run side by side, and
    // lowering its priority evicts it between their reads.
    GemmArgs args = a;
    {
        constexpr long long PANEL_BYTES = 33ll << 20;
        const long long slab = 2ll * BM * a.K * 2;
        long long g = PANEL_BYTES / (slab > 0 ? slab : 1);
        if (g < 8) g = 8;
        const long long gm = g < num_m ? g : num_m, gn = g < num_n ? g : num_n;
        const long long groups_m = (num_m + gm - 1) / gm, groups_n = (num_n + gn - 1) / gn;
        const double bytes_a = 2.0 * a.M * a.K, bytes_w = 2.0 * a.K * a.N;
        const bool along_n = a.group_offsets == nullptr && bytes_w + bytes_a * groups_n < bytes_a + bytes_w * groups_m;
        args.group_along_n = along_n ? 1 : 0;
        args.group_m = (int)(along_n ? gn : gm);
    }
    // up to two work items per tile (see work_plan): small problems get both halves of a tile onto
    // different clusters
    const long long most = a.row_partials == 0 ? 2 * num_tiles : num_tiles;
    const int clusters = most < max_clusters ? (int)most : max_clusters;
    const dim3 grid(2 * clusters), block(THREADS);
    switch (a.act) {
    case ACT_GELU_ERF:  gemm_bf16_kernel<ACT_GELU_ERF><<<grid, block, SMEM_BYTES, stream>>>(tmA, tmB, args); break;
    case ACT_GELU_TANH: gemm_bf16_kernel<ACT_GELU_TANH><<<grid, block, SMEM_BYTES, stream>>>(tmA, tmB, args); break;
    case ACT_SILU:      gemm_bf16_kernel<ACT_SILU><<<grid, block, SMEM_BYTES, stream>>>(tmA, tmB, args); break;
    default:            gemm_bf16_kernel<ACT_NONE><<<grid, block, SMEM_BYTES, stream>>>(tmA, tmB, args); break;
    }
    return cudaGetLastError();
}

}  // namespace pike
