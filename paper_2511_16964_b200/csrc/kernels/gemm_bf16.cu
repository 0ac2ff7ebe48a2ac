// bf16 x bf16 -> fp32 GEMM on the 5th-generation tensor cores with the whole
// pointwise epilogue applied in registers before one store.
//
//   out[m,n] = scale * act( sum_k A[m,k] * W[k,n] + bias[n] ) + residual[m,n]
//
// Persistent clusters of two CTAs (cta_group::2), one cluster per SM pair, each cluster
// walking over 256 x 256 output tiles; warp roles and the shared building blocks are in
// gemm_tile.cuh.  The epilogue warps apply bias/activation/scale/residual in registers and
// store; optionally they emit per-row partials - (max, sum exp) or (mean, sum of squared
// deviations) - for a softmax / LayerNorm split across N tiles.  The epilogue of one tile runs
// under the next tile's K loop (two accumulator stages).
// The pair halves the W traffic each SM's shared memory sees compared with a 128x256
// single-CTA tile, which was shared-memory-bandwidth bound.
#include "gemm_tile.cuh"

namespace pike {
using namespace gemm;
namespace {

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
// Grouped mode: row tiles are counted group by group - group e (rows off[e] .. off[e+1]) has
// ceil(len_e / 256) of them - a tile's rows stop at the end of its group, and `group` selects the weight matrix
// and bias row.  The exclusive prefix sums first[e] of the tile counts are built once per CTA in shared memory
// (build_group_table) and the owner of an index is found by bisection over them: O(log G) shared-memory reads per
// tile, and no index is wasted, so the tiles of one group and column block stay neighbours in the round-robin deal
// (they share a slab of W through L2).  With more groups than the table holds the owner is found by bisection
// over the offsets themselves, with group e owning the indices from off[e]/256 + e - ranges that never overlap
// but leave some indices EMPTY (row0 == row_end): every warp role skips such an item.
// Offsets come from device memory the host cannot check, so each one is clamped to [0, M] (and an end
// to at least its start): whatever a router wrote there, no row outside the tensors is touched.
constexpr int MAX_TABLE_GROUPS = 4096;
constexpr size_t SMEM_BYTES_GEMM = SMEM_BYTES + (MAX_TABLE_GROUPS + 1) * sizeof(int);

struct RowTile { int row0, row_end, group; };
__device__ __forceinline__ int clamp_offset(const int *offsets, int i, int lo, int hi)
{
    return min(max(__ldg(offsets + i), lo), hi);
}
__device__ __forceinline__ int group_tiles(const GemmArgs &p, int e)
{
    const int first = clamp_offset(p.group_offsets, e, 0, p.M);
    return (clamp_offset(p.group_offsets, e + 1, first, p.M) - first + 2 * BM - 1) / (2 * BM);
}
// first[0 .. G]: exclusive prefix sums of the groups' tile counts (all threads of the CTA call this; warp 0 scans)
__device__ __forceinline__ void build_group_table(const GemmArgs &p, int *first)
{
    if (p.group_offsets == nullptr || p.num_groups > MAX_TABLE_GROUPS) return;
    if (threadIdx.x < 32) {
        int carry = 0;
        for (int e0 = 0; e0 < p.num_groups; e0 += 32) {
            const int e = e0 + (int)threadIdx.x;
            const int n = e < p.num_groups ? group_tiles(p, e) : 0;
            int incl = n;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, incl, o);
                if ((int)threadIdx.x >= o) incl += up;
            }
            if (e < p.num_groups) first[e] = carry + incl - n;
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (threadIdx.x == 0) first[p.num_groups] = carry;
    }
    __syncthreads();
}
__device__ __forceinline__ RowTile row_tile(const GemmArgs &p, const int *first_tile, int m_lin)
{
    if (p.group_offsets == nullptr) return RowTile{m_lin * 2 * BM, p.M, 0};
    const bool table = p.num_groups <= MAX_TABLE_GROUPS;
    int lo = 0, hi = p.num_groups - 1;      // the owner is the last group whose first index is <= m_lin
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        const int t_mid = table ? first_tile[mid] : clamp_offset(p.group_offsets, mid, 0, p.M) / (2 * BM) + mid;
        if (t_mid <= m_lin) lo = mid; else hi = mid - 1;
    }
    const int first = clamp_offset(p.group_offsets, lo, 0, p.M);
    const int end = clamp_offset(p.group_offsets, lo + 1, first, p.M);
    const long long local = (long long)m_lin - (table ? first_tile[lo] : first / (2 * BM) + lo);
    const long long row0 = first + local * (2 * BM);
    if (local < 0 || row0 >= end) return RowTile{p.M, p.M, 0};
    return RowTile{(int)row0, end, lo};
}
__device__ __forceinline__ int count_row_tiles(const GemmArgs &p, const int *first_tile)
{
    if (p.group_offsets == nullptr) return (p.M + 2 * BM - 1) / (2 * BM);
    if (p.num_groups <= MAX_TABLE_GROUPS) return first_tile[p.num_groups];
    return clamp_offset(p.group_offsets, p.num_groups, 0, p.M) / (2 * BM) + p.num_groups;
}

template <int ACT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmArgs p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(tiles + (size_t)STAGES * STAGE_BYTES);

    int *first_tile = reinterpret_cast<int *>(ctrl + 1);      // grouped mode: prefix sums of the groups' row tiles

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();           // 0 = leader
    const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
    // barriers, tensor memory and the wait for the previous kernel of the stream first: the group offsets below are
    // device data that kernel may have written
    const uint32_t tmem_base = pair_setup(ctrl, &tmA, &tmB, warp);
    const WaitCtx ctx{p.status, &ctrl->abort, p.limit_ns, KID_GEMM};
    build_group_table(p, first_tile);
    const int num_m = count_row_tiles(p, first_tile), num_n = (p.N + BN - 1) / BN;
    const int num_tiles = num_m * num_n;
    const int num_kb = (p.K + BK - 1) / BK;
    const WorkPlan plan = work_plan(num_tiles, num_clusters, p.row_partials == 0);

    if (warp == 0) {
        // -------------------- TMA producer (warp-uniform loop, one elected lane issues)
        const bool leader = elect_one();
        RingPos rp{0, 0};
        for (int w = cluster_id; w < plan.items && !p.test_withhold_loads; w += num_clusters) {
            const Work wk = work_item(plan, w);
            int m_blk, n_blk;
            tile_coords(wk.tile, num_m, num_n, p.group_m, p.group_along_n, m_blk, n_blk);
            const RowTile rt = row_tile(p, first_tile, m_blk);
            if (rt.row0 >= rt.row_end) continue;        // empty row tile (grouped mode): every role skips it
            // this CTA stages its half of the item's W columns; for a half tile the boxes keep their size
            // (the bytes a stage waits for stay the same) and only their first 64 columns are used
            produce_tile(tiles, ctrl, &tmA, &tmB, rp, num_kb, rt.row0 + (int)rank * BM,
                         n_blk * BN + wk.col_off + (int)rank * (wk.ncols / 2), rt.group, p.w_is_nk != 0, rank, leader, ctx,
                         p.alternate_k != 0 && (((w - cluster_id) / num_clusters) & 1) != 0);
        }
    } else if (warp == 1) {
        // ---------- MMA issuer (leader CTA only; warp-uniform loop, one elected lane issues)
        if (rank == 0) {
            const bool leader = elect_one();
            const uint32_t idesc_full = make_idesc_bf16(2 * BM, BN, false, !p.w_is_nk, p.f16 != 0);
            const uint32_t idesc_half = make_idesc_bf16(2 * BM, BN / 2, false, !p.w_is_nk, p.f16 != 0);
            const MmaDescs md = make_mma_descs(tiles, p.w_is_nk != 0);
            RingPos rp{0, 0};
            int it = 0;
            for (int w = cluster_id; w < plan.items; w += num_clusters) {
                const Work wk = work_item(plan, w);
                if (p.group_offsets != nullptr) {
                    int m_blk, n_blk;
                    tile_coords(wk.tile, num_m, num_n, p.group_m, p.group_along_n, m_blk, n_blk);
                    const RowTile rt = row_tile(p, first_tile, m_blk);
                    if (rt.row0 >= rt.row_end) continue;
                }
                const int acc = it & 1;
                const uint32_t aph = (it >> 1) & 1;
                mbar_wait_cluster(&ctrl->tmem_empty[acc], aph ^ 1, ctx, BAR_TMEM_EMPTY);
                tc_fence_after();
                mma_tile(ctrl, md, rp, num_kb, tmem_base + acc * BN, wk.ncols == BN ? idesc_full : idesc_half,
                         &ctrl->tmem_full[acc], leader, ctx);
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
            const RowTile rt = row_tile(p, first_tile, m_blk);
            if (rt.row0 >= rt.row_end) continue;
            const int acc = it & 1;
            const uint32_t aph = (it >> 1) & 1;
            const int n0 = n_blk * BN + wk.col_off;      // first output column of this item
            const int row = rt.row0 + (int)rank * BM + q * 32 + lane;
            const bool row_ok = row < rt.row_end;

            stage_bias(p, ctrl, n0, rt.group, et);
            mbar_wait(&ctrl->tmem_full[acc], aph, ctx, BAR_TMEM_FULL);
            tc_fence_after();

            // softmax: running (max, sum exp); LayerNorm: running (mean, sum of squared deviations)
            float run_m = p.row_partials == 2 ? 0.0f : -INFINITY, run_l = 0.0f;
#pragma unroll 1
            for (int c = 0; c < wk.ncols / 32; ++c) {
                const int nc = n0 + c * 32;
                if (nc >= p.N) break;
                float v[32];
                chunk_values<ACT>(p, ctrl, tmem_base + acc * BN + c * 32 + (static_cast<uint32_t>(q * 32) << 16), row,
                                  row_ok, nc, c, f16, v);

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
                    softmax_fold(v, nc, p.N, run_m, run_l);
                }
                if (row_ok) store_chunk(p, row, nc, f16, v);
            }
            // accumulator drained: one arrival per epilogue warp on the LEADER's barrier
            release_accumulator(ctrl, acc, lane);

            if (p.row_partials && row_ok) p.partials[(long long)row * num_n + n_blk] = make_float2(run_m, run_l);
            ++it;
        }
    }

    pair_teardown(ctrl, tmem_base, warp);
}

}  // namespace

template <typename Kern>
static cudaError_t setup_one(Kern kern, int num_sms, int *max_clusters)
{
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES_GEMM);
    if (e != cudaSuccess) return e;
    // how many CTA pairs the device can hold at once (one CTA per SM at this shared-memory size)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (num_sms / 2));
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES_GEMM;
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
    // (every group can add one partly filled tile)
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
        // The clusters that run side by side (74 = about 8 x 9 tiles) read about 17 slabs per round.  Where those
        // no longer fit in half the L2, a round's slabs are gone from it when the next round - which shares the
        // panel's slabs - begins, except their ends: each cluster then walks k in alternating directions (measured
        // on 8192x16384x4096: 1665 -> 1505 MB read; with 2 MB slabs, which stay resident anyway, the alternation only
        // costs sharing between clusters that are a round apart: +4 %, so it stays off there).
        args.alternate_k = 17 * slab > (64ll << 20) ? 1 : 0;
    }
    // up to two work items per tile (see work_plan): small problems get both halves of a tile onto
    // different clusters
    const long long most = a.row_partials == 0 ? 2 * num_tiles : num_tiles;
    const int clusters = most < max_clusters ? (int)most : max_clusters;
    const dim3 grid(2 * clusters), block(THREADS);
    switch (a.act) {
    case ACT_GELU_ERF:  return launch_kernel(gemm_bf16_kernel<ACT_GELU_ERF>, grid, block, SMEM_BYTES_GEMM, stream, a.pdl != 0, tmA, tmB, args);
    case ACT_GELU_TANH: return launch_kernel(gemm_bf16_kernel<ACT_GELU_TANH>, grid, block, SMEM_BYTES_GEMM, stream, a.pdl != 0, tmA, tmB, args);
    case ACT_SILU:      return launch_kernel(gemm_bf16_kernel<ACT_SILU>, grid, block, SMEM_BYTES_GEMM, stream, a.pdl != 0, tmA, tmB, args);
    default:            return launch_kernel(gemm_bf16_kernel<ACT_NONE>, grid, block, SMEM_BYTES_GEMM, stream, a.pdl != 0, tmA, tmB, args);
    }
}

}  // namespace pike
