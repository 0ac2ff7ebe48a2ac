// Logits + row softmax in ONE pass over the output:  out[m,:] = softmax_n( scale * act( A W + bias ) + residual ).
//
// The split-row softmax of the general GEMM kernel writes the un-normalised values, and a second kernel reads them
// back once the row maximum and sum are known.  Here a 256-row STRIPE of logits stays in tensor memory until its
// statistics are complete: the 74 CTA pairs hold two 256 x 256 fp32 accumulators each, 148 tiles, so a stripe of up to
// 148 column tiles (N <= 37888) fits on the chip at once.  Per stripe every cluster computes its one or two tiles, the
// epilogue warps read the accumulators a first time and publish one (max, sum exp) pair per row and tile to global
// memory (tile-major, [tile][row]), every CTA counts itself in on the stripe's counter, waits (bounded) until all CTAs of the stripe have, folds
// the row's pairs into (m, l), reads the accumulators a second time and writes exp(v - m) / l - each probability
// exactly once, no un-normalised value ever reaches HBM.
//
// CTAs wait on one another inside this kernel, so it is launched cooperatively (all CTAs resident); the wait has the
// same time limit and status word as every other wait of the library.  Same building blocks as the general kernel
// (gemm_tile.cuh).
#include "gemm_tile.cuh"

namespace pike {
using namespace gemm;
namespace {

template <int ACT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
gemm_softmax_onepass_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                            const GemmArgs p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Ctrl *ctrl = reinterpret_cast<Ctrl *>(tiles + (size_t)STAGES * STAGE_BYTES);
    __shared__ uint32_t stripe_ok;                 // epilogue thread 0 -> the other epilogue threads

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();           // 0 = leader
    const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
    const int num_stripes = (p.M + 2 * BM - 1) / (2 * BM), num_n = (p.N + BN - 1) / BN;
    const int num_kb = (p.K + BK - 1) / BK;
    // this cluster's column tiles of every stripe: cluster_id and cluster_id + num_clusters (accumulator stages 0, 1)
    const int my_tiles = (cluster_id < num_n ? 1 : 0) + (cluster_id + num_clusters < num_n ? 1 : 0);

    const uint32_t tmem_base = pair_setup(ctrl, &tmA, &tmB, warp);
    const WaitCtx ctx{p.status, &ctrl->abort, p.limit_ns, KID_GEMM};

    if (warp == 0) {
        // -------------------- TMA producer
        const bool leader = elect_one();
        RingPos rp{0, 0};
        for (int s = 0; s < num_stripes && !p.test_withhold_loads; ++s)
            for (int i = 0; i < my_tiles; ++i)
                produce_tile(tiles, ctrl, &tmA, &tmB, rp, num_kb, s * 2 * BM + (int)rank * BM,
                             (cluster_id + i * num_clusters) * BN + (int)rank * BN_HALF, 0, p.w_is_nk != 0, rank, leader, ctx);
    } else if (warp == 1) {
        // ---------- MMA issuer (leader CTA only): tile i of a stripe goes into accumulator stage i, which the
        // epilogue hands back only after the stripe has been normalised and stored
        if (rank == 0) {
            const bool leader = elect_one();
            const uint32_t idesc = make_idesc_bf16(2 * BM, BN, false, !p.w_is_nk, p.f16 != 0);
            const MmaDescs md = make_mma_descs(tiles, p.w_is_nk != 0);
            RingPos rp{0, 0};
            for (int s = 0; s < num_stripes; ++s)
                for (int i = 0; i < my_tiles; ++i) {
                    mbar_wait_cluster(&ctrl->tmem_empty[i], (uint32_t)(s & 1) ^ 1, ctx, BAR_TMEM_EMPTY);
                    tc_fence_after();
                    mma_tile(ctrl, md, rp, num_kb, tmem_base + i * BN, idesc, &ctrl->tmem_full[i], leader, ctx);
                }
        }
    } else if (my_tiles > 0) {
        // ---------------------------------------------------------------- epilogue
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        const int et = threadIdx.x - 64;        // 0..127
        const bool f16 = p.f16 != 0;
        const uint32_t lane_addr = static_cast<uint32_t>(q * 32) << 16;
        const unsigned participants = 2u * (unsigned)min(num_clusters, num_n);    // CTAs that own tiles of a stripe
        for (int s = 0; s < num_stripes; ++s) {
            const int row = s * 2 * BM + (int)rank * BM + q * 32 + lane;
            const bool row_ok = row < p.M;
            // ---- first reading of the accumulators: one (max, sum exp) pair per row and tile
            for (int i = 0; i < my_tiles; ++i) {
                const int n_blk = cluster_id + i * num_clusters, n0 = n_blk * BN;
                stage_bias(p, ctrl, n0, 0, et);
                mbar_wait(&ctrl->tmem_full[i], (uint32_t)(s & 1), ctx, BAR_TMEM_FULL);
                tc_fence_after();
                float run_m = -INFINITY, run_l = 0.0f;
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    const int nc = n0 + c * 32;
                    if (nc >= p.N) break;
                    float v[32];
                    chunk_values<ACT>(p, ctrl, tmem_base + i * BN + c * 32 + lane_addr, row, row_ok, nc, c, f16, v);
                    softmax_fold(v, nc, p.N, run_m, run_l);
                }
                if (row_ok) p.partials[(long long)n_blk * p.M + row] = make_float2(run_m, run_l);   // tile-major
            }
            // ---- count this CTA in, wait for the stripe's other CTAs
            __threadfence();                               // the pairs are visible device-wide before the count is
            named_bar_sync(2, EPI_THREADS);
            if (et == 0) {
                if (!(p.test_withhold_partials && blockIdx.x == 0)) atomicAdd(p.stripe_counters + s, 1u);
                stripe_ok = counter_wait(p.stripe_counters + s, participants, ctx, BAR_STRIPE) ? 1u : 0u;
            }
            named_bar_sync(2, EPI_THREADS);
            // ---- the row's statistics from all tiles' pairs (written by other SMs: read through L2).  The pairs are
            // laid out tile-major ([tile][row]), so the lanes of a warp - consecutive rows - read consecutive
            // addresses, and every thread folds its own row; sixteen loads are issued before the first is used.
            float m = 0.0f, inv_l = 1.0f;
            if (row_ok && stripe_ok) {
                const float2 *pr = p.partials + row;
                float mm = -INFINITY, l = 0.0f;
                for (int t0 = 0; t0 < num_n; t0 += 16) {
                    float2 pt[16];
#pragma unroll
                    for (int u = 0; u < 16; ++u)
                        pt[u] = t0 + u < num_n ? __ldcg(pr + (long long)(t0 + u) * p.M) : make_float2(-INFINITY, 0.0f);
#pragma unroll
                    for (int u = 0; u < 16; ++u) {
                        const float nm = fmaxf(mm, pt[u].x);
                        if (nm != -INFINITY) l = l * __expf(mm - nm) + pt[u].y * __expf(pt[u].x - nm);
                        mm = nm;
                    }
                }
                m = mm;
                inv_l = 1.0f / l;
            }
            // ---- second reading: probabilities, written once; then the accumulator goes back to the MMA warp
            for (int i = 0; i < my_tiles; ++i) {
                const int n_blk = cluster_id + i * num_clusters, n0 = n_blk * BN;
                if (my_tiles > 1) stage_bias(p, ctrl, n0, 0, et);      // the staged bias is the other tile's
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    const int nc = n0 + c * 32;
                    if (nc >= p.N) break;
                    float v[32];
                    chunk_values<ACT>(p, ctrl, tmem_base + i * BN + c * 32 + lane_addr, row, row_ok, nc, c, f16, v);
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __expf(v[j] - m) * inv_l;
                    if (row_ok) store_chunk(p, row, nc, f16, v);
                }
                release_accumulator(ctrl, i, lane);
            }
        }
    }

    pair_teardown(ctrl, tmem_base, warp);
}

}  // namespace

cudaError_t setup_gemm_softmax_onepass()
{
    cudaError_t e;
    e = cudaFuncSetAttribute(gemm_softmax_onepass_kernel<ACT_NONE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_softmax_onepass_kernel<ACT_GELU_ERF>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_softmax_onepass_kernel<ACT_GELU_TANH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(gemm_softmax_onepass_kernel<ACT_SILU>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
}

bool gemm_softmax_onepass_fits(int N, int max_clusters)
{
    return max_clusters > 0 && (long long)(N + BN - 1) / BN <= 2ll * max_clusters;
}

cudaError_t launch_gemm_softmax_onepass(const CUtensorMap &tmA, const CUtensorMap &tmB, const GemmArgs &a, int max_clusters,
                                        cudaStream_t stream)
{
    if (a.M <= 0) return cudaSuccess;
    if (!gemm_softmax_onepass_fits(a.N, max_clusters)) return cudaErrorInvalidValue;
    // every CTA of a stripe waits for the others: all clusters must be resident, which a cooperative launch guarantees
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (unsigned)max_clusters);
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    switch (a.act) {
    case ACT_GELU_ERF:  return cudaLaunchKernelEx(&cfg, gemm_softmax_onepass_kernel<ACT_GELU_ERF>, tmA, tmB, a);
    case ACT_GELU_TANH: return cudaLaunchKernelEx(&cfg, gemm_softmax_onepass_kernel<ACT_GELU_TANH>, tmA, tmB, a);
    case ACT_SILU:      return cudaLaunchKernelEx(&cfg, gemm_softmax_onepass_kernel<ACT_SILU>, tmA, tmB, a);
    default:            return cudaLaunchKernelEx(&cfg, gemm_softmax_onepass_kernel<ACT_NONE>, tmA, tmB, a);
    }
}

}  // namespace pike
