// Building blocks shared by the tcgen05 GEMM kernels (the general chain kernel and the one-pass logits + softmax
// kernel): tile constants, the control block in shared memory, set-up and tear-down of a CTA pair, the producer's
// and the MMA issuer's K loops for one tile, and the epilogue's per-chunk value computation and stores.
//
// A cluster of two CTAs (cta_group::2) computes a 256 x 256 output tile.  Per CTA (192 threads):
//   warp 0      TMA producer: this CTA's 128 rows of A and its 128 of the tile's 256 W columns, 64 k at a time, into
//               a 6-stage 128-byte-swizzled ring (32 KiB per stage); both CTAs' loads complete on the LEADER's barrier
//   warp 1      allocates 512 tensor-memory columns (two 128x256 fp32 accumulator stages per CTA); in the leader CTA
//               one thread issues tcgen05.mma.cta_group::2 (256x256x16) for the pair and commits to both CTAs
//   warps 2..5  epilogue: tcgen05.ld this CTA's accumulator rows (thread = row, 32 columns at a time)
// No TMA multicast is used.  Every mbarrier wait is bounded (see mbar_wait).
#pragma once
#include "../device/act.cuh"
#include "../device/ptx.cuh"
#include "kernels.h"

namespace pike {
namespace gemm {

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

enum : uint32_t { BAR_EMPTY = 1, BAR_FULL = 2, BAR_TMEM_EMPTY = 3, BAR_TMEM_FULL = 4, BAR_STRIPE = 5 };

// position in the operand ring, carried from tile to tile by the producer and by the MMA issuer
struct RingPos { int s; uint32_t ph; };

// Barriers, tensor memory and the rendezvous of the pair; returns the accumulators' base address.
__device__ __forceinline__ uint32_t pair_setup(Ctrl *ctrl, const CUtensorMap *tmA, const CUtensorMap *tmB, int warp)
{
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&ctrl->full[s], 1); mbar_init(&ctrl->empty[s], 1); }
        for (int a = 0; a < NUM_ACC; ++a) { mbar_init(&ctrl->tmem_full[a], 1); mbar_init(&ctrl->tmem_empty[a], 2 * EPI_WARPS); }
        ctrl->abort = 0;
        fence_barrier_init();
        tma_prefetch_desc(tmA);
        tma_prefetch_desc(tmB);
    }
    if (warp == 1) {
        tmem_alloc_pair(&ctrl->tmem_base, TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();          // the peer's barriers are initialised before anything signals them
    tc_fence_after();
    pdl_wait();                  // everything above touched no global tensor; from here on the previous kernel's output is read
    return ctrl->tmem_base;
}

__device__ __forceinline__ void pair_teardown(Ctrl *ctrl, uint32_t tmem_base, int warp)
{
    tc_fence_before();
    __syncthreads();
    if (ctrl->abort) abort_drain();
    cluster_sync_all();          // neither CTA frees tensor memory while the pair may still use it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

// Producer warp, one tile: this CTA's 128 rows of A from row0 and its W columns from col0 (weight matrix `group`),
// all k-blocks, through the ring.  Warp-uniform; `leader` is the one elected lane that issues.  With `descending`
// the k-blocks are fetched last to first (the sum does not care): a cluster alternates the direction from one of
// its tiles to the next, so a tile that shares a slab with the previous one starts on the part of it that was read
// last and is still in L2.
__device__ __forceinline__ void produce_tile(uint8_t *tiles, Ctrl *ctrl, const CUtensorMap *tmA, const CUtensorMap *tmB,
                                             RingPos &rp, int num_kb, int row0, int col0, int group, bool w_is_nk,
                                             uint32_t rank, bool leader, const WaitCtx &ctx, bool descending = false)
{
    for (int i = 0; i < num_kb; ++i) {
        const int kb = descending ? num_kb - 1 - i : i;
        mbar_wait(&ctrl->empty[rp.s], rp.ph ^ 1, ctx, BAR_EMPTY);
        uint8_t *a_s = tiles + (size_t)rp.s * STAGE_BYTES;
        uint8_t *b_s = a_s + A_BYTES;
        const uint32_t full_leader = mapa_shared(smem_u32(&ctrl->full[rp.s]), 0);
        if (leader) {
            if (rank == 0) mbar_arrive_expect_tx(&ctrl->full[rp.s], 2 * STAGE_BYTES);
            tma_load_2d_pair(a_s, tmA, full_leader, kb * BK, row0);
            if (w_is_nk) {
                tma_load_3d_pair(b_s, tmB, full_leader, kb * BK, col0, group);
            } else {
#pragma unroll
                for (int i = 0; i < BN_HALF / 64; ++i)
                    tma_load_3d_pair(b_s + i * (64 * BK * 2), tmB, full_leader, col0 + i * 64, kb * BK, group);
            }
        }
        __syncwarp();
        if (++rp.s == STAGES) { rp.s = 0; rp.ph ^= 1; }
    }
}

// Shared-memory descriptors of ring stage 0 (a stage is a constant number of bytes further) and the byte step of
// W per 16 k inside a stage.
struct MmaDescs { uint64_t a0, b0; uint32_t b_kstep; };
__device__ __forceinline__ MmaDescs make_mma_descs(const uint8_t *tiles, bool w_is_nk)
{
    const uint32_t a_addr0 = smem_u32(tiles), b_addr0 = a_addr0 + A_BYTES;
    MmaDescs d;
    d.a0 = make_smem_desc_sw128(a_addr0, 0, 1024);
    d.b0 = w_is_nk ? make_smem_desc_sw128(b_addr0, 0, 1024) : make_smem_desc_sw128(b_addr0, 64 * BK * 2, 1024);
    d.b_kstep = w_is_nk ? 32u : 2048u;
    return d;
}

// MMA warp of the leader CTA, one tile: all k-blocks into the accumulator at d_tmem, then the commit that tells
// both CTAs' epilogue warps.  Warp-uniform; `leader` is the one elected lane that issues.
__device__ __forceinline__ void mma_tile(Ctrl *ctrl, const MmaDescs &md, RingPos &rp, int num_kb, uint32_t d_tmem,
                                         uint32_t idesc, uint64_t *tmem_full, bool leader, const WaitCtx &ctx)
{
    for (int kb = 0; kb < num_kb; ++kb) {
        mbar_wait_cluster(&ctrl->full[rp.s], rp.ph, ctx, BAR_FULL);
        tc_fence_after();
        const uint64_t adesc = desc_advance(md.a0, (uint32_t)rp.s * STAGE_BYTES);
        const uint64_t bdesc = desc_advance(md.b0, (uint32_t)rp.s * STAGE_BYTES);
        if (leader) {
#pragma unroll
            for (int k = 0; k < BK / 16; ++k)
                umma_ss_pair(d_tmem, desc_advance(adesc, k * 32), desc_advance(bdesc, k * md.b_kstep), idesc,
                             (kb | k) != 0 ? 1u : 0u);
            umma_commit_pair(&ctrl->empty[rp.s], 0x3);
        }
        __syncwarp();
        if (++rp.s == STAGES) { rp.s = 0; rp.ph ^= 1; }
    }
    if (leader) umma_commit_pair(tmem_full, 0x3);
    __syncwarp();
}

// Epilogue threads: stage the tile's bias as fp32 in shared memory (columns n0 .. n0 + BN of bias row `group`).
__device__ __forceinline__ void stage_bias(const GemmArgs &p, Ctrl *ctrl, int n0, int group, int et)
{
    const long long bias0 = (long long)group * p.N + n0;    // bias is [num_groups, N] in grouped mode
    named_bar_sync(1, EPI_THREADS);
    for (int i = et; i < BN; i += EPI_THREADS) {
        float b = 0.0f;
        if (p.bias != nullptr && n0 + i < p.N)
            b = p.bias_f32 ? static_cast<const float *>(p.bias)[bias0 + i] : h16_at(p.bias, bias0 + i, p.f16 != 0);
        ctrl->bias[i] = b;
    }
    named_bar_sync(1, EPI_THREADS);
}

// One chunk of 32 columns of this thread's row (columns nc .. nc+31 of the output, chunk c of the tile):
//   v[j] = scale * act(acc + bias) + residual,  everything in registers.  taddr = the chunk's tensor-memory address.
template <int ACT>
__device__ __forceinline__ void chunk_values(const GemmArgs &p, const Ctrl *ctrl, uint32_t taddr, int row, bool row_ok,
                                             int nc, int c, bool f16, float (&v)[32])
{
    uint32_t r[32];
    tmem_ld32(taddr, r);

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
}

// Store one chunk of 32 values of this thread's row.  Thread = row, so one store instruction of a warp touches 32
// different rows: where the chunk lies fully inside N and starts on a 32-byte boundary it is written with 32-byte
// stores (whole sectors, half as many instructions), else with 16-byte ones.
__device__ __forceinline__ void store_chunk(const GemmArgs &p, int row, int nc, bool f16, const float (&v)[32])
{
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
                    *reinterpret_cast<float4 *>(op + g * 4) = make_float4(v[g * 4], v[g * 4 + 1], v[g * 4 + 2], v[g * 4 + 3]);
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
                    *reinterpret_cast<uint4 *>(op + g * 8) = make_uint4(w[g * 4], w[g * 4 + 1], w[g * 4 + 2], w[g * 4 + 3]);
        }
    }
}

// Running (max, sum exp) of a row over the chunks of a tile: fold in one chunk's values (columns nc .. nc+31, those
// past N excluded).
__device__ __forceinline__ void softmax_fold(const float (&v)[32], int nc, int N, float &run_m, float &run_l)
{
    float cm = -INFINITY;
#pragma unroll
    for (int j = 0; j < 32; ++j)
        if (nc + j < N) cm = fmaxf(cm, v[j]);
    const float nm = fmaxf(run_m, cm);
    float s = 0.0f;
#pragma unroll
    for (int j = 0; j < 32; ++j)
        if (nc + j < N) s += __expf(v[j] - nm);
    run_l = run_l * __expf(run_m - nm) + s;
    run_m = nm;
}

// The epilogue warps of both CTAs tell the leader's MMA warp that accumulator stage `acc` has been read out.
__device__ __forceinline__ void release_accumulator(Ctrl *ctrl, int acc, int lane)
{
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&ctrl->tmem_empty[acc]), 0));
}

}  // namespace gemm
}  // namespace pike
