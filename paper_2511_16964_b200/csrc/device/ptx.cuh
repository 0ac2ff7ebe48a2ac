// Device primitives for sm_100a: mbarrier with bounded waits, TMA tile loads,
// tcgen05 (tensor memory allocation, MMA issue, commit, loads), UMMA descriptors.
// Everything here is written against the public PTX ISA (8.7) documentation.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace pike {

// Device status word: 0 = ok, otherwise (kernel id << 16 | barrier id) of the
// first wait that ran out.  status[1] keeps the block index for diagnosis.
struct WaitCtx {
    unsigned int *status;      // global, may be nullptr
    volatile uint32_t *abort;  // shared, one word per CTA
    unsigned long long limit_ns;
    uint32_t kernel_id;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ unsigned long long globaltimer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// ---------------------------------------------------------------- mbarrier ----
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// The bookkeeping of a bounded wait, out of line: a wait is inlined at dozens of places and only its polling
// loop has to be there; this part runs once per 32 failed polls.  It looks at the CTA's abort word, reads the clock
// every 1024 polls (a slow system register) and, once limit_ns have passed since the first reading, records where
// the wait stopped and raises the abort word.  Returns the (possibly updated) time of the first reading, or
// WAIT_GAVE_UP when the caller must stop waiting.
constexpr unsigned long long WAIT_GAVE_UP = ~0ull;
static __device__ __noinline__ unsigned long long wait_bookkeeping(unsigned int *status, volatile uint32_t *abort,
                                                            unsigned long long limit_ns, uint32_t status_word,
                                                            uint32_t spins, unsigned long long t0)
{
    if (*abort) return WAIT_GAVE_UP;            // another thread of the CTA gave up
    if ((spins & 0x3FF) != 0) return t0;
    const unsigned long long now = globaltimer_ns();
    if (t0 == 0) return now;
    if (now - t0 <= limit_ns) return t0;
    *abort = 1;
    if (status != nullptr) {
        if (atomicCAS(status, 0u, status_word) == 0u) status[1] = blockIdx.x;
    }
    return WAIT_GAVE_UP;
}

// Wait for the phase with the given parity to complete.  Never spins forever:
// after ctx.limit_ns (or as soon as another thread of the CTA gave up) it records
// where it stopped, raises the CTA's abort word and returns false.  Callers keep
// going with whatever data they have, so the kernel always runs to its end,
// releases tensor memory and returns; the host sees PIKE_ERR_TIMEOUT.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, const WaitCtx &ctx, uint32_t barrier_id)
{
    if (mbar_try_wait(bar, parity)) return true;
    uint32_t spins = 0;
    unsigned long long t0 = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x1F) == 0) {
            t0 = wait_bookkeeping(ctx.status, ctx.abort, ctx.limit_ns, (ctx.kernel_id << 16) | barrier_id, spins, t0);
            if (t0 == WAIT_GAVE_UP) return false;
        }
    }
    return true;
}

// Wait until a counter in global memory that other CTAs increment has reached `target` (acquire at device scope).
// Bounded like mbar_wait: after ctx.limit_ns, or when another thread of the CTA gave up, it records where it
// stopped, raises the CTA's abort word and returns false.  Only for kernels whose CTAs are all resident.
__device__ __forceinline__ bool counter_wait(const unsigned int *counter, unsigned int target, const WaitCtx &ctx,
                                             uint32_t barrier_id)
{
    uint32_t spins = 0;
    unsigned long long t0 = 0;
    for (;;) {
        unsigned int seen;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
        if (seen >= target) return true;
        if ((++spins & 0xF) == 0) {
            if (*ctx.abort) return false;
            const unsigned long long now = globaltimer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > ctx.limit_ns) {
                *ctx.abort = 1;
                if (ctx.status != nullptr) {
                    if (atomicCAS(ctx.status, 0u, (ctx.kernel_id << 16) | barrier_id) == 0u)
                        ctx.status[1] = blockIdx.x;
                }
                return false;
            }
        }
        __nanosleep(100);
    }
}

// Give copies that may still be in flight time to land before the CTA exits on
// the abort path (about one millisecond, bounded).
__device__ __forceinline__ void abort_drain()
{
#pragma unroll 1
    for (int i = 0; i < 1000; ++i) __nanosleep(1000);
}

// ------------------------------------------------ programmatic dependent launch ----
// A grid launched with the programmatic-stream-serialisation attribute may be scheduled while the previous kernel
// of its stream still runs: its CTAs take the SMs that kernel's CTAs have left.  pdl_wait() returns once that kernel
// has completed and its writes are visible; every kernel executes it after a prologue that touches no global tensor
// (barrier initialisation, tensor-memory allocation, descriptor prefetch) and before its first global access.  It
// is a no-op in a launch without the attribute.  No kernel here signals its dependents early
// (griddepcontrol.launch_dependents): with the signal at kernel start the next kernel's CTAs sat beside the GEMM's
// for its whole run and the logits + softmax chain got 3 % slower; leaving it to each CTA's exit keeps the gain
// (launch latency and prologue hidden in the previous kernel's tail) without that cost.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// --------------------------------------------------------------------- TMA ----
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap *map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
// Untiled bulk copy global -> shared (no tensor map): both addresses 16-byte aligned, bytes a multiple of 16;
// completion is signalled on the mbarrier as transferred bytes.
__device__ __forceinline__ void bulk_load_1d(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// 2-D tile load; x (innermost coordinate) times the element size must be a
// multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y, int z)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y, int z, int w)
{
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z), "r"(w)
        : "memory");
}
// Asynchronous copies global -> shared issued by every thread (no tensor map, no barrier object): all of a
// thread's copies are in flight at once and one wait covers them.  `valid` false writes zeros instead
// (nothing is read, but src must still be an address inside the tensor).
__device__ __forceinline__ void cp_async_16(void *dst, const void *src, bool valid)   // both 16-byte aligned
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(valid ? 16 : 0)
                 : "memory");
}
__device__ __forceinline__ void cp_async_4(void *dst, const void *src, bool valid)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(valid ? 4 : 0)
                 : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
// generic-proxy writes to shared memory -> visible to the async proxy (MMA/TMA)
__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ----------------------------------------------------------------- tcgen05 ----
__device__ __forceinline__ void tmem_alloc(uint32_t *smem_result, uint32_t ncols)  // whole warp
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish()  // whole warp
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)  // whole warp
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], kind::f16 (bf16 x bf16 -> fp32), issued by ONE thread.
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on an mbarrier once every MMA issued so far by this thread has finished
// (implies tcgen05.fence::before_thread_sync).
__device__ __forceinline__ void umma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread t of the warp gets lane
// (lane field of taddr + t), registers r[0..31] = columns c..c+31.  The lane
// field must be 32 * (warp index within its warpgroup).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Mirror of tmem_ld32: thread t writes registers r[0..31] to lane (lane field + t), columns c..c+31.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
// 16-column form of tmem_st32
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[tmem] * B[smem]: the A operand (M = 128 rows on the 128 lanes, 16-bit elements
// packed two per 32-bit column, K-major) is read from tensor memory.  Issued by ONE thread.
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Warpgroup-wide register re-partitioning (all four warps of the warpgroup execute it).
template <int N>
__device__ __forceinline__ void setmaxnreg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void setmaxnreg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

// ------------------------------------------------ CTA pairs (cta_group::2) ----
// A cluster of two CTAs on two SMs works on one 256-row tile: each CTA stages its own
// half of A and of B, one thread of the even ("leader") CTA issues the MMA for both, and
// each CTA's tensor memory receives the accumulator rows of its half.
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_nctas()   // CTAs per cluster (x extent; clusters here are one-dimensional)
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctaid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()  // every thread of every CTA of the cluster
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The two halves of a cluster barrier on their own: a relaxed arrival orders no memory accesses (enough
// when the barrier only has to say "I no longer read your shared memory") and lets work go on until the wait.
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.aligned;" ::: "memory"); }
// shared::cta address of this CTA -> shared::cluster address of the same offset in CTA `rank`
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// 8-byte load from any CTA's shared memory of the cluster (address from mapa_shared)
__device__ __forceinline__ float2 ld_shared_cluster_f32x2(uint32_t cluster_addr)
{
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(cluster_addr) : "memory");
    return v;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Tile load whose completion is signalled on an mbarrier given by its shared::cluster
// address (the leader's barrier, also when the peer CTA issues the load).  No multicast.
__device__ __forceinline__ void tma_load_2d_pair(void *dst, const CUtensorMap *map, uint32_t bar_cluster_addr, int x,
                                                 int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(void *dst, const CUtensorMap *map, uint32_t bar_cluster_addr, int x,
                                                 int y, int z)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(x), "r"(y), "r"(z)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t *smem_result, uint32_t ncols)  // one warp in EACH CTA
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// 256 x N x 16 MMA over the CTA pair; descriptors hold the leader's shared-memory offsets,
// which the hardware applies in both CTAs.  Issued by ONE thread of the leader CTA.
__device__ __forceinline__ void umma_ss_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on the mbarrier at this shared-memory offset in every CTA of `cta_mask` once all
// MMAs issued so far by this thread have finished.
__device__ __forceinline__ void umma_commit_pair(uint64_t *bar, uint16_t cta_mask)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(smem_u32(bar)), "h"(cta_mask)
        : "memory");
}

// Same, for a barrier that threads of the peer CTA arrive on (cluster-scope acquire).
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t *bar, uint32_t parity, const WaitCtx &ctx, uint32_t barrier_id)
{
    if (mbar_try_wait_cluster(bar, parity)) return true;
    uint32_t spins = 0;
    unsigned long long t0 = 0;
    while (!mbar_try_wait_cluster(bar, parity)) {
        if ((++spins & 0x1F) == 0) {
            t0 = wait_bookkeeping(ctx.status, ctx.abort, ctx.limit_ns, (ctx.kernel_id << 16) | barrier_id, spins, t0);
            if (t0 == WAIT_GAVE_UP) return false;
        }
    }
    return true;
}

// ------------------------------------------------------- UMMA descriptors ----
// Shared-memory matrix descriptor (64 bit):
//   [0,14)  start address >> 4        [16,30) leading-dimension byte offset >> 4
//   [32,46) stride-dimension byte offset >> 4      [46,48) = 1 (descriptor version)
//   [49,52) base offset (0: tiles are 1024-byte aligned)   [61,64) swizzle (2 = 128 B)
// 128-byte swizzle, K-major operand (rows of 64 bf16 = 128 B): SBO = distance
//   between 8-row groups (1024 B for dense rows), LBO unused.
// 128-byte swizzle, MN-major operand (k-rows of 64 contiguous MN elements):
//   LBO = distance between 64-element blocks along MN, SBO = distance between
//   8-k groups (1024 B).
__device__ __forceinline__ uint64_t make_smem_desc_sw128(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}

// Advancing a descriptor's start address by `bytes` (a multiple of 16 that stays inside the 256 KiB
// window, so the 14-bit address field cannot carry into its neighbours) is one 64-bit add.  The MMA
// issue loop runs on ONE thread, so descriptors are built once and only advanced per instruction.
__device__ __forceinline__ constexpr uint64_t desc_advance(uint64_t desc, uint32_t bytes)
{
    return desc + static_cast<uint64_t>(bytes >> 4);
}

// Instruction descriptor for kind::f16 with 16-bit operands (both bf16, or both f16) and fp32 accumulator:
//   [4,6) D format (1 = f32)  [7,10) A format (0 = f16, 1 = bf16)  [10,13) B format (same as A)
//   bit 15 A is MN-major   bit 16 B is MN-major   [17,23) N >> 3   [24,29) M >> 4
__host__ __device__ constexpr uint32_t make_idesc_bf16(int M, int N, bool a_mn_major, bool b_mn_major, bool f16 = false)
{
    return (1u << 4) | (f16 ? 0u : ((1u << 7) | (1u << 10))) | (a_mn_major ? (1u << 15) : 0u) |
           (b_mn_major ? (1u << 16) : 0u) | (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}

// ------------------------------------------------------------------ misc ----
// One lane of a fully active warp.  Role loops are run by the WHOLE warp (so addresses, descriptors
// and loop state stay warp-uniform and live in uniform registers) and only the single-thread
// instructions (TMA issue, tcgen05.mma, tcgen05.commit) are predicated on this.
__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}

__device__ __forceinline__ void named_bar_sync(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);  // .x = lo (low 16 bits)
    return *reinterpret_cast<uint32_t *>(&v);
}
// The 16-bit storage type of a tensor is bf16 or IEEE half (f16 == true); both are computed in fp32.
__device__ __forceinline__ float h16_lo(uint32_t u, bool f16)
{
    return f16 ? __half2float(__ushort_as_half(static_cast<unsigned short>(u & 0xFFFFu))) : bf16_lo(u);
}
__device__ __forceinline__ float h16_hi(uint32_t u, bool f16)
{
    return f16 ? __half2float(__ushort_as_half(static_cast<unsigned short>(u >> 16))) : bf16_hi(u);
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi)
{
    __half2 v = __floats2half2_rn(lo, hi);             // .x = lo (low 16 bits)
    return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ uint32_t pack_h16x2(float lo, float hi, bool f16)
{
    return f16 ? pack_f16x2(lo, hi) : pack_bf16x2(lo, hi);
}
// Two fp32 lanes per instruction (sm_100 packed arithmetic): half the issue slots of the scalar forms, which
// is what row-wise code bound by instruction issue (softmax, LayerNorm) needs.
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t mul_f32x2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
// the two 16-bit values of a word as an fp32 pair (low half first)
__device__ __forceinline__ uint64_t h16x2_to_f32x2(uint32_t u, bool f16)
{
    return pack_f32x2(h16_lo(u, f16), h16_hi(u, f16));
}
// one 256-bit store (sm_100); dst must be 32-byte aligned
__device__ __forceinline__ void st_global_32B(void *dst, const uint32_t *w)
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                 "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]) : "memory");
}
// one 256-bit load (sm_100); src must be 32-byte aligned
__device__ __forceinline__ void ld_global_32B(const void *src, uint32_t *w)
{
    asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                 : "l"(src));
}
// element i of a 16-bit vector as fp32
__device__ __forceinline__ float h16_at(const void *p, long long i, bool f16)
{
    const unsigned short u = static_cast<const unsigned short *>(p)[i];
    return f16 ? __half2float(__ushort_as_half(u)) : __uint_as_float(static_cast<uint32_t>(u) << 16);
}

}  // namespace pike
