/*
 * pike.h — C ABI of the fused operator-chain library for NVIDIA B200 (sm_100a).
 *
 * The paper (arxiv 2511.16964, Section 5.3 "Task-wise Benchmark Analysis") names
 * the optimisation pattern this library implements: fuse a heavy operator (a
 * dense GEMM) with the pointwise and row-reduction operators that follow it into
 * one kernel, so intermediates never round-trip through HBM and launch overhead
 * disappears, and replace naive attention by a flash-attention kernel with
 * on-the-fly causal masking (Appendix C, "VisionAttention", "MinGPT",
 * "HunyuanVideo").  The paper gives no formulas for the operators; each entry
 * point below states the textbook definition it computes.
 *
 * Conventions
 *  - Plain C, no exceptions cross the boundary; every function returns
 *    pike_status_t (PIKE_OK == 0).
 *  - Every tensor is CALLER-OWNED DEVICE MEMORY on the handle's device, borrowed
 *    until the enqueued work has finished.  Tensors are row-major with element
 *    strides; the innermost stride must be 1 and the base address 16-byte
 *    aligned.  The library never allocates per call: scratch comes from a caller
 *    supplied workspace (device memory, 256-byte aligned) whose size the matching
 *    *_workspace query returns.
 *  - Calls enqueue on the caller's CUDA stream (a cudaStream_t passed as void*,
 *    NULL = default stream) and return without synchronising.  The return value
 *    reports host-detectable errors only.  Device-detected conditions (a bounded
 *    wait inside a kernel that ran out) land in a status word that
 *    pike_get_last_device_status reads after the caller has synchronised.
 *    A chain call only launches kernels (no allocation, no copy, no event unless
 *    profiling is on), so a sequence of calls on a capturing stream becomes a CUDA
 *    graph that can be replayed on new contents of the same buffers.
 *  - There is no CPU or library fallback: a device that is not compute
 *    capability 10.x yields PIKE_ERR_ARCH, an unsupported shape or combination
 *    PIKE_ERR_UNSUPPORTED.
 */
#ifndef PIKE_H_
#define PIKE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PIKE_OK = 0,
    PIKE_ERR_NULL = 1,        /* a required pointer is NULL                              */
    PIKE_ERR_SHAPE = 2,       /* ranks / extents do not fit together                     */
    PIKE_ERR_DTYPE = 3,       /* dtype combination not accepted by this entry point      */
    PIKE_ERR_ALIGNMENT = 4,   /* base pointer or row pitch not 16-byte aligned           */
    PIKE_ERR_STRIDE = 5,      /* innermost stride != 1 or a non-dense layout             */
    PIKE_ERR_UNSUPPORTED = 6, /* valid request outside the implemented envelope          */
    PIKE_ERR_WORKSPACE = 7,   /* workspace NULL / misaligned / too small                 */
    PIKE_ERR_ARCH = 8,        /* device is not sm_100                                    */
    PIKE_ERR_CUDA = 9,        /* a CUDA runtime or driver call failed                    */
    PIKE_ERR_TIMEOUT = 10     /* device status only: a bounded in-kernel wait ran out    */
} pike_status_t;

/* Element types.  PIKE_BF16 and PIKE_F16 (IEEE binary16, the reduced precision the paper's winning
 * solutions use: Section 5.3 and Appendix C, "VisionAttention", "MinGPT") select the same tensor-core
 * kernels with fp32 accumulation; wherever the text below says "16-bit" either may be used, but one
 * call never mixes the two: every 16-bit tensor of a call has the dtype of x (or q), anything else
 * is PIKE_ERR_DTYPE.  F16 has the narrower range (largest finite value 65504): values that overflow
 * it on output become infinities, as in any f16 computation. */
typedef enum { PIKE_F32 = 0, PIKE_BF16 = 1, PIKE_F16 = 2 } pike_dtype_t;

/* A view of caller-owned device memory.  stride[] is in elements. */
typedef struct {
    void *data;
    pike_dtype_t dtype;
    int32_t ndim;             /* 1..4 */
    int64_t shape[4];
    int64_t stride[4];
} pike_tensor_t;

typedef enum { PIKE_ACT_NONE = 0, PIKE_ACT_GELU_ERF = 1, PIKE_ACT_GELU_TANH = 2, PIKE_ACT_SILU = 3 } pike_act_t;
typedef enum { PIKE_REDUCE_NONE = 0, PIKE_REDUCE_LAYERNORM = 1, PIKE_REDUCE_SOFTMAX = 2 } pike_reduce_t;

#define PIKE_FLAG_W_IS_NK 0x1u /* weight tensors are [N,K] ("out,in") instead of [K,N]   */
#define PIKE_FLAG_CAUSAL  0x2u /* attention: key j takes part for query i only if j <= i */
#define PIKE_FLAG_ONE_PASS 0x4u /* pike_linear_epilogue, 16-bit path, reduce == SOFTMAX: one kernel, every      */
                               /* probability written exactly once (see pike_linear_epilogue)                 */

/* Epilogue descriptor: what follows the GEMM inside the same kernel. */
typedef struct {
    uint32_t struct_size;     /* sizeof(pike_epilogue_t), for forward compatibility      */
    pike_act_t act;           /* activation applied to (acc + bias)                      */
    float scale;              /* multiplies the activation (1.0f = off); attention: the  */
                              /* factor applied to q.k before the softmax                */
    pike_reduce_t reduce;     /* row reduction over N applied last                       */
    float eps;                /* LayerNorm epsilon (inside the square root)              */
    pike_dtype_t out_dtype;   /* must equal out->dtype                                   */
    uint32_t flags;           /* PIKE_FLAG_*                                             */
} pike_epilogue_t;

typedef struct pike_handle_s *pike_handle_t;

/* Create / destroy a handle for CUDA device `device`.  pike_create makes that
 * device current, prepares every kernel for it (shared-memory limits, how many
 * CTA pairs fit) and stores what it learns in the handle: the library keeps no
 * per-device state outside handles, so handles on different devices or host
 * threads never interfere.  The handle owns a 16-byte device status word (its
 * only device allocation), one non-blocking stream for reading it, and a small
 * cache of encoded TMA tensor maps keyed by (pointer, extents, pitches, box), so
 * repeated calls on the same buffers skip the encoding.  A handle is not
 * thread-safe; use one per host thread.  PIKE_ERR_ARCH if the device is not
 * compute capability 10.x.  With PIKE_LOG=1 in the environment when the handle is
 * created, every kernel selection made through it is written to stderr as one line
 * (kernel, shapes, layout, epilogue): host-side only, nothing changes on the device.
 * Kernels are launched with the programmatic-stream-serialisation attribute: a
 * kernel's CTAs may be scheduled onto SMs the previous kernel of the stream has
 * already left and run their prologue there; each waits for that kernel to complete
 * before it touches a tensor, so stream order is kept.  PIKE_PDL=0 in the
 * environment at creation takes the attribute off (results are identical). */
pike_status_t pike_create(pike_handle_t *handle, int device);
pike_status_t pike_destroy(pike_handle_t handle);

/* Static, never-freed description of a status code. */
const char *pike_status_string(pike_status_t status);

/* Reads (and clears) the device status word.  It waits for no kernel: the
 * caller synchronises the stream(s) whose status it wants first; the read
 * itself travels on the handle's own stream.  *status is PIKE_OK or
 * PIKE_ERR_TIMEOUT; *where identifies the wait that gave up
 * (kernel id << 16 | barrier id). */
pike_status_t pike_get_last_device_status(pike_handle_t handle, pike_status_t *status, uint32_t *where);

/* Test hook: upper bound, in nanoseconds, for every in-kernel wait of kernels
 * launched through this handle afterwards (default 2e9).  0 restores the default. */
pike_status_t pike_set_wait_limit_ns(pike_handle_t handle, uint64_t ns);

/* Test hook for the failure-detection path (no counterpart in the paper): the NEXT bf16 GEMM launched
 * through this handle issues no operand loads (the next fp32 chain, if that comes first: none of the bulk copies
 * its small-problem kernel stages 16-byte aligned operands with), so its first wait for data runs out after the wait limit,
 * the kernel records where, skips its remaining waits, runs to its end (the output is garbage) and
 * pike_get_last_device_status reports PIKE_ERR_TIMEOUT.  Nothing faults, traps or hangs; the context and
 * the handle stay usable.  Use with a small pike_set_wait_limit_ns. */
pike_status_t pike_test_withhold_loads(pike_handle_t handle);

/* Test hook for the cross-CTA wait of the one-pass softmax (PIKE_FLAG_ONE_PASS; no counterpart in the paper): in the
 * NEXT such launch through this handle one CTA never counts itself in on the stripe counters, so its peers' waits run
 * out after the wait limit, the kernel records where, runs to its end (the output is garbage) and
 * pike_get_last_device_status reports PIKE_ERR_TIMEOUT.  Nothing faults, traps or hangs.  Use with a small
 * pike_set_wait_limit_ns. */
pike_status_t pike_test_withhold_partials(pike_handle_t handle);

/*
 * Per-kernel device timing, following the paper's timing protocol (Section 4.6:
 * timed runs bracketed on the device, synchronisation inside the timed region).
 * Between pike_profile_begin and pike_profile_end every kernel the handle launches
 * is bracketed by two CUDA events on the caller's stream.  pike_profile_end
 * synchronises the device and fills out[PIKE_KERNEL_COUNT] (caller-owned host
 * memory) with the launch count and the summed device time of each kernel.
 */
typedef enum {
    PIKE_KERNEL_FP32_CHAIN = 0,     /* fp32 linear + epilogue + row reduction          */
    PIKE_KERNEL_GEMM_BF16 = 1,      /* tcgen05 GEMM + register epilogue                */
    PIKE_KERNEL_LAYERNORM_BF16 = 2, /* MLP block prologue                              */
    PIKE_KERNEL_SOFTMAX_FINISH = 3, /* combine split-row partials, normalise in place  */
    PIKE_KERNEL_ATTENTION_BF16 = 4, /* GEMM -> online softmax -> GEMM                  */
    PIKE_KERNEL_COUNT = 5
} pike_kernel_t;
typedef struct { uint64_t launches; double device_ms; } pike_kernel_profile_t;
pike_status_t pike_profile_begin(pike_handle_t handle);
pike_status_t pike_profile_end(pike_handle_t handle, pike_kernel_profile_t *out);

/*
 * Linear + epilogue chain (the "operator fusion" pattern of Section 5.3):
 *
 *   v[m,n]   = scale * act( sum_k x[m,k] * w[k,n] + bias[n] ) + residual[m,n]
 *   out[m,:] = v[m,:]                                   reduce == NONE
 *            = (v - mean)/sqrt(var + eps) * gamma + beta reduce == LAYERNORM (biased var)
 *            = exp(v - max v) / sum exp(v - max v)       reduce == SOFTMAX
 *
 * x [M,K]; w [K,N] (or [N,K] with PIKE_FLAG_W_IS_NK); bias, gamma, beta [N];
 * residual, out [M,N].  bias, residual, gamma, beta may be NULL (0, 0, 1, 0).
 *
 * fp32 path (x, w, out all PIKE_F32; bias/residual/gamma/beta F32): true fp32
 *   FMA on the CUDA cores; any M, K; N <= 1024; every reduce mode.
 * 16-bit path (x, w both PIKE_BF16 or both PIKE_F16; bias/residual/gamma/beta of
 *   that type or F32): tcgen05 tensor-core GEMM with fp32 accumulation; K and N
 *   multiples of 8; out of that 16-bit type or F32.  A row reduction on this path is split across the GEMM's 256-column
 *   tiles: the epilogue writes the un-reduced values plus one pair per (row, tile)
 *   to the workspace - (max, sum exp) for SOFTMAX, (mean, sum of squared
 *   deviations) for LAYERNORM - and a second kernel combines the pairs and
 *   finishes the rows in place.  SOFTMAX needs out F32; LAYERNORM takes 16-bit or F32
 *   (with a 16-bit out the un-reduced values are rounded once before normalisation).
 *   With PIKE_FLAG_ONE_PASS a SOFTMAX on this path runs as ONE kernel that never writes an un-normalised value
 *   (Section 5.3: "eliminating intermediate memory writes"): a 256-row stripe of logits stays in tensor memory
 *   across all CTA pairs of the device until its per-tile (max, sum exp) pairs have been exchanged through the
 *   workspace, then every probability is written once.  The kernel's CTAs wait for one another, so it is
 *   launched cooperatively (it needs the whole device; the wait is bounded like every other and reports
 *   PIKE_ERR_TIMEOUT through the status word).  Needs ceil(N/256) <= 2 x (CTA pairs the device holds), i.e.
 *   N <= 37888 on a 148-SM part, else PIKE_ERR_UNSUPPORTED; the workspace also holds one counter per stripe.
 *   On the benchmark's logits chain it is SLOWER than the two-kernel form (measured; see profiles/), which is
 *   why it is an option and not the default.
 * out must not alias any input (PIKE_ERR_UNSUPPORTED if the ranges overlap).
 *
 * Workspace: pike_linear_epilogue_workspace returns the bytes needed (0 unless a
 * row reduction is requested on the 16-bit path); it reads only shapes and dtypes.
 * For every entry point that takes one, a workspace that is NULL, not 256-byte
 * aligned, too small, or that overlaps any tensor of the call is PIKE_ERR_WORKSPACE.
 */
pike_status_t pike_linear_epilogue_workspace(pike_handle_t handle, const pike_tensor_t *x,
                                             const pike_tensor_t *w, const pike_epilogue_t *epi,
                                             size_t *bytes);
pike_status_t pike_linear_epilogue(pike_handle_t handle, const pike_tensor_t *x, const pike_tensor_t *w,
                                   const pike_tensor_t *bias, const pike_tensor_t *residual,
                                   const pike_tensor_t *gamma, const pike_tensor_t *beta,
                                   const pike_epilogue_t *epi, pike_tensor_t *out, void *workspace,
                                   size_t workspace_bytes, void *cuda_stream);

/*
 * Logits + row softmax with the columns split over several GPUs (the paper's "Future Work" section names
 * multi-GPU inference as the next step for these chains; a vocabulary projection is the chain whose
 * weight is sharded column-wise in practice).  GPU r of R holds the column slice w_r [K,N_r] (and bias_r)
 * and every GPU holds the same x [M,K]; together they compute
 *
 *   out[m, slice r] = exp(v[m,n] - max_n v[m,:]) / sum_n exp(v[m,n] - max_n v[m,:]),
 *   v[m,n] = scale * act( sum_k x[m,k] * w[k,n] + bias[n] )
 *
 * with the maximum and the sum taken over ALL N = sum_r N_r columns.  Two calls per GPU with one
 * exchange between them (the only data that crosses GPUs is one (max, sum) pair per row and GPU):
 *
 *  1. pike_linear_softmax_shard_local: out_r [M,N_r] F32 receives the un-normalised v of this slice and
 *     row_stats[m] = ( max_n v[m, slice r], sum_n exp(v[m,n] - that max) ), M pairs of floats in DEVICE
 *     memory (8-byte aligned).  Same kernels, dtypes (x, w both BF16 or both F16; bias that type or F32 or
 *     NULL) and envelope (K, N_r multiples of 8) as pike_linear_epilogue with reduce == SOFTMAX;
 *     epi->reduce must be PIKE_REDUCE_SOFTMAX and epi->out_dtype PIKE_F32.  Workspace as returned by
 *     pike_linear_softmax_shard_workspace (the per-tile pairs).
 *  2. The caller gathers every GPU's row_stats into all_stats [R, M] pairs, shard-major - exactly what an
 *     all-gather of the R row_stats arrays produces (8*M bytes per GPU; NCCL or any other transport;
 *     the library itself does no communication).
 *  3. pike_linear_softmax_shard_finish: combines the R pairs of each row,
 *     m = max_r m_r, l = sum_r l_r * exp(m_r - m), and overwrites out_r with exp(out_r - m) / l.
 *     all_stats is DEVICE memory, 8-byte aligned; num_shards = R >= 1.  out_r must still hold the values
 *     step 1 wrote.  With R == 1 the two calls compute the same result as pike_linear_epilogue.
 *
 * The order of the shards in all_stats does not matter (max and sum commute), but every GPU must use the
 * same x, scale, act and a disjoint slice of the columns.  Errors as for pike_linear_epilogue.
 */
pike_status_t pike_linear_softmax_shard_workspace(pike_handle_t handle, const pike_tensor_t *x,
                                                  const pike_tensor_t *w, const pike_epilogue_t *epi,
                                                  size_t *bytes);
pike_status_t pike_linear_softmax_shard_local(pike_handle_t handle, const pike_tensor_t *x, const pike_tensor_t *w,
                                              const pike_tensor_t *bias, const pike_epilogue_t *epi,
                                              pike_tensor_t *out, float *row_stats, void *workspace,
                                              size_t workspace_bytes, void *cuda_stream);
pike_status_t pike_linear_softmax_shard_finish(pike_handle_t handle, pike_tensor_t *out, const float *all_stats,
                                               int32_t num_shards, void *cuda_stream);

/*
 * Logits + row softmax for callers that cannot allocate device memory.  (The paper has
 * no counterpart to this entry point; it exists for how the library gets embedded.)
 *
 *   out[m,:] = softmax_n( scale * act( sum_k x[m,k] * w[k,n] + bias[n] ) )
 *
 * Same arithmetic, kernels and bf16 envelope as pike_linear_epilogue with
 * reduce == PIKE_REDUCE_SOFTMAX (x, w PIKE_BF16, bias BF16/F32 or NULL, out PIKE_F32,
 * K and N multiples of 8, M >= 1; epi->reduce must be PIKE_REDUCE_SOFTMAX and
 * epi->out_dtype PIKE_F32), but it takes no workspace: some hosts of this library
 * cannot produce one -- a server that gave the whole device heap to its own pool, a
 * plugin running inside another framework's step, a latency-critical thread that may
 * not enter cudaMalloc (it locks and can synchronise the device).  The per-(row,
 * 256-column tile) partial (max, sum) pairs go to an array built into the library
 * image instead.  The call itself performs no cudaMalloc/cudaFree and calls no
 * allocating routine.  What follows from the built-in array:
 *  - Capacity: M * ceil(N/256) <= PIKE_NOALLOC_MAX_PARTIALS (2 MiB of pairs, resident
 *    on every GPU that loads the library until the process exits).  A larger problem
 *    returns PIKE_ERR_WORKSPACE and enqueues nothing.
 *  - The first call on a device looks up the array's device address
 *    (cudaGetSymbolAddress); make that first call outside any stream capture.
 *  - All calls on a device share the array.  Calls that can overlap on the GPU (issued
 *    to different streams without an ordering between them) race on it and produce
 *    wrong results; calls on one stream are safe.  The array keeps the previous call's
 *    values, which is harmless: each call writes every pair before reading it.
 */
#define PIKE_NOALLOC_MAX_PARTIALS 262144
pike_status_t pike_linear_softmax_noalloc(pike_handle_t handle, const pike_tensor_t *x, const pike_tensor_t *w,
                                          const pike_tensor_t *bias, const pike_epilogue_t *epi, pike_tensor_t *out,
                                          void *cuda_stream);

/*
 * Grouped linear + epilogue: many small GEMMs with different weights in ONE launch (Appendix C,
 * "DeepSeek3MOESmallBatch": the per-expert loop of a mixture-of-experts layer replaced by one
 * grouped matrix multiplication over packed expert weights):
 *
 *   for group g and every row r in [group_offsets[g], group_offsets[g+1]):
 *     out[r,:] = scale * act( x[r,:] @ w[g] + bias[g,:] ) + residual[r,:]
 *
 * x [T,K] 16-bit (BF16 or F16) with the rows of one group stored together; w [G,K,N] (or [G,N,K] with
 * PIKE_FLAG_W_IS_NK) of the same type; bias [G,N] that type or F32, or NULL; residual, out [T,N] (that type or F32);
 * K and N multiples of 8; reduce must be NONE.  group_offsets points to G+1 int32 values in DEVICE
 * memory (non-decreasing, first 0, last T; empty groups are fine): the kernel reads them itself, so
 * the host never has to wait for a router's counts.  No workspace.  Rows outside
 * [0, group_offsets[G]) are not written.  The host cannot check the offsets, so the kernel clamps each
 * one to [0, T] and each group's end to at least its start: offsets that break the contract give
 * meaningless values in the rows concerned, never an access outside the tensors.  The group that owns
 * a row tile is found by bisection over prefix sums each CTA builds once in shared memory (up to 4096
 * groups; beyond that over the offsets themselves), so G up to 65536 costs no scan per tile.
 */
pike_status_t pike_grouped_linear_epilogue(pike_handle_t handle, const pike_tensor_t *x, const pike_tensor_t *w,
                                           const pike_tensor_t *bias, const pike_tensor_t *residual,
                                           const int32_t *group_offsets, const pike_epilogue_t *epi, pike_tensor_t *out,
                                           void *cuda_stream);

/*
 * Pre-LayerNorm transformer MLP block (sub-graph fusion, Section 5.3):
 *
 *   z   = LayerNorm(x; gamma, beta, eps)            over the last dimension D
 *   h   = act( z @ w1 + b1 )                         [M,F]
 *   out = x + h @ w2 + b2                            [M,D]   (residual = un-normalised x)
 *
 * All tensors 16-bit, all BF16 or all F16 (gamma, beta, b1, b2 may be F32); x, out [M,D]; w1 [D,F];
 * w2 [F,D] (or transposed with PIKE_FLAG_W_IS_NK); D, F multiples of 8, D <= 16384.
 * epi->act selects the activation, epi->eps the LayerNorm epsilon; scale must be 1
 * and reduce NONE.  z and h are rounded to the 16-bit type and live in the workspace
 * (M*D*2 + M*F*2 bytes, each part 256-byte aligned).  Three kernels are enqueued
 * on the stream.
 */
pike_status_t pike_mlp_block_workspace(pike_handle_t handle, const pike_tensor_t *x, const pike_tensor_t *w1,
                                       const pike_epilogue_t *epi, size_t *bytes);
pike_status_t pike_mlp_block(pike_handle_t handle, const pike_tensor_t *x, const pike_tensor_t *gamma,
                             const pike_tensor_t *beta, const pike_tensor_t *w1, const pike_tensor_t *b1,
                             const pike_tensor_t *w2, const pike_tensor_t *b2, const pike_epilogue_t *epi,
                             pike_tensor_t *out, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Attention chain (flash attention with on-the-fly causal masking, Appendix C):
 *
 *   s[i,j]  = epi->scale * sum_d q[i,d] * k[j,d]
 *   out[i,:] = sum_j softmax_j(s[i,.])[j] * v[j,:]   (j <= i only with PIKE_FLAG_CAUSAL)
 *
 * per (batch, head).  q, out are [B,H,S,D] and k, v [B,H,Sk,D] 16-bit views (all BF16 or all F16), D == 128 or 64, any
 * S, Sk >= 1; Sk != S (cross attention) only without PIKE_FLAG_CAUSAL.  Rows must be contiguous (stride[3] == 1); the batch, head and row strides may be anything
 * that is a multiple of 8 elements and at least D, so dense [B,H,S,D], a [B,S,H,D] tensor viewed as
 * [B,H,S,D], or the q / k / v slices of a packed [B,S,3,H,D] projection output all work without a copy.  The score matrix lives in tensor memory and registers
 * only; probabilities are rounded to the 16-bit type before the second GEMM.  Workspace: 0
 * bytes (the query exists for symmetry).
 */
pike_status_t pike_attention_chain_workspace(pike_handle_t handle, const pike_tensor_t *q,
                                             const pike_epilogue_t *epi, size_t *bytes);
pike_status_t pike_attention_chain(pike_handle_t handle, const pike_tensor_t *q, const pike_tensor_t *k,
                                   const pike_tensor_t *v, const pike_epilogue_t *epi, pike_tensor_t *out,
                                   void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Pre-LayerNorm attention block with fused input and output projections (Appendix C, "VisionAttention":
 * the largest win reported is flash attention plus fused projection kernels; "MinGPT": causal blocks):
 *
 *   z   = LayerNorm(x; gamma, beta, eps)                     over the last dimension E
 *   qkv = z @ w_qkv + b_qkv                                  [B,S,3E], columns ordered q | k | v, each H heads of 128
 *   a   = softmax(scale * q k^T [+ causal mask]) v           per (batch, head), written as [B,S,H,128]
 *   out = x + a @ w_o + b_o                                  [B,S,E]
 *
 * x, out dense [B,S,E] 16-bit (BF16 or F16) with E = H*128 <= 4096; w_qkv [E,3E], w_o [E,E] of that type (or transposed
 * with PIKE_FLAG_W_IS_NK); gamma, beta [E], b_qkv [3E], b_o [E] of that type or F32, each may be NULL.  epi->eps is
 * the LayerNorm epsilon, epi->scale (> 0) the factor on q.k, PIKE_FLAG_CAUSAL the mask; act must be NONE and
 * reduce NONE.  The attention kernel reads q, k, v as strided views of the projection output and writes its
 * result in the layout the output projection reads, so no transpose or copy kernel runs: four kernels are
 * enqueued (LayerNorm, GEMM+bias, attention, GEMM+bias+residual).  z, qkv and a are 16-bit in the workspace
 * (2*B*S*E*2 + B*S*3E*2 bytes, each part 256-byte aligned).
 */
pike_status_t pike_attention_block_workspace(pike_handle_t handle, const pike_tensor_t *x, const pike_epilogue_t *epi,
                                             size_t *bytes);
pike_status_t pike_attention_block(pike_handle_t handle, const pike_tensor_t *x, const pike_tensor_t *gamma,
                                   const pike_tensor_t *beta, const pike_tensor_t *w_qkv, const pike_tensor_t *b_qkv,
                                   const pike_tensor_t *w_o, const pike_tensor_t *b_o, const pike_epilogue_t *epi,
                                   pike_tensor_t *out, void *workspace, size_t workspace_bytes, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* PIKE_H_ */
