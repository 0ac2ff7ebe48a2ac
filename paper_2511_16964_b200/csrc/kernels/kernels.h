// Host-side launchers of the chain kernels (internal to the library).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

namespace pike {

// One kernel launch on `stream`.  With `pdl` the launch carries the programmatic-stream-serialisation attribute:
// the grid may be scheduled while the previous kernel in the stream is still running (its CTAs take the SMs that
// kernel's CTAs have left), which hides the launch latency and the prologue between the kernels of a chain and
// between calls.  Every kernel of this library executes griddepcontrol.wait before its first access to a global
// tensor, so the attribute is safe behind any predecessor.
template <typename... P, typename... A>
inline cudaError_t launch_kernel(void (*kern)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool pdl,
                                 A &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<A>(args)...);
}

enum : uint32_t {
    KID_GEMM = 1,
    KID_ATTN = 2,
    KID_LAYERNORM = 3,
    KID_FP32_CHAIN = 4,
};

// ---- fp32 CUDA-core chain: out = reduce(scale*act(x@w+b)+res) ------------------
struct Fp32ChainArgs {
    const float *x, *w, *bias, *residual, *gamma, *beta;
    float *out;
    int M, K, N;
    long long ldx, ldw, ldr, ldo;
    int w_is_nk;
    int act, reduce;
    float scale, eps;
    int pdl;        // launch with programmatic stream serialisation (see launch_kernel)
    unsigned int *status;            // device status word and the bound of the kernel's wait for its tiled copies
    unsigned long long limit_ns;
    int test_withhold_loads;         // test hook: the tiled copies are not issued, so the wait for them runs out
};
// How a problem is laid over the chip: rows per thread (1 = the split-k kernel for small problems, 8 rows per
// cluster; 2, 4 = 16 or 32 rows), 32 cw columns per CTA, cn CTAs per cluster, kc = k per staged chunk.  tma_x / tma_w:
// the split-k kernel fetches that operand through a tensor map (fp32, no swizzle, zero fill) with the box given
// here - x as {K, M} with box {kc, 8}, w [K,N] as {N, K} with box {32 cw, kc}; the caller encodes the maps, or
// clears the flag to fall back to per-thread copies.
struct Fp32ChainPlan {
    int rpt, cw, cn, kc;
    int tma_x, tma_w;
    uint32_t x_box[2], w_box[2];
};
Fp32ChainPlan plan_fp32_chain(const Fp32ChainArgs &a, int num_sms);
cudaError_t launch_fp32_chain(const Fp32ChainArgs &a, const Fp32ChainPlan &plan, const CUtensorMap *tm_x,
                              const CUtensorMap *tm_w, cudaStream_t stream);

// ---- once per device (with that device current): function attributes and launch limits ------------
// Each setup_* raises the dynamic shared-memory limit of its kernels on the current device, so that
// the launchers make no attribute call per launch, and reports what the launchers need to know.
cudaError_t setup_fp32_chain();
cudaError_t setup_gemm_bf16(int num_sms, int *max_clusters);   // CTA pairs the device holds at once
cudaError_t setup_row_kernels();
cudaError_t setup_attention_bf16(bool *regs_ok);               // false: compiled with too few registers for the in-kernel split

// ---- 16-bit (bf16 or f16) tcgen05 GEMM + epilogue --------------------------------
struct GemmArgs {
    int M, N, K;
    int w_is_nk;
    int f16;               // every 16-bit tensor (x, w and any 16-bit bias/residual/out) is IEEE half, not bf16
    const void *bias;      int bias_f32;
    const void *residual;  int residual_f32;  long long ldr;
    void *out;             int out_f32;       long long ldo;
    int act;
    float scale;
    int row_partials;      // per-(row, n-tile) pairs for a row reduction split across tiles: 0 none,
                           // 1 softmax (max, sum exp), 2 LayerNorm (mean, sum of squared deviations)
    float2 *partials;
    unsigned int *status;
    unsigned long long limit_ns;
    // grouped mode (group_offsets != nullptr): rows [group_offsets[e], group_offsets[e+1]) of A use weight
    // matrix e (third coordinate of the W tensor map) and bias row e; M is the total row count
    const int *group_offsets;  // device, num_groups + 1 ints
    int num_groups;
    // set by the launcher: the rasterisation (see tile_coords)
    int group_m;              // blocks per rasterisation group (row blocks, or column blocks if group_along_n)
    int group_along_n;        // 0: groups of row blocks, W streams; 1: groups of column blocks, A streams
    int test_withhold_loads;  // test hook: the producers issue no loads, so the first "full" wait runs out
    // one-pass logits + softmax kernel only
    unsigned int *stripe_counters;   // device, one per 256-row stripe, zero at launch
    int test_withhold_partials;      // test hook: block 0 never counts itself in, so every stripe wait runs out
    int pdl;                         // launch with programmatic stream serialisation (see launch_kernel); not for the one-pass kernel
    int alternate_k;                 // set by the launcher: a cluster walks k downwards on every other of its tiles
};
// A CTA pair computes a (2*GEMM_BM) x GEMM_BN tile; each CTA stages GEMM_BM rows of A and half of
// the tile's W columns.  Tensor-map boxes: A {GEMM_BK, GEMM_BM}; W as [N,K] {GEMM_BK, GEMM_BN/2};
// W as [K,N] {64, GEMM_BK}.
constexpr int GEMM_BM = 128, GEMM_BN = 256, GEMM_BK = 64;
cudaError_t launch_gemm_bf16(const CUtensorMap &tmA, const CUtensorMap &tmB, const GemmArgs &a, int max_clusters,
                             cudaStream_t stream);

// One-pass logits + softmax (gemm_softmax_onepass.cu): a.partials holds M * ceil(N/256) pairs, a.stripe_counters
// ceil(M/256) zeroed words; out is fp32.  Needs ceil(N/256) <= 2 * max_clusters (a stripe's tiles fit the chip's
// tensor memory); launched cooperatively with exactly max_clusters CTA pairs.
cudaError_t setup_gemm_softmax_onepass();
bool gemm_softmax_onepass_fits(int N, int max_clusters);
cudaError_t launch_gemm_softmax_onepass(const CUtensorMap &tmA, const CUtensorMap &tmB, const GemmArgs &a,
                                        int max_clusters, cudaStream_t stream);

// ---- row kernels -------------------------------------------------------------------
// z = LayerNorm(x) rows, 16-bit in/out (f16 != 0: IEEE half, else bf16), fp32 statistics; gamma/beta of
// the same 16-bit type or f32 or null.
// (status / limit_ns: the device status word and the bound of the kernel's waits for its row copies)
cudaError_t launch_layernorm_bf16(const void *x, long long ldx, void *z, long long ldz, const void *gamma,
                                  int gamma_f32, const void *beta, int beta_f32, float eps, int M, int D, int f16,
                                  unsigned int *status, unsigned long long limit_ns, int num_sms, cudaStream_t stream,
                                  bool pdl = false);
// p[m,:] = exp(v[m,:] - m_row) / l_row in place, (m_row, l_row) combined from the partials
// Pair t of row m sits at partials[m*pair_row_stride + t*pair_tile_stride] (pair_row_stride 0 = num_n_tiles,
// the layout the GEMM epilogue writes; {1, M} reads pairs stored [t][m], as an all-gather over GPUs lays them).
cudaError_t launch_softmax_finish(float *v, long long ldv, const float2 *partials, int num_n_tiles, int M, int N,
                                  cudaStream_t stream, long long pair_row_stride = 0, long long pair_tile_stride = 1,
                                  bool pdl = false);
// stats[m] = the row's per-tile (max, sum exp) pairs [M, num_n_tiles] folded into one pair
cudaError_t launch_softmax_row_stats(const float2 *partials, int num_n_tiles, float2 *stats, int M, cudaStream_t stream,
                                     bool pdl = false);

// out = (v - mean)/sqrt(var + eps)*gamma + beta in place (v 16-bit or f32), statistics combined from the
// per-(row, n-tile) (mean, sum of squared deviations) pairs; tile_n = columns per tile
cudaError_t launch_layernorm_finish(void *v, int out_f32, long long ldv, const float2 *partials, int num_n_tiles,
                                    int tile_n, int M, int N, const void *gamma, int gamma_f32, const void *beta,
                                    int beta_f32, float eps, int f16, cudaStream_t stream, bool pdl = false);

// ---- attention ---------------------------------------------------------------------
struct AttnArgs {
    int BH, H, S;   // BH = batch * H; tensor maps are 4-D {D, S or Sk, H, batch}
    int Sk, D;      // key/value length (== S unless cross attention) and head dimension (64 or 128)
    float scale;
    int causal;
    int f16;        // q, k, v and out are IEEE half instead of bf16
    void *out;      // 16-bit; element (b, h, s, d) at out + b*out_b + h*out_h + s*out_s + d
    long long out_b, out_h, out_s;
    unsigned int *status;
    unsigned long long limit_ns;
    int pdl;        // launch with programmatic stream serialisation (see launch_kernel)
};
cudaError_t launch_attention_bf16(const CUtensorMap &tmQ, const CUtensorMap &tmK, const CUtensorMap &tmV,
                                  const AttnArgs &a, int num_sms, bool regs_ok, cudaStream_t stream);

}  // namespace pike
