// C ABI of the library: argument validation, TMA tensor-map encoding, kernel
// selection and launch.  Host code only; every arithmetic step runs in the kernels.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cudaTypedefs.h>
#include <math.h>
#include <string.h>

#include <new>
#include <vector>

#include "../../../include/pike.h"
#include "../kernels/kernels.h"

#include "handle.h"

#include "validate.h"

using namespace pike_api;

namespace {

constexpr unsigned long long DEFAULT_LIMIT_NS = 2000000000ull;

size_t softmax_partials_bytes(const LinearShape &s)
{
    const int64_t num_n = (s.N + pike::GEMM_BN - 1) / pike::GEMM_BN;
    return align256((size_t)s.M * (size_t)num_n * sizeof(float2));
}

}  // namespace

namespace pike_api {

// Launch one 16-bit GEMM + epilogue; w's dtype (bf16 or f16) is the chain's.  All tensors validated by the caller.
pike_status_t run_gemm(pike_handle_t h, const void *a_ptr, int64_t lda, const pike_tensor_t *w, bool w_is_nk, int64_t M,
                       int64_t K, int64_t N, const pike_tensor_t *bias, const void *res_ptr, bool res_f32, int64_t ldr,
                       void *out_ptr, bool out_f32, int64_t ldo, int act, float scale, float2 *partials,
                       cudaStream_t stream, int partials_mode, const int *group_offsets, int num_groups)
{
    CUtensorMap tmA, tmB;
    if (pike_status_t st = make_map_2d(h, &tmA, w->dtype, a_ptr, (uint64_t)M, (uint64_t)K, (uint64_t)lda, pike::GEMM_BK, pike::GEMM_BM))
        return st;
    // w is [K,N] / [N,K], or [groups,K,N] / [groups,N,K] in grouped mode (the last two dimensions are the matrix)
    const int wd = w->ndim - 2;
    const uint64_t groups = wd == 1 ? (uint64_t)w->shape[0] : 1, gpitch = wd == 1 ? (uint64_t)w->stride[0] : 0;
    if (w_is_nk) {
        if (pike_status_t st = make_map_w(h, &tmB, w->dtype, w->data, groups, (uint64_t)N, (uint64_t)K, (uint64_t)w->stride[wd],
                                          gpitch, pike::GEMM_BK, pike::GEMM_BN / 2))
            return st;
    } else {
        if (pike_status_t st = make_map_w(h, &tmB, w->dtype, w->data, groups, (uint64_t)K, (uint64_t)N, (uint64_t)w->stride[wd],
                                          gpitch, 64, pike::GEMM_BK))
            return st;
    }
    pike::GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.pdl = h->pdl ? 1 : 0;
    g.M = (int)M; g.N = (int)N; g.K = (int)K;
    g.w_is_nk = w_is_nk ? 1 : 0;
    g.f16 = w->dtype == PIKE_F16 ? 1 : 0;
    g.bias = bias ? bias->data : nullptr;
    g.bias_f32 = bias && bias->dtype == PIKE_F32;
    g.residual = res_ptr; g.residual_f32 = res_f32 ? 1 : 0; g.ldr = ldr;
    g.out = out_ptr; g.out_f32 = out_f32 ? 1 : 0; g.ldo = ldo;
    g.act = act; g.scale = scale;
    g.row_partials = partials == nullptr ? 0 : partials_mode;
    g.group_offsets = group_offsets;
    g.num_groups = num_groups;
    g.partials = partials;
    g.status = h->status;
    g.limit_ns = h->limit_ns;
    g.test_withhold_loads = h->withhold_next ? 1 : 0;
    h->withhold_next = false;
    PIKE_LOGF(h, "gemm_bf16_kernel M=%lld K=%lld N=%lld %s w=%s act=%d out=%s%s%s partials=%d groups=%d clusters<=%d",
              (long long)M, (long long)K, (long long)N, g.f16 ? "f16" : "bf16", w_is_nk ? "[N,K]" : "[K,N]", act,
              out_f32 ? "f32" : "16-bit", bias ? " +bias" : "", res_ptr ? " +residual" : "", g.row_partials, num_groups,
              h->gemm_max_clusters);
    TimedLaunch timed(h, PIKE_KERNEL_GEMM_BF16, stream);
    return pike::launch_gemm_bf16(tmA, tmB, g, h->gemm_max_clusters, stream) == cudaSuccess ? PIKE_OK : PIKE_ERR_CUDA;
}

size_t onepass_workspace_bytes(int64_t M, int64_t N)
{
    const int64_t num_n = (N + pike::GEMM_BN - 1) / pike::GEMM_BN, stripes = (M + 2 * pike::GEMM_BM - 1) / (2 * pike::GEMM_BM);
    return align256((size_t)M * (size_t)num_n * sizeof(float2)) + align256((size_t)stripes * sizeof(unsigned int));
}

pike_status_t run_gemm_softmax_onepass(pike_handle_t h, const pike_tensor_t *x, const pike_tensor_t *w, bool w_is_nk,
                                       int64_t M, int64_t K, int64_t N, const pike_tensor_t *bias,
                                       const pike_tensor_t *residual, pike_tensor_t *out, int act, float scale,
                                       void *workspace, cudaStream_t stream)
{
    CUtensorMap tmA, tmB;
    if (pike_status_t st = make_map_2d(h, &tmA, w->dtype, x->data, (uint64_t)M, (uint64_t)K, (uint64_t)x->stride[0],
                                       pike::GEMM_BK, pike::GEMM_BM))
        return st;
    if (pike_status_t st = w_is_nk ? make_map_w(h, &tmB, w->dtype, w->data, 1, (uint64_t)N, (uint64_t)K, (uint64_t)w->stride[0],
                                                0, pike::GEMM_BK, pike::GEMM_BN / 2)
                                   : make_map_w(h, &tmB, w->dtype, w->data, 1, (uint64_t)K, (uint64_t)N, (uint64_t)w->stride[0],
                                                0, 64, pike::GEMM_BK))
        return st;
    const int64_t num_n = (N + pike::GEMM_BN - 1) / pike::GEMM_BN, stripes = (M + 2 * pike::GEMM_BM - 1) / (2 * pike::GEMM_BM);
    pike::GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.M = (int)M; g.N = (int)N; g.K = (int)K;
    g.w_is_nk = w_is_nk ? 1 : 0;
    g.f16 = w->dtype == PIKE_F16 ? 1 : 0;
    g.bias = bias ? bias->data : nullptr;
    g.bias_f32 = bias && bias->dtype == PIKE_F32;
    g.residual = residual ? residual->data : nullptr;
    g.residual_f32 = residual && residual->dtype == PIKE_F32;
    g.ldr = residual ? residual->stride[0] : 0;
    g.out = out->data; g.out_f32 = 1; g.ldo = out->stride[0];
    g.act = act; g.scale = scale;
    g.row_partials = 1;
    g.partials = static_cast<float2 *>(workspace);
    g.stripe_counters = reinterpret_cast<unsigned int *>(static_cast<uint8_t *>(workspace) +
                                                         align256((size_t)M * (size_t)num_n * sizeof(float2)));
    g.status = h->status;
    g.limit_ns = h->limit_ns;
    g.test_withhold_loads = h->withhold_next ? 1 : 0;
    g.test_withhold_partials = h->withhold_partials_next ? 1 : 0;
    h->withhold_next = h->withhold_partials_next = false;
    // the counters start at zero for every launch (a memset node on the caller's stream, no allocation)
    if (cudaMemsetAsync(g.stripe_counters, 0, (size_t)stripes * sizeof(unsigned int), stream) != cudaSuccess) return PIKE_ERR_CUDA;
    PIKE_LOGF(h, "gemm_softmax_onepass_kernel M=%lld K=%lld N=%lld stripes=%lld tiles_per_stripe=%lld clusters=%d (cooperative)",
              (long long)M, (long long)K, (long long)N, (long long)stripes, (long long)num_n, h->gemm_max_clusters);
    TimedLaunch timed(h, PIKE_KERNEL_GEMM_BF16, stream);
    return pike::launch_gemm_softmax_onepass(tmA, tmB, g, h->gemm_max_clusters, stream) == cudaSuccess ? PIKE_OK : PIKE_ERR_CUDA;
}

// Second half of the split-row softmax: combine the per-tile pairs, normalise `out` in place.
pike_status_t run_softmax_finish(pike_handle_t h, pike_tensor_t *out, const float2 *partials, int64_t M, int64_t N,
                                 cudaStream_t stream)
{
    const int num_n = (int)((N + pike::GEMM_BN - 1) / pike::GEMM_BN);
    PIKE_LOGF(h, "softmax_finish_kernel M=%lld N=%lld pairs_per_row=%d", (long long)M, (long long)N, num_n);
    TimedLaunch timed(h, PIKE_KERNEL_SOFTMAX_FINISH, stream);
    return pike::launch_softmax_finish(static_cast<float *>(out->data), out->stride[0], partials, num_n, (int)M, (int)N,
                                       stream, 0, 1, h->pdl) == cudaSuccess ? PIKE_OK : PIKE_ERR_CUDA;
}

}  // namespace pike_api

extern "C" {

const char *pike_status_string(pike_status_t s)
{
    switch (s) {
    case PIKE_OK:              return "ok";
    case PIKE_ERR_NULL:        return "a required pointer is NULL";
    case PIKE_ERR_SHAPE:       return "tensor ranks or extents do not fit together";
    case PIKE_ERR_DTYPE:       return "dtype combination not accepted";
    case PIKE_ERR_ALIGNMENT:   return "base pointer or row pitch is not 16-byte aligned";
    case PIKE_ERR_STRIDE:      return "innermost stride is not 1 or the layout is not dense enough";
    case PIKE_ERR_UNSUPPORTED: return "request is outside the implemented envelope";
    case PIKE_ERR_WORKSPACE:   return "workspace is NULL, misaligned or too small";
    case PIKE_ERR_ARCH:        return "device is not compute capability 10.x (sm_100)";
    case PIKE_ERR_CUDA:        return "a CUDA runtime or driver call failed";
    case PIKE_ERR_TIMEOUT:     return "a bounded in-kernel wait ran out";
    }
    return "unknown status";
}

pike_status_t pike_create(pike_handle_t *handle, int device)
{
    if (handle == nullptr) return PIKE_ERR_NULL;
    *handle = nullptr;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { cudaGetLastError(); return PIKE_ERR_CUDA; }
    if (prop.major != 10) return PIKE_ERR_ARCH;
    if (cudaSetDevice(device) != cudaSuccess) return PIKE_ERR_CUDA;
    pike_handle_s *h = new (std::nothrow) pike_handle_s();
    if (h == nullptr) return PIKE_ERR_CUDA;
    h->device = device;
    h->num_sms = prop.multiProcessorCount;
    h->limit_ns = DEFAULT_LIMIT_NS;
    h->profiling = false;
    h->withhold_next = false;
    h->withhold_partials_next = false;
    {
        const char *env = getenv("PIKE_LOG");
        h->log = env != nullptr && env[0] != '\0' && env[0] != '0';
        env = getenv("PIKE_PDL");
        h->pdl = !(env != nullptr && env[0] == '0');
    }
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || fn == nullptr) {
        delete h;
        return PIKE_ERR_CUDA;
    }
    h->encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
    h->status = nullptr;
    h->aux_stream = nullptr;
    h->noalloc_partials = nullptr;
    h->map_cache.reserve(pike_handle_s::MAP_CACHE_SIZE);
    // per-device kernel set-up, once, here: shared-memory limits of every kernel on this device and the launch
    // limits the launchers need, so that no launch pays for an attribute call or reads a process-wide variable
    if (pike::setup_fp32_chain() != cudaSuccess || pike::setup_gemm_bf16(h->num_sms, &h->gemm_max_clusters) != cudaSuccess ||
        pike::setup_gemm_softmax_onepass() != cudaSuccess ||
        pike::setup_row_kernels() != cudaSuccess || pike::setup_attention_bf16(&h->attention_regs_ok) != cudaSuccess ||
        cudaStreamCreateWithFlags(&h->aux_stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaMalloc(&h->status, 4 * sizeof(unsigned int)) != cudaSuccess ||
        cudaMemset(h->status, 0, 4 * sizeof(unsigned int)) != cudaSuccess) {
        cudaGetLastError();
        if (h->status != nullptr) cudaFree(h->status);
        if (h->aux_stream != nullptr) cudaStreamDestroy(h->aux_stream);
        delete h;
        return PIKE_ERR_CUDA;
    }
    *handle = h;
    return PIKE_OK;
}

pike_status_t pike_destroy(pike_handle_t h)
{
    if (h == nullptr) return PIKE_ERR_NULL;
    cudaFree(h->status);
    cudaStreamDestroy(h->aux_stream);
    for (int k = 0; k < PIKE_KERNEL_COUNT; ++k) {
        for (cudaEvent_t e : h->ev_start[k]) cudaEventDestroy(e);
        for (cudaEvent_t e : h->ev_stop[k]) cudaEventDestroy(e);
    }
    for (cudaEvent_t e : h->ev_pool) cudaEventDestroy(e);
    delete h;
    return PIKE_OK;
}

pike_status_t pike_profile_begin(pike_handle_t h)
{
    if (h == nullptr) return PIKE_ERR_NULL;
    for (int k = 0; k < PIKE_KERNEL_COUNT; ++k) {
        for (cudaEvent_t e : h->ev_start[k]) h->ev_pool.push_back(e);
        for (cudaEvent_t e : h->ev_stop[k]) h->ev_pool.push_back(e);
        h->ev_start[k].clear();
        h->ev_stop[k].clear();
    }
    h->profiling = true;
    return PIKE_OK;
}

pike_status_t pike_profile_end(pike_handle_t h, pike_kernel_profile_t *out)
{
    if (h == nullptr || out == nullptr) return PIKE_ERR_NULL;
    h->profiling = false;
    if (cudaDeviceSynchronize() != cudaSuccess) return PIKE_ERR_CUDA;
    pike_status_t rc = PIKE_OK;
    for (int k = 0; k < PIKE_KERNEL_COUNT; ++k) {
        out[k].launches = h->ev_stop[k].size();
        out[k].device_ms = 0.0;
        for (size_t i = 0; i < h->ev_stop[k].size(); ++i) {
            float ms = 0.0f;
            if (cudaEventElapsedTime(&ms, h->ev_start[k][i], h->ev_stop[k][i]) != cudaSuccess) rc = PIKE_ERR_CUDA;
            out[k].device_ms += ms;
        }
        for (cudaEvent_t e : h->ev_start[k]) h->ev_pool.push_back(e);
        for (cudaEvent_t e : h->ev_stop[k]) h->ev_pool.push_back(e);
        h->ev_start[k].clear();
        h->ev_stop[k].clear();
    }
    return rc;
}

pike_status_t pike_get_last_device_status(pike_handle_t h, pike_status_t *status, uint32_t *where)
{
    if (h == nullptr || status == nullptr) return PIKE_ERR_NULL;
    unsigned int host[4] = {0, 0, 0, 0};
    // The read (and the clearing write) travel on the handle's own non-blocking stream: they wait for no
    // kernel of the caller, who has synchronised the streams whose status is of interest beforehand.
    if (cudaMemcpyAsync(host, h->status, sizeof(host), cudaMemcpyDeviceToHost, h->aux_stream) != cudaSuccess ||
        cudaStreamSynchronize(h->aux_stream) != cudaSuccess)
        return PIKE_ERR_CUDA;
    if (host[0] != 0 && (cudaMemsetAsync(h->status, 0, sizeof(host), h->aux_stream) != cudaSuccess ||
                         cudaStreamSynchronize(h->aux_stream) != cudaSuccess))
        return PIKE_ERR_CUDA;
    *status = host[0] != 0 ? PIKE_ERR_TIMEOUT : PIKE_OK;
    if (where != nullptr) *where = host[0];
    return PIKE_OK;
}

pike_status_t pike_set_wait_limit_ns(pike_handle_t h, uint64_t ns)
{
    if (h == nullptr) return PIKE_ERR_NULL;
    h->limit_ns = ns == 0 ? DEFAULT_LIMIT_NS : ns;
    return PIKE_OK;
}

pike_status_t pike_test_withhold_loads(pike_handle_t h)
{
    if (h == nullptr) return PIKE_ERR_NULL;
    h->withhold_next = true;
    return PIKE_OK;
}

pike_status_t pike_test_withhold_partials(pike_handle_t h)
{
    if (h == nullptr) return PIKE_ERR_NULL;
    h->withhold_partials_next = true;
    return PIKE_OK;
}

pike_status_t pike_linear_epilogue_workspace(pike_handle_t h, const pike_tensor_t *x, const pike_tensor_t *w,
                                             const pike_epilogue_t *epi, size_t *bytes)
{
    if (h == nullptr || bytes == nullptr) return PIKE_ERR_NULL;
    LinearShape s;
    if (pike_status_t st = linear_shape(x, w, epi, s)) return st;
    const bool one_pass = (epi->flags & PIKE_FLAG_ONE_PASS) != 0;
    if (one_pass) {
        if (s.fp32_path || epi->reduce != PIKE_REDUCE_SOFTMAX) return PIKE_ERR_UNSUPPORTED;
        if (!pike::gemm_softmax_onepass_fits((int)s.N, h->gemm_max_clusters)) return PIKE_ERR_UNSUPPORTED;
        *bytes = onepass_workspace_bytes(s.M, s.N);
        return PIKE_OK;
    }
    *bytes = (!s.fp32_path && epi->reduce != PIKE_REDUCE_NONE) ? softmax_partials_bytes(s) : 0;
    return PIKE_OK;
}

pike_status_t pike_linear_epilogue(pike_handle_t h, const pike_tensor_t *x, const pike_tensor_t *w,
                                   const pike_tensor_t *bias, const pike_tensor_t *residual,
                                   const pike_tensor_t *gamma, const pike_tensor_t *beta, const pike_epilogue_t *epi,
                                   pike_tensor_t *out, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (h == nullptr || out == nullptr) return PIKE_ERR_NULL;
    LinearShape s;
    if (pike_status_t st = linear_shape(x, w, epi, s)) return st;
    const bool p16 = !s.fp32_path;  // the fp32 kernel uses scalar accesses: any row pitch is fine
    if (pike_status_t st = check_matrix(x, s.M, s.K, p16)) return st;
    if (pike_status_t st = check_matrix(w, s.w_is_nk ? s.N : s.K, s.w_is_nk ? s.K : s.N, p16)) return st;
    if (pike_status_t st = check_matrix(out, s.M, s.N, p16)) return st;
    if (out->dtype != epi->out_dtype) return PIKE_ERR_DTYPE;
    if (pike_status_t st = check_vector(bias, s.N)) return st;
    if (pike_status_t st = check_vector(gamma, s.N)) return st;
    if (pike_status_t st = check_vector(beta, s.N)) return st;
    if (residual != nullptr)
        if (pike_status_t st = check_matrix(residual, s.M, s.N, p16)) return st;
    const pike_tensor_t *ins[6] = {x, w, bias, residual, gamma, beta};
    for (const pike_tensor_t *t : ins)
        if (overlaps(out, t)) return PIKE_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaSetDevice(h->device) != cudaSuccess) return PIKE_ERR_CUDA;
    if (s.M == 0) return PIKE_OK;

    if (s.fp32_path) {
        for (const pike_tensor_t *t : {bias, residual, gamma, beta})
            if (t != nullptr && t->dtype != PIKE_F32) return PIKE_ERR_DTYPE;
        pike::Fp32ChainArgs a;
        memset(&a, 0, sizeof(a));
        a.pdl = h->pdl ? 1 : 0;
        a.x = static_cast<const float *>(x->data);
        a.w = static_cast<const float *>(w->data);
        a.bias = bias ? static_cast<const float *>(bias->data) : nullptr;
        a.residual = residual ? static_cast<const float *>(residual->data) : nullptr;
        a.gamma = gamma ? static_cast<const float *>(gamma->data) : nullptr;
        a.beta = beta ? static_cast<const float *>(beta->data) : nullptr;
        a.out = static_cast<float *>(out->data);
        a.M = (int)s.M; a.K = (int)s.K; a.N = (int)s.N;
        a.ldx = x->stride[0]; a.ldw = w->stride[0]; a.ldr = residual ? residual->stride[0] : 0; a.ldo = out->stride[0];
        a.w_is_nk = s.w_is_nk;
        a.act = (int)epi->act; a.reduce = (int)epi->reduce;
        a.scale = epi->scale; a.eps = epi->eps;
        a.status = h->status; a.limit_ns = h->limit_ns;
        a.test_withhold_loads = h->withhold_next ? 1 : 0;
        h->withhold_next = false;
        PIKE_LOGF(h, "fp32_chain_kernel M=%d K=%d N=%d act=%d reduce=%d w=%s", a.M, a.K, a.N, a.act, a.reduce,
                  a.w_is_nk ? "[N,K]" : "[K,N]");
        pike::Fp32ChainPlan plan = pike::plan_fp32_chain(a, h->num_sms);
        CUtensorMap tm_x, tm_w;
        // a map that cannot be encoded (a pitch beyond the format's range, say) only means per-thread copies
        if (plan.tma_x && make_map_2d_f32(h, &tm_x, a.x, (uint64_t)a.M, (uint64_t)a.K, (uint64_t)a.ldx, plan.x_box[0],
                                          plan.x_box[1]) != PIKE_OK)
            plan.tma_x = 0;
        if (plan.tma_w && make_map_2d_f32(h, &tm_w, a.w, (uint64_t)a.K, (uint64_t)a.N, (uint64_t)a.ldw, plan.w_box[0],
                                          plan.w_box[1]) != PIKE_OK)
            plan.tma_w = 0;
        PIKE_LOGF(h, "fp32_chain plan rows/thread=%d cols/cta=%d cluster=%d kc=%d tiled x=%d w=%d", plan.rpt, 32 * plan.cw,
                  plan.cn, plan.kc, plan.tma_x, plan.tma_w);
        TimedLaunch timed(h, PIKE_KERNEL_FP32_CHAIN, stream);
        return pike::launch_fp32_chain(a, plan, &tm_x, &tm_w, stream) == cudaSuccess ? PIKE_OK : PIKE_ERR_CUDA;
    }

    for (const pike_tensor_t *t : {bias, residual, gamma, beta})
        if (!side_ok(t, x->dtype)) return PIKE_ERR_DTYPE;
    if (epi->flags & PIKE_FLAG_ONE_PASS) {
        // the softmax in one kernel: a stripe's logits stay in tensor memory until its statistics are known
        if (epi->reduce != PIKE_REDUCE_SOFTMAX) return PIKE_ERR_UNSUPPORTED;
        if (!pike::gemm_softmax_onepass_fits((int)s.N, h->gemm_max_clusters)) return PIKE_ERR_UNSUPPORTED;
        const pike_tensor_t *all[5] = {x, w, bias, residual, out};
        if (pike_status_t st = check_workspace(workspace, workspace_bytes, onepass_workspace_bytes(s.M, s.N), all, 5)) return st;
        return run_gemm_softmax_onepass(h, x, w, s.w_is_nk, s.M, s.K, s.N, bias, residual, out, (int)epi->act, epi->scale,
                                        workspace, stream);
    }
    // a row reduction on this path is split across the GEMM's column tiles: per-(row, tile) pairs go to the
    // workspace, a second kernel combines them and finishes the rows in place
    float2 *partials = nullptr;
    if (epi->reduce != PIKE_REDUCE_NONE) {
        const pike_tensor_t *all[7] = {x, w, bias, residual, gamma, beta, out};
        if (pike_status_t st = check_workspace(workspace, workspace_bytes, softmax_partials_bytes(s), all, 7)) return st;
        partials = static_cast<float2 *>(workspace);
    }
    const bool layernorm = epi->reduce == PIKE_REDUCE_LAYERNORM;
    if (pike_status_t st = run_gemm(h, x->data, x->stride[0], w, s.w_is_nk, s.M, s.K, s.N, bias,
                                    residual ? residual->data : nullptr, residual && residual->dtype == PIKE_F32,
                                    residual ? residual->stride[0] : 0, out->data, out->dtype == PIKE_F32,
                                    out->stride[0], (int)epi->act, epi->scale, partials, stream, layernorm ? 2 : 1))
        return st;
    if (partials != nullptr) {
        const int num_n = (int)((s.N + pike::GEMM_BN - 1) / pike::GEMM_BN);
        if (layernorm) {
            TimedLaunch timed(h, PIKE_KERNEL_LAYERNORM_BF16, stream);
            if (pike::launch_layernorm_finish(out->data, out->dtype == PIKE_F32, out->stride[0], partials, num_n,
                                              pike::GEMM_BN, (int)s.M, (int)s.N, gamma ? gamma->data : nullptr,
                                              gamma && gamma->dtype == PIKE_F32, beta ? beta->data : nullptr,
                                              beta && beta->dtype == PIKE_F32, epi->eps, x->dtype == PIKE_F16,
                                              stream, h->pdl) != cudaSuccess)
                return PIKE_ERR_CUDA;
        } else {
            return run_softmax_finish(h, out, partials, s.M, s.N, stream);
        }
    }
    return PIKE_OK;
}

// Validation shared by the two halves of the column-sharded softmax.
static pike_status_t shard_shape(const pike_tensor_t *x, const pike_tensor_t *w, const pike_epilogue_t *epi,
                                 LinearShape &s)
{
    if (pike_status_t st = linear_shape(x, w, epi, s)) return st;
    if (s.fp32_path) return PIKE_ERR_DTYPE;
    if (epi->reduce != PIKE_REDUCE_SOFTMAX || epi->out_dtype != PIKE_F32) return PIKE_ERR_UNSUPPORTED;
    return PIKE_OK;
}

pike_status_t pike_linear_softmax_shard_workspace(pike_handle_t h, const pike_tensor_t *x, const pike_tensor_t *w,
                                                  const pike_epilogue_t *epi, size_t *bytes)
{
    if (h == nullptr || bytes == nullptr) return PIKE_ERR_NULL;
    LinearShape s;
    if (pike_status_t st = shard_shape(x, w, epi, s)) return st;
    *bytes = softmax_partials_bytes(s);
    return PIKE_OK;
}

pike_status_t pike_linear_softmax_shard_local(pike_handle_t h, const pike_tensor_t *x, const pike_tensor_t *w,
                                              const pike_tensor_t *bias, const pike_epilogue_t *epi,
                                              pike_tensor_t *out, float *row_stats, void *workspace,
                                              size_t workspace_bytes, void *cuda_stream)
{
    if (h == nullptr || out == nullptr || row_stats == nullptr) return PIKE_ERR_NULL;
    LinearShape s;
    if (pike_status_t st = shard_shape(x, w, epi, s)) return st;
    if (pike_status_t st = check_matrix(x, s.M, s.K)) return st;
    if (pike_status_t st = check_matrix(w, s.w_is_nk ? s.N : s.K, s.w_is_nk ? s.K : s.N)) return st;
    if (pike_status_t st = check_matrix(out, s.M, s.N)) return st;
    if (out->dtype != PIKE_F32) return PIKE_ERR_DTYPE;
    if (pike_status_t st = check_vector(bias, s.N)) return st;
    if (!side_ok(bias, x->dtype)) return PIKE_ERR_DTYPE;
    if (reinterpret_cast<uintptr_t>(row_stats) % 8 != 0) return PIKE_ERR_ALIGNMENT;
    for (const pike_tensor_t *t : {x, w, bias})
        if (overlaps(out, t)) return PIKE_ERR_UNSUPPORTED;
    {
        const pike_tensor_t *all[4] = {x, w, bias, out};
        if (pike_status_t st = check_workspace(workspace, workspace_bytes, softmax_partials_bytes(s), all, 4)) return st;
        if (s.M > 0 && overlaps_bytes(out, row_stats, (size_t)s.M * 8)) return PIKE_ERR_UNSUPPORTED;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaSetDevice(h->device) != cudaSuccess) return PIKE_ERR_CUDA;
    if (s.M == 0) return PIKE_OK;
    float2 *partials = static_cast<float2 *>(workspace);
    if (pike_status_t st = run_gemm(h, x->data, x->stride[0], w, s.w_is_nk, s.M, s.K, s.N, bias, nullptr, false, 0,
                                    out->data, true, out->stride[0], (int)epi->act, epi->scale, partials, stream, 1))
        return st;
    const int num_n = (int)((s.N + pike::GEMM_BN - 1) / pike::GEMM_BN);
    TimedLaunch timed(h, PIKE_KERNEL_SOFTMAX_FINISH, stream);
    return pike::launch_softmax_row_stats(partials, num_n, reinterpret_cast<float2 *>(row_stats), (int)s.M,
                                          stream, h->pdl) == cudaSuccess ? PIKE_OK : PIKE_ERR_CUDA;
}

pike_status_t pike_linear_softmax_shard_finish(pike_handle_t h, pike_tensor_t *out, const float *all_stats,
                                               int32_t num_shards, void *cuda_stream)
{
    if (h == nullptr || out == nullptr || all_stats == nullptr) return PIKE_ERR_NULL;
    if (num_shards < 1) return PIKE_ERR_SHAPE;
    if (out->ndim != 2 || out->shape[0] < 0 || out->shape[1] < 1) return PIKE_ERR_SHAPE;
    if (out->shape[0] > 0x7fffffff || out->shape[1] > 0x7fffffff) return PIKE_ERR_UNSUPPORTED;
    if (out->shape[1] % 8 != 0) return PIKE_ERR_UNSUPPORTED;
    if (pike_status_t st = check_matrix(out, out->shape[0], out->shape[1])) return st;
    if (out->dtype != PIKE_F32) return PIKE_ERR_DTYPE;
    if (reinterpret_cast<uintptr_t>(all_stats) % 8 != 0) return PIKE_ERR_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaSetDevice(h->device) != cudaSuccess) return PIKE_ERR_CUDA;
    const int64_t M = out->shape[0];
    if (M == 0) return PIKE_OK;
    TimedLaunch timed(h, PIKE_KERNEL_SOFTMAX_FINISH, stream);
    // pair of (row m, shard r) at all_stats[(r*M + m)*2]: row stride 1 pair, "tile" stride M pairs
    return pike::launch_softmax_finish(static_cast<float *>(out->data), out->stride[0],
                                       reinterpret_cast<const float2 *>(all_stats), (int)num_shards, (int)M,
                                       (int)out->shape[1], stream, 1, M, h->pdl) == cudaSuccess ? PIKE_OK : PIKE_ERR_CUDA;
}

pike_status_t pike_grouped_linear_epilogue(pike_handle_t h, const pike_tensor_t *x, const pike_tensor_t *w,
                                           const pike_tensor_t *bias, const pike_tensor_t *residual,
                                           const int32_t *group_offsets, const pike_epilogue_t *epi, pike_tensor_t *out,
                                           void *cuda_stream)
{
    if (h == nullptr || x == nullptr || w == nullptr || out == nullptr || group_offsets == nullptr) return PIKE_ERR_NULL;
    if (pike_status_t st = check_epilogue(epi)) return st;
    if (x->ndim != 2 || w->ndim != 3) return PIKE_ERR_SHAPE;
    if (!is_16bit(x->dtype) || w->dtype != x->dtype) return PIKE_ERR_DTYPE;
    if (epi->out_dtype != PIKE_F32 && epi->out_dtype != x->dtype) return PIKE_ERR_DTYPE;
    if (!side_ok(bias, x->dtype) || !side_ok(residual, x->dtype)) return PIKE_ERR_DTYPE;
    if (epi->reduce != PIKE_REDUCE_NONE) return PIKE_ERR_UNSUPPORTED;
    const bool nk = (epi->flags & PIKE_FLAG_W_IS_NK) != 0;
    const int64_t T = x->shape[0], K = x->shape[1], G = w->shape[0];
    const int64_t N = nk ? w->shape[1] : w->shape[2];
    if ((nk ? w->shape[2] : w->shape[1]) != K) return PIKE_ERR_SHAPE;
    if (T < 0 || K < 1 || N < 1 || G < 1) return PIKE_ERR_SHAPE;
    if (T > 0x7fffffff || K > 0x7fffffff || N > 0x7fffffff || G > 65536 || K % 8 != 0 || N % 8 != 0)
        return PIKE_ERR_UNSUPPORTED;
    if (pike_status_t st = check_matrix(x, T, K)) return st;
    if (pike_status_t st = check_matrix(out, T, N)) return st;
    if (out->dtype != epi->out_dtype) return PIKE_ERR_DTYPE;
    if (residual != nullptr)
        if (pike_status_t st = check_matrix(residual, T, N)) return st;
    // weights: G dense matrices, innermost stride 1, 16-byte aligned pitches
    if (w->data == nullptr) return PIKE_ERR_NULL;
    if (w->stride[2] != 1 || w->stride[1] < w->shape[2] || w->stride[0] < w->shape[1] * w->stride[1]) return PIKE_ERR_STRIDE;
    if (reinterpret_cast<uintptr_t>(w->data) % 16 != 0 || (w->stride[1] * 2) % 16 != 0 || (w->stride[0] * 2) % 16 != 0)
        return PIKE_ERR_ALIGNMENT;
    if (bias != nullptr) {
        if (bias->data == nullptr) return PIKE_ERR_NULL;
        if (!valid_dtype(bias->dtype)) return PIKE_ERR_DTYPE;
        if (bias->ndim != 2 || bias->shape[0] != G || bias->shape[1] != N) return PIKE_ERR_SHAPE;
        if (bias->stride[1] != 1 || bias->stride[0] != N) return PIKE_ERR_STRIDE;
    }
    const pike_tensor_t *ins[4] = {x, w, bias, residual};
    for (const pike_tensor_t *t : ins)
        if (overlaps(out, t)) return PIKE_ERR_UNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaSetDevice(h->device) != cudaSuccess) return PIKE_ERR_CUDA;
    if (T == 0) return PIKE_OK;
    return run_gemm(h, x->data, x->stride[0], w, nk, T, K, N, bias, residual ? residual->data : nullptr,
                    residual && residual->dtype == PIKE_F32, residual ? residual->stride[0] : 0, out->data,
                    out->dtype == PIKE_F32, out->stride[0], (int)epi->act, epi->scale, nullptr, stream, 0, group_offsets,
                    (int)G);
}

static pike_status_t mlp_shape(const pike_tensor_t *x, const pike_tensor_t *w1, const pike_epilogue_t *epi, int64_t &M,
                               int64_t &D, int64_t &F, bool &nk)
{
    if (x == nullptr || w1 == nullptr) return PIKE_ERR_NULL;
    if (pike_status_t st = check_epilogue(epi)) return st;
    if (x->ndim != 2 || w1->ndim != 2) return PIKE_ERR_SHAPE;
    if (!is_16bit(x->dtype) || w1->dtype != x->dtype || epi->out_dtype != x->dtype) return PIKE_ERR_DTYPE;
    if (epi->reduce != PIKE_REDUCE_NONE || epi->scale != 1.0f) return PIKE_ERR_UNSUPPORTED;
    nk = (epi->flags & PIKE_FLAG_W_IS_NK) != 0;
    M = x->shape[0];
    D = x->shape[1];
    F = nk ? w1->shape[0] : w1->shape[1];
    if ((nk ? w1->shape[1] : w1->shape[0]) != D) return PIKE_ERR_SHAPE;
    if (M < 0 || D < 1 || F < 1) return PIKE_ERR_SHAPE;
    if (D % 8 != 0 || F % 8 != 0 || D > 16384) return PIKE_ERR_UNSUPPORTED;
    if (M > 0x7fffffff || F > 0x7fffffff) return PIKE_ERR_UNSUPPORTED;
    return PIKE_OK;
}

pike_status_t pike_mlp_block_workspace(pike_handle_t h, const pike_tensor_t *x, const pike_tensor_t *w1,
                                       const pike_epilogue_t *epi, size_t *bytes)
{
    if (h == nullptr || bytes == nullptr) return PIKE_ERR_NULL;
    int64_t M, D, F;
    bool nk;
    if (pike_status_t st = mlp_shape(x, w1, epi, M, D, F, nk)) return st;
    *bytes = align256((size_t)M * D * 2) + align256((size_t)M * F * 2);
    return PIKE_OK;
}

pike_status_t pike_mlp_block(pike_handle_t h, const pike_tensor_t *x, const pike_tensor_t *gamma,
                             const pike_tensor_t *beta, const pike_tensor_t *w1, const pike_tensor_t *b1,
                             const pike_tensor_t *w2, const pike_tensor_t *b2, const pike_epilogue_t *epi,
                             pike_tensor_t *out, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (h == nullptr || out == nullptr || w2 == nullptr) return PIKE_ERR_NULL;
    int64_t M, D, F;
    bool nk;
    if (pike_status_t st = mlp_shape(x, w1, epi, M, D, F, nk)) return st;
    if (pike_status_t st = check_matrix(x, M, D)) return st;
    if (pike_status_t st = check_matrix(w1, nk ? F : D, nk ? D : F)) return st;
    if (pike_status_t st = check_matrix(w2, nk ? D : F, nk ? F : D)) return st;
    if (pike_status_t st = check_matrix(out, M, D)) return st;
    if (w2->dtype != x->dtype || out->dtype != x->dtype) return PIKE_ERR_DTYPE;
    for (const pike_tensor_t *t : {gamma, beta, b1, b2})
        if (!side_ok(t, x->dtype)) return PIKE_ERR_DTYPE;
    if (pike_status_t st = check_vector(gamma, D)) return st;
    if (pike_status_t st = check_vector(beta, D)) return st;
    if (pike_status_t st = check_vector(b1, F)) return st;
    if (pike_status_t st = check_vector(b2, D)) return st;
    const pike_tensor_t *ins[7] = {x, gamma, beta, w1, b1, w2, b2};
    for (const pike_tensor_t *t : ins)
        if (overlaps(out, t)) return PIKE_ERR_UNSUPPORTED;
    const size_t z_bytes = align256((size_t)M * D * 2), h_bytes = align256((size_t)M * F * 2);
    if (M > 0) {
        const pike_tensor_t *all[8] = {x, gamma, beta, w1, b1, w2, b2, out};
        if (pike_status_t st = check_workspace(workspace, workspace_bytes, z_bytes + h_bytes, all, 8)) return st;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaSetDevice(h->device) != cudaSuccess) return PIKE_ERR_CUDA;
    if (M == 0) return PIKE_OK;

    void *z = workspace;
    void *hbuf = static_cast<uint8_t *>(workspace) + z_bytes;
    {
        TimedLaunch timed(h, PIKE_KERNEL_LAYERNORM_BF16, stream);
        if (pike::launch_layernorm_bf16(x->data, x->stride[0], z, D, gamma ? gamma->data : nullptr,
                                        gamma && gamma->dtype == PIKE_F32, beta ? beta->data : nullptr,
                                        beta && beta->dtype == PIKE_F32, epi->eps, (int)M, (int)D,
                                        x->dtype == PIKE_F16, h->status, h->limit_ns, h->num_sms, stream,
                                        h->pdl) != cudaSuccess)
            return PIKE_ERR_CUDA;
    }
    // h = act(z @ w1 + b1), rounded to the chain's 16-bit type
    if (pike_status_t st = run_gemm(h, z, D, w1, nk, M, D, F, b1, nullptr, false, 0, hbuf, false, F, (int)epi->act,
                                    1.0f, nullptr, stream))
        return st;
    // out = h @ w2 + b2 + x
    return run_gemm(h, hbuf, F, w2, nk, M, F, D, b2, x->data, false, x->stride[0], out->data, false, out->stride[0],
                    PIKE_ACT_NONE, 1.0f, nullptr, stream);
}

static pike_status_t attn_shape(const pike_tensor_t *q, const pike_epilogue_t *epi)
{
    if (q == nullptr) return PIKE_ERR_NULL;
    if (pike_status_t st = check_epilogue(epi)) return st;
    if (q->ndim != 4) return PIKE_ERR_SHAPE;
    if (!is_16bit(q->dtype) || epi->out_dtype != q->dtype) return PIKE_ERR_DTYPE;
    if (q->shape[3] != 128 && q->shape[3] != 64) return PIKE_ERR_UNSUPPORTED;
    if (q->shape[0] < 0 || q->shape[1] < 0 || q->shape[2] < 0) return PIKE_ERR_SHAPE;
    if (q->shape[0] * q->shape[1] > 0x7fffff || q->shape[2] > 0x7fffff00) return PIKE_ERR_UNSUPPORTED;
    if (!(epi->scale > 0.0f)) return PIKE_ERR_UNSUPPORTED;
    if (epi->act != PIKE_ACT_NONE || epi->reduce != PIKE_REDUCE_NONE) return PIKE_ERR_UNSUPPORTED;
    return PIKE_OK;
}

static pike_status_t check_bhsd(const pike_tensor_t *t, const pike_tensor_t *like, bool own_length = false)
{
    if (t == nullptr) return PIKE_ERR_NULL;
    if (t->dtype != like->dtype) return PIKE_ERR_DTYPE;
    if (t->ndim != 4) return PIKE_ERR_SHAPE;
    for (int i = 0; i < 4; ++i)
        if (t->shape[i] != like->shape[i] && !(own_length && i == 2)) return PIKE_ERR_SHAPE;   // keys may have their own length
    if (t->shape[0] * t->shape[1] * t->shape[2] == 0) return PIKE_OK;  // empty: no storage needed
    if (t->data == nullptr) return PIKE_ERR_NULL;
    // any [B,H,S,D] view whose rows are contiguous and whose other strides keep 16-byte alignment
    // (dense [B,H,S,D], [B,S,H,D] seen as [B,H,S,D], a slice of a packed qkv buffer, ...)
    if (t->stride[3] != 1) return PIKE_ERR_STRIDE;
    for (int i = 0; i < 3; ++i)
        if (t->shape[i] > 1 && (t->stride[i] < t->shape[3] || t->stride[i] % 8 != 0)) return PIKE_ERR_STRIDE;
    if (reinterpret_cast<uintptr_t>(t->data) % 16 != 0) return PIKE_ERR_ALIGNMENT;
    return PIKE_OK;
}

// stride of dimension i, or a harmless multiple of 16 bytes when the extent is 1
static uint64_t eff_stride(const pike_tensor_t *t, int i) { return t->shape[i] > 1 ? (uint64_t)t->stride[i] : 128u; }

static pike_status_t run_attention(pike_handle_t h, const pike_tensor_t *q, const pike_tensor_t *k, const pike_tensor_t *v,
                                   const pike_tensor_t *out, float scale, bool causal, cudaStream_t stream)
{
    const uint64_t B = q->shape[0], H = q->shape[1], S = q->shape[2], Sk = k->shape[2], D = q->shape[3];
    CUtensorMap tmQ, tmK, tmV;
    if (pike_status_t st = make_map_bhsd(h, &tmQ, q->dtype, q->data, B, H, S, D, eff_stride(q, 0), eff_stride(q, 1), eff_stride(q, 2))) return st;
    if (pike_status_t st = make_map_bhsd(h, &tmK, q->dtype, k->data, B, H, Sk, D, eff_stride(k, 0), eff_stride(k, 1), eff_stride(k, 2))) return st;
    if (pike_status_t st = make_map_bhsd(h, &tmV, q->dtype, v->data, B, H, Sk, D, eff_stride(v, 0), eff_stride(v, 1), eff_stride(v, 2))) return st;
    pike::AttnArgs a;
    memset(&a, 0, sizeof(a));
    a.pdl = h->pdl ? 1 : 0;
    a.BH = (int)(B * H); a.H = (int)H; a.S = (int)S; a.Sk = (int)Sk; a.D = (int)D;
    a.scale = scale;
    a.causal = causal ? 1 : 0;
    a.f16 = q->dtype == PIKE_F16 ? 1 : 0;
    a.out = out->data;
    a.out_b = (long long)eff_stride(out, 0); a.out_h = (long long)eff_stride(out, 1); a.out_s = (long long)eff_stride(out, 2);
    a.status = h->status;
    a.limit_ns = h->limit_ns;
    PIKE_LOGF(h, "attention_bf16_kernel B*H=%d S=%d Sk=%d D=%d %s%s scale=%g", a.BH, a.S, a.Sk, a.D, a.f16 ? "f16" : "bf16",
              causal ? " causal" : "", (double)scale);
    TimedLaunch timed(h, PIKE_KERNEL_ATTENTION_BF16, stream);
    return pike::launch_attention_bf16(tmQ, tmK, tmV, a, h->num_sms, h->attention_regs_ok, stream) == cudaSuccess
               ? PIKE_OK : PIKE_ERR_CUDA;
}

pike_status_t pike_attention_chain_workspace(pike_handle_t h, const pike_tensor_t *q, const pike_epilogue_t *epi,
                                             size_t *bytes)
{
    if (h == nullptr || bytes == nullptr) return PIKE_ERR_NULL;
    if (pike_status_t st = attn_shape(q, epi)) return st;
    *bytes = 0;
    return PIKE_OK;
}

pike_status_t pike_attention_chain(pike_handle_t h, const pike_tensor_t *q, const pike_tensor_t *k,
                                   const pike_tensor_t *v, const pike_epilogue_t *epi, pike_tensor_t *out,
                                   void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    (void)workspace;
    (void)workspace_bytes;
    if (h == nullptr) return PIKE_ERR_NULL;
    if (pike_status_t st = attn_shape(q, epi)) return st;
    if (pike_status_t st = check_bhsd(q, q)) return st;
    if (pike_status_t st = check_bhsd(k, q, true)) return st;
    if (pike_status_t st = check_bhsd(v, k)) return st;
    if (pike_status_t st = check_bhsd(out, q)) return st;
    // keys of another length (cross attention) have no causal alignment with the queries
    if (k->shape[2] != q->shape[2] && (epi->flags & PIKE_FLAG_CAUSAL)) return PIKE_ERR_UNSUPPORTED;
    if (k->shape[2] > 0x7fffff00) return PIKE_ERR_UNSUPPORTED;
    const pike_tensor_t *ins[3] = {q, k, v};
    for (const pike_tensor_t *t : ins)
        if (overlaps(out, t)) return PIKE_ERR_UNSUPPORTED;
    const int64_t BH = q->shape[0] * q->shape[1], S = q->shape[2];
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaSetDevice(h->device) != cudaSuccess) return PIKE_ERR_CUDA;
    if (BH == 0 || S == 0) return PIKE_OK;
    if (k->shape[2] == 0) return PIKE_ERR_SHAPE;               // a softmax over no keys is undefined
    return run_attention(h, q, k, v, out, epi->scale, (epi->flags & PIKE_FLAG_CAUSAL) != 0, stream);
}

static pike_status_t block_shape(const pike_tensor_t *x, const pike_epilogue_t *epi, int64_t &B, int64_t &S, int64_t &E)
{
    if (x == nullptr) return PIKE_ERR_NULL;
    if (pike_status_t st = check_epilogue(epi)) return st;
    if (x->ndim != 3) return PIKE_ERR_SHAPE;
    if (!is_16bit(x->dtype) || epi->out_dtype != x->dtype) return PIKE_ERR_DTYPE;
    B = x->shape[0]; S = x->shape[1]; E = x->shape[2];
    if (B < 0 || S < 0 || E < 1) return PIKE_ERR_SHAPE;
    if (E % 128 != 0 || E > 4096) return PIKE_ERR_UNSUPPORTED;          // heads of 128; LayerNorm row in one warp
    if (B * S > 0x7fffffff || B * (E / 128) > 0x7fffff) return PIKE_ERR_UNSUPPORTED;
    if (!(epi->scale > 0.0f)) return PIKE_ERR_UNSUPPORTED;
    if (epi->act != PIKE_ACT_NONE || epi->reduce != PIKE_REDUCE_NONE) return PIKE_ERR_UNSUPPORTED;
    return PIKE_OK;
}

static pike_status_t check_dense_bse(const pike_tensor_t *t, pike_dtype_t dt, int64_t B, int64_t S, int64_t E)
{
    if (t == nullptr) return PIKE_ERR_NULL;
    if (t->dtype != dt) return PIKE_ERR_DTYPE;
    if (t->ndim != 3 || t->shape[0] != B || t->shape[1] != S || t->shape[2] != E) return PIKE_ERR_SHAPE;
    if (B * S == 0) return PIKE_OK;
    if (t->data == nullptr) return PIKE_ERR_NULL;
    if (t->stride[2] != 1 || (S > 1 && t->stride[1] != E) || (B > 1 && t->stride[0] != S * E)) return PIKE_ERR_STRIDE;
    if (reinterpret_cast<uintptr_t>(t->data) % 16 != 0) return PIKE_ERR_ALIGNMENT;
    return PIKE_OK;
}

pike_status_t pike_attention_block_workspace(pike_handle_t h, const pike_tensor_t *x, const pike_epilogue_t *epi,
                                             size_t *bytes)
{
    if (h == nullptr || bytes == nullptr) return PIKE_ERR_NULL;
    int64_t B, S, E;
    if (pike_status_t st = block_shape(x, epi, B, S, E)) return st;
    const size_t M = (size_t)(B * S);
    *bytes = 2 * align256(M * E * 2) + align256(M * 3 * E * 2);
    return PIKE_OK;
}

pike_status_t pike_attention_block(pike_handle_t h, const pike_tensor_t *x, const pike_tensor_t *gamma,
                                   const pike_tensor_t *beta, const pike_tensor_t *w_qkv, const pike_tensor_t *b_qkv,
                                   const pike_tensor_t *w_o, const pike_tensor_t *b_o, const pike_epilogue_t *epi,
                                   pike_tensor_t *out, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (h == nullptr || w_qkv == nullptr || w_o == nullptr || out == nullptr) return PIKE_ERR_NULL;
    int64_t B, S, E;
    if (pike_status_t st = block_shape(x, epi, B, S, E)) return st;
    const bool nk = (epi->flags & PIKE_FLAG_W_IS_NK) != 0;
    if (pike_status_t st = check_dense_bse(x, x->dtype, B, S, E)) return st;
    if (pike_status_t st = check_dense_bse(out, x->dtype, B, S, E)) return st;
    if (w_qkv->dtype != x->dtype || w_o->dtype != x->dtype) return PIKE_ERR_DTYPE;
    for (const pike_tensor_t *t : {gamma, beta, b_qkv, b_o})
        if (!side_ok(t, x->dtype)) return PIKE_ERR_DTYPE;
    if (pike_status_t st = check_matrix(w_qkv, nk ? 3 * E : E, nk ? E : 3 * E)) return st;
    if (pike_status_t st = check_matrix(w_o, E, E)) return st;
    if (pike_status_t st = check_vector(gamma, E)) return st;
    if (pike_status_t st = check_vector(beta, E)) return st;
    if (pike_status_t st = check_vector(b_qkv, 3 * E)) return st;
    if (pike_status_t st = check_vector(b_o, E)) return st;
    const pike_tensor_t *ins[7] = {x, gamma, beta, w_qkv, b_qkv, w_o, b_o};
    for (const pike_tensor_t *t : ins)
        if (overlaps(out, t)) return PIKE_ERR_UNSUPPORTED;
    const int64_t M = B * S, H = E / 128;
    const size_t z_bytes = align256((size_t)M * E * 2), qkv_bytes = align256((size_t)M * 3 * E * 2);
    if (M > 0) {
        const pike_tensor_t *all[8] = {x, gamma, beta, w_qkv, b_qkv, w_o, b_o, out};
        if (pike_status_t st = check_workspace(workspace, workspace_bytes, 2 * z_bytes + qkv_bytes, all, 8)) return st;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaSetDevice(h->device) != cudaSuccess) return PIKE_ERR_CUDA;
    if (M == 0) return PIKE_OK;

    uint8_t *ws = static_cast<uint8_t *>(workspace);
    void *z = ws, *qkv = ws + z_bytes, *att = ws + z_bytes + qkv_bytes;
    {   // z = LayerNorm(x)
        TimedLaunch timed(h, PIKE_KERNEL_LAYERNORM_BF16, stream);
        if (pike::launch_layernorm_bf16(x->data, E, z, E, gamma ? gamma->data : nullptr, gamma && gamma->dtype == PIKE_F32,
                                        beta ? beta->data : nullptr, beta && beta->dtype == PIKE_F32, epi->eps, (int)M,
                                        (int)E, x->dtype == PIKE_F16, h->status, h->limit_ns, h->num_sms, stream,
                                        h->pdl) != cudaSuccess)
            return PIKE_ERR_CUDA;
    }
    // qkv = z @ w_qkv + b_qkv, laid out [B, S, 3, H, 128]
    if (pike_status_t st = run_gemm(h, z, E, w_qkv, nk, M, E, 3 * E, b_qkv, nullptr, false, 0, qkv, false, 3 * E,
                                    PIKE_ACT_NONE, 1.0f, nullptr, stream))
        return st;
    // attention straight on the packed buffer: q, k, v are [B,H,S,128] views of it, the result is written as [B,S,H,128]
    pike_tensor_t view[4];
    for (int i = 0; i < 4; ++i) {
        view[i].dtype = x->dtype;
        view[i].ndim = 4;
        view[i].shape[0] = B; view[i].shape[1] = H; view[i].shape[2] = S; view[i].shape[3] = 128;
        view[i].stride[3] = 1; view[i].stride[1] = 128;
        if (i < 3) {
            view[i].data = static_cast<uint16_t *>(qkv) + (int64_t)i * E;
            view[i].stride[0] = S * 3 * E; view[i].stride[2] = 3 * E;
        } else {
            view[i].data = att;
            view[i].stride[0] = S * E; view[i].stride[2] = E;
        }
    }
    if (pike_status_t st = run_attention(h, &view[0], &view[1], &view[2], &view[3], epi->scale,
                                         (epi->flags & PIKE_FLAG_CAUSAL) != 0, stream))
        return st;
    // out = x + att @ w_o + b_o
    return run_gemm(h, att, E, w_o, nk, M, E, E, b_o, x->data, false, E, out->data, false, E, PIKE_ACT_NONE, 1.0f, nullptr,
                    stream);
}

}  // extern "C"
