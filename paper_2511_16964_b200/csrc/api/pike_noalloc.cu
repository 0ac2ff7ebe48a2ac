// pike_linear_softmax_noalloc: the bf16 logits + row-softmax chain for callers that
// must not allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits or unwanted -- a
// serving loop that has handed the whole device heap to its own pool allocator, a
// plugin called from inside another framework's execution step, a real-time thread
// that may not take the allocator's locks or an implicit device synchronisation.
// pike_linear_epilogue asks such callers for a workspace they have no way to get.
// Here the scratch (the per-row, per-column-tile (max, sum-exp) pairs of the split
// softmax) lives in a fixed array inside the library image instead, so the caller
// passes only inputs and the output.
//
// Consequences of a single built-in array, all of which the header repeats:
//  - it has a fixed capacity (PIKE_NOALLOC_MAX_PARTIALS pairs, 2 MiB) that every GPU
//    loading the library carries until the process exits; larger problems are refused;
//  - every call on a device uses the same array, so two calls that may overlap on the
//    GPU (different streams, no ordering between them) race on it;
//  - it keeps the previous call's contents.  Nothing has to be cleared: every pair the
//    normalising kernel reads is written by the GEMM kernel of the same call first.
#include <string.h>

#include "../kernels/kernels.h"
#include "handle.h"

namespace {

// Scratch for the split-row softmax.  In host code this name is only a handle for the
// runtime's symbol table, never a device address: its address is looked up once per
// device with cudaGetSymbolAddress and that pointer is what the kernels receive.
static __device__ __align__(256) float2 g_noalloc_partials[PIKE_NOALLOC_MAX_PARTIALS];

constexpr int MAX_DEVICES = 64;
float2 *g_partials_ptr[MAX_DEVICES];  // device address of g_noalloc_partials, per device (nullptr = not set up)

// First call on a device: resolve the array's device address with that device current.
pike_status_t scratch_for_device(int device, float2 **out)
{
    if (device < 0 || device >= MAX_DEVICES) return PIKE_ERR_UNSUPPORTED;
    if (g_partials_ptr[device] == nullptr) {
        float2 *ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_noalloc_partials) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return PIKE_ERR_CUDA;
        }
        g_partials_ptr[device] = ptr;
    }
    *out = g_partials_ptr[device];
    return PIKE_OK;
}

pike_status_t check_bf16_matrix(const pike_tensor_t *t, int64_t rows, int64_t cols, pike_dtype_t dtype)
{
    if (t == nullptr || t->data == nullptr) return PIKE_ERR_NULL;
    if (t->dtype != dtype) return PIKE_ERR_DTYPE;
    if (t->ndim != 2 || t->shape[0] != rows || t->shape[1] != cols) return PIKE_ERR_SHAPE;
    if (t->stride[1] != 1 || t->stride[0] < cols) return PIKE_ERR_STRIDE;
    const int64_t esz = dtype == PIKE_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(t->data) % 16 != 0 || (t->stride[0] * esz) % 16 != 0) return PIKE_ERR_ALIGNMENT;
    return PIKE_OK;
}

// rank 2 for the activations, rank 3 (one matrix) for the weights, as the GEMM kernel expects
pike_status_t encode_2d(pike_handle_t h, CUtensorMap *map, const void *ptr, uint64_t rows, uint64_t cols,
                        uint64_t pitch_elems, uint32_t box_cols, uint32_t box_rows, int rank = 2)
{
    const cuuint64_t dims[3] = {cols, rows, 1};
    const cuuint64_t strides[2] = {pitch_elems * 2, rows * pitch_elems * 2};
    const cuuint32_t box[3] = {box_cols, box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = h->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void *>(ptr), dims, strides, box,
                                 estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PIKE_OK : PIKE_ERR_CUDA;
}

bool ranges_overlap(const pike_tensor_t *a, const pike_tensor_t *b)
{
    auto span = [](const pike_tensor_t *t, uintptr_t &lo, uintptr_t &hi) {
        int64_t last = 0;
        for (int i = 0; i < t->ndim; ++i) last += (t->shape[i] - 1) * t->stride[i];
        lo = reinterpret_cast<uintptr_t>(t->data);
        hi = lo + (uintptr_t)(last + 1) * (t->dtype == PIKE_F32 ? 4 : 2);
    };
    uintptr_t alo, ahi, blo, bhi;
    span(a, alo, ahi);
    span(b, blo, bhi);
    return alo < bhi && blo < ahi;
}

}  // namespace

extern "C" pike_status_t pike_linear_softmax_noalloc(pike_handle_t h, const pike_tensor_t *x, const pike_tensor_t *w,
                                                     const pike_tensor_t *bias, const pike_epilogue_t *epi,
                                                     pike_tensor_t *out, void *cuda_stream)
{
    if (h == nullptr || x == nullptr || w == nullptr || epi == nullptr || out == nullptr) return PIKE_ERR_NULL;
    if (epi->struct_size != sizeof(pike_epilogue_t)) return PIKE_ERR_UNSUPPORTED;
    if (epi->reduce != PIKE_REDUCE_SOFTMAX || epi->out_dtype != PIKE_F32) return PIKE_ERR_UNSUPPORTED;
    if ((int)epi->act < 0 || (int)epi->act > 3 || !(epi->scale == epi->scale)) return PIKE_ERR_UNSUPPORTED;
    if (x->ndim != 2 || w->ndim != 2) return PIKE_ERR_SHAPE;
    const bool nk = (epi->flags & PIKE_FLAG_W_IS_NK) != 0;
    const int64_t M = x->shape[0], K = x->shape[1];
    const int64_t N = nk ? w->shape[0] : w->shape[1];
    if ((nk ? w->shape[1] : w->shape[0]) != K) return PIKE_ERR_SHAPE;
    if (M < 1 || K < 1 || N < 1) return PIKE_ERR_SHAPE;
    if (M > 0x7fffffff || K > 0x7fffffff || N > 0x7fffffff || K % 8 != 0 || N % 8 != 0) return PIKE_ERR_UNSUPPORTED;
    if (pike_status_t st = check_bf16_matrix(x, M, K, PIKE_BF16)) return st;
    if (pike_status_t st = check_bf16_matrix(w, nk ? N : K, nk ? K : N, PIKE_BF16)) return st;
    if (pike_status_t st = check_bf16_matrix(out, M, N, PIKE_F32)) return st;
    if (bias != nullptr) {
        if (bias->data == nullptr) return PIKE_ERR_NULL;
        if (bias->dtype != PIKE_BF16 && bias->dtype != PIKE_F32) return PIKE_ERR_DTYPE;
        if (bias->ndim != 1 || bias->shape[0] != N) return PIKE_ERR_SHAPE;
        if (bias->stride[0] != 1) return PIKE_ERR_STRIDE;
    }
    if (ranges_overlap(out, x) || ranges_overlap(out, w) || (bias != nullptr && ranges_overlap(out, bias)))
        return PIKE_ERR_UNSUPPORTED;

    // the built-in scratch has a fixed size: refuse what does not fit
    const int64_t num_n = (N + pike::GEMM_BN - 1) / pike::GEMM_BN;
    if (M * num_n > (int64_t)PIKE_NOALLOC_MAX_PARTIALS) return PIKE_ERR_WORKSPACE;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaSetDevice(h->device) != cudaSuccess) return PIKE_ERR_CUDA;
    float2 *partials = nullptr;
    if (pike_status_t st = scratch_for_device(h->device, &partials)) return st;

    CUtensorMap tmA, tmB;
    if (pike_status_t st = encode_2d(h, &tmA, x->data, (uint64_t)M, (uint64_t)K, (uint64_t)x->stride[0], pike::GEMM_BK,
                                     pike::GEMM_BM))
        return st;
    if (pike_status_t st = nk ? encode_2d(h, &tmB, w->data, (uint64_t)N, (uint64_t)K, (uint64_t)w->stride[0],
                                          pike::GEMM_BK, pike::GEMM_BN / 2, 3)
                              : encode_2d(h, &tmB, w->data, (uint64_t)K, (uint64_t)N, (uint64_t)w->stride[0], 64,
                                          pike::GEMM_BK, 3))
        return st;
    pike::GemmArgs g;
    memset(&g, 0, sizeof(g));
    g.M = (int)M; g.N = (int)N; g.K = (int)K;
    g.w_is_nk = nk ? 1 : 0;
    g.bias = bias ? bias->data : nullptr;
    g.bias_f32 = bias && bias->dtype == PIKE_F32;
    g.out = out->data; g.out_f32 = 1; g.ldo = out->stride[0];
    g.act = (int)epi->act; g.scale = epi->scale;
    g.row_partials = 1;
    g.partials = partials;
    g.status = h->status;
    g.limit_ns = h->limit_ns;
    if (pike::launch_gemm_bf16(tmA, tmB, g, h->num_sms, stream) != cudaSuccess) return PIKE_ERR_CUDA;
    if (pike::launch_softmax_finish(static_cast<float *>(out->data), out->stride[0], partials, (int)num_n, (int)M, (int)N,
                                    stream) != cudaSuccess)
        return PIKE_ERR_CUDA;
    return PIKE_OK;
}
