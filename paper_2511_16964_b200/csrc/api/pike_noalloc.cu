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
//
// Validation, tensor maps, the launch itself and its profiling events are the same
// code the workspace entry point runs (validate.h, run_gemm): the two differ only in
// where the pairs live.
#include <string.h>

#include "../kernels/kernels.h"
#include "handle.h"
#include "validate.h"

using namespace pike_api;

namespace {

// Scratch for the split-row softmax.  In host code this name is only a handle for the
// runtime's symbol table, never a device address: its address on the handle's device is
// looked up with cudaGetSymbolAddress and that pointer is what the kernels receive.
static __device__ __align__(256) float2 g_noalloc_partials[PIKE_NOALLOC_MAX_PARTIALS];

// First call through a handle: resolve the array's address on the handle's device (which the
// caller has made current) and keep it in the handle.
pike_status_t scratch_of(pike_handle_t h, float2 **out)
{
    if (h->noalloc_partials == nullptr) {
        float2 *ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_noalloc_partials) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return PIKE_ERR_CUDA;
        }
        h->noalloc_partials = ptr;
    }
    *out = h->noalloc_partials;
    return PIKE_OK;
}

}  // namespace

extern "C" pike_status_t pike_linear_softmax_noalloc(pike_handle_t h, const pike_tensor_t *x, const pike_tensor_t *w,
                                                     const pike_tensor_t *bias, const pike_epilogue_t *epi,
                                                     pike_tensor_t *out, void *cuda_stream)
{
    if (h == nullptr || out == nullptr) return PIKE_ERR_NULL;
    LinearShape s;
    if (pike_status_t st = linear_shape(x, w, epi, s)) return st;
    if (x->dtype != PIKE_BF16) return PIKE_ERR_DTYPE;
    if (epi->reduce != PIKE_REDUCE_SOFTMAX || epi->out_dtype != PIKE_F32) return PIKE_ERR_UNSUPPORTED;
    if (s.M < 1) return PIKE_ERR_SHAPE;
    if (pike_status_t st = check_matrix(x, s.M, s.K)) return st;
    if (pike_status_t st = check_matrix(w, s.w_is_nk ? s.N : s.K, s.w_is_nk ? s.K : s.N)) return st;
    if (pike_status_t st = check_matrix(out, s.M, s.N)) return st;
    if (out->dtype != PIKE_F32) return PIKE_ERR_DTYPE;
    if (pike_status_t st = check_vector(bias, s.N)) return st;
    if (!side_ok(bias, PIKE_BF16)) return PIKE_ERR_DTYPE;
    for (const pike_tensor_t *t : {x, w, bias})
        if (overlaps(out, t)) return PIKE_ERR_UNSUPPORTED;

    // the built-in scratch has a fixed size: refuse what does not fit
    const int64_t num_n = (s.N + pike::GEMM_BN - 1) / pike::GEMM_BN;
    if (s.M * num_n > (int64_t)PIKE_NOALLOC_MAX_PARTIALS) return PIKE_ERR_WORKSPACE;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaSetDevice(h->device) != cudaSuccess) return PIKE_ERR_CUDA;
    float2 *partials = nullptr;
    if (pike_status_t st = scratch_of(h, &partials)) return st;
    if (pike_status_t st = run_gemm(h, x->data, x->stride[0], w, s.w_is_nk, s.M, s.K, s.N, bias, nullptr, false, 0,
                                    out->data, true, out->stride[0], (int)epi->act, epi->scale, partials, stream, 1))
        return st;
    return run_softmax_finish(h, out, partials, s.M, s.N, stream);
}
