// Argument validation shared by every entry point of the C ABI (host code only).
#pragma once
#include <math.h>
#include <stdint.h>

#include "../../../include/pike.h"

namespace pike_api {

inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }
inline size_t elem_size(pike_dtype_t t) { return t == PIKE_F32 ? 4 : 2; }

inline bool valid_dtype(pike_dtype_t t) { return t == PIKE_F32 || t == PIKE_BF16 || t == PIKE_F16; }
inline bool is_16bit(pike_dtype_t t) { return t == PIKE_BF16 || t == PIKE_F16; }
// an optional side tensor of a 16-bit chain is fp32 or of the chain's own 16-bit type (bf16 and f16 never mix)
inline bool side_ok(const pike_tensor_t *t, pike_dtype_t chain) { return t == nullptr || t->dtype == PIKE_F32 || t->dtype == chain; }

// a dense-enough 2-D view: innermost stride 1, row pitch >= columns, 16-byte aligned base and pitch
inline pike_status_t check_matrix(const pike_tensor_t *t, int64_t rows, int64_t cols, bool pitch16 = true)
{
    if (t == nullptr) return PIKE_ERR_NULL;
    if (!valid_dtype(t->dtype)) return PIKE_ERR_DTYPE;
    if (t->ndim != 2 || t->shape[0] != rows || t->shape[1] != cols) return PIKE_ERR_SHAPE;
    if (rows == 0 || cols == 0) return PIKE_OK;  // an empty tensor may have no storage
    if (t->data == nullptr) return PIKE_ERR_NULL;
    if (t->stride[1] != 1 || t->stride[0] < cols) return PIKE_ERR_STRIDE;
    if (reinterpret_cast<uintptr_t>(t->data) % 16 != 0) return PIKE_ERR_ALIGNMENT;
    if (pitch16 && (t->stride[0] * (int64_t)elem_size(t->dtype)) % 16 != 0) return PIKE_ERR_ALIGNMENT;
    return PIKE_OK;
}

inline pike_status_t check_vector(const pike_tensor_t *t, int64_t n)
{
    if (t == nullptr) return PIKE_OK;  // optional
    if (t->data == nullptr) return PIKE_ERR_NULL;
    if (!valid_dtype(t->dtype)) return PIKE_ERR_DTYPE;
    if (t->ndim != 1 || t->shape[0] != n) return PIKE_ERR_SHAPE;
    if (t->stride[0] != 1) return PIKE_ERR_STRIDE;
    if (reinterpret_cast<uintptr_t>(t->data) % 16 != 0) return PIKE_ERR_ALIGNMENT;
    return PIKE_OK;
}

// [lo, hi): the bytes a tensor view can touch
inline void byte_range(const pike_tensor_t *t, uintptr_t &lo, uintptr_t &hi)
{
    int64_t last = 0;
    bool empty = false;
    for (int i = 0; i < t->ndim; ++i) {
        if (t->shape[i] <= 0) empty = true;
        last += (t->shape[i] - 1) * t->stride[i];
    }
    lo = reinterpret_cast<uintptr_t>(t->data);
    hi = empty ? lo : lo + (uintptr_t)(last + 1) * elem_size(t->dtype);
}

inline bool overlaps(const pike_tensor_t *a, const pike_tensor_t *b)
{
    if (a == nullptr || b == nullptr || a->data == nullptr || b->data == nullptr) return false;
    uintptr_t alo, ahi, blo, bhi;
    byte_range(a, alo, ahi);
    byte_range(b, blo, bhi);
    return alo < bhi && blo < ahi;
}

// does the tensor touch any of the `bytes` bytes at `p`? (a workspace against the call's tensors)
inline bool overlaps_bytes(const pike_tensor_t *t, const void *p, size_t bytes)
{
    if (t == nullptr || t->data == nullptr || p == nullptr || bytes == 0) return false;
    uintptr_t lo, hi;
    byte_range(t, lo, hi);
    const uintptr_t plo = reinterpret_cast<uintptr_t>(p);
    return lo < plo + bytes && plo < hi;
}

// A workspace of at least `need` bytes, 256-byte aligned, that none of the call's tensors touches.
inline pike_status_t check_workspace(const void *ws, size_t ws_bytes, size_t need, const pike_tensor_t *const *tensors,
                                     int count)
{
    if (need == 0) return PIKE_OK;
    if (ws == nullptr || reinterpret_cast<uintptr_t>(ws) % 256 != 0 || ws_bytes < need) return PIKE_ERR_WORKSPACE;
    for (int i = 0; i < count; ++i)
        if (overlaps_bytes(tensors[i], ws, need)) return PIKE_ERR_WORKSPACE;
    return PIKE_OK;
}

inline pike_status_t check_epilogue(const pike_epilogue_t *e)
{
    if (e == nullptr) return PIKE_ERR_NULL;
    if (e->struct_size != sizeof(pike_epilogue_t)) return PIKE_ERR_UNSUPPORTED;
    if ((int)e->act < 0 || (int)e->act > 3 || (int)e->reduce < 0 || (int)e->reduce > 2) return PIKE_ERR_UNSUPPORTED;
    if (!valid_dtype(e->out_dtype)) return PIKE_ERR_DTYPE;
    if (!isfinite(e->scale)) return PIKE_ERR_UNSUPPORTED;
    return PIKE_OK;
}

struct LinearShape {
    int64_t M, K, N;
    bool w_is_nk;
    bool fp32_path;
};

// shapes and dtypes of x, w and the descriptor of a linear chain (reads no data pointers)
inline pike_status_t linear_shape(const pike_tensor_t *x, const pike_tensor_t *w, const pike_epilogue_t *epi, LinearShape &s)
{
    if (x == nullptr || w == nullptr) return PIKE_ERR_NULL;
    if (pike_status_t st = check_epilogue(epi)) return st;
    if (x->ndim != 2 || w->ndim != 2) return PIKE_ERR_SHAPE;
    if (!valid_dtype(x->dtype) || x->dtype != w->dtype) return PIKE_ERR_DTYPE;
    s.w_is_nk = (epi->flags & PIKE_FLAG_W_IS_NK) != 0;
    s.M = x->shape[0];
    s.K = x->shape[1];
    s.N = s.w_is_nk ? w->shape[0] : w->shape[1];
    if ((s.w_is_nk ? w->shape[1] : w->shape[0]) != s.K) return PIKE_ERR_SHAPE;
    if (s.M < 0 || s.K < 1 || s.N < 1) return PIKE_ERR_SHAPE;
    if (s.M > 0x7fffffff || s.K > 0x7fffffff || s.N > 0x7fffffff) return PIKE_ERR_UNSUPPORTED;
    s.fp32_path = x->dtype == PIKE_F32;
    if (s.fp32_path) {
        if (s.N > 1024) return PIKE_ERR_UNSUPPORTED;
        if (epi->out_dtype != PIKE_F32) return PIKE_ERR_DTYPE;
    } else {
        if (s.K % 8 != 0 || s.N % 8 != 0) return PIKE_ERR_UNSUPPORTED;
        if (epi->out_dtype != PIKE_F32 && epi->out_dtype != x->dtype) return PIKE_ERR_DTYPE;
        if (epi->reduce == PIKE_REDUCE_SOFTMAX && epi->out_dtype != PIKE_F32) return PIKE_ERR_UNSUPPORTED;
    }
    return PIKE_OK;
}

}  // namespace pike_api
