// The library handle (internal): everything the library knows per device lives here - device
// properties, the launch limits of the kernels on that device, the status word, the tensor-map
// encoder entry point with a small cache of encoded maps, and the per-kernel timing state.
// Nothing per-device is kept in function-local or file-scope variables, so handles on different
// devices (or on different host threads) never see each other's values.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cudaTypedefs.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "../../../include/pike.h"

// A tensor map is a pure function of these fields, so an encoded map can be reused whenever they
// all match (same pointer, extents, pitches and box).
struct TensorMapKey {
    const void *ptr;
    uint64_t dims[4];
    uint64_t strides[3];   // bytes
    uint32_t box[4];
    uint32_t rank;
    uint32_t dtype;        // CUtensorMapDataType
};

struct pike_handle_s {
    int device;
    int num_sms;
    unsigned int *status;  // device, 4 words
    unsigned long long limit_ns;
    bool withhold_next;    // pike_test_withhold_loads: applies to the next bf16 GEMM or fp32 chain launch only
    bool withhold_partials_next;   // pike_test_withhold_partials: applies to the next one-pass softmax launch only
    PFN_cuTensorMapEncodeTiled_v12000 encode;
    cudaStream_t aux_stream;      // non-blocking; carries the status-word reads so that they wait for nobody's kernels
    // launch limits, filled by pike_create with the handle's device current
    int gemm_max_clusters;        // CTA pairs of the GEMM kernel the device holds at once
    bool attention_regs_ok;       // the attention kernels were compiled with the registers their setmaxnreg split needs
    float2 *noalloc_partials;     // device address of the built-in scratch of pike_linear_softmax_noalloc (set on its first call)
    bool log;                     // PIKE_LOG=1 in the environment at pike_create: one stderr line per kernel selection
    bool pdl;                     // launches carry the programmatic-stream-serialisation attribute (off with PIKE_PDL=0)
    // encoded tensor maps, most recent use first (a model calls the same few GEMMs on the same buffers over and over)
    static constexpr size_t MAP_CACHE_SIZE = 48;
    struct CachedMap { TensorMapKey key; CUtensorMap map; };
    std::vector<CachedMap> map_cache;
    // per-kernel device timing (pike_profile_begin / pike_profile_end)
    bool profiling;
    std::vector<cudaEvent_t> ev_pool;                       // recycled events
    std::vector<cudaEvent_t> ev_start[PIKE_KERNEL_COUNT];
    std::vector<cudaEvent_t> ev_stop[PIKE_KERNEL_COUNT];
};

namespace pike_api {

// Host-side kernel-selection log (PIKE_LOG=1): what was launched, on which shapes.  Never on unless asked for.
#define PIKE_LOGF(h, ...)                                  \
    do {                                                   \
        if ((h)->log) {                                    \
            fprintf(stderr, "[pike] " __VA_ARGS__);        \
            fputc('\n', stderr);                           \
        }                                                  \
    } while (0)

// Brackets one kernel launch with CUDA events on the caller's stream while profiling is on.
struct TimedLaunch {
    pike_handle_t h;
    pike_kernel_t kid;
    cudaStream_t stream;
    static cudaEvent_t get(pike_handle_t h)
    {
        cudaEvent_t e = nullptr;
        if (!h->ev_pool.empty()) { e = h->ev_pool.back(); h->ev_pool.pop_back(); }
        else if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); e = nullptr; }
        return e;
    }
    TimedLaunch(pike_handle_t h_, pike_kernel_t kid_, cudaStream_t s) : h(h_), kid(kid_), stream(s)
    {
        if (!h->profiling) return;
        cudaEvent_t e = get(h);
        if (e != nullptr) { cudaEventRecord(e, stream); h->ev_start[kid].push_back(e); }
    }
    ~TimedLaunch()
    {
        if (!h->profiling || h->ev_start[kid].size() == h->ev_stop[kid].size()) return;
        cudaEvent_t e = get(h);
        if (e != nullptr) { cudaEventRecord(e, stream); h->ev_stop[kid].push_back(e); }
        else { h->ev_pool.push_back(h->ev_start[kid].back()); h->ev_start[kid].pop_back(); }
    }
};

// Encode (or fetch from the handle's cache) a tiled tensor map: 128-byte swizzle over 16-bit elements, no swizzle
// over fp32 elements (the fp32 chain reads its tiles with plain shared-memory loads).
inline pike_status_t tensor_map(pike_handle_t h, CUtensorMap *out, const TensorMapKey &key)
{
    for (size_t i = 0; i < h->map_cache.size(); ++i) {
        if (memcmp(&h->map_cache[i].key, &key, sizeof(key)) == 0) {
            if (i != 0) {   // move to the front
                pike_handle_s::CachedMap hit = h->map_cache[i];
                h->map_cache.erase(h->map_cache.begin() + (long)i);
                h->map_cache.insert(h->map_cache.begin(), hit);
            }
            *out = h->map_cache[0].map;
            return PIKE_OK;
        }
    }
    cuuint64_t dims[4], strides[3];
    cuuint32_t box[4], estr[4] = {1, 1, 1, 1};
    for (int i = 0; i < 4; ++i) { dims[i] = key.dims[i]; box[i] = key.box[i]; }
    for (int i = 0; i < 3; ++i) strides[i] = key.strides[i];
    const CUresult r = h->encode(out, static_cast<CUtensorMapDataType>(key.dtype), key.rank, const_cast<void *>(key.ptr),
                                 dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                 key.dtype == CU_TENSOR_MAP_DATA_TYPE_FLOAT32 ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return PIKE_ERR_CUDA;
    if (h->map_cache.size() >= pike_handle_s::MAP_CACHE_SIZE) h->map_cache.pop_back();
    h->map_cache.insert(h->map_cache.begin(), pike_handle_s::CachedMap{key, *out});
    return PIKE_OK;
}

inline TensorMapKey make_key(const void *ptr, pike_dtype_t dt, uint32_t rank)
{
    TensorMapKey k;
    memset(&k, 0, sizeof(k));   // padding bytes too: keys are compared with memcmp
    k.ptr = ptr;
    k.rank = rank;
    k.dtype = dt == PIKE_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    return k;
}

// 16-bit [rows, cols] row-major matrix -> tensor map with a (box_cols x box_rows) box
inline pike_status_t make_map_2d(pike_handle_t h, CUtensorMap *map, pike_dtype_t dt, const void *ptr, uint64_t rows,
                                 uint64_t cols, uint64_t pitch_elems, uint32_t box_cols, uint32_t box_rows)
{
    TensorMapKey k = make_key(ptr, dt, 2);
    k.dims[0] = cols; k.dims[1] = rows;
    k.strides[0] = pitch_elems * 2;
    k.box[0] = box_cols; k.box[1] = box_rows;
    return tensor_map(h, map, k);
}

// fp32 [rows, cols] row-major matrix -> unswizzled tensor map with a (box_cols x box_rows) box
inline pike_status_t make_map_2d_f32(pike_handle_t h, CUtensorMap *map, const void *ptr, uint64_t rows, uint64_t cols,
                                     uint64_t pitch_elems, uint32_t box_cols, uint32_t box_rows)
{
    TensorMapKey k = make_key(ptr, PIKE_BF16, 2);
    k.dtype = CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    k.dims[0] = cols; k.dims[1] = rows;
    k.strides[0] = pitch_elems * 4;
    k.box[0] = box_cols; k.box[1] = box_rows;
    return tensor_map(h, map, k);
}

// 16-bit weights [groups, rows, cols] (dense matrices `group_pitch` elements apart; groups == 1 for a plain
// GEMM) -> 3-D map with a (box_cols x box_rows x 1) box
inline pike_status_t make_map_w(pike_handle_t h, CUtensorMap *map, pike_dtype_t dt, const void *ptr, uint64_t groups,
                                uint64_t rows, uint64_t cols, uint64_t pitch_elems, uint64_t group_pitch,
                                uint32_t box_cols, uint32_t box_rows)
{
    TensorMapKey k = make_key(ptr, dt, 3);
    k.dims[0] = cols; k.dims[1] = rows; k.dims[2] = groups;
    k.strides[0] = pitch_elems * 2;
    k.strides[1] = (groups > 1 ? group_pitch : rows * pitch_elems) * 2;
    k.box[0] = box_cols; k.box[1] = box_rows; k.box[2] = 1;
    return tensor_map(h, map, k);
}

// 16-bit attention operand, element (b, h, s, d) at ptr + b*sb + h*sh + s*ss + d (strides in elements, multiples
// of 8) -> 4-D map {D, S, H, B} with a (64 x 128 x 1 x 1) box
inline pike_status_t make_map_bhsd(pike_handle_t h, CUtensorMap *map, pike_dtype_t dt, const void *ptr, uint64_t B,
                                   uint64_t H, uint64_t S, uint64_t D, uint64_t sb, uint64_t sh, uint64_t ss)
{
    TensorMapKey k = make_key(ptr, dt, 4);
    k.dims[0] = D; k.dims[1] = S; k.dims[2] = H; k.dims[3] = B;
    k.strides[0] = ss * 2; k.strides[1] = sh * 2; k.strides[2] = sb * 2;
    k.box[0] = 64; k.box[1] = 128; k.box[2] = 1; k.box[3] = 1;
    return tensor_map(h, map, k);
}

// Defined in pike_api.cu, shared with the other translation units of the API.
// One 16-bit GEMM + epilogue launch (tensor maps from the handle's cache, profiling events, test hook); the
// caller has validated every tensor.  partials_mode: 1 softmax pairs, 2 LayerNorm pairs (used if partials != null).
pike_status_t run_gemm(pike_handle_t h, const void *a_ptr, int64_t lda, const pike_tensor_t *w, bool w_is_nk, int64_t M,
                       int64_t K, int64_t N, const pike_tensor_t *bias, const void *res_ptr, bool res_f32, int64_t ldr,
                       void *out_ptr, bool out_f32, int64_t ldo, int act, float scale, float2 *partials,
                       cudaStream_t stream, int partials_mode = 1, const int *group_offsets = nullptr, int num_groups = 0);
// The one-pass logits + softmax kernel (PIKE_FLAG_ONE_PASS); `workspace` holds the pairs, then the stripe counters.
size_t onepass_workspace_bytes(int64_t M, int64_t N);
pike_status_t run_gemm_softmax_onepass(pike_handle_t h, const pike_tensor_t *x, const pike_tensor_t *w, bool w_is_nk,
                                       int64_t M, int64_t K, int64_t N, const pike_tensor_t *bias,
                                       const pike_tensor_t *residual, pike_tensor_t *out, int act, float scale,
                                       void *workspace, cudaStream_t stream);
pike_status_t run_softmax_finish(pike_handle_t h, pike_tensor_t *out, const float2 *partials, int64_t M, int64_t N,
                                 cudaStream_t stream);

}  // namespace pike_api
