// The library handle (internal): device properties, the status word, the tensor-map
// encoder entry point and the per-kernel timing state.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cudaTypedefs.h>

#include <vector>

#include "../../../include/pike.h"

struct pike_handle_s {
    int device;
    int num_sms;
    unsigned int *status;  // device, 4 words
    unsigned long long limit_ns;
    bool withhold_next;    // pike_test_withhold_loads: applies to the next bf16 GEMM launch only
    PFN_cuTensorMapEncodeTiled_v12000 encode;
    // per-kernel device timing (pike_profile_begin / pike_profile_end)
    bool profiling;
    std::vector<cudaEvent_t> ev_pool;                       // recycled events
    std::vector<cudaEvent_t> ev_start[PIKE_KERNEL_COUNT];
    std::vector<cudaEvent_t> ev_stop[PIKE_KERNEL_COUNT];
};
