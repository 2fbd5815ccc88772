// Host-side cache object behind the opaque svlm_cache handle (private to the library).
#pragma once
#include <cuda_runtime.h>

#include <vector>

#include "svlm_dev.h"

struct svlm_cache {
    SvlmCacheDev dev;
    cudaStream_t stream = nullptr;
    int device = 0;
    std::vector<void*> allocs;
    long long appended = 0;       // tokens accepted by the host checks so far
    int pending_n = 0;            // n of the latest metadata append (layers 1.. must match)
    bool configured_locked = false;
    // staging for the *_host entry points
    void* stage = nullptr;
    size_t stage_bytes = 0;
};
