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
    unsigned wait_limit_host = 0;  // source buffer of svlm_debug_set_wait_limit's copy
    unsigned char* decode_tagged = nullptr;   // per-layer decode kernel: epochs and tagged records (device memory)
    // What the latest enqueued operation was, for the decode step's early loads: a decode of one layer
    // may start reading its pages while the previous kernel still runs only if that kernel was a decode
    // of another layer of this cache (which writes neither the metadata nor this layer's pages).
    int last_decode_layer = -1;   // layer of the latest operation if it was a single-layer decode, else -1
    int calls_since_decode = 0;   // library calls on this cache's stream since that decode that left the record alone (projections)
    int last_decode_batch = 0;    // how many caches that launch served, and the first of them
    const svlm_cache* last_decode_first = nullptr;
    SvlmCacheDev* dev_copy = nullptr;   // `dev` in device memory, for the batched kernels
    // staging for the *_host entry points
    void* stage = nullptr;
    size_t stage_bytes = 0;
    void* hstage = nullptr;       // page-locked host buffer: small inputs of a host-buffer call are gathered here for one copy
    size_t hstage_bytes = 0;
    // copy streams and per-layer events of the pipelined host-buffer chunk prefill (created on first use)
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_start = nullptr;
    std::vector<cudaEvent_t> ev_in, ev_done;
};
