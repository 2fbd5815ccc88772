// Host-side launchers of the kernels (one translation unit per kernel family).
#pragma once
#include <cuda_runtime.h>

#include <atomic>

#include "svlm_dev.h"

void svlm_count_launch();

// Raises a kernel's dynamic shared-memory limit, once per device (the attribute belongs to the device's
// context) and safe to call from several host threads.  The current device is the one the launch goes to.
template <auto Kernel>
cudaError_t svlm_allow_smem(size_t bytes) {
    static std::atomic<unsigned long long> done{0};   // one bit per device, one word per kernel instantiation
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 64 && ((done.load(std::memory_order_acquire) >> dev) & 1ull)) return cudaSuccess;
    e = cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess && dev < 64) done.fetch_or(1ull << dev, std::memory_order_release);
    return e;
}

// metadata (svlm_meta.cu)
void svlm_launch_append_meta(const SvlmCacheDev& cd, const unsigned char* types, const int* pos, int n, cudaStream_t st);
void svlm_launch_evict_meta(const SvlmCacheDev& cd, cudaStream_t st);
// batched forms, one block per cache: types [n_caches][n], pos [n_caches][n](x3)
void svlm_launch_append_meta_batch(const SvlmCacheList& list, const unsigned char* types, const int* pos, int n,
                                   cudaStream_t st);
void svlm_launch_evict_meta_batch(const SvlmCacheList& list, cudaStream_t st);

// key/value movement (svlm_kv.cu)
// layer < 0: K,V are [layers][n][kv_heads][d]; otherwise [n][kv_heads][d] for that layer.
void svlm_launch_kv_write(const SvlmCacheDev& cd, int layer, const void* K, const void* V, int n, cudaStream_t st);
void svlm_launch_evict_rotate(const SvlmCacheDev& cd, cudaStream_t st);
// every cache of the list has the geometry of geom
void svlm_launch_evict_rotate_batch(const SvlmCacheList& list, const SvlmCacheDev& geom, cudaStream_t st);

// attention (svlm_attend_simple.cu)
// Q, out: [n_caches][n_layers][n_q][q_heads][d]; q_pos: [n_caches][n_q](x3)
void svlm_launch_attend_simple(const SvlmAttendBatch& b, int layer0, int n_layers, const void* Q, const int* q_pos,
                               int n_q, int q_heads, void* out, cudaStream_t st);

// split-KV decode, n_q = 1 (svlm_decode.cu)
size_t svlm_decode_ws_floats(int layers_in_launch, int kv_heads, int head_dim, int splits);
int svlm_decode_splits(int n_pages, int kv_heads, int problems);
// The kernel keeps the list of active pages in shared memory: caches with more pages take the general kernel.
bool svlm_decode_supported(int n_pages);
// Knew/Vnew non-null: fused decode step, the latest appended token's key and value ([caches*layers][kv_heads][d],
// un-rotated) are written to the cache by this launch.  early_loads != 0: the caller vouches that no kernel
// enqueued since the one before the previous launch on this stream wrote this cache's metadata or the pages of the
// layers attended here, so the kernel may read them before the previous kernel has finished.
// early_loads == 2: moreover that previous kernel was itself a decode step of this cache (the per-layer kernel then
// paces its read-ahead, one unit's worth per warp at a time).
// tagged: the cache's area of svlm_decode_tagged_bytes(kv_heads, head_dim, splits) bytes for a launch of one cache
// and one layer (the per-layer kernel, whose splits hand their partial results over in tagged words); null, or
// several problems in the launch: the streaming kernel with its arrival counters in the view's scratch.
cudaError_t svlm_launch_decode(const SvlmAttendBatch& b, int layer0, int n_layers, const void* Q, const int* q_pos,
                               int q_heads, void* out, int splits, const void* Knew, const void* Vnew, int early_loads,
                               void* tagged, cudaStream_t st);
size_t svlm_decode_tagged_bytes(int kv_heads, int head_dim, int splits);

// Q/K/V projection with the append as its epilogue, head_dim 128 (svlm_qkv_sm100.cu).  tmX, tmW: host copies of
// the CUtensorMap of X [n][hidden] (64 x 128 box) and W [(q_heads + 2 kv_heads) * 128][hidden] (64 x 256 box), 128-byte swizzle.
// with_append = false: the plain projection Y = X W^T with q_heads blocks of 128 output columns, all written to Q_out.
cudaError_t svlm_launch_qkv_append(const void* tmX, const void* tmW, const SvlmCacheDev& cd, int layer, int n, int hidden,
                                   int q_heads, bool with_append, void* Q_out, cudaStream_t st);

// Y = X W^T for a few rows of X (decode-time projections), a bandwidth kernel (svlm_gemv.cu)
bool svlm_gemv_supported(int n, int in_dim);
cudaError_t svlm_launch_gemv(const void* X, const void* W, void* Y, int n, int in_dim, int out_dim, cudaStream_t st);

// tcgen05/TMEM/TMA chunk prefill, n_q >= 2 (svlm_prefill_sm100.cu)
bool svlm_prefill_supported(int n_pages, int group);
cudaError_t svlm_launch_prefill(const SvlmAttendBatch& b, int layer0, int n_layers, const void* Q, const int* q_pos,
                                int n_q, int q_heads, void* out, cudaStream_t st);
