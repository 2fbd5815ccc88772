// Host runtime behind the C ABI of include/svlm.h: owns the device allocations of a cache,
// validates arguments, and enqueues the kernels on the cache's stream.  No host synchronisation on
// the hot path: everything the kernels need to know about the stream's state lives in the device
// control block.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstddef>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/svlm.h"
#include "svlm_dev.h"
#include "svlm_host.h"
#include "svlm_launch.h"

static std::atomic<long long> g_launches{0};
void svlm_count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

namespace {

#define SVLM_CUDA(call)                          \
    do {                                         \
        cudaError_t e_ = (call);                 \
        if (e_ != cudaSuccess) return SVLM_ERR_CUDA; \
    } while (0)

struct DeviceGuard {
    int prev = -1;
    explicit DeviceGuard(int dev) {
        cudaGetDevice(&prev);
        if (prev != dev) cudaSetDevice(dev);
        else prev = -1;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

template <typename T>
int dev_alloc(svlm_cache* c, T** p, size_t count, bool zero = true) {
    void* q = nullptr;
    if (cudaMalloc(&q, std::max<size_t>(count, 1) * sizeof(T)) != cudaSuccess) return SVLM_ERR_NOMEM;
    c->allocs.push_back(q);
    if (zero && cudaMemset(q, 0, std::max<size_t>(count, 1) * sizeof(T)) != cudaSuccess) return SVLM_ERR_CUDA;
    *p = static_cast<T*>(q);
    return SVLM_OK;
}

void fill_theta(SvlmCacheDev& d, double base) {
    for (int i = 0; i < d.head_dim / 2; ++i) d.theta[i] = std::pow(base, -2.0 * i / d.head_dim);
}

int ensure_stage(svlm_cache* c, size_t bytes) {
    if (bytes <= c->stage_bytes) return SVLM_OK;
    SVLM_CUDA(cudaStreamSynchronize(c->stream));
    if (c->stage) cudaFree(c->stage);
    c->stage = nullptr;
    c->stage_bytes = 0;
    if (cudaMalloc(&c->stage, bytes) != cudaSuccess) return SVLM_ERR_NOMEM;
    c->stage_bytes = bytes;
    return SVLM_OK;
}

// The page-locked gathering buffer.  A host-buffer call that uses it ends with a synchronisation of the cache's
// stream, so the buffer is free again when the next call starts.
int ensure_hstage(svlm_cache* c, size_t bytes) {
    if (bytes <= c->hstage_bytes) return SVLM_OK;
    SVLM_CUDA(cudaStreamSynchronize(c->stream));
    if (c->hstage) cudaFreeHost(c->hstage);
    c->hstage = nullptr;
    c->hstage_bytes = 0;
    bytes = std::max<size_t>(bytes, 64 << 10);
    if (cudaHostAlloc(&c->hstage, bytes, cudaHostAllocDefault) != cudaSuccess) return SVLM_ERR_NOMEM;
    c->hstage_bytes = bytes;
    return SVLM_OK;
}

void fill_view(const svlm_cache* c, SvlmAttendView& v) {
    v.K = c->dev.K;
    v.V = c->dev.V;
    v.ctrl = c->dev.ctrl;
    v.tiles = c->dev.tiles;
    v.slot_gid = c->dev.slot_gid;
    v.ws = c->dev.ws;
    v.tmaps = c->dev.tmaps;
    v.new_slot = c->dev.new_slot;
    v.slot_c = c->dev.slot_c;
}

// Rotation table: (cos, sin)(k * 256^level * theta_i) in fp32 from fp64 (see svlm_rope.cuh).
int upload_rope_table(svlm_cache* c) {
    const SvlmCacheDev& d = c->dev;
    const int half = d.head_dim / 2;
    std::vector<float> tab((size_t)3 * 256 * half * 2);
    for (int level = 0; level < 3; ++level)
        for (int k = 0; k < 256; ++k)
            for (int i = 0; i < half; ++i) {
                const double ang = (double)k * std::pow(256.0, level) * d.theta[i];
                tab[(((size_t)level * 256 + k) * half + i) * 2] = (float)std::cos(ang);
                tab[(((size_t)level * 256 + k) * half + i) * 2 + 1] = (float)std::sin(ang);
            }
    if (cudaMemcpy(d.rope_tab, tab.data(), tab.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess)
        return SVLM_ERR_CUDA;
    return SVLM_OK;
}

// TMA descriptors of the K and V slabs: a 2D view [layers*kv_heads*n_slots rows][head_dim] with a
// 64-element x 128-row box and 128-byte swizzle (one box = half a page of one head at head_dim 128).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn tensor_map_encoder() {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
        return nullptr;
    return reinterpret_cast<EncodeTiledFn>(fn);
}

// Map of a row-major bf16 matrix [rows][cols] with a 64-column x box_rows box and 128-byte swizzle.
bool encode_matrix_map(EncodeTiledFn encode, CUtensorMap* map, const void* base, long long rows, long long cols, int box_rows) {
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int make_tensor_maps(svlm_cache* c) {
    EncodeTiledFn encode = tensor_map_encoder();
    if (!encode) return SVLM_ERR_CUDA;
    const SvlmCacheDev& d = c->dev;
    alignas(64) CUtensorMap maps[4];
    for (int which = 0; which < 4; ++which) {   // K, V with a whole-page box; K, V with a 32-row box
        cuuint64_t dims[2] = {(cuuint64_t)d.head_dim, (cuuint64_t)d.layers * d.kv_heads * d.n_slots};
        cuuint64_t strides[1] = {(cuuint64_t)d.head_dim * 2};
        cuuint32_t box[2] = {64, which < 2 ? (cuuint32_t)SVLM_PAGE : 32u};
        cuuint32_t estr[2] = {1, 1};
        if (encode(&maps[which], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (which & 1) ? (void*)d.V : (void*)d.K, dims, strides, box,
                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return SVLM_ERR_CUDA;
    }
    if (cudaMemcpy(d.tmaps, maps, sizeof maps, cudaMemcpyHostToDevice) != cudaSuccess) return SVLM_ERR_CUDA;
    return SVLM_OK;
}

void fill_batch_geometry(const svlm_cache* c, SvlmAttendBatch& b) {
    b.layers = c->dev.layers;
    b.kv_heads = c->dev.kv_heads;
    b.head_dim = c->dev.head_dim;
    b.n_slots = c->dev.n_slots;
    b.rope_mode = c->dev.rope_mode;
    b.sec_t = c->dev.sec_t;
    b.sec_th = c->dev.sec_th;
    std::memcpy(b.theta, c->dev.theta, sizeof b.theta);
    b.rope_tab = c->dev.rope_tab;
    b.q_varlen = 0;
}

// Caches that may share one launch: same shape, rotary settings, device and stream.
bool same_geometry(const svlm_cache* c, const svlm_cache* c0) {
    return c->stream == c0->stream && c->dev.layers == c0->dev.layers && c->dev.kv_heads == c0->dev.kv_heads &&
           c->dev.head_dim == c0->dev.head_dim && c->dev.n_slots == c0->dev.n_slots &&
           c->dev.rope_mode == c0->dev.rope_mode && c->dev.sec_t == c0->dev.sec_t && c->dev.sec_th == c0->dev.sec_th &&
           c->dev.theta[1] == c0->dev.theta[1] && c->device == c0->device;
}

// The descriptor copy in device memory that the batched kernels read (refreshed by every call that
// changes the configuration; the configuration is frozen by the first append).
int sync_dev_copy(svlm_cache* c) {
    if (cudaMemcpy(c->dev_copy, &c->dev, sizeof(SvlmCacheDev), cudaMemcpyHostToDevice) != cudaSuccess) return SVLM_ERR_CUDA;
    return SVLM_OK;
}

// Kernel parameter naming the caches of a batched call; all must be distinct and share a geometry.
int make_list(svlm_cache* const* caches, int n_caches, SvlmCacheList& list) {
    if (!caches || n_caches < 1 || n_caches > SVLM_MAX_BATCH || !caches[0]) return SVLM_ERR_ARG;
    list.n = n_caches;
    for (int i = 0; i < n_caches; ++i) {
        if (!caches[i] || !same_geometry(caches[i], caches[0])) return SVLM_ERR_ARG;
        for (int j = 0; j < i; ++j)
            if (caches[j] == caches[i]) return SVLM_ERR_ARG;
        list.cd[i] = caches[i]->dev_copy;
    }
    return SVLM_OK;
}

int attend_common(svlm_cache* const* caches, int n_caches, int layer, const void* Q, const int32_t* q_pos, int n_q,
                  int q_heads, void* out, const void* Knew = nullptr, const void* Vnew = nullptr) {
    svlm_cache* c0 = caches[0];
    if (!Q || !q_pos || !out || n_q < 1 || q_heads < 1) return SVLM_ERR_ARG;
    if (q_heads % c0->dev.kv_heads) return SVLM_ERR_ARG;
    if (layer < -1 || layer >= c0->dev.layers) return SVLM_ERR_ARG;
    SvlmAttendBatch b;
    b.n_caches = n_caches;
    fill_batch_geometry(c0, b);
    for (int i = 0; i < n_caches; ++i) {
        const svlm_cache* c = caches[i];
        if (!c) return SVLM_ERR_ARG;
        if (!same_geometry(c, c0)) return SVLM_ERR_ARG;
        if (n_q > c->appended) return SVLM_ERR_ORDER;
        fill_view(c, b.view[i]);
    }
    DeviceGuard guard(c0->device);
    const int layer0 = layer < 0 ? 0 : layer;
    const int n_layers = layer < 0 ? c0->dev.layers : 1;
    const int group = q_heads / c0->dev.kv_heads;
    int early = 0;
    if (n_q == 1 && layer >= 0) {
        // early loads: the kernel directly before this one on the stream was a decode of another layer that
        // covered exactly these caches (it wrote neither their metadata nor this layer's pages)
        early = 1;
        for (int i = 0; i < n_caches; ++i) {
            svlm_cache* c = caches[i];
            if (c->last_decode_layer < 0 || c->last_decode_layer == layer || c->last_decode_batch != n_caches ||
                c->last_decode_first != c0 || c->stream != c0->stream)
                early = 0;
        }
        // 2: nothing but that decode ran since (a chain of decode steps): the read-ahead has a whole layer-step of
        // time and is paced; 1: other kernels ran in between (projections): read ahead at once
        if (early && c0->calls_since_decode == 0) early = 2;
        for (int i = 0; i < n_caches; ++i) {
            caches[i]->last_decode_layer = layer;
            caches[i]->last_decode_batch = n_caches;
            caches[i]->last_decode_first = c0;
            caches[i]->calls_since_decode = 0;
        }
    } else {
        for (int i = 0; i < n_caches; ++i) caches[i]->last_decode_layer = -1;
    }
    if (n_q == 1 && group <= 8 && svlm_decode_supported(c0->dev.n_pages)) {
        // split-KV decode; every cache's scratch was sized for this launch shape at creation
        const int splits = svlm_decode_splits(c0->dev.n_pages, c0->dev.kv_heads, n_caches * n_layers);
        SVLM_CUDA(svlm_launch_decode(b, layer0, n_layers, Q, q_pos, q_heads, out, splits, Knew, Vnew, early, c0->decode_tagged, c0->stream));
        return SVLM_OK;
    }
    if (Knew) return SVLM_ERR_ARG;   // the fused step exists for the split-KV kernel only
    if (n_q >= 2 && svlm_prefill_supported(c0->dev.n_pages, group)) {
        SVLM_CUDA(svlm_launch_prefill(b, layer0, n_layers, Q, q_pos, n_q, q_heads, out, c0->stream));
        return SVLM_OK;
    }
    svlm_launch_attend_simple(b, layer0, n_layers, Q, q_pos, n_q, q_heads, out, c0->stream);
    SVLM_CUDA(cudaGetLastError());
    return SVLM_OK;
}

}  // namespace

extern "C" {

int svlm_cache_create(svlm_cache** out, int layers, int kv_heads, int head_dim, int n_sink, int vision_window,
                      int text_window, int capacity) {
    if (!out) return SVLM_ERR_ARG;
    *out = nullptr;
    if (layers < 1 || kv_heads < 1 || (head_dim != 64 && head_dim != 128) || n_sink < 0 || vision_window < 0 ||
        text_window < 0 || capacity < 1)
        return SVLM_ERR_ARG;
    svlm_cache* c = new (std::nothrow) svlm_cache;
    if (!c) return SVLM_ERR_NOMEM;
    if (cudaGetDevice(&c->device) != cudaSuccess) { delete c; return SVLM_ERR_CUDA; }
    SvlmCacheDev& d = c->dev;
    std::memset(&d, 0, sizeof d);
    d.layers = layers; d.kv_heads = kv_heads; d.head_dim = head_dim;
    d.n_sink = n_sink; d.vision_window = vision_window; d.text_window = text_window; d.capacity = capacity;
    d.n_sink_pages = (std::min(n_sink, capacity) + SVLM_PAGE - 1) / SVLM_PAGE;
    // two rings, each with at most one partial page at either end
    d.n_pages = d.n_sink_pages + (capacity + SVLM_PAGE - 1) / SVLM_PAGE + 4;
    d.n_slots = d.n_pages * SVLM_PAGE;
    d.pt_size = 1;
    while (d.pt_size <= d.n_pages) d.pt_size <<= 1;
    d.rope_mode = SVLM_ROPE_1D; d.sink_any = 0; d.contiguous = 1;
    d.sec_t = d.sec_th = head_dim / 2;
    fill_theta(d, 10000.0);

    int rc = SVLM_OK;
    const size_t slab = (size_t)layers * kv_heads * d.n_slots * head_dim;
    auto A = [&](int r) { if (rc == SVLM_OK) rc = r; };
    A(dev_alloc(c, &d.ctrl, 1));
    A(dev_alloc(c, &d.free_stack, d.n_pages));
    A(dev_alloc(c, &d.page_table[0], d.pt_size));
    A(dev_alloc(c, &d.page_table[1], d.pt_size));
    A(dev_alloc(c, &d.slot_gid, d.n_slots));
    A(dev_alloc(c, &d.slot_c, 3 * (size_t)d.n_slots));
    A(dev_alloc(c, &d.slot_a, d.n_slots));
    A(dev_alloc(c, &d.slot_delta, d.n_slots));
    A(dev_alloc(c, &d.slot_type, d.n_slots));
    A(dev_alloc(c, &d.tiles, d.n_pages));
    A(dev_alloc(c, &d.new_slot, capacity));
    A(dev_alloc(c, &d.new_c, 3 * (size_t)capacity));
    for (int t = 0; t < 2; ++t) {
        A(dev_alloc(c, &d.ev_gid[t], capacity));
        A(dev_alloc(c, &d.ev_pref[t], (size_t)capacity + 1));
    }
    {   // split-KV scratch: the larger of a one-layer launch and an all-layers launch
        const size_t one = svlm_decode_ws_floats(layers, kv_heads, head_dim, svlm_decode_splits(d.n_pages, kv_heads, 1));
        const size_t all = svlm_decode_ws_floats(layers, kv_heads, head_dim, svlm_decode_splits(d.n_pages, kv_heads, layers));
        A(dev_alloc(c, &d.ws, std::max(one, all)));
        // the per-layer kernel's tagged records: zero-filled here, afterwards written by that kernel alone
        A(dev_alloc(c, &c->decode_tagged, svlm_decode_tagged_bytes(kv_heads, head_dim, svlm_decode_splits(d.n_pages, kv_heads, 1))));
    }
    A(dev_alloc(c, &d.K, slab));
    A(dev_alloc(c, &d.V, slab));
    {
        unsigned char* tm = nullptr;
        A(dev_alloc(c, &tm, 512));
        d.tmaps = tm;
    }
    A(dev_alloc(c, &d.rope_tab, (size_t)3 * 256 * (head_dim / 2) * 2, false));
    A(dev_alloc(c, &c->dev_copy, 1));
    if (rc == SVLM_OK) rc = make_tensor_maps(c);
    if (rc == SVLM_OK) rc = upload_rope_table(c);
    if (rc == SVLM_OK) rc = sync_dev_copy(c);
    if (rc == SVLM_OK) {
        // pool pages on the free stack (top of the stack = lowest page number)
        std::vector<int> stack;
        for (int p = d.n_pages - 1; p >= d.n_sink_pages; --p) stack.push_back(p);
        SvlmCtrl ctrl;
        std::memset(&ctrl, 0, sizeof ctrl);
        ctrl.free_top = (int)stack.size();
        ctrl.wait_limit = 1u << 20;   // polls; seconds at worst
        std::vector<long long> minus1(d.n_slots, -1);
        if (cudaMemcpy(d.free_stack, stack.data(), stack.size() * sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(d.ctrl, &ctrl, sizeof ctrl, cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(d.slot_gid, minus1.data(), minus1.size() * sizeof(long long), cudaMemcpyHostToDevice) !=
                cudaSuccess)
            rc = SVLM_ERR_CUDA;
    }
    if (rc != SVLM_OK) {
        for (void* p : c->allocs) cudaFree(p);
        delete c;
        return rc;
    }
    *out = c;
    return SVLM_OK;
}

void svlm_cache_destroy(svlm_cache* c) {
    if (!c) return;
    DeviceGuard guard(c->device);
    cudaStreamSynchronize(c->stream);
    for (void* p : c->allocs) cudaFree(p);
    if (c->stage) cudaFree(c->stage);
    if (c->hstage) cudaFreeHost(c->hstage);
    if (c->copy_in) { cudaStreamSynchronize(c->copy_in); cudaStreamDestroy(c->copy_in); }
    if (c->copy_out) { cudaStreamSynchronize(c->copy_out); cudaStreamDestroy(c->copy_out); }
    if (c->ev_start) cudaEventDestroy(c->ev_start);
    for (cudaEvent_t e : c->ev_in) cudaEventDestroy(e);
    for (cudaEvent_t e : c->ev_done) cudaEventDestroy(e);
    delete c;
}

int svlm_cache_set_rope(svlm_cache* c, int mode, double base, const int sections[3]) {
    if (!c || !(base > 1.0) || (mode != SVLM_ROPE_1D && mode != SVLM_ROPE_MROPE)) return SVLM_ERR_ARG;
    if (c->configured_locked) return SVLM_ERR_ORDER;
    const int half = c->dev.head_dim / 2;
    if (mode == SVLM_ROPE_MROPE) {
        if (!sections || sections[0] < 0 || sections[1] < 0 || sections[2] < 0 ||
            sections[0] + sections[1] + sections[2] != half)
            return SVLM_ERR_ARG;
        c->dev.sec_t = sections[0];
        c->dev.sec_th = sections[0] + sections[1];
    } else {
        c->dev.sec_t = c->dev.sec_th = half;
    }
    c->dev.rope_mode = mode;
    fill_theta(c->dev, base);
    DeviceGuard guard(c->device);
    const int rc = upload_rope_table(c);
    return rc != SVLM_OK ? rc : sync_dev_copy(c);
}

int svlm_cache_set_policy(svlm_cache* c, int sink_any_type, int contiguous) {
    if (!c) return SVLM_ERR_ARG;
    if (c->configured_locked) return SVLM_ERR_ORDER;
    c->dev.sink_any = sink_any_type ? 1 : 0;
    c->dev.contiguous = contiguous ? 1 : 0;
    DeviceGuard guard(c->device);
    return sync_dev_copy(c);
}

int svlm_cache_set_stream(svlm_cache* c, void* cuda_stream) {
    if (!c) return SVLM_ERR_ARG;
    c->stream = static_cast<cudaStream_t>(cuda_stream);
    return SVLM_OK;
}

int svlm_cache_append(svlm_cache* c, int layer, const void* K, const void* V, const uint8_t* token_type,
                      const int32_t* pos, int n) {
    if (!c || !K || !V || n < 1 || layer < -1 || layer >= c->dev.layers) return SVLM_ERR_ARG;
    DeviceGuard guard(c->device);
    c->last_decode_layer = -1;
    if (layer <= 0) {
        if (!token_type || !pos) return SVLM_ERR_ARG;
        if (n > c->dev.capacity) return SVLM_ERR_CAPACITY;
        c->configured_locked = true;
        svlm_launch_append_meta(c->dev, token_type, pos, n, c->stream);
        c->appended += n;
        c->pending_n = n;
    } else if (n != c->pending_n) {
        return SVLM_ERR_ORDER;
    }
    svlm_launch_kv_write(c->dev, layer, K, V, n, c->stream);
    SVLM_CUDA(cudaGetLastError());
    return SVLM_OK;
}

int svlm_qkv_append(svlm_cache* c, int layer, const void* X, const void* W, int hidden, int q_heads,
                    const uint8_t* token_type, const int32_t* pos, int n, void* Q_out) {
    if (!c || !X || !W || !Q_out || n < 1 || layer < 0 || layer >= c->dev.layers) return SVLM_ERR_ARG;
    if (c->dev.head_dim != 128 || hidden < 64 || hidden % 64 || q_heads < 1 || q_heads % c->dev.kv_heads) return SVLM_ERR_ARG;
    if (((uintptr_t)X | (uintptr_t)W | (uintptr_t)Q_out) & 15) return SVLM_ERR_ARG;      // TMA and 16-byte stores
    DeviceGuard guard(c->device);
    static const EncodeTiledFn encode = tensor_map_encoder();
    if (!encode) return SVLM_ERR_CUDA;
    alignas(64) CUtensorMap tmX, tmW;
    if (!encode_matrix_map(encode, &tmX, X, n, hidden, 128) ||
        !encode_matrix_map(encode, &tmW, W, (long long)(q_heads + 2 * c->dev.kv_heads) * 128, hidden, 256))
        return SVLM_ERR_CUDA;
    c->last_decode_layer = -1;
    if (layer == 0) {
        if (!token_type || !pos) return SVLM_ERR_ARG;
        if (n > c->dev.capacity) return SVLM_ERR_CAPACITY;
        c->configured_locked = true;
        svlm_launch_append_meta(c->dev, token_type, pos, n, c->stream);
        c->appended += n;
        c->pending_n = n;
    } else if (n != c->pending_n) {
        return SVLM_ERR_ORDER;
    }
    SVLM_CUDA(svlm_launch_qkv_append(&tmX, &tmW, c->dev, layer, n, hidden, q_heads, true, Q_out, c->stream));
    return SVLM_OK;
}

int svlm_out_proj(svlm_cache* c, const void* A, const void* Wo, int in_dim, int out_dim, int n, void* Y) {
    if (!c || !A || !Wo || !Y || n < 1 || in_dim < 64 || in_dim % 64 || out_dim < 128 || out_dim % 128) return SVLM_ERR_ARG;
    if (((uintptr_t)A | (uintptr_t)Wo | (uintptr_t)Y) & 15) return SVLM_ERR_ARG;
    DeviceGuard guard(c->device);
    // The cache's record of its latest decode launch stays as it is: this call neither reads nor writes the
    // cache, so a decode step that follows may still fetch its pages early.  It does remember that something ran in
    // between: the decode then has less time before its inputs are ready and does not pace its read-ahead.
    ++c->calls_since_decode;
    if (svlm_gemv_supported(n, in_dim)) {      // a few tokens (decode): reading Wo once is all the work
        SVLM_CUDA(svlm_launch_gemv(A, Wo, Y, n, in_dim, out_dim, c->stream));
        return SVLM_OK;
    }
    static const EncodeTiledFn encode = tensor_map_encoder();
    if (!encode) return SVLM_ERR_CUDA;
    alignas(64) CUtensorMap tmA, tmW;
    if (!encode_matrix_map(encode, &tmA, A, n, in_dim, 128) || !encode_matrix_map(encode, &tmW, Wo, out_dim, in_dim, 256))
        return SVLM_ERR_CUDA;
    SVLM_CUDA(svlm_launch_qkv_append(&tmA, &tmW, c->dev, 0, n, in_dim, out_dim / 128, false, Y, c->stream));
    return SVLM_OK;
}

int svlm_cache_evict(svlm_cache* c) {
    if (!c) return SVLM_ERR_ARG;
    DeviceGuard guard(c->device);
    c->last_decode_layer = -1;
    svlm_launch_evict_meta(c->dev, c->stream);
    if (c->dev.contiguous) svlm_launch_evict_rotate(c->dev, c->stream);
    SVLM_CUDA(cudaGetLastError());
    return SVLM_OK;
}

int svlm_cache_evict_batched(svlm_cache* const* caches, int n_caches) {
    SvlmCacheList list;
    const int rc = make_list(caches, n_caches, list);
    if (rc != SVLM_OK) return rc;
    svlm_cache* c0 = caches[0];
    DeviceGuard guard(c0->device);
    bool rotate = false;
    for (int i = 0; i < n_caches; ++i) {
        caches[i]->last_decode_layer = -1;
        rotate = rotate || caches[i]->dev.contiguous;   // a cache with native positions never sets evict_moved
    }
    svlm_launch_evict_meta_batch(list, c0->stream);
    if (rotate) svlm_launch_evict_rotate_batch(list, c0->dev, c0->stream);
    SVLM_CUDA(cudaGetLastError());
    return SVLM_OK;
}

int svlm_attend(svlm_cache* c, int layer, const void* Q, const int32_t* q_pos, int n_q, int q_heads, void* out) {
    if (!c) return SVLM_ERR_ARG;
    svlm_cache* one[1] = {c};
    return attend_common(one, 1, layer, Q, q_pos, n_q, q_heads, out);
}

int svlm_decode_step(svlm_cache* c, int layer, const void* K, const void* V, const uint8_t* token_type,
                     const int32_t* pos, const void* Q, int q_heads, void* out) {
    if (!c || !K || !V || !pos || !Q || !out || layer < -1 || layer >= c->dev.layers || q_heads < 1) return SVLM_ERR_ARG;
    if (q_heads % c->dev.kv_heads || q_heads / c->dev.kv_heads > 8) return SVLM_ERR_ARG;
    if (!svlm_decode_supported(c->dev.n_pages)) return SVLM_ERR_ARG;   // more pages than the fused kernel's page list holds
    DeviceGuard guard(c->device);
    if (layer <= 0) {
        if (!token_type) return SVLM_ERR_ARG;
        c->configured_locked = true;
        c->last_decode_layer = -1;
        svlm_launch_append_meta(c->dev, token_type, pos, 1, c->stream);
        c->appended += 1;
        c->pending_n = 1;
    } else if (c->pending_n != 1) {
        return SVLM_ERR_ORDER;
    }
    svlm_cache* one[1] = {c};
    return attend_common(one, 1, layer, Q, pos, 1, q_heads, out, K, V);
}

int svlm_decode_step_batched(svlm_cache* const* caches, int n_caches, int layer, const void* K, const void* V,
                             const uint8_t* token_type, const int32_t* pos, const void* Q, int q_heads, void* out) {
    SvlmCacheList list;
    const int rc = make_list(caches, n_caches, list);
    if (rc != SVLM_OK) return rc;
    svlm_cache* c0 = caches[0];
    if (!K || !V || !pos || !Q || !out || layer < 0 || layer >= c0->dev.layers || q_heads < 1) return SVLM_ERR_ARG;
    if (q_heads % c0->dev.kv_heads || q_heads / c0->dev.kv_heads > 8) return SVLM_ERR_ARG;
    if (!svlm_decode_supported(c0->dev.n_pages)) return SVLM_ERR_ARG;
    DeviceGuard guard(c0->device);
    if (layer == 0) {
        if (!token_type) return SVLM_ERR_ARG;
        for (int i = 0; i < n_caches; ++i) {
            svlm_cache* c = caches[i];
            c->configured_locked = true;
            c->last_decode_layer = -1;
            c->appended += 1;
            c->pending_n = 1;
        }
        svlm_launch_append_meta_batch(list, token_type, pos, 1, c0->stream);
    } else {
        for (int i = 0; i < n_caches; ++i)
            if (caches[i]->pending_n != 1) return SVLM_ERR_ORDER;
    }
    return attend_common(caches, n_caches, layer, Q, pos, 1, q_heads, out, K, V);
}

int svlm_attend_batched_varlen(svlm_cache* const* caches, int n_caches, int layer, const void* Q, const int32_t* q_pos,
                               const int32_t* n_q, int q_heads, void* out) {
    SvlmCacheList list;   // only for its checks: distinct caches of one geometry
    int rc = make_list(caches, n_caches, list);
    if (rc != SVLM_OK) return rc;
    svlm_cache* c0 = caches[0];
    if (!Q || !q_pos || !n_q || !out || q_heads < 1 || layer < 0 || layer >= c0->dev.layers) return SVLM_ERR_ARG;
    if (q_heads % c0->dev.kv_heads || !svlm_prefill_supported(c0->dev.n_pages, q_heads / c0->dev.kv_heads)) return SVLM_ERR_ARG;
    SvlmAttendBatch b;
    b.n_caches = n_caches;
    fill_batch_geometry(c0, b);
    b.q_varlen = 1;
    long long off = 0;
    int n_max = 0;
    for (int i = 0; i < n_caches; ++i) {
        if (n_q[i] < 1) return SVLM_ERR_ARG;
        if (n_q[i] > caches[i]->appended) return SVLM_ERR_ORDER;
        b.q_off[i] = (int)off;
        b.q_cnt[i] = n_q[i];
        off += n_q[i];
        n_max = std::max(n_max, n_q[i]);
        fill_view(caches[i], b.view[i]);
        caches[i]->last_decode_layer = -1;
    }
    if (off > 0x7fffffffll) return SVLM_ERR_ARG;
    DeviceGuard guard(c0->device);
    SVLM_CUDA(svlm_launch_prefill(b, layer, 1, Q, q_pos, n_max, q_heads, out, c0->stream));
    return SVLM_OK;
}

int svlm_attend_batched(svlm_cache* const* caches, int n_caches, int layer, const void* Q, const int32_t* q_pos,
                        int n_q, int q_heads, void* out) {
    if (!caches || n_caches < 1 || n_caches > SVLM_MAX_BATCH || layer < 0) return SVLM_ERR_ARG;
    if (!caches[0]) return SVLM_ERR_ARG;
    return attend_common(caches, n_caches, layer, Q, q_pos, n_q, q_heads, out);
}

int svlm_cache_append_host(svlm_cache* c, int layer, const void* K_host, const void* V_host,
                           const uint8_t* token_type_host, const int32_t* pos_host, int n) {
    if (!c || !K_host || !V_host || n < 1 || layer < -1 || layer >= c->dev.layers) return SVLM_ERR_ARG;
    if (layer <= 0 && (!token_type_host || !pos_host)) return SVLM_ERR_ARG;
    DeviceGuard guard(c->device);
    const int nl = layer < 0 ? c->dev.layers : 1;
    const size_t kv_bytes = (size_t)nl * n * c->dev.kv_heads * c->dev.head_dim * 2;
    const size_t pos_bytes = (size_t)n * (c->dev.rope_mode == SVLM_ROPE_1D ? 1 : 3) * sizeof(int32_t);
    const size_t ty_off = 2 * kv_bytes, pos_off = (ty_off + n + 255) / 256 * 256;
    int rc = ensure_stage(c, pos_off + pos_bytes);
    if (rc != SVLM_OK) return rc;
    char* s = static_cast<char*>(c->stage);
    SVLM_CUDA(cudaMemcpyAsync(s, K_host, kv_bytes, cudaMemcpyHostToDevice, c->stream));
    SVLM_CUDA(cudaMemcpyAsync(s + kv_bytes, V_host, kv_bytes, cudaMemcpyHostToDevice, c->stream));
    if (layer <= 0) {
        SVLM_CUDA(cudaMemcpyAsync(s + ty_off, token_type_host, n, cudaMemcpyHostToDevice, c->stream));
        SVLM_CUDA(cudaMemcpyAsync(s + pos_off, pos_host, pos_bytes, cudaMemcpyHostToDevice, c->stream));
    }
    return svlm_cache_append(c, layer, s, s + kv_bytes, reinterpret_cast<const uint8_t*>(s + ty_off),
                             reinterpret_cast<const int32_t*>(s + pos_off), n);
}

int svlm_attend_host(svlm_cache* c, int layer, const void* Q_host, const int32_t* q_pos_host, int n_q, int q_heads,
                     void* out_host) {
    if (!c || !Q_host || !q_pos_host || !out_host || n_q < 1 || q_heads < 1 || layer < -1 || layer >= c->dev.layers)
        return SVLM_ERR_ARG;
    DeviceGuard guard(c->device);
    const int nl = layer < 0 ? c->dev.layers : 1;
    const size_t q_bytes = ((size_t)nl * n_q * q_heads * c->dev.head_dim * 2 + 255) / 256 * 256;
    const size_t pos_bytes = ((size_t)n_q * (c->dev.rope_mode == SVLM_ROPE_1D ? 1 : 3) * sizeof(int32_t) + 255) / 256 * 256;
    int rc = ensure_stage(c, 2 * q_bytes + pos_bytes);
    if (rc != SVLM_OK) return rc;
    char* s = static_cast<char*>(c->stage);
    if (layer < 0 && nl > 1 && n_q >= 2) {
        // All layers of a chunk: the layers' queries go up, are attended and their outputs come down as a
        // pipeline over three streams, so that the copies of one layer hide behind the attention of another.
        if (!c->copy_in) {
            SVLM_CUDA(cudaStreamCreateWithFlags(&c->copy_in, cudaStreamNonBlocking));
            SVLM_CUDA(cudaStreamCreateWithFlags(&c->copy_out, cudaStreamNonBlocking));
            SVLM_CUDA(cudaEventCreateWithFlags(&c->ev_start, cudaEventDisableTiming));
        }
        while ((int)c->ev_in.size() < nl) {
            cudaEvent_t a = nullptr, b = nullptr;
            SVLM_CUDA(cudaEventCreateWithFlags(&a, cudaEventDisableTiming));
            c->ev_in.push_back(a);
            SVLM_CUDA(cudaEventCreateWithFlags(&b, cudaEventDisableTiming));
            c->ev_done.push_back(b);
        }
        const size_t layer_bytes = (size_t)n_q * q_heads * c->dev.head_dim * 2;
        const size_t pos_n = (size_t)n_q * (c->dev.rope_mode == SVLM_ROPE_1D ? 1 : 3) * sizeof(int32_t);
        // the staging buffer may still be in use by earlier work on the cache's stream
        SVLM_CUDA(cudaEventRecord(c->ev_start, c->stream));
        SVLM_CUDA(cudaStreamWaitEvent(c->copy_in, c->ev_start, 0));
        SVLM_CUDA(cudaMemcpyAsync(s + 2 * q_bytes, q_pos_host, pos_n, cudaMemcpyHostToDevice, c->stream));
        for (int l = 0; l < nl; ++l) {
            SVLM_CUDA(cudaMemcpyAsync(s + l * layer_bytes, static_cast<const char*>(Q_host) + l * layer_bytes, layer_bytes,
                                      cudaMemcpyHostToDevice, c->copy_in));
            SVLM_CUDA(cudaEventRecord(c->ev_in[l], c->copy_in));
        }
        for (int l = 0; l < nl; ++l) {
            SVLM_CUDA(cudaStreamWaitEvent(c->stream, c->ev_in[l], 0));
            rc = svlm_attend(c, l, s + l * layer_bytes, reinterpret_cast<const int32_t*>(s + 2 * q_bytes), n_q, q_heads,
                             s + q_bytes + l * layer_bytes);
            if (rc != SVLM_OK) break;
            SVLM_CUDA(cudaEventRecord(c->ev_done[l], c->stream));
            SVLM_CUDA(cudaStreamWaitEvent(c->copy_out, c->ev_done[l], 0));
            SVLM_CUDA(cudaMemcpyAsync(static_cast<char*>(out_host) + l * layer_bytes, s + q_bytes + l * layer_bytes, layer_bytes,
                                      cudaMemcpyDeviceToHost, c->copy_out));
        }
        SVLM_CUDA(cudaStreamSynchronize(c->copy_in));
        SVLM_CUDA(cudaStreamSynchronize(c->stream));
        SVLM_CUDA(cudaStreamSynchronize(c->copy_out));
        return rc;
    }
    SVLM_CUDA(cudaMemcpyAsync(s, Q_host, (size_t)nl * n_q * q_heads * c->dev.head_dim * 2, cudaMemcpyHostToDevice,
                              c->stream));
    SVLM_CUDA(cudaMemcpyAsync(s + 2 * q_bytes, q_pos_host,
                              (size_t)n_q * (c->dev.rope_mode == SVLM_ROPE_1D ? 1 : 3) * sizeof(int32_t),
                              cudaMemcpyHostToDevice, c->stream));
    rc = svlm_attend(c, layer, s, reinterpret_cast<const int32_t*>(s + 2 * q_bytes), n_q, q_heads, s + q_bytes);
    if (rc != SVLM_OK) return rc;
    SVLM_CUDA(cudaMemcpyAsync(out_host, s + q_bytes, (size_t)nl * n_q * q_heads * c->dev.head_dim * 2,
                              cudaMemcpyDeviceToHost, c->stream));
    SVLM_CUDA(cudaStreamSynchronize(c->stream));
    return SVLM_OK;
}

// The device's view of a host buffer that is page-locked and mapped (as pinned allocations are under unified
// addressing), else null.
static void* mapped_alias(const void* host) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, host) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return a.type == cudaMemoryTypeHost ? a.devicePointer : nullptr;
}

int svlm_decode_step_host(svlm_cache* c, int layer, const void* K_host, const void* V_host, const uint8_t* token_type_host,
                          const int32_t* pos_host, const void* Q_host, int q_heads, void* out_host) {
    if (!c || !K_host || !V_host || !pos_host || !Q_host || !out_host || q_heads < 1 || layer < -1 || layer >= c->dev.layers)
        return SVLM_ERR_ARG;
    if (layer <= 0 && !token_type_host) return SVLM_ERR_ARG;
    DeviceGuard guard(c->device);
    if (layer < 0) {
        // All layers of a generated token in one launch: the inputs are a few KB per layer, and when all of them sit
        // in pinned, mapped host memory the kernels read them where they are and write the output where it belongs,
        // which costs one bus round trip inside the kernel instead of five small copies in front of it and one
        // behind (7.4-7.8 -> 6.2 ms per chunk end to end on the config-3 step).  Not for a single layer: there all
        // 37 CTAs of a KV head would fetch the same query over the bus (measured: 36 against 32 ms per chunk).
        // Anything else goes through the staging buffer below.
        void* dK = mapped_alias(K_host);
        void* dV = dK ? mapped_alias(V_host) : nullptr;
        void* dQ = dV ? mapped_alias(Q_host) : nullptr;
        void* dP = dQ ? mapped_alias(pos_host) : nullptr;
        void* dO = dP ? mapped_alias(out_host) : nullptr;
        void* dT = dO ? mapped_alias(token_type_host) : nullptr;
        if (dT && !(((uintptr_t)dK | (uintptr_t)dV | (uintptr_t)dQ | (uintptr_t)dO) & 15) && !((uintptr_t)dP & 3)) {
            const int rc = svlm_decode_step(c, layer, dK, dV, static_cast<const uint8_t*>(dT), static_cast<const int32_t*>(dP), dQ,
                                            q_heads, dO);
            if (rc != SVLM_OK) return rc;
            SVLM_CUDA(cudaStreamSynchronize(c->stream));
            return SVLM_OK;
        }
    }
    const int nl = layer < 0 ? c->dev.layers : 1;
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    const size_t kv_bytes = (size_t)nl * c->dev.kv_heads * c->dev.head_dim * 2, q_bytes = (size_t)nl * q_heads * c->dev.head_dim * 2;
    const size_t pos_bytes = (c->dev.rope_mode == SVLM_ROPE_1D ? 1 : 3) * sizeof(int32_t);
    const size_t oK = 0, oV = up(kv_bytes), oQ = oV + up(kv_bytes), oP = oQ + up(q_bytes), oT = oP + 256, oO = oT + 256;
    int rc = ensure_stage(c, oO + up(q_bytes));
    if (rc != SVLM_OK) return rc;
    char* s = static_cast<char*>(c->stage);
    if (oO <= (256 << 10)) {
        // the step's inputs are small: gathered in page-locked memory they go up in one copy instead of five
        rc = ensure_hstage(c, oO);
        if (rc != SVLM_OK) return rc;
        char* h = static_cast<char*>(c->hstage);
        std::memcpy(h + oK, K_host, kv_bytes);
        std::memcpy(h + oV, V_host, kv_bytes);
        std::memcpy(h + oQ, Q_host, q_bytes);
        std::memcpy(h + oP, pos_host, pos_bytes);
        if (layer <= 0) h[oT] = static_cast<char>(*token_type_host);
        SVLM_CUDA(cudaMemcpyAsync(s, h, oT + 16, cudaMemcpyHostToDevice, c->stream));
    } else {
        SVLM_CUDA(cudaMemcpyAsync(s + oK, K_host, kv_bytes, cudaMemcpyHostToDevice, c->stream));
        SVLM_CUDA(cudaMemcpyAsync(s + oV, V_host, kv_bytes, cudaMemcpyHostToDevice, c->stream));
        SVLM_CUDA(cudaMemcpyAsync(s + oQ, Q_host, q_bytes, cudaMemcpyHostToDevice, c->stream));
        SVLM_CUDA(cudaMemcpyAsync(s + oP, pos_host, pos_bytes, cudaMemcpyHostToDevice, c->stream));
        if (layer <= 0) SVLM_CUDA(cudaMemcpyAsync(s + oT, token_type_host, 1, cudaMemcpyHostToDevice, c->stream));
    }
    rc = svlm_decode_step(c, layer, s + oK, s + oV, reinterpret_cast<const uint8_t*>(s + oT), reinterpret_cast<const int32_t*>(s + oP),
                          s + oQ, q_heads, s + oO);
    if (rc != SVLM_OK) return rc;
    SVLM_CUDA(cudaMemcpyAsync(out_host, s + oO, q_bytes, cudaMemcpyDeviceToHost, c->stream));
    SVLM_CUDA(cudaStreamSynchronize(c->stream));
    return SVLM_OK;
}

// Host mirror of the stored tokens in stream order: (gid, slot) pairs sorted by gid.
static int snapshot(svlm_cache* c, std::vector<std::pair<long long, int>>& order, SvlmCtrl& ctrl) {
    const SvlmCacheDev& d = c->dev;
    SVLM_CUDA(cudaStreamSynchronize(c->stream));
    SVLM_CUDA(cudaMemcpy(&ctrl, d.ctrl, sizeof ctrl, cudaMemcpyDeviceToHost));
    std::vector<SvlmTile> tiles(std::max(ctrl.n_tiles, 1));
    std::vector<long long> gid(d.n_slots);
    SVLM_CUDA(cudaMemcpy(tiles.data(), d.tiles, ctrl.n_tiles * sizeof(SvlmTile), cudaMemcpyDeviceToHost));
    SVLM_CUDA(cudaMemcpy(gid.data(), d.slot_gid, gid.size() * sizeof(long long), cudaMemcpyDeviceToHost));
    order.clear();
    for (int t = 0; t < ctrl.n_tiles; ++t)
        for (int o = tiles[t].lo; o < tiles[t].hi; ++o) {
            const int slot = tiles[t].page * SVLM_PAGE + o;
            order.emplace_back(gid[slot], slot);
        }
    std::sort(order.begin(), order.end());
    return SVLM_OK;
}

int svlm_cache_query(svlm_cache* c, int64_t* n_kept, int64_t* gids, int32_t* pos, uint8_t* types,
                     int64_t* shift_total) {
    if (!c) return SVLM_ERR_ARG;
    DeviceGuard guard(c->device);
    const SvlmCacheDev& d = c->dev;
    std::vector<std::pair<long long, int>> order;
    SvlmCtrl ctrl;
    int rc = snapshot(c, order, ctrl);
    if (rc != SVLM_OK) return rc;
    std::vector<int> cpos(3 * (size_t)d.n_slots);
    std::vector<unsigned char> ty(d.n_slots);
    SVLM_CUDA(cudaMemcpy(cpos.data(), d.slot_c, cpos.size() * sizeof(int), cudaMemcpyDeviceToHost));
    SVLM_CUDA(cudaMemcpy(ty.data(), d.slot_type, ty.size(), cudaMemcpyDeviceToHost));
    if ((long long)order.size() != ctrl.n_stored) return SVLM_ERR_CUDA;   // tile list and count disagree
    for (size_t i = 0; i < order.size(); ++i) {
        const int slot = order[i].second;
        if (gids) gids[i] = order[i].first;
        if (types) types[i] = ty[slot];
        if (pos) for (int k = 0; k < 3; ++k) pos[3 * i + k] = cpos[(size_t)k * d.n_slots + slot];
    }
    if (n_kept) *n_kept = (int64_t)order.size();
    if (shift_total) *shift_total = ctrl.shift_total;
    return SVLM_OK;
}

int svlm_cache_read_kv(svlm_cache* c, int layer, void* K_host, void* V_host) {
    if (!c || layer < 0 || layer >= c->dev.layers) return SVLM_ERR_ARG;
    DeviceGuard guard(c->device);
    const SvlmCacheDev& d = c->dev;
    std::vector<std::pair<long long, int>> order;
    SvlmCtrl ctrl;
    int rc = snapshot(c, order, ctrl);
    if (rc != SVLM_OK) return rc;
    const size_t per_layer = (size_t)d.kv_heads * d.n_slots * d.head_dim;
    std::vector<uint16_t> slab(per_layer);
    for (int which = 0; which < 2; ++which) {
        uint16_t* dst = static_cast<uint16_t*>(which ? V_host : K_host);
        if (!dst) continue;
        const uint16_t* src = (which ? d.V : d.K) + (size_t)layer * per_layer;
        SVLM_CUDA(cudaMemcpy(slab.data(), src, per_layer * sizeof(uint16_t), cudaMemcpyDeviceToHost));
        for (size_t i = 0; i < order.size(); ++i)
            for (int h = 0; h < d.kv_heads; ++h)
                std::memcpy(dst + (i * d.kv_heads + h) * d.head_dim,
                            slab.data() + ((size_t)h * d.n_slots + order[i].second) * d.head_dim,
                            d.head_dim * sizeof(uint16_t));
    }
    return SVLM_OK;
}

int svlm_cache_status(svlm_cache* c) {
    if (!c) return SVLM_ERR_ARG;
    DeviceGuard guard(c->device);
    SVLM_CUDA(cudaStreamSynchronize(c->stream));
    SvlmCtrl ctrl;
    SVLM_CUDA(cudaMemcpy(&ctrl, c->dev.ctrl, sizeof ctrl, cudaMemcpyDeviceToHost));
    return ctrl.status;
}

int svlm_debug_set_wait_limit(svlm_cache* c, unsigned polls) {
    if (!c) return SVLM_ERR_ARG;
    DeviceGuard guard(c->device);
    c->wait_limit_host = polls;   // the copy reads this field when the stream reaches it
    SVLM_CUDA(cudaMemcpyAsync(reinterpret_cast<char*>(c->dev.ctrl) + offsetof(SvlmCtrl, wait_limit), &c->wait_limit_host,
                              sizeof(unsigned), cudaMemcpyHostToDevice, c->stream));
    SVLM_CUDA(cudaStreamSynchronize(c->stream));
    return SVLM_OK;
}

int64_t svlm_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* svlm_strerror(int status) {
    switch (status) {
        case SVLM_OK: return "ok";
        case SVLM_ERR_ARG: return "bad argument";
        case SVLM_ERR_CAPACITY: return "cache capacity exceeded";
        case SVLM_ERR_ORDER: return "call out of order";
        case SVLM_ERR_CUDA: return "CUDA call failed";
        case SVLM_ERR_TIMEOUT: return "bounded device wait ran out";
        case SVLM_ERR_NOMEM: return "out of memory";
        case SVLM_ERR_TOO_LARGE: return "problem exceeds the fixed scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

}  // extern "C"
