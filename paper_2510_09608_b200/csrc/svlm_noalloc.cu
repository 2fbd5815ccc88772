// svlm_attend_decode_noalloc: single-query (decode) attention whose split-KV scratch is a fixed array
// inside the library image instead of memory obtained from the CUDA allocator.
//
// Who needs this: a caller that must not, or cannot, allocate device memory at the moment it wants
// to attend.  Typical cases are a serving process that has handed all free device memory to its own
// pool after start-up (a later cudaMalloc fails or fragments the pool), a latency-critical loop that
// must not take the allocator's device-wide lock, and code running where the CUDA allocation calls
// are not permitted at all.  The regular path sizes its scratch when the cache is created; this one
// works with any cache, including one whose creator gave it no scratch, because it brings its own.
//
// The array lives in every GPU that loads the library until the process exits (512 KiB per device).
// All calls on a device share it, and it keeps whatever the previous call left behind: the arrival
// counters are cleared on the stream before every launch, the partial results are fully rewritten
// before they are read.  Two calls whose kernels overlap on the GPU (different streams) would race
// on it; serialise them.
#include <cuda_runtime.h>

#include <cstring>
#include <mutex>

#include "../../include/svlm.h"
#include "svlm_dev.h"
#include "svlm_host.h"
#include "svlm_launch.h"

namespace {

constexpr size_t kScratchBytes = SVLM_NOALLOC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// Device-side storage.  In host code this name is only a handle for the symbol, not an address a
// kernel can use: the device address is looked up once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_decode_scratch[kScratchBytes];

std::mutex g_mu;
float* g_scratch_addr[kMaxDevices] = {};   // device address of g_decode_scratch, per device

// Device address of the array on `device`, which must be the current device.  The first call per
// device asks the runtime for it (this may initialise the module on that device, so it should
// happen outside any stream capture); later calls return the cached pointer.
int scratch_for_device(int device, float** out) {
    if (device < 0 || device >= kMaxDevices) return SVLM_ERR_ARG;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[device]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_decode_scratch) != cudaSuccess || !p) return SVLM_ERR_CUDA;
        g_scratch_addr[device] = static_cast<float*>(p);
    }
    *out = g_scratch_addr[device];
    return SVLM_OK;
}

}  // namespace

extern "C" int svlm_attend_decode_noalloc(svlm_cache* c, int layer, const void* Q, const int32_t* q_pos, int q_heads,
                                          void* out) {
    if (!c || !Q || !q_pos || !out || q_heads < 1) return SVLM_ERR_ARG;
    const SvlmCacheDev& d = c->dev;
    if (layer < 0 || layer >= d.layers || q_heads % d.kv_heads) return SVLM_ERR_ARG;
    const int group = q_heads / d.kv_heads;
    if (group > 8) return SVLM_ERR_ARG;                 // the split-KV kernel packs at most 8 query heads per KV head
    if (c->appended < 1) return SVLM_ERR_ORDER;
    if (!svlm_decode_supported(d.n_pages)) return SVLM_ERR_TOO_LARGE;   // more pages than the kernel's page list holds

    const int splits = svlm_decode_splits(d.n_pages, d.kv_heads, 1);
    // counters for every (layer, kv head) of the cache, then one layer's partials
    auto up4 = [](size_t x) { return (x + 3) & ~(size_t)3; };
    const size_t need = (up4((size_t)d.layers * d.kv_heads) - up4((size_t)d.kv_heads) +
                         svlm_decode_ws_floats(1, d.kv_heads, d.head_dim, splits)) * sizeof(float);
    if (need > kScratchBytes) return SVLM_ERR_TOO_LARGE;

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return SVLM_ERR_CUDA;
    if (prev != c->device && cudaSetDevice(c->device) != cudaSuccess) return SVLM_ERR_CUDA;
    int rc = SVLM_OK;
    float* scratch = nullptr;
    rc = scratch_for_device(c->device, &scratch);
    // What this call enqueues is not "a decode step of another layer" in the sense the regular entry points use to
    // let their next launch read early: forget the record.
    c->last_decode_layer = -1;
    if (rc == SVLM_OK) {
        // counters first in the scratch: they must be zero when the kernel starts
        const size_t counter_bytes = (size_t)d.layers * d.kv_heads * sizeof(unsigned);
        if (cudaMemsetAsync(scratch, 0, counter_bytes, c->stream) != cudaSuccess) rc = SVLM_ERR_CUDA;
    }
    if (rc == SVLM_OK) {
        SvlmAttendBatch b;
        b.n_caches = 1;
        b.layers = d.layers; b.kv_heads = d.kv_heads; b.head_dim = d.head_dim; b.n_slots = d.n_slots;
        b.rope_mode = d.rope_mode; b.sec_t = d.sec_t; b.sec_th = d.sec_th;
        std::memcpy(b.theta, d.theta, sizeof b.theta);
        SvlmAttendView& v = b.view[0];
        v.K = d.K; v.V = d.V; v.ctrl = d.ctrl; v.tiles = d.tiles; v.slot_gid = d.slot_gid; v.tmaps = d.tmaps; v.new_slot = d.new_slot; v.slot_c = d.slot_c;
        b.rope_tab = d.rope_tab;
        b.q_varlen = 0;
        v.ws = scratch;
        if (svlm_launch_decode(b, layer, 1, Q, q_pos, q_heads, out, splits, nullptr, nullptr, 0, nullptr, c->stream) != cudaSuccess)
            rc = SVLM_ERR_CUDA;
    }
    if (prev != c->device) cudaSetDevice(prev);
    return rc;
}
