// Key/value movement: writing appended tokens into their slots with the first rotation, and the
// in-place re-rotation of retained keys after an eviction (paper Section 2.1, "Contiguous RoPE":
// the indices of later tokens are shifted left; a stored key R(c)k becomes R(c-E)k = R(-E)R(c)k).
// Both are streaming kernels: 16-byte accesses, no reuse, bound by HBM bandwidth.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "svlm_dev.h"
#include "svlm_launch.h"
#include "svlm_rope.cuh"

namespace {

struct __align__(16) Bf16x8 { __nv_bfloat162 v[4]; };

// Rotate 8 consecutive pairs (lo[j], hi[j]) by (cs[j], sn[j]) in fp32, round to bf16.
__device__ __forceinline__ void rotate8(Bf16x8& lo, Bf16x8& hi, const float* cs, const float* sn) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float2 a = __bfloat1622float2(lo.v[j]);
        const float2 b = __bfloat1622float2(hi.v[j]);
        float2 ra, rb;
        ra.x = a.x * cs[2 * j] - b.x * sn[2 * j];
        rb.x = b.x * cs[2 * j] + a.x * sn[2 * j];
        ra.y = a.y * cs[2 * j + 1] - b.y * sn[2 * j + 1];
        rb.y = b.y * cs[2 * j + 1] + a.y * sn[2 * j + 1];
        lo.v[j] = __float22bfloat162_rn(ra);
        hi.v[j] = __float22bfloat162_rn(rb);
    }
}

// One thread per (token, group of 8 pairs); it serves the kv heads of its share of the layers
// (grid.y splits the layers when layer < 0), so the rotation factors are looked up once (table, see
// svlm_rope.cuh).  The source rows do not depend on the metadata, so the loads of the first rows are
// issued before the chain slot -> position -> factors is walked.
template <int UNROLL>
__global__ void __launch_bounds__(256) kv_write_kernel(SvlmCacheDev cd, int layer, const uint16_t* __restrict__ K,
                                                       const uint16_t* __restrict__ V, int n, int layers_per_block) {
    const int half = cd.head_dim / 2;
    const int groups = half / 8;          // threads per token
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int i = t / groups, g = t % groups;
    if (i >= n) return;
    const int d = cd.head_dim;
    const int l0 = layer < 0 ? blockIdx.y * layers_per_block : layer;
    const int l1 = layer < 0 ? min(cd.layers, l0 + layers_per_block) : layer + 1;
    const int row0 = l0 * cd.kv_heads, row1 = l1 * cd.kv_heads;      // rows of [layer][kv_head]
    // source of row r: [layer (only when all layers are given)][token][kv_head]
    auto src_of = [&](int r) {
        const int l = r / cd.kv_heads, h = r % cd.kv_heads;
        return (((size_t)(layer < 0 ? l : 0) * n + i) * cd.kv_heads + h) * d + g * 8;
    };
    Bf16x8 lo[UNROLL], hi[UNROLL];
    uint4 vlo[UNROLL], vhi[UNROLL];
    auto load_rows = [&](int r) {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            if (r + u < row1) {
                const size_t src = src_of(r + u);
                lo[u] = *reinterpret_cast<const Bf16x8*>(K + src);
                hi[u] = *reinterpret_cast<const Bf16x8*>(K + src + half);
                vlo[u] = *reinterpret_cast<const uint4*>(V + src);
                vhi[u] = *reinterpret_cast<const uint4*>(V + src + half);
            }
    };
    load_rows(row0);
    if (cd.ctrl->append_n != n) return;   // the metadata append was dropped (capacity) or does not match
    const int slot = cd.new_slot[i];
    // A layer's keys may arrive after an eviction has already shifted these tokens (layers are
    // computed one after another): rotate at the slot's CURRENT position, and skip a token that
    // the eviction has dropped in the meantime.
    if (cd.slot_gid[slot] != cd.ctrl->n_total - n + i) return;
    float cs[8], sn[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int pair = g * 8 + j;
        const int axis = cd.rope_mode == 0 ? 0 : (pair < cd.sec_t ? 0 : (pair < cd.sec_th ? 1 : 2));
        const float2 f = svlm_rope_cs(reinterpret_cast<const float2*>(cd.rope_tab), half, pair,
                                      cd.slot_c[axis * cd.n_slots + slot], cd.theta[pair]);
        cs[j] = f.x;
        sn[j] = f.y;
    }
    for (int r = row0; r < row1; r += UNROLL) {
        if (r != row0) load_rows(r);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            if (r + u < row1) {
                const size_t dst = ((size_t)(r + u) * cd.n_slots + slot) * d + g * 8;
                rotate8(lo[u], hi[u], cs, sn);
                *reinterpret_cast<Bf16x8*>(cd.K + dst) = lo[u];
                *reinterpret_cast<Bf16x8*>(cd.K + dst + half) = hi[u];
                *reinterpret_cast<uint4*>(cd.V + dst) = vlo[u];
                *reinterpret_cast<uint4*>(cd.V + dst + half) = vhi[u];
            }
    }
}

// Re-rotation after an eviction.  grid.x covers the slots, grid.y splits the layers.  A thread owns
// (slot, group of 8 pairs) and walks its share of the [layer][kv_head] rows with the same sines;
// the angle -E*theta is identical on the three MRoPE axes because all three indices of a token
// shift by the same E.
template <int UNROLL>
__device__ __forceinline__ void evict_rotate_body(const SvlmCacheDev& cd, int layers_per_block) {
    if (!cd.ctrl->evict_moved) return;
    const int half = cd.head_dim / 2;
    const int groups = half / 8;
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int slot = t / groups, g = t % groups;
    if (slot >= cd.n_slots) return;
    const int delta = cd.slot_delta[slot];
    if (delta == 0) return;
    float cs[8], sn[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float2 f = svlm_rope_cs(reinterpret_cast<const float2*>(cd.rope_tab), half, g * 8 + j, -(long long)delta,
                                      cd.theta[g * 8 + j]);
        cs[j] = f.x;
        sn[j] = f.y;
    }
    const int d = cd.head_dim;
    const int row0 = blockIdx.y * layers_per_block * cd.kv_heads;
    const int row1 = min(cd.layers, (blockIdx.y + 1) * layers_per_block) * cd.kv_heads;
    const size_t stride = (size_t)cd.n_slots * d;
    uint16_t* base = cd.K + (size_t)slot * d + g * 8;
    for (int r = row0; r < row1; r += UNROLL) {
        Bf16x8 lo[UNROLL], hi[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            if (r + u < row1) {
                lo[u] = *reinterpret_cast<const Bf16x8*>(base + (r + u) * stride);
                hi[u] = *reinterpret_cast<const Bf16x8*>(base + (r + u) * stride + half);
            }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            if (r + u < row1) {
                rotate8(lo[u], hi[u], cs, sn);
                *reinterpret_cast<Bf16x8*>(base + (r + u) * stride) = lo[u];
                *reinterpret_cast<Bf16x8*>(base + (r + u) * stride + half) = hi[u];
            }
    }
}

template <int UNROLL>
__global__ void __launch_bounds__(256) evict_rotate_kernel(SvlmCacheDev cd, int layers_per_block) {
    evict_rotate_body<UNROLL>(cd, layers_per_block);
}

// Batched form: blockIdx.z selects the cache, whose descriptor is first copied to shared memory.
template <int UNROLL>
__global__ void __launch_bounds__(256) evict_rotate_batch_kernel(SvlmCacheList list, int layers_per_block) {
    __shared__ SvlmCacheDev s_cd;
    svlm_load_desc(&s_cd, list.cd[blockIdx.z]);
    evict_rotate_body<UNROLL>(s_cd, layers_per_block);
}

// Layers per block in y: enough blocks to fill the machine a few times over, at least 4 rows per thread.
int rotate_layers_per_block(int layers, int kv_heads) {
    int splits = 1;
    while (splits < layers && (layers + splits - 1) / splits * kv_heads > 8) ++splits;
    return (layers + splits - 1) / splits;
}

}  // namespace

void svlm_launch_kv_write(const SvlmCacheDev& cd, int layer, const void* K, const void* V, int n, cudaStream_t st) {
    const int groups = cd.head_dim / 16;
    const int threads = n * groups;
    const int lpb = rotate_layers_per_block(cd.layers, cd.kv_heads);
    dim3 grid((threads + 255) / 256, layer < 0 ? (cd.layers + lpb - 1) / lpb : 1);
    kv_write_kernel<4><<<grid, 256, 0, st>>>(cd, layer, (const uint16_t*)K, (const uint16_t*)V, n, lpb);
    svlm_count_launch();
}

void svlm_launch_evict_rotate(const SvlmCacheDev& cd, cudaStream_t st) {
    const int groups = cd.head_dim / 16;
    const int threads = cd.n_slots * groups;
    const int lpb = rotate_layers_per_block(cd.layers, cd.kv_heads);
    dim3 grid((threads + 255) / 256, (cd.layers + lpb - 1) / lpb);
    evict_rotate_kernel<4><<<grid, 256, 0, st>>>(cd, lpb);
    svlm_count_launch();
}

void svlm_launch_evict_rotate_batch(const SvlmCacheList& list, const SvlmCacheDev& geom, cudaStream_t st) {
    const int threads = geom.n_slots * (geom.head_dim / 16);
    const int lpb = rotate_layers_per_block(geom.layers, geom.kv_heads);
    dim3 grid((threads + 255) / 256, (geom.layers + lpb - 1) / lpb, list.n);
    evict_rotate_batch_kernel<4><<<grid, 256, 0, st>>>(list, lpb);
    svlm_count_launch();
}
