// Q/K/V projection whose epilogue appends to the cache (sm_100a): the step on the input side of the
// per-chunk path.  For the n new tokens of a layer, Y = X W^T with W = [W_q; W_k; W_v]; the query columns
// go to the caller's Q buffer, the key columns are rotated at each token's contiguous position
// (paper Section 2.1, "Contiguous RoPE") and written, with the value columns, straight into the
// token's cache slot: K and V never make a round trip through global memory between the GEMM and
// the cache.
//
// A dense contraction, so it runs on the tensor cores: one CTA per 128 x 256 output tile (128 tokens x
// two heads: head_dim is 128, so the rotation partners j and j + 64 of a key sit in the same tile; with
// 128 x 128 tiles the operand stream out of L2, 64 flop per byte, bounded the kernel at ~700 TFLOP/s),
// X and W tiles by TMA (128-byte swizzle) through a 4-stage ring, one thread issuing
// tcgen05.mma (M128 N256 K16) into a 256-column TMEM accumulator, four epilogue warps reading the
// accumulator with tcgen05.ld, one row per thread, one head after the other.  Every mbarrier wait is bounded; on expiry the CTA
// records SVLM_ERR_TIMEOUT, drains its copies, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "svlm_dev.h"
#include "svlm_launch.h"
#include "svlm_ptx.cuh"
#include "svlm_rope.cuh"
#include "svlm_tc.cuh"

namespace {

using namespace svlm_ptx;
using namespace svlm_tc;

constexpr int QK_STAGES = 4;
constexpr int QK_BK = 64;                       // k-block: 64 bf16 = one 128-byte swizzle row
constexpr int QK_TILE = 128 * QK_BK * 2;        // bytes of the X tile (128 rows); the W tile (256 rows) is twice that
constexpr int QK_STAGE = 3 * QK_TILE;
constexpr int QK_THREADS = 192;                 // warp 0: TMA, warp 1: MMA issue + TMEM, warps 2-5: epilogue

// Out of line: the rare fp64 path of the look-up would otherwise be copied into every unrolled pair.
__device__ __noinline__ float2 rope_cs_call(const float2* tab, int pair, long long c, double theta) {
    return svlm_rope_cs(tab, 64, pair, c, theta);
}

// The table look-up without the fp64 path: |c| < 2^24 (see svlm_rope.cuh).
__device__ __forceinline__ float2 rope_cs_fast(const float2* __restrict__ tab, int pair, int c) {
    const unsigned u = (unsigned)(c < 0 ? -c : c);
    float2 r = __ldg(tab + (size_t)(u & 255u) * 64 + pair);
    if (u >> 8) {
        r = svlm_cmul(r, __ldg(tab + (size_t)(256 + ((u >> 8) & 255u)) * 64 + pair));
        if (u >> 16) r = svlm_cmul(r, __ldg(tab + (size_t)(512 + (u >> 16)) * 64 + pair));
    }
    if (c < 0) r.y = -r.y;
    return r;
}

struct QkShared {
    unsigned long long full[QK_STAGES], empty[QK_STAGES], acc_full;
    unsigned tmem_base;
    int abort_flag;
};

// kv_heads_used = cd.kv_heads for the projection with append; 0 turns the kernel into the plain projection
// Y = X W^T (the output projection after attention): every 128-column block is then a "query head" and goes to Q_out.
__global__ void __launch_bounds__(QK_THREADS, 1)
qkv_append_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, SvlmCacheDev cd,
                  int layer, int n, int hidden, int q_heads, int kv_heads_used, uint16_t* __restrict__ Q_out) {
    constexpr int D = 128, HALF = 64;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* ring = smem_raw;                                      // [stage][X tile | W tile]
    QkShared& sh = *reinterpret_cast<QkShared*>(ring + QK_STAGES * QK_STAGE);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int head0 = 2 * blockIdx.x;            // the tile's two heads, in the order query heads, key heads, value heads
    const int n_heads = q_heads + 2 * kv_heads_used;
    const int m0 = blockIdx.y * 128;             // first token of the tile
    const int n_kb = hidden / QK_BK;
    volatile int* abort_flag = &sh.abort_flag;
    const unsigned wait_limit = cd.ctrl->wait_limit;   // written at creation only, never by a kernel

    if (smem_u32(smem_raw) & 1023) {             // swizzled tiles need a 1024-byte aligned base; same in every CTA
        if (threadIdx.x == 0) atomicCAS(&cd.ctrl->status, 0, -4);   // SVLM_ERR_CUDA
        return;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < QK_STAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        mbar_init(&sh.acc_full, 1);
        sh.abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(256));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem = sh.tmem_base;

    if (warp == 0) {
        // ================= TMA producer =================
        if (lane == 0) {
            for (int kb = 0; kb < n_kb; ++kb) {
                const int st = kb % QK_STAGES;
                if (!mbar_wait(&sh.empty[st], ((kb / QK_STAGES) & 1) ^ 1, abort_flag, wait_limit)) break;   // first pass: already free
                unsigned char* dst = ring + st * QK_STAGE;
                mbar_expect_tx(&sh.full[st], QK_STAGE);
                tma_load_2d(dst, &tmX, kb * QK_BK, m0, &sh.full[st]);                 // rows past the end read as zeros
                tma_load_2d(dst + QK_TILE, &tmW, kb * QK_BK, head0 * D, &sh.full[st]);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ================= MMA issuer =================
        if (lane == 0) {
            constexpr unsigned IDESC = make_idesc(128, 256, 0);
            bool ok = true;
            for (int kb = 0; kb < n_kb && ok; ++kb) {
                const int st = kb % QK_STAGES;
                ok = mbar_wait(&sh.full[st], (kb / QK_STAGES) & 1, abort_flag, wait_limit);
                if (!ok) break;
                tc_fence_after();
                const unsigned long long da = smem_desc(smem_u32(ring + st * QK_STAGE), 16, 1024);
                const unsigned long long db = smem_desc(smem_u32(ring + st * QK_STAGE + QK_TILE), 16, 1024);
#pragma unroll
                for (int ks = 0; ks < QK_BK / 16; ++ks)
                    tc_mma_ss(tmem, da + (unsigned)(ks * 32 >> 4), db + (unsigned)(ks * 32 >> 4), IDESC, (kb | ks) != 0);
                tc_commit(&sh.empty[st]);
            }
            if (ok) tc_commit(&sh.acc_full);
        }
        __syncwarp();
    } else {
        // ================= epilogue: one thread per token of the tile =================
        const int quad = warp & 3;                               // the TMEM lane quadrant this warp may read
        const int row = quad * 32 + lane;
        const int i = m0 + row;
        // where the token lives (key and value heads): the append's slot, if the append stood
        int slot = -1;
        if (head0 + 1 >= q_heads && i < n && cd.ctrl->append_n == n) {
            const int s = cd.new_slot[i];
            if (cd.slot_gid[s] == cd.ctrl->n_total - n + i) slot = s;
        }
        // A tile with key heads: the token's 64 rotation factors are looked up into registers now, while the
        // tensor pipe is still busy with the tile (64 dependent-latency look-ups after it took longer than the GEMM).
        const float2* tab = reinterpret_cast<const float2*>(cd.rope_tab);
        float2 cs[HALF];
        bool have_cs = false;
        int cpos[3] = {0, 0, 0};
        if (slot >= 0 && head0 < q_heads + kv_heads_used) {
            cpos[0] = cd.slot_c[slot]; cpos[1] = cd.slot_c[cd.n_slots + slot]; cpos[2] = cd.slot_c[2 * cd.n_slots + slot];
            const int lim = 1 << 24;
            have_cs = cpos[0] > -lim && cpos[0] < lim && cpos[1] > -lim && cpos[1] < lim && cpos[2] > -lim && cpos[2] < lim;
            if (have_cs) {
#pragma unroll
                for (int pair = 0; pair < HALF; ++pair) {
                    const int axis = cd.rope_mode == 0 ? 0 : (pair < cd.sec_t ? 0 : (pair < cd.sec_th ? 1 : 2));
                    cs[pair] = rope_cs_fast(tab, pair, axis == 0 ? cpos[0] : (axis == 1 ? cpos[1] : cpos[2]));
                }
            }
        }
        const bool ok = mbar_wait(&sh.acc_full, 0, abort_flag, wait_limit);
        tc_fence_after();
#pragma unroll 1
        for (int hh = 0; hh < 2 && ok; ++hh) {
            const int head = head0 + hh;
            if (head >= n_heads) break;                          // odd head count: the last tile is half empty
            const unsigned tacc = tmem + ((unsigned)(quad * 32) << 16) + hh * D;
            const int kv = head - q_heads;                       // < 0: query head; < kv_heads: key head; else value head
            if (kv >= 0 && kv < cd.kv_heads) {
                // key: pairs (j, j + 64), rotated at the slot's current position, 32 pairs at a time
                uint16_t* dst = cd.K + (((size_t)layer * cd.kv_heads + kv) * cd.n_slots + (slot >= 0 ? slot : 0)) * D;
#pragma unroll
                for (int c32 = 0; c32 < 2; ++c32) {
                    float lo[32], hi[32];
                    tmem_ld32(tacc + c32 * 32, lo);
                    tmem_ld32(tacc + HALF + c32 * 32, hi);
                    tmem_wait_ld();
                    if (slot >= 0) {
#pragma unroll
                        for (int k = 0; k < 32; ++k) {
                            const int pair = c32 * 32 + k;
                            float2 f;
                            if (have_cs) {
                                f = cs[pair];
                            } else {   // a position beyond the table's range (native positions of a very long stream)
                                const int axis = cd.rope_mode == 0 ? 0 : (pair < cd.sec_t ? 0 : (pair < cd.sec_th ? 1 : 2));
                                f = rope_cs_call(tab, pair, axis == 0 ? cpos[0] : (axis == 1 ? cpos[1] : cpos[2]), cd.theta[pair]);
                            }
                            const float x = lo[k], y = hi[k];
                            lo[k] = x * f.x - y * f.y;
                            hi[k] = y * f.x + x * f.y;
                        }
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            *reinterpret_cast<uint4*>(dst + c32 * 32 + 8 * k) =
                                make_uint4(pack2(lo[8 * k], lo[8 * k + 1]), pack2(lo[8 * k + 2], lo[8 * k + 3]),
                                           pack2(lo[8 * k + 4], lo[8 * k + 5]), pack2(lo[8 * k + 6], lo[8 * k + 7]));
                            *reinterpret_cast<uint4*>(dst + HALF + c32 * 32 + 8 * k) =
                                make_uint4(pack2(hi[8 * k], hi[8 * k + 1]), pack2(hi[8 * k + 2], hi[8 * k + 3]),
                                           pack2(hi[8 * k + 4], hi[8 * k + 5]), pack2(hi[8 * k + 6], hi[8 * k + 7]));
                        }
                    }
                }
            } else {
                // query head -> the caller's buffer; value head -> the cache slot: a plain bf16 copy of the row
                uint16_t* dst = nullptr;
                if (kv < 0) { if (i < n) dst = Q_out + ((size_t)i * q_heads + head) * D; }
                else if (slot >= 0) dst = cd.V + (((size_t)layer * cd.kv_heads + (kv - cd.kv_heads)) * cd.n_slots + slot) * D;
#pragma unroll 1
                for (int c32 = 0; c32 < 4; ++c32) {
                    float v[32];
                    tmem_ld32(tacc + c32 * 32, v);
                    tmem_wait_ld();
                    if (dst) {
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            *reinterpret_cast<uint4*>(dst + c32 * 32 + 8 * k) =
                                make_uint4(pack2(v[8 * k], v[8 * k + 1]), pack2(v[8 * k + 2], v[8 * k + 3]),
                                           pack2(v[8 * k + 4], v[8 * k + 5]), pack2(v[8 * k + 6], v[8 * k + 7]));
                    }
                }
            }
        }
    }

    // ---- teardown ------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (sh.abort_flag) {
        if (threadIdx.x == 0) {   // copies already issued still land here: give every stage a bounded chance to complete
            for (int s = 0; s < QK_STAGES; ++s)
                for (unsigned p = 0; p < 2; ++p)
                    for (unsigned w = 0; w < (1u << 16) && !mbar_test(&sh.full[s], p); ++w) __nanosleep(32);
            atomicCAS(&cd.ctrl->status, 0, -5);   // SVLM_ERR_TIMEOUT
        }
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256));
    }
}

constexpr size_t qkv_smem() { return (size_t)QK_STAGES * QK_STAGE + sizeof(QkShared); }

}  // namespace

cudaError_t svlm_launch_qkv_append(const void* tmX, const void* tmW, const SvlmCacheDev& cd, int layer, int n, int hidden,
                                   int q_heads, bool with_append, void* Q_out, cudaStream_t st) {
    cudaError_t e = svlm_allow_smem<qkv_append_kernel>(qkv_smem());
    if (e != cudaSuccess) return e;
    const int kv = with_append ? cd.kv_heads : 0;
    const dim3 grid((q_heads + 2 * kv + 1) / 2, (n + 127) / 128);
    qkv_append_kernel<<<grid, QK_THREADS, qkv_smem(), st>>>(*static_cast<const CUtensorMap*>(tmX), *static_cast<const CUtensorMap*>(tmW),
                                                             cd, layer, n, hidden, q_heads, kv, static_cast<uint16_t*>(Q_out));
    svlm_count_launch();
    return cudaGetLastError();
}
