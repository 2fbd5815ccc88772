// Split-KV decode attention (one query token per cache/layer attends over the whole retained cache;
// paper Section 3.3: per-token latency over a fixed-length context is the figure of merit), optionally
// fused with the append of that token's own key and value (one "decode step" of a layer).
//
// The step reads every stored key and value exactly once, so it is bound by HBM bandwidth; at
// 19 MB per layer the data time is a few microseconds and everything serial around it counts:
//   * grid = (splits, kv_heads, caches*layers), about one CTA per SM; a CTA owns a contiguous run of
//     32-key sub-tiles of the active-page list;
//   * one producer thread streams the sub-tiles with TMA (2D boxes of 32 keys x 64 dims, 128-byte
//     swizzle) through a ring of shared-memory stages, each with a full and an empty mbarrier;
//     the whole first ring-load is in flight before anything else happens;
//   * six consumer warps take sub-tiles round-robin, each through its own ring stage; the G <= 8 query heads that share a KV head
//     ride in the N dimension of m16n8k16 MMAs (S^T = K Q^T, O^T += V^T P^T), so K and V are read
//     once for the whole group; per-warp online softmax with warp-shuffle reductions;
//   * rotation factors come from a small table (no sincos in the kernel);
//   * fused append: the warp that owns the sub-tile holding the new token's slot rotates the new key,
//     patches the row in shared memory and writes key and value to the cache, so the token needs no
//     launch of its own and is never read from the cache by the step that writes it;
//   * split partials (o, m, l) go to scratch; the last CTA of a (cache, layer, kv head) to arrive
//     combines them (arrival counter, nobody waits);
//   * with programmatic dependent launch the next layer's kernel starts its loads while this one
//     finishes: everything that depends on earlier kernels (query, scratch) is read after the
//     grid-dependency wait, the cache pages are not (the caller's contract, see the launcher).
// Every mbarrier wait is bounded; on expiry the CTA records SVLM_ERR_TIMEOUT, drains its copies
// and leaves.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "svlm_dev.h"
#include "svlm_launch.h"
#include "svlm_ptx.cuh"
#include "svlm_rope.cuh"

namespace {

using namespace svlm_ptx;

constexpr int DEC_CWARPS = 6;                       // consumer warps
constexpr int DEC_THREADS = (DEC_CWARPS + 1) * 32;  // + one producer warp
// One ring stage per consumer warp: a warp meets every phase of its stage's barriers in turn.  (With
// a stage shared between warps a waiter would skip phases, and a parity wait cannot tell the phase
// it wants from the one two earlier.)
constexpr int DEC_STAGES = DEC_CWARPS;
constexpr int SUB = 32;                             // keys per sub-tile
constexpr int DEC_MAX_TILES = 512;

__device__ __forceinline__ void ldmatrix_x4(unsigned& r0, unsigned& r1, unsigned& r2, unsigned& r3, const void* p) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(p);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(s));
}
__device__ __forceinline__ void ldmatrix_x4_trans(unsigned& r0, unsigned& r1, unsigned& r2, unsigned& r3,
                                                  const void* p) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(p);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(s));
}
__device__ __forceinline__ unsigned movmatrix_trans(unsigned a) {
    unsigned d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ void mma_bf16(float* c, unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0,
                                         unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                 "{%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<unsigned*>(&v);
}

// Scratch layout per cache: arrival counters [layers*kv_heads] (kept at zero between launches),
// then per (layer in launch, kv head): splits records { o[8][D] bf16, m[8] f32, l[8] f32 }.  The
// un-normalised partial outputs travel as bf16 (their error is of the size of the final rounding of
// the output), which lets the combining CTA stage every record in shared memory in one round trip.
template <int D>
__host__ __device__ constexpr int rec_bytes() { return 8 * D * 2 + 64; }
template <int D>
__host__ __device__ constexpr int partial_floats() { return rec_bytes<D>() / 4; }

struct DecShared {
    unsigned long long full[DEC_STAGES], empty[DEC_STAGES];
    int abort_flag;
    int last;
    unsigned tile_pk[DEC_MAX_TILES];   // page | lo << 16 | hi << 24
};

// Position of a 16-byte chunk inside a stage: 64-dim panels of [32 keys][128 B], chunks XOR-swizzled
// by the key's low three bits (the layout the 128-byte-swizzle TMA box writes).
__device__ __forceinline__ int sw_off(int key, int chunk) {
    return (chunk >> 3) * (SUB * 128) + key * 128 + (((chunk & 7) ^ (key & 7)) << 4);
}

template <int D>
__global__ void __launch_bounds__(DEC_THREADS, 2)
decode_kernel(SvlmAttendBatch b, int layer0, int n_layers, const uint16_t* __restrict__ Q,
              const int* __restrict__ q_pos, int q_heads, uint16_t* __restrict__ out, int splits,
              const uint16_t* __restrict__ Knew, const uint16_t* __restrict__ Vnew, int early_loads) {
    constexpr int KB = D / 64;                       // 64-dim panels per row
    constexpr int PANEL_BYTES = SUB * 128;
    constexpr int STAGE_BYTES = 2 * KB * PANEL_BYTES;   // K panels then V panels
    constexpr int KSTEPS = D / 16;
    constexpr int DBLK = D / 16;
    constexpr int HALF = D / 2;
    extern __shared__ unsigned char smem_raw[];
    DecShared& sh = *reinterpret_cast<DecShared*>(smem_raw);
    unsigned char* ring = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + sizeof(DecShared) + 1023) & ~(uintptr_t)1023);
    uint16_t* s_q = reinterpret_cast<uint16_t*>(ring + DEC_STAGES * STAGE_BYTES);   // [8][D] bf16
    uint16_t* s_new = s_q + 8 * D;       // fused step: the new token's rotated key [D], then its value [D]

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int split = blockIdx.x, hk = blockIdx.y;
    const int prob = blockIdx.z;
    const int ci = prob / n_layers, li = prob % n_layers;
    const int layer = layer0 + li;
    const SvlmAttendView& vw = b.view[ci];
    const int G = q_heads / b.kv_heads;
    volatile int* abort_flag = &sh.abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < DEC_STAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        sh.abort_flag = 0;
        mbar_init_fence();
    }
    // The metadata was written by an earlier kernel in the stream.  When the launcher vouches that
    // the kernel directly before this one did not write it (early_loads), it is read at once;
    // otherwise after the grid-dependency wait.  A kernel that has to wait does so BEFORE it lets its
    // successor start: a successor with early loads then only ever runs behind a completed metadata
    // kernel (whatever that kernel's own trigger), not merely behind one that has been launched.
    if (!early_loads) pdl_wait();
    pdl_launch_dependents();
    const int n_tiles = min(__ldcg(&vw.ctrl->n_tiles), DEC_MAX_TILES);
    for (int i = threadIdx.x; i < n_tiles; i += DEC_THREADS) {
        const int4 tl = __ldcg(reinterpret_cast<const int4*>(vw.tiles + i));   // page, lo, hi, pad
        sh.tile_pk[i] = (unsigned)tl.x | ((unsigned)tl.y << 16) | ((unsigned)tl.z << 24);
    }
    if (early_loads && threadIdx.x < 3) {
        // Bring the call's own small inputs towards L2 while the previous kernel still runs (a hint:
        // they are read for real only after the grid-dependency wait).
        const size_t qoff = ((size_t)prob * q_heads + (size_t)hk * G) * D, koff = ((size_t)prob * b.kv_heads + hk) * D;
        const void* p = threadIdx.x == 0 ? (const void*)(Q + qoff) : threadIdx.x == 1 ? (const void*)(Knew ? Knew + koff : Q + qoff)
                                                                                     : (const void*)(Vnew ? Vnew + koff : Q + qoff);
        const int bytes = threadIdx.x == 0 ? G * D * 2 : D * 2;
        for (int o = 0; o < bytes; o += 128)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(p) + o));
    }
    const long long shift = __ldcg(&vw.ctrl->shift_total);
    // the new token of a fused step: where it lives and whether it is still stored there
    int new_slot = -1;
    if (Knew && warp < DEC_CWARPS) {
        const int s = __ldcg(vw.new_slot);
        if (__ldcg(&vw.ctrl->append_n) == 1 && __ldcg(vw.slot_gid + s) == __ldcg(&vw.ctrl->n_total) - 1) new_slot = s;
    }
    __syncthreads();

    const int total_q = 4 * n_tiles;
    const int q0 = (int)((long long)split * total_q / splits), q1 = (int)((long long)(split + 1) * total_q / splits);
    const size_t head_row0 = ((size_t)layer * b.kv_heads + hk) * b.n_slots;
    constexpr int REC = rec_bytes<D>();
    unsigned char* ws_parts = reinterpret_cast<unsigned char*>(vw.ws + (((size_t)b.layers * b.kv_heads + 3) & ~(size_t)3));
    unsigned char* part = ws_parts + ((size_t)(li * b.kv_heads + hk) * splits + split) * REC;   // 16-byte aligned

    auto sub_valid = [&](int q, int& page, int& lo, int& hi) {
        const unsigned pk = sh.tile_pk[q >> 2];
        page = pk & 0xFFFF; lo = (pk >> 16) & 0xFF; hi = pk >> 24;
        const int k0 = (q & 3) * SUB;
        return k0 < hi && k0 + SUB > lo;
    };

    if (warp == DEC_CWARPS) {
        // ================= producer =================
        if (lane == 0) {
            const unsigned char* maps = reinterpret_cast<const unsigned char*>(vw.tmaps);
            const void* tmK = maps + 256;
            const void* tmV = maps + 384;
            int it = 0;
            for (int q = q0; q < q1; ++q) {
                int page, lo, hi;
                if (!sub_valid(q, page, lo, hi)) continue;
                const int st = it % DEC_STAGES;
                if (it == DEC_STAGES && early_loads && gridDim.z == 1) {
                    // The ring is full and frees up only once the consumers have the query (after the wait for
                    // the previous kernel): bring the rest of this CTA's sub-tiles into L2 meanwhile (9.56 ->
                    // 9.31 us per layer-step).  Only for one problem per launch behind another decode: a batched
                    // launch streams many ring-loads per CTA and gains nothing from the hint.
                    for (int q2 = q, n2 = 0; q2 < q1 && n2 < DEC_STAGES; ++q2) {   // at most one more ring-load
                        int pg, l2, h2;
                        if (!sub_valid(q2, pg, l2, h2)) continue;
                        ++n2;
                        const int y2 = (int)(head_row0 + (size_t)pg * SVLM_PAGE + (q2 & 3) * SUB);
#pragma unroll
                        for (int kb = 0; kb < KB; ++kb) {
                            tma_prefetch_2d(tmK, kb * 64, y2);
                            tma_prefetch_2d(tmV, kb * 64, y2);
                        }
                    }
                }
                if (!mbar_wait(&sh.empty[st], ((it / DEC_STAGES) & 1) ^ 1, abort_flag)) break;
                unsigned char* dst = ring + st * STAGE_BYTES;
                const int y = (int)(head_row0 + (size_t)page * SVLM_PAGE + (q & 3) * SUB);
                mbar_expect_tx(&sh.full[st], STAGE_BYTES);
#pragma unroll
                for (int kb = 0; kb < KB; ++kb) {
                    tma_load_2d(dst + kb * PANEL_BYTES, tmK, kb * 64, y, &sh.full[st]);
                    tma_load_2d(dst + (KB + kb) * PANEL_BYTES, tmV, kb * 64, y, &sh.full[st]);
                }
                ++it;
            }
        }
    } else {
        // ================= consumers =================
        const float2* tab = reinterpret_cast<const float2*>(b.rope_tab);
        // ---- query rows: rotate at q_pos - shift_total, round to bf16, park in shared memory ----
        {
            const int pair = threadIdx.x & (HALF - 1);
            const int axis = b.rope_mode == 0 ? 0 : (pair < b.sec_t ? 0 : (pair < b.sec_th ? 1 : 2));
            float2 cs;
            if (new_slot >= 0) {
                // fused step: the query is the appended token, its position is already in the metadata,
                // so the rotation factors do not have to wait for the previous kernel
                cs = svlm_rope_cs(tab, HALF, pair, __ldcg(vw.slot_c + (size_t)axis * b.n_slots + new_slot), b.theta[pair]);
                if (early_loads) pdl_wait();
            } else {
                if (early_loads) pdl_wait();
                const int* qp = q_pos + (size_t)ci * (b.rope_mode == 0 ? 1 : 3);
                cs = svlm_rope_cs(tab, HALF, pair, (long long)qp[b.rope_mode == 0 ? 0 : axis] - shift, b.theta[pair]);
            }
            constexpr int HSTEP = (DEC_CWARPS * 32) / HALF, HN = (8 + HSTEP - 1) / HSTEP;   // heads per thread
            uint16_t qx[HN], qy[HN];
            // fused step: the new token's key and value rows come in with the query (same round trip); the key is
            // rotated with the query's factors (same token, same position) and both wait in shared memory for the
            // warp whose sub-tile holds the token's slot
            const bool prep_new = new_slot >= 0 && threadIdx.x < HALF;
            uint16_t kx = 0, ky = 0, vx = 0, vy = 0;
            if (prep_new) {
                const size_t noff = ((size_t)prob * b.kv_heads + hk) * D;
                kx = Knew[noff + pair]; ky = Knew[noff + pair + HALF];
                vx = Vnew[noff + pair]; vy = Vnew[noff + pair + HALF];
            }
#pragma unroll
            for (int k = 0; k < HN; ++k) {      // all loads first: one round trip
                const int h = threadIdx.x / HALF + k * HSTEP;
                const size_t off = (((size_t)prob) * q_heads + hk * G + (h < G ? h : 0)) * D;   // n_q = 1
                qx[k] = Q[off + pair];
                qy[k] = Q[off + pair + HALF];
            }
#pragma unroll
            for (int k = 0; k < HN; ++k) {
                const int h = threadIdx.x / HALF + k * HSTEP;
                if (h >= 8) continue;
                const float x = h < G ? __bfloat162float(__ushort_as_bfloat16(qx[k])) : 0.f;
                const float y = h < G ? __bfloat162float(__ushort_as_bfloat16(qy[k])) : 0.f;
                s_q[h * D + pair] = __bfloat16_as_ushort(__float2bfloat16_rn(x * cs.x - y * cs.y));
                s_q[h * D + pair + HALF] = __bfloat16_as_ushort(__float2bfloat16_rn(y * cs.x + x * cs.y));
            }
            if (prep_new) {
                const float x = __bfloat162float(__ushort_as_bfloat16(kx)), y = __bfloat162float(__ushort_as_bfloat16(ky));
                s_new[pair] = __bfloat16_as_ushort(__float2bfloat16_rn(x * cs.x - y * cs.y));
                s_new[pair + HALF] = __bfloat16_as_ushort(__float2bfloat16_rn(y * cs.x + x * cs.y));
                s_new[D + pair] = vx;
                s_new[D + pair + HALF] = vy;
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(DEC_CWARPS * 32));   // consumer warps only
        unsigned qf[KSTEPS][2];   // B fragments of Q^T: (d = ks*16 + 2t.., head g)
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            qf[ks][0] = *reinterpret_cast<const unsigned*>(s_q + g * D + ks * 16 + 2 * t);
            qf[ks][1] = *reinterpret_cast<const unsigned*>(s_q + g * D + ks * 16 + 2 * t + 8);
        }

        const float scale = 1.4426950408889634f * rsqrtf((float)D);
        float o[DBLK][4];
#pragma unroll
        for (int i = 0; i < DBLK; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};   // heads 2t, 2t+1 (l: this thread's share)

        int it = 0;
        bool ok = true;
        for (int q = q0; q < q1 && ok; ++q) {
            int page, lo, hi;
            if (!sub_valid(q, page, lo, hi)) continue;
            const int my = (it % DEC_CWARPS) == warp;
            const int st = it % DEC_STAGES;
            const unsigned par = (it / DEC_STAGES) & 1;
            ++it;
            if (!my) continue;
            ok = mbar_wait(&sh.full[st], par, abort_flag);
            if (!ok) break;
            unsigned char* sk = ring + st * STAGE_BYTES;
            unsigned char* sv = sk + KB * PANEL_BYTES;
            const int k0 = (q & 3) * SUB;

            if (new_slot >= 0 && (new_slot >> 7) == page && ((new_slot & 127) >> 5) == (q & 3)) {
                // fused append: rotate the new key at its position, put key and value into the
                // shared-memory row and into the cache
                const int r = new_slot & 31;
                uint16_t* kdst = const_cast<uint16_t*>(vw.K) + (head_row0 + new_slot) * D;
                uint16_t* vdst = const_cast<uint16_t*>(vw.V) + (head_row0 + new_slot) * D;
                for (int pair = lane; pair < HALF; pair += 32) {
                    const uint16_t klo = s_new[pair], khi = s_new[pair + HALF];
                    const uint16_t vlo = s_new[D + pair], vhi = s_new[D + pair + HALF];
                    kdst[pair] = klo; kdst[pair + HALF] = khi;
                    vdst[pair] = vlo; vdst[pair + HALF] = vhi;
                    const int e0 = pair, e1 = pair + HALF;
                    *reinterpret_cast<uint16_t*>(sk + sw_off(r, e0 >> 3) + (e0 & 7) * 2) = klo;
                    *reinterpret_cast<uint16_t*>(sk + sw_off(r, e1 >> 3) + (e1 & 7) * 2) = khi;
                    *reinterpret_cast<uint16_t*>(sv + sw_off(r, e0 >> 3) + (e0 & 7) * 2) = vlo;
                    *reinterpret_cast<uint16_t*>(sv + sw_off(r, e1 >> 3) + (e1 & 7) * 2) = vhi;
                }
                __syncwarp();
            }

            // S^T[32 keys x 8 heads] = K Q^T
            float s[2][4];
#pragma unroll
            for (int mb = 0; mb < 2; ++mb) {
                s[mb][0] = s[mb][1] = s[mb][2] = s[mb][3] = 0.f;
#pragma unroll
                for (int ks = 0; ks < KSTEPS; ++ks) {
                    const int i = lane >> 3, r = lane & 7;
                    const int key = mb * 16 + (i & 1) * 8 + r;
                    const int chunk = ks * 2 + (i >> 1);
                    unsigned a0, a1, a2, a3;
                    ldmatrix_x4(a0, a1, a2, a3, sk + sw_off(key, chunk));
                    mma_bf16(s[mb], a0, a1, a2, a3, qf[ks][0], qf[ks][1]);
                }
            }
            // scale, mask slots outside [lo, hi), column (head) maxima over the 32 keys
            float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int mb = 0; mb < 2; ++mb)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int key = k0 + mb * 16 + g + (e >> 1) * 8;
                    const bool in = key >= lo && key < hi;
                    s[mb][e] = in ? s[mb][e] * scale : -INFINITY;
                    mx[e & 1] = fmaxf(mx[e & 1], s[mb][e]);
                }
#pragma unroll
            for (int sft = 4; sft < 32; sft <<= 1) {
                mx[0] = fmaxf(mx[0], __shfl_xor_sync(0xffffffffu, mx[0], sft));
                mx[1] = fmaxf(mx[1], __shfl_xor_sync(0xffffffffu, mx[1], sft));
            }
            float corr[2], mu[2];
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const float mn = fmaxf(m[c], mx[c]);
                mu[c] = mn == -INFINITY ? 0.f : mn;
                corr[c] = exp2f(m[c] - mu[c]);      // m = -inf gives 0
                m[c] = mn;
                l[c] *= corr[c];
            }
            unsigned pb[2][2];   // P^T as B fragments: [key block of 16][k halves]
#pragma unroll
            for (int mb = 0; mb < 2; ++mb) {
                float p[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    p[e] = exp2f(s[mb][e] - mu[e & 1]);
                    l[e & 1] += p[e];
                }
                pb[mb][0] = movmatrix_trans(pack_bf16(p[0], p[1]));
                pb[mb][1] = movmatrix_trans(pack_bf16(p[2], p[3]));
            }
            // O^T[D x 8 heads] = O^T * corr + V^T P^T
#pragma unroll
            for (int db = 0; db < DBLK; ++db) {
                o[db][0] *= corr[0]; o[db][2] *= corr[0];
                o[db][1] *= corr[1]; o[db][3] *= corr[1];
#pragma unroll
                for (int kb = 0; kb < 2; ++kb) {
                    const int i = lane >> 3, r = lane & 7;
                    const int key = kb * 16 + (i >> 1) * 8 + r;
                    const int chunk = db * 2 + (i & 1);
                    unsigned a0, a1, a2, a3;
                    ldmatrix_x4_trans(a0, a1, a2, a3, sv + sw_off(key, chunk));
                    mma_bf16(o[db], a0, a1, a2, a3, pb[kb][0], pb[kb][1]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.empty[st]);
        }
        // l: sum the shares of the 8 lane groups that hold the same heads
#pragma unroll
        for (int sft = 4; sft < 32; sft <<= 1) {
            l[0] += __shfl_xor_sync(0xffffffffu, l[0], sft);
            l[1] += __shfl_xor_sync(0xffffffffu, l[1], sft);
        }
        // ---- merge the consumer warps through shared memory (the ring is free once all are here) ----
        asm volatile("bar.sync 1, %0;" ::"n"(DEC_CWARPS * 32));
        float* s_o = reinterpret_cast<float*>(ring);          // [warp][8 heads][D]
        float* s_m = s_o + DEC_CWARPS * 8 * D;                // [warp][8]
        float* s_l = s_m + DEC_CWARPS * 8;
#pragma unroll
        for (int db = 0; db < DBLK; ++db) {
            float* base = s_o + (size_t)warp * 8 * D;
            base[(2 * t) * D + db * 16 + g] = o[db][0];
            base[(2 * t + 1) * D + db * 16 + g] = o[db][1];
            base[(2 * t) * D + db * 16 + g + 8] = o[db][2];
            base[(2 * t + 1) * D + db * 16 + g + 8] = o[db][3];
        }
        if (g == 0) {
            s_m[warp * 8 + 2 * t] = m[0]; s_m[warp * 8 + 2 * t + 1] = m[1];
            s_l[warp * 8 + 2 * t] = l[0]; s_l[warp * 8 + 2 * t + 1] = l[1];
        }
        asm volatile("bar.sync 1, %0;" ::"n"(DEC_CWARPS * 32));
        const int ct = threadIdx.x;   // 0 .. DEC_CWARPS*32-1
        if (ct < D) {                 // eight consecutive output elements of one head
            const int h = ct / (D / 8), d0 = (ct % (D / 8)) * 8;
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < DEC_CWARPS; ++w) M = fmaxf(M, s_m[w * 8 + h]);
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            if (M > -INFINITY)
#pragma unroll
                for (int w = 0; w < DEC_CWARPS; ++w) {
                    const float f = exp2f(s_m[w * 8 + h] - M);
                    const float4 a = *reinterpret_cast<const float4*>(s_o + (size_t)w * 8 * D + h * D + d0);
                    const float4 c = *reinterpret_cast<const float4*>(s_o + (size_t)w * 8 * D + h * D + d0 + 4);
                    acc[0] += a.x * f; acc[1] += a.y * f; acc[2] += a.z * f; acc[3] += a.w * f;
                    acc[4] += c.x * f; acc[5] += c.y * f; acc[6] += c.z * f; acc[7] += c.w * f;
                }
            uint4 pk;
            pk.x = pack_bf16(acc[0], acc[1]); pk.y = pack_bf16(acc[2], acc[3]);
            pk.z = pack_bf16(acc[4], acc[5]); pk.w = pack_bf16(acc[6], acc[7]);
            *reinterpret_cast<uint4*>(part + (size_t)(h * D + d0) * 2) = pk;
        } else if (ct < D + 8) {
            const int h = ct - D;
            float M = -INFINITY, L = 0.f;
#pragma unroll
            for (int w = 0; w < DEC_CWARPS; ++w) M = fmaxf(M, s_m[w * 8 + h]);
            if (M > -INFINITY)
#pragma unroll
                for (int w = 0; w < DEC_CWARPS; ++w) L += s_l[w * 8 + h] * exp2f(s_m[w * 8 + h] - M);
            float* ml = reinterpret_cast<float*>(part + 8 * D * 2);
            ml[h] = M;
            ml[8 + h] = L;
        }
    }

    // ---- last CTA of this (cache, layer, kv head) combines the splits -----------------------------
    __syncthreads();
    if (sh.abort_flag) {
        // Somebody gave up.  Copies already issued still land in this CTA's shared memory: give every
        // full barrier a bounded chance to complete before the memory is released.
        if (threadIdx.x == 0) {
            for (int s = 0; s < DEC_STAGES; ++s)
                for (unsigned p = 0; p < 2; ++p)
                    for (unsigned w = 0; w < (1u << 16) && !mbar_test(&sh.full[s], p); ++w) __nanosleep(32);
            atomicCAS(const_cast<int*>(&vw.ctrl->status), 0, -5);   // SVLM_ERR_TIMEOUT
        }
        __syncthreads();
        return;
    }
    // The barrier above ordered every thread's partial-result stores before thread 0's release.
    unsigned* counter = reinterpret_cast<unsigned*>(vw.ws) + li * b.kv_heads + hk;
    if (threadIdx.x == 0) {
        unsigned prev;
        asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(prev) : "l"(counter) : "memory");
        sh.last = (prev == (unsigned)splits - 1);
        if (sh.last) *counter = 0;   // ready for the next launch
    }
    __syncthreads();
    if (!sh.last) return;
    // Stage the splits' records in shared memory with independent 16-byte loads by every thread (one
    // round trip to L2 for as many records as fit, normally all), then two threads per group of eight
    // output elements merge them (even and odd records) and add up through a shuffle.
    const unsigned char* parts = ws_parts + (size_t)(li * b.kv_heads + hk) * splits * REC;
    constexpr int PER_ROUND = DEC_STAGES * STAGE_BYTES / REC;
    const int pairs = G * (D / 8);                      // groups of eight output elements
    const bool two = pairs * 2 <= DEC_THREADS;          // otherwise one thread takes all records of its group
    const int grp = two ? threadIdx.x >> 1 : threadIdx.x, sub = two ? threadIdx.x & 1 : 0, stride = two ? 2 : 1;
    const bool owner = grp < pairs;
    const int h = grp / (D / 8), d0 = (grp % (D / 8)) * 8;
    float M = -INFINITY, L = 0.f;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int sp0 = 0; sp0 < splits; sp0 += PER_ROUND) {
        const int n = min(PER_ROUND, splits - sp0);
        __syncthreads();   // the ring is free (first round: merge buffers; later: previous round read)
        {
            // asynchronous 16-byte copies straight into shared memory: no registers, all in flight at once
            const unsigned char* src = parts + (size_t)sp0 * REC;
            const int n16 = n * (REC / 16);
            for (int i = threadIdx.x; i < n16; i += DEC_THREADS)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(ring + (size_t)i * 16)),
                             "l"(src + (size_t)i * 16) : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        if (owner) {
            float bm = -INFINITY;
            for (int r = 0; r < n; ++r) bm = fmaxf(bm, *reinterpret_cast<const float*>(ring + (size_t)r * REC + 8 * D * 2 + h * 4));
            const float Mn = fmaxf(M, bm);
            if (Mn > -INFINITY) {
                const float resc = exp2f(M - Mn);   // M = -inf gives 0
                L *= resc;
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] *= resc;
#pragma unroll 4
                for (int r = sub; r < n; r += stride) {
                    const unsigned char* rec = ring + (size_t)r * REC;
                    const float w = exp2f(*reinterpret_cast<const float*>(rec + 8 * D * 2 + h * 4) - Mn);
                    L += *reinterpret_cast<const float*>(rec + 8 * D * 2 + 32 + h * 4) * w;
                    const uint4 v = *reinterpret_cast<const uint4*>(rec + (size_t)(h * D + d0) * 2);
                    acc[0] += __uint_as_float(v.x << 16) * w; acc[1] += __uint_as_float(v.x & 0xffff0000u) * w;
                    acc[2] += __uint_as_float(v.y << 16) * w; acc[3] += __uint_as_float(v.y & 0xffff0000u) * w;
                    acc[4] += __uint_as_float(v.z << 16) * w; acc[5] += __uint_as_float(v.z & 0xffff0000u) * w;
                    acc[6] += __uint_as_float(v.w << 16) * w; acc[7] += __uint_as_float(v.w & 0xffff0000u) * w;
                }
                M = Mn;
            }
        }
    }
    // even + odd records (both threads of a pair used the same maximum)
    if (two) {
        L += __shfl_xor_sync(0xffffffffu, L, 1);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], 1);
    }
    if (owner && sub == 0) {
        const float inv = L > 0.f ? 1.f / L : 0.f;
        uint4 pk;
        pk.x = pack_bf16(acc[0] * inv, acc[1] * inv); pk.y = pack_bf16(acc[2] * inv, acc[3] * inv);
        pk.z = pack_bf16(acc[4] * inv, acc[5] * inv); pk.w = pack_bf16(acc[6] * inv, acc[7] * inv);
        *reinterpret_cast<uint4*>(out + ((size_t)prob * q_heads + hk * G + h) * D + d0) = pk;
    }
}

template <int D>
constexpr size_t decode_smem() {
    return sizeof(DecShared) + 1024 + (size_t)DEC_STAGES * 2 * SUB * D * 2 + 8 * D * 2 + 2 * D * 2;
}

}  // namespace

// Scratch floats needed per cache for `splits` splits (all layers at once is the largest launch).
size_t svlm_decode_ws_floats(int layers, int kv_heads, int head_dim, int splits) {
    const size_t pf = head_dim == 128 ? partial_floats<128>() : partial_floats<64>();
    return (((size_t)layers * kv_heads + 3) & ~(size_t)3) + (size_t)layers * kv_heads * splits * pf;
}

bool svlm_decode_supported(int n_pages) { return n_pages <= DEC_MAX_TILES; }

int svlm_decode_splits(int n_pages, int kv_heads, int problems) {
    // One problem (a single stream's layer): one CTA per SM, since the combine reads every split's
    // partial once and more splits than needed to fill the machine only lengthen the tail.  Several
    // problems in one launch: up to two resident CTAs per SM (measured on 16 streams x 4 KV heads:
    // 256 CTAs 64 us, 128 CTAs 70 us, 384 CTAs, which no longer fit at once, 74 us).
    int splits = (problems > 1 ? 296 : 148) / (kv_heads * problems);
    splits = splits < 1 ? 1 : splits;
    return splits > 4 * n_pages ? 4 * n_pages : splits;
}

cudaError_t svlm_launch_decode(const SvlmAttendBatch& b, int layer0, int n_layers, const void* Q, const int* q_pos,
                               int q_heads, void* out, int splits, const void* Knew, const void* Vnew, int early_loads,
                               cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(splits, b.kv_heads, b.n_caches * n_layers);
    cfg.blockDim = dim3(DEC_THREADS);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const uint16_t* Qp = (const uint16_t*)Q;
    uint16_t* Op = (uint16_t*)out;
    const uint16_t* Kn = (const uint16_t*)Knew;
    const uint16_t* Vn = (const uint16_t*)Vnew;
    cudaError_t e;
    if (b.head_dim == 128) {
        e = svlm_allow_smem<decode_kernel<128>>(decode_smem<128>());
        if (e != cudaSuccess) return e;
        cfg.dynamicSmemBytes = decode_smem<128>();
        e = cudaLaunchKernelEx(&cfg, decode_kernel<128>, b, layer0, n_layers, Qp, q_pos, q_heads, Op, splits, Kn, Vn,
                               early_loads);
    } else {
        e = svlm_allow_smem<decode_kernel<64>>(decode_smem<64>());
        if (e != cudaSuccess) return e;
        cfg.dynamicSmemBytes = decode_smem<64>();
        e = cudaLaunchKernelEx(&cfg, decode_kernel<64>, b, layer0, n_layers, Qp, q_pos, q_heads, Op, splits, Kn, Vn,
                               early_loads);
    }
    svlm_count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}
