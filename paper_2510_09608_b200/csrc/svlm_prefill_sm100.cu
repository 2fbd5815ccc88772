// Chunk-prefill attention for sm_100a: the new chunk's queries (n_q >= 2 rows) attend over the
// retained cache plus, causally, the chunk itself (paper Section 2.1: the retained KV is reused, only
// the new second of tokens is computed).  This is the one dense contraction of the path, so it runs
// on the 5th-generation tensor cores:
//   * the G query heads that share a KV head are packed along M (row = (token, head-in-group)), so a
//     128-row tile reads each key/value tile once for the whole group;
//   * K and V tiles (one 128-slot page each) arrive by TMA (128-byte swizzle) into a 2-stage ring;
//   * S = Q K^T is issued by one thread with tcgen05.mma into one of two 128-column TMEM buffers, so
//     the tensor core computes tile j+1 while the softmax warps work on tile j;
//   * four softmax warps (one thread per row) read S with tcgen05.ld, keep a lazily updated running
//     maximum (O is rescaled only when the maximum grows by more than 2^8), write P as bf16 into
//     swizzled shared memory, and O += P V accumulates in TMEM (V is the MN-major B operand);
//   * causal and partial-page masking only touches the few tiles that hold new-chunk tokens or a
//     ring's ragged end; whole tiles that no row of the CTA may see are skipped.
// Every wait is bounded: on expiry the CTA records SVLM_ERR_TIMEOUT in the cache's status word,
// drains its outstanding copies, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "svlm_dev.h"
#include "svlm_launch.h"

namespace {

constexpr int PF_THREADS = 192;       // warps 0-3 softmax/epilogue, warp 4 TMA, warp 5 MMA issue
constexpr int PF_STAGES = 2;
constexpr int PF_MAX_TILES = 512;
constexpr unsigned WAIT_LIMIT = 1u << 20;

// ---- PTX wrappers ----------------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(void* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(void* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(void* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(void* bar, unsigned parity) {
    unsigned ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit ran out or another thread of the CTA already gave up.
__device__ __forceinline__ bool mbar_wait(void* bar, unsigned parity, volatile int* abort_flag) {
    for (unsigned it = 0; it < WAIT_LIMIT; ++it) {
        if (mbar_test(bar, parity)) return true;
        if ((it & 63) == 63) {
            if (*abort_flag) return false;
            __nanosleep(64);
        }
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const void* tmap, int x, int y, void* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(dst)), "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(void* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_mma(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                       unsigned idesc, unsigned accumulate) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.u32 p, %4, 0;\n"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld32(unsigned taddr, float* v) {
    unsigned* r = reinterpret_cast<unsigned*>(v);
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(unsigned taddr, const float* v) {
    const unsigned* r = reinterpret_cast<const unsigned*>(v);
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
                 "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
                   "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
                   "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
                 : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle, version 1 (sm_100).  Offsets in bytes.
__device__ __forceinline__ unsigned long long smem_desc(unsigned addr, unsigned lbo, unsigned sbo) {
    return (unsigned long long)((addr & 0x3FFFF) >> 4) | ((unsigned long long)(lbo >> 4) << 16) |
           ((unsigned long long)(sbo >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// kind::f16 instruction descriptor: bf16 x bf16 -> f32, A K-major, B K-major or MN-major.
__host__ __device__ constexpr unsigned make_idesc(int M, int N, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((unsigned)b_mn_major << 16) | ((unsigned)(N >> 3) << 17) |
           ((unsigned)(M >> 4) << 24);
}

__device__ __forceinline__ unsigned pack2(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<unsigned*>(&v);
}

struct PfShared {            // control part of shared memory (tiles follow, 1024-byte aligned)
    unsigned long long k_full[PF_STAGES], k_empty[PF_STAGES], v_full[PF_STAGES], v_empty[PF_STAGES];
    unsigned long long s_full[2], s_empty[2], p_full, pv_done, mask_bar;
    unsigned tmem_base;
    int abort_flag;
    int tile[PF_MAX_TILES];  // page | mask<<29 | skip<<30
    int minrow[2][SVLM_PAGE];
};

template <int D>
__global__ void __launch_bounds__(PF_THREADS, 1)
prefill_kernel(SvlmAttendBatch b, int layer0, int n_layers, const uint16_t* __restrict__ Q,
               const int* __restrict__ q_pos, int n_q, int q_heads, uint16_t* __restrict__ out) {
    constexpr int KB = D / 64;                 // 64-element (128-byte) blocks along d
    constexpr int TILE_BYTES = 128 * D * 2;    // one K or V page of one head
    extern __shared__ unsigned char smem_raw[];
    PfShared& sh = *reinterpret_cast<PfShared*>(smem_raw);
    unsigned char* tiles_base = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + sizeof(PfShared) + 1023) & ~(uintptr_t)1023);
    unsigned char* sQ = tiles_base;                           // [KB][128 rows][128 B]
    unsigned char* sK = sQ + TILE_BYTES;                      // [stage][KB][128 keys][128 B]
    unsigned char* sV = sK + PF_STAGES * TILE_BYTES;          // [stage][KB][128 keys][128 B]
    unsigned char* sP = sV + PF_STAGES * TILE_BYTES;          // [2][128 rows][128 B] (keys 0-63, 64-127)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = q_heads / b.kv_heads;
    const int hk = blockIdx.y;
    const int prob = blockIdx.z;
    const int ci = prob / n_layers, li = prob % n_layers;
    const int layer = layer0 + li;
    const SvlmAttendView& vw = b.view[ci];
    const int m_total = n_q * G;
    const int m0 = blockIdx.x * 128;
    const int r_lo = m0 / G, r_hi = min(n_q - 1, (m0 + 127) / G);

    const int n_tiles = min(vw.ctrl->n_tiles, PF_MAX_TILES);
    const long long gid_q0 = vw.ctrl->n_total - n_q;
    const long long shift = vw.ctrl->shift_total;

    // ---- set-up: barriers, TMEM, tile list ------------------------------------------------------
    if (threadIdx.x == 0) {
        for (int s = 0; s < PF_STAGES; ++s) {
            mbar_init(&sh.k_full[s], 1); mbar_init(&sh.k_empty[s], 1);
            mbar_init(&sh.v_full[s], 1); mbar_init(&sh.v_empty[s], 1);
        }
        for (int s = 0; s < 2; ++s) { mbar_init(&sh.s_full[s], 1); mbar_init(&sh.s_empty[s], 128); }
        mbar_init(&sh.p_full, 128);
        mbar_init(&sh.pv_done, 1);
        mbar_init(&sh.mask_bar, 128);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = threadIdx.x; i < n_tiles; i += PF_THREADS) {
        const SvlmTile tl = vw.tiles[i];
        const int skip = tl.min_gid > gid_q0 + r_hi;
        const int mask = tl.lo > 0 || tl.hi < SVLM_PAGE || tl.max_gid > gid_q0 + r_lo;
        sh.tile[i] = tl.page | (mask << 29) | (skip << 30);
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }

    // ---- query tile: rotate at q_pos - shift_total, round to bf16, store K-major swizzled ---------
    if (warp < 4) {
        const int m = threadIdx.x;                 // row of the tile
        const int mg = m0 + m;
        const bool live = mg < m_total;
        const int r = live ? mg / G : 0, h = live ? mg % G : 0;
        const uint16_t* src = Q + ((((size_t)prob) * n_q + r) * q_heads + hk * G + h) * D;
        const int* qp = q_pos + ((size_t)ci * n_q + r) * (b.rope_mode == 0 ? 1 : 3);
        long long c3[3];
        c3[0] = (long long)qp[0] - shift;
        c3[1] = b.rope_mode == 0 ? c3[0] : (long long)qp[1] - shift;
        c3[2] = b.rope_mode == 0 ? c3[0] : (long long)qp[2] - shift;
        constexpr int HALF = D / 2;
#pragma unroll 1
        for (int c8 = 0; c8 < HALF / 8; ++c8) {    // 8 pairs at a time: chunk c8 of the low half, same of the high half
            uint4 lo4 = make_uint4(0, 0, 0, 0), hi4 = make_uint4(0, 0, 0, 0);
            if (live) {
                lo4 = *reinterpret_cast<const uint4*>(src + c8 * 8);
                hi4 = *reinterpret_cast<const uint4*>(src + HALF + c8 * 8);
            }
            const unsigned* lw = reinterpret_cast<const unsigned*>(&lo4);
            const unsigned* hw = reinterpret_cast<const unsigned*>(&hi4);
            unsigned lo_o[4], hi_o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float xl[2] = {__uint_as_float(lw[j] << 16), __uint_as_float(lw[j] & 0xffff0000u)};
                float xh[2] = {__uint_as_float(hw[j] << 16), __uint_as_float(hw[j] & 0xffff0000u)};
                float ol[2], oh[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int pair = c8 * 8 + 2 * j + e;
                    const int axis = b.rope_mode == 0 ? 0 : (pair < b.sec_t ? 0 : (pair < b.sec_th ? 1 : 2));
                    double sn, cs;
                    sincos((double)c3[axis] * b.theta[pair], &sn, &cs);
                    ol[e] = xl[e] * (float)cs - xh[e] * (float)sn;
                    oh[e] = xh[e] * (float)cs + xl[e] * (float)sn;
                }
                lo_o[j] = pack2(ol[0], ol[1]);
                hi_o[j] = pack2(oh[0], oh[1]);
            }
            // element e of the row lives in block e/64, 16-byte chunk (e%64)/8, XOR-swizzled by row&7
            const int e_lo = c8 * 8, e_hi = HALF + c8 * 8;
            unsigned char* dl = sQ + (e_lo / 64) * (128 * 128) + m * 128 + ((((e_lo % 64) / 8) ^ (m & 7)) << 4);
            unsigned char* dh = sQ + (e_hi / 64) * (128 * 128) + m * 128 + ((((e_hi % 64) / 8) ^ (m & 7)) << 4);
            *reinterpret_cast<uint4*>(dl) = make_uint4(lo_o[0], lo_o[1], lo_o[2], lo_o[3]);
            *reinterpret_cast<uint4*>(dh) = make_uint4(hi_o[0], hi_o[1], hi_o[2], hi_o[3]);
        }
        fence_proxy_async();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem = sh.tmem_base;
    const unsigned tmem_S[2] = {tmem, tmem + 128};
    const unsigned tmem_O = tmem + 256;
    volatile int* abort_flag = &sh.abort_flag;

    const size_t head_row0 = ((size_t)layer * b.kv_heads + hk) * b.n_slots;

    if (warp == 4) {
        // ================= TMA producer =================
        if (lane == 0) {
            const void* tmK = vw.tmaps;
            const void* tmV = reinterpret_cast<const unsigned char*>(vw.tmaps) + 128;
            int it = 0;
            bool ok = true;
            for (int j = 0; j < n_tiles && ok; ++j) {
                const int t = sh.tile[j];
                if (t & (1 << 30)) continue;
                const int st = it % PF_STAGES;
                const unsigned par = ((it / PF_STAGES) & 1) ^ 1;      // first pass over a stage: already free
                const int y = (int)(head_row0 + (size_t)(t & 0xFFFFF) * SVLM_PAGE);
                ok = mbar_wait(&sh.k_empty[st], par, abort_flag);
                if (!ok) break;
                mbar_expect_tx(&sh.k_full[st], TILE_BYTES);
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
                    tma_load_2d(sK + st * TILE_BYTES + kb * (128 * 128), tmK, kb * 64, y, &sh.k_full[st]);
                ok = mbar_wait(&sh.v_empty[st], par, abort_flag);
                if (!ok) break;
                mbar_expect_tx(&sh.v_full[st], TILE_BYTES);
#pragma unroll
                for (int kb = 0; kb < KB; ++kb)
                    tma_load_2d(sV + st * TILE_BYTES + kb * (128 * 128), tmV, kb * 64, y, &sh.v_full[st]);
                ++it;
            }
        }
    } else if (warp == 5) {
        // ================= MMA issuer =================
        if (lane == 0) {
            constexpr unsigned IDESC_S = make_idesc(128, 128, 0);
            constexpr unsigned IDESC_O = make_idesc(128, D, 1);
            const unsigned q_addr = smem_u32(sQ), k_addr = smem_u32(sK), v_addr = smem_u32(sV), p_addr = smem_u32(sP);
            auto issue_S = [&](int it) {        // S[it%2] = Q K^T for the it-th processed tile
                const int st = it % PF_STAGES;
                if (!mbar_wait(&sh.k_full[st], (it / PF_STAGES) & 1, abort_flag)) return false;
                if (!mbar_wait(&sh.s_empty[it & 1], ((it >> 1) & 1) ^ 1, abort_flag)) return false;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const unsigned off = (ks / 4) * (128 * 128) + (ks % 4) * 32;
                    tc_mma(tmem_S[it & 1], smem_desc(q_addr + off, 16, 1024),
                           smem_desc(k_addr + st * TILE_BYTES + off, 16, 1024), IDESC_S, ks > 0);
                }
                tc_commit(&sh.s_full[it & 1]);
                tc_commit(&sh.k_empty[st]);
                return true;
            };
            int n_proc = 0;
            for (int j = 0; j < n_tiles; ++j) n_proc += !(sh.tile[j] & (1 << 30));
            bool ok = n_proc > 0 ? issue_S(0) : true;
            for (int it = 0; it < n_proc && ok; ++it) {
                if (it + 1 < n_proc) ok = issue_S(it + 1);
                if (!ok) break;
                const int st = it % PF_STAGES;
                ok = mbar_wait(&sh.v_full[st], (it / PF_STAGES) & 1, abort_flag) &&
                     mbar_wait(&sh.p_full, it & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {   // 128 keys, 16 per MMA
                    const unsigned a_off = (ks / 4) * (128 * 128) + (ks % 4) * 32;
                    const unsigned b_off = st * TILE_BYTES + ks * 2048;   // 16 keys x 128 B
                    tc_mma(tmem_O, smem_desc(p_addr + a_off, 16, 1024), smem_desc(v_addr + b_off, 128 * 128, 1024),
                           IDESC_O, (it > 0) || (ks > 0));
                }
                tc_commit(&sh.pv_done);
                tc_commit(&sh.v_empty[st]);
            }
        }
    } else {
        // ================= softmax, correction, epilogue (one thread per row) =================
        const int m = threadIdx.x;
        const int mg = m0 + m;
        const int r = min(mg / G, n_q - 1);
        const unsigned lane_base = (unsigned)(warp * 32) << 16;
        const float c = 1.4426950408889634f * rsqrtf((float)D);
        float m_ref = -INFINITY, l = 0.f;
        int it = 0, n_masked = 0;
        bool ok = true;
        for (int j = 0; j < n_tiles && ok; ++j) {
            const int t = sh.tile[j];
            if (t & (1 << 30)) continue;
            const bool masked = t & (1 << 29);
            if (masked) {   // per-column visibility threshold for this tile
                const SvlmTile tl = vw.tiles[j];
                const int slot = tl.page * SVLM_PAGE + m;
                int mr = 0x7fffffff;
                if (m >= tl.lo && m < tl.hi) {
                    const long long rel = vw.slot_gid[slot] - gid_q0;
                    mr = rel <= 0 ? 0 : (rel > 0x7ffffff0ll ? 0x7fffffff : (int)rel);
                }
                sh.minrow[n_masked & 1][m] = mr;
                mbar_arrive(&sh.mask_bar);                  // the 128 softmax threads meet here (bounded)
                ok = mbar_wait(&sh.mask_bar, n_masked & 1, abort_flag);
                if (!ok) break;
            }
            ok = mbar_wait(&sh.s_full[it & 1], (it >> 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            float s[128];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) tmem_ld32(tmem_S[it & 1] + lane_base + q4 * 32, s + q4 * 32);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(&sh.s_empty[it & 1]);
            if (masked) {
                const int* mr = sh.minrow[n_masked & 1];
#pragma unroll
                for (int k = 0; k < 128; ++k) s[k] = (r >= mr[k]) ? s[k] : -INFINITY;
                ++n_masked;
            }
            float mx = s[0];
#pragma unroll
            for (int k = 1; k < 128; ++k) mx = fmaxf(mx, s[k]);
            mx *= c;
            // lazy running maximum: only move the reference when it would be exceeded by 2^8
            const bool grow = mx > m_ref + 8.f;
            const float m_new = grow ? mx : m_ref;
            const float m_use = m_new == -INFINITY ? 0.f : m_new;
            float rowsum = 0.f;
            unsigned pk[64];
#pragma unroll
            for (int k = 0; k < 64; ++k) {
                const float p0 = exp2f(fmaf(s[2 * k], c, -m_use));
                const float p1 = exp2f(fmaf(s[2 * k + 1], c, -m_use));
                rowsum += p0 + p1;
                pk[k] = pack2(p0, p1);
            }
            // P's buffer and O are free once the previous tile's P V has completed
            if (it > 0) {
                ok = mbar_wait(&sh.pv_done, (it - 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
            }
            const float corr = grow ? exp2f(m_ref - m_use) : 1.f;   // m_ref = -inf gives 0
            if (it > 0 && __any_sync(0xffffffffu, grow)) {
#pragma unroll 1
                for (int q4 = 0; q4 < D / 32; ++q4) {
                    float o[32];
                    tmem_ld32(tmem_O + lane_base + q4 * 32, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int k = 0; k < 32; ++k) o[k] *= corr;
                    tmem_st32(tmem_O + lane_base + q4 * 32, o);
                }
                tmem_wait_st();
            }
            l = l * corr + rowsum;
            m_ref = m_new;
#pragma unroll
            for (int ch = 0; ch < 16; ++ch) {   // 16 chunks of 8 keys
                unsigned char* dst = sP + (ch / 8) * (128 * 128) + m * 128 + (((ch % 8) ^ (m & 7)) << 4);
                *reinterpret_cast<uint4*>(dst) = make_uint4(pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2], pk[4 * ch + 3]);
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(&sh.p_full);
            ++it;
        }
        // epilogue: O / l -> bf16 -> out[r][head]
        if (ok && it > 0) ok = mbar_wait(&sh.pv_done, (it - 1) & 1, abort_flag);
        if (ok) {
            tc_fence_after();
            const float inv = l > 0.f ? 1.f / l : 0.f;
            const bool live = mg < m_total;
            uint16_t* dst = out + ((((size_t)prob) * n_q + r) * q_heads + hk * G + (mg % G)) * D;
#pragma unroll 1
            for (int q4 = 0; q4 < D / 32; ++q4) {
                float o[32];
                if (it > 0) {
                    tmem_ld32(tmem_O + lane_base + q4 * 32, o);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int k = 0; k < 32; ++k) o[k] = 0.f;
                }
                if (live) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        uint4 v;
                        v.x = pack2(o[8 * k] * inv, o[8 * k + 1] * inv);
                        v.y = pack2(o[8 * k + 2] * inv, o[8 * k + 3] * inv);
                        v.z = pack2(o[8 * k + 4] * inv, o[8 * k + 5] * inv);
                        v.w = pack2(o[8 * k + 6] * inv, o[8 * k + 7] * inv);
                        *reinterpret_cast<uint4*>(dst + q4 * 32 + 8 * k) = v;
                    }
                }
            }
        }
    }

    // ---- teardown ------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (sh.abort_flag) {
        // Somebody gave up.  Copies already issued still land in this CTA's shared memory: give
        // every full-barrier a bounded chance to complete before the memory is released.
        if (threadIdx.x == 0) {
            for (int s = 0; s < PF_STAGES; ++s)
                for (unsigned p = 0; p < 2; ++p) {
                    for (unsigned w = 0; w < (1u << 16) && !mbar_test(&sh.k_full[s], p); ++w) __nanosleep(32);
                    for (unsigned w = 0; w < (1u << 16) && !mbar_test(&sh.v_full[s], p); ++w) __nanosleep(32);
                }
            atomicCAS(const_cast<int*>(&vw.ctrl->status), 0, -5);   // SVLM_ERR_TIMEOUT
        }
        __syncthreads();
    }
    if (warp == 4) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
    }
}

template <int D>
constexpr size_t prefill_smem() { return sizeof(PfShared) + 1024 + (size_t)(1 + 2 * PF_STAGES + 1) * 128 * D * 2 + (D == 64 ? 128 * 128 : 0); }

}  // namespace

bool svlm_prefill_supported(int n_pages, int group) { return n_pages <= PF_MAX_TILES && group >= 1; }

cudaError_t svlm_launch_prefill(const SvlmAttendBatch& b, int layer0, int n_layers, const void* Q, const int* q_pos,
                                int n_q, int q_heads, void* out, cudaStream_t st) {
    const int G = q_heads / b.kv_heads;
    dim3 grid((n_q * G + 127) / 128, b.kv_heads, b.n_caches * n_layers);
    cudaError_t e;
    if (b.head_dim == 128) {
        static bool once = false;
        if (!once) {
            e = cudaFuncSetAttribute(prefill_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)prefill_smem<128>());
            if (e != cudaSuccess) return e;
            once = true;
        }
        prefill_kernel<128><<<grid, PF_THREADS, prefill_smem<128>(), st>>>(b, layer0, n_layers, (const uint16_t*)Q, q_pos,
                                                                        n_q, q_heads, (uint16_t*)out);
    } else {
        static bool once = false;
        if (!once) {
            e = cudaFuncSetAttribute(prefill_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)prefill_smem<64>());
            if (e != cudaSuccess) return e;
            once = true;
        }
        prefill_kernel<64><<<grid, PF_THREADS, prefill_smem<64>(), st>>>(b, layer0, n_layers, (const uint16_t*)Q, q_pos,
                                                                      n_q, q_heads, (uint16_t*)out);
    }
    svlm_count_launch();
    return cudaGetLastError();
}
