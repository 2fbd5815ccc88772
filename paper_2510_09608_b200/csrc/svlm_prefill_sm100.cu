// Chunk-prefill attention for sm_100a: the new chunk's queries (n_q >= 2 rows) attend over the
// retained cache plus, causally, the chunk itself (paper Section 2.1: the retained KV is reused, only
// the new second of tokens is computed).  This is the one dense contraction of the path, so it runs
// on the 5th-generation tensor cores:
//   * the G query heads that share a KV head are packed along M (row = (token, head-in-group));
//   * a CTA owns 256 such rows as two 128-row tiles A and B.  Both tiles use every K/V page the CTA
//     streams, which halves the bytes per flop that have to come out of L2 (with 128 rows per CTA
//     the K/V stream alone took as long as the whole kernel should);
//   * the K/V pages of one (tile pair, KV head) are split between the two CTAs of a thread-block
//     cluster; at the end each CTA hands the un-normalised result of one tile to the other through
//     distributed shared memory and merges and writes the tile it keeps;
//   * K and V pages (128 slots) arrive by TMA (128-byte swizzle) into one 5-stage ring, K(j) V(j)
//     K(j+1) ..., in the order the tensor pipe consumes them;
//   * one thread issues tcgen05.mma: S_A, S_B = Q K^T into two 128-column TMEM buffers, O_A, O_B += P V
//     into two TMEM accumulators, in the order PV_A(j) S_A(j+1) PV_B(j) S_B(j+1), so the tensor
//     pipe works for one tile while the other tile's softmax warpgroup exponentiates;
//   * two softmax warpgroups (one thread per row) read S with tcgen05.ld in 32-column chunks (a first
//     pass for the row maximum, a second for the exponentials, the next chunk always in flight),
//     write P as bf16 back into the TMEM columns of S, where it is the A operand of P V (no
//     shared-memory round trip); the running maximum moves lazily (O is rescaled only when the
//     maximum grows by more than 2^8);
//   * rotation factors of the queries come from a table; causal and partial-page masking only
//     touches the few pages that hold new-chunk tokens or a ring's ragged end; pages that no row
//     of the CTA may see are skipped.
// Every mbarrier wait is bounded: on expiry the CTA records SVLM_ERR_TIMEOUT in the cache's status
// word, drains its outstanding copies, frees its TMEM and returns (both CTAs of a cluster still meet
// at the hardware cluster barriers, which every thread reaches on every path).
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

#ifndef PF_ISSUERS
#define PF_ISSUERS 1                  // threads that issue tcgen05.mma (two interleaving streams measured slower)
#endif
constexpr int PF_THREADS = 288 + 32 * PF_ISSUERS;   // warps 0-3: softmax of tile A, 4-7: tile B; warp 8: TMA; warp 9 (, 10): MMA issue
constexpr int PF_RING = 5;            // K/V page stages
constexpr int PF_MAX_TILES = 512;
constexpr int PF_ROWS = 256;          // rows per CTA

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One page of one row: S (128 fp32 columns at tS, this thread's TMEM lane) -> P (bf16 pairs in the first 64
// columns of the same buffer), with the lazily moving reference maximum.  Two passes over S in halves of
// 64 columns (two 32-column loads in flight at a time): row maximum, then exponentials.  P chunk ch
// (16 columns) lands where S columns [16 ch, 16 ch + 16) were; those have been read by then and the
// loads still in flight lie beyond them.  On MASKED pages the row sees the columns [vlo, vlo + vlen): stream
// ordinals grow with the offset inside a page, so the valid and causally visible columns of a row are one interval.
template <bool MASKED>
__device__ __noinline__ void softmax_page(unsigned tS, unsigned tO, int D, unsigned vlo, unsigned vlen,
                                             float c, float m_ref, bool have_o, float& rowsum, float& corr, float& m_new) {
    auto visible = [&](int k) { return (unsigned)k - vlo < vlen; };
    float ca[32], cb[32];
    // ---- pass 1: row maximum
    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
        tmem_ld32(tS + hf * 64, ca);
        tmem_ld32(tS + hf * 64 + 32, cb);
        tmem_wait_ld();
#pragma unroll
        for (int k = 0; k < 32; ++k) {
            const float a = MASKED ? (visible(hf * 64 + k) ? ca[k] : -INFINITY) : ca[k];
            const float bq = MASKED ? (visible(hf * 64 + 32 + k) ? cb[k] : -INFINITY) : cb[k];
            mx4[k & 3] = fmaxf(mx4[k & 3], fmaxf(a, bq));
        }
    }
    tmem_ld32(tS, ca);            // first half again, for pass 2
    tmem_ld32(tS + 32, cb);
    const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * c;
    // lazy running maximum: only move the reference when it would be exceeded by 2^8
    const bool grow = mx > m_ref + 8.f;
    m_new = grow ? mx : m_ref;
    const float m_use = m_new == -INFINITY ? 0.f : m_new;
    corr = grow ? exp2f(m_ref - m_use) : 1.f;   // m_ref = -inf gives 0
    tmem_wait_ld();
    if (have_o && __any_sync(0xffffffffu, grow)) {
        // S of this page was issued after P V of the previous one: O is quiescent
#pragma unroll 1
        for (int q4 = 0; q4 < D / 32; ++q4) {
            float o[32];
            tmem_ld32(tO + q4 * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int k = 0; k < 32; ++k) o[k] *= corr;
            tmem_st32(tO + q4 * 32, o);
        }
    }
    // ---- pass 2: exponentials in stages (all scale-subtracts, all ex2, then sums and packing), so
    //      that the special-function pipe always has independent work queued
    float rs4[4] = {0.f, 0.f, 0.f, 0.f};
    auto exp_chunk = [&](float* x, int ch) {
#pragma unroll
        for (int k = 0; k < 32; ++k) x[k] = fmaf(x[k], c, -m_use);
#pragma unroll
        for (int k = 0; k < 32; ++k) x[k] = ex2(x[k]);
        if (MASKED) {
#pragma unroll
            for (int k = 0; k < 32; ++k) x[k] = visible(ch * 32 + k) ? x[k] : 0.f;
        }
        unsigned pk[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            rs4[k & 3] += x[2 * k] + x[2 * k + 1];
            pk[k] = pack2(x[2 * k], x[2 * k + 1]);
        }
        tmem_st16(tS + ch * 16, pk);
    };
    exp_chunk(ca, 0);
    exp_chunk(cb, 1);
    tmem_ld32(tS + 64, ca);       // columns 64..127 are untouched by P (columns 0..63)
    tmem_ld32(tS + 96, cb);
    tmem_wait_ld();
    exp_chunk(ca, 2);
    exp_chunk(cb, 3);
    rowsum = (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]);
}

struct PfShared {            // control part of shared memory (tiles follow, 1024-byte aligned)
    unsigned long long full[PF_RING], empty[PF_RING];
    unsigned long long s_full[2], p_full[2], all_done;
    unsigned tmem_base;
    int abort_flag;
    unsigned short tile[PF_MAX_TILES];     // page | mask << 14 | skip << 15
    unsigned short minrow[2][SVLM_PAGE];   // per softmax group: first query token that may see the column
};
static_assert(sizeof(PfShared) <= 2040, "control block must leave room for the tiles");

template <int D>
__global__ void __launch_bounds__(PF_THREADS, 1)
prefill_kernel(SvlmAttendBatch b, int layer0, int n_layers, const uint16_t* __restrict__ Q,
               const int* __restrict__ q_pos, int n_q_arg, int q_heads, uint16_t* __restrict__ out) {
    constexpr int KB = D / 64;                 // 64-element (128-byte) blocks along d
    constexpr int TILE_BYTES = 128 * D * 2;    // one K or V page of one head, or one 128-row Q tile
    constexpr int HALF = D / 2;
    extern __shared__ unsigned char smem_raw[];
    PfShared& sh = *reinterpret_cast<PfShared*>(smem_raw);
    unsigned char* tiles_base = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + sizeof(PfShared) + 1023) & ~(uintptr_t)1023);
    unsigned char* sQ = tiles_base;                           // [2 tiles][KB][128 rows][128 B]
    unsigned char* ring = sQ + 2 * TILE_BYTES;                // [stage][KB][128 keys][128 B]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = q_heads / b.kv_heads;
    const int hk = blockIdx.y;
    const int prob = blockIdx.z;
    const int ci = prob / n_layers, li = prob % n_layers;
    const int layer = layer0 + li;
    const SvlmAttendView& vw = b.view[ci];
    // rows of this problem: n_q_arg per problem, or (caches with chunks of different lengths) the cache's own count
    const int n_q = b.q_varlen ? b.q_cnt[ci] : n_q_arg;
    const size_t q_row0 = b.q_varlen ? (size_t)b.q_off[ci] : (size_t)prob * n_q_arg;   // first row in Q and out
    const size_t p_row0 = b.q_varlen ? (size_t)b.q_off[ci] : (size_t)ci * n_q_arg;     // first row in q_pos
    if ((int)(blockIdx.x >> 1) * PF_ROWS >= n_q * G) return;   // a shorter chunk: both CTAs of the pair leave at once
    const int m_total = n_q * G;
    const unsigned rank = cluster_rank();      // which half of the pages this CTA takes
    const int m0 = (blockIdx.x >> 1) * PF_ROWS;
    const int r_lo = m0 / G, r_hi = min(n_q - 1, (m0 + PF_ROWS - 1) / G);

    // The CTA's query rows and positions are read a few microseconds from now, in four dependent rounds of loads:
    // ask for their lines now, so that those rounds find them in L2 (one token's G heads are G * D * 2 contiguous bytes).
    {
        const int line_per_tok = (G * D * 2 + 127) / 128;
        for (int i = threadIdx.x; i < (r_hi - r_lo + 1) * line_per_tok; i += PF_THREADS) {
            const int tk = i / line_per_tok, ln = i % line_per_tok;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(Q + ((q_row0 + r_lo + tk) * q_heads + hk * G) * D) + ln * 128));
        }
        if (threadIdx.x < 32)
            for (int i = threadIdx.x * 32; i < (r_hi - r_lo + 1) * (b.rope_mode == 0 ? 1 : 3); i += 32 * 32)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(q_pos + (p_row0 + r_lo) * (b.rope_mode == 0 ? 1 : 3) + i));
    }
    const int n_tiles = min(vw.ctrl->n_tiles, PF_MAX_TILES);
    const long long gid_q0 = vw.ctrl->n_total - n_q;
    const long long shift = vw.ctrl->shift_total;
    const unsigned wait_limit = vw.ctrl->wait_limit;

    // ---- set-up: barriers, TMEM, page list ------------------------------------------------------
    if (threadIdx.x == 0) {
        for (int s = 0; s < PF_RING; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], PF_ISSUERS); }   // every issuer releases a page
        for (int s = 0; s < 2; ++s) { mbar_init(&sh.s_full[s], 1); mbar_init(&sh.p_full[s], 128); }
        mbar_init(&sh.all_done, PF_ISSUERS);
        sh.abort_flag = 0;
        mbar_init_fence();
    }
    for (int i = threadIdx.x; i < n_tiles; i += PF_THREADS) {
        const SvlmTile tl = vw.tiles[i];
        const int skip = tl.min_gid > gid_q0 + r_hi;
        const int mask = tl.lo > 0 || tl.hi < SVLM_PAGE || tl.max_gid > gid_q0 + r_lo;
        sh.tile[i] = (unsigned short)(tl.page | (mask << 14) | (skip << 15));
    }
    if (warp == 8) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }

    __syncthreads();   // barriers and page list are ready: the producer may start

    const size_t head_row0 = ((size_t)layer * b.kv_heads + hk) * b.n_slots;
    // this CTA's share of the processed pages: [p0, p1) of the non-skipped ones
    int n_all = 0;
    for (int j = 0; j < n_tiles; ++j) n_all += !(sh.tile[j] >> 15);
    const int half = (n_all + 1) / 2;
    const int p0 = rank == 0 ? 0 : half, p1 = rank == 0 ? half : n_all;
    const int n_proc = p1 - p0;
    volatile int* abort_flag = &sh.abort_flag;

    // K/V producer state (warp 8, lane 0); the first PF_RING - 2 loads go out before the query prologue,
    // the last two stages are borrowed by the prologue for the rotation factors
    int pr_j = 0, pr_pi = 0, pr_n = 0;
    bool pr_ok = true;
    auto produce = [&](int limit) {   // issue loads until `limit` ring items have been issued in total
        const void* tmK = vw.tmaps;
        const void* tmV = reinterpret_cast<const unsigned char*>(vw.tmaps) + 128;
        while (pr_ok && pr_n < limit && pr_j < n_tiles) {
            const unsigned t = sh.tile[pr_j];
            if (t >> 15) { ++pr_j; continue; }
            if (pr_pi < p0 || pr_pi >= p1) { ++pr_pi; ++pr_j; continue; }
            const int y = (int)(head_row0 + (size_t)(t & 0x3FFF) * SVLM_PAGE);
            const int kv = pr_n & 1;      // even items are K pages, odd items V pages of the same page
            const int st = pr_n % PF_RING;
            pr_ok = mbar_wait(&sh.empty[st], ((pr_n / PF_RING) & 1) ^ 1, abort_flag, wait_limit);   // first pass: already free
            if (!pr_ok) break;
            mbar_expect_tx(&sh.full[st], TILE_BYTES);
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
                tma_load_2d(ring + st * TILE_BYTES + kb * (128 * 128), kv ? tmV : tmK, kb * 64, y, &sh.full[st]);
            ++pr_n;
            if (kv) { ++pr_pi; ++pr_j; }
        }
    };
    if (warp == 8 && lane == 0) produce(PF_RING - 2);

    // ---- query tiles: rotate at q_pos - shift_total, round to bf16, store K-major swizzled -------
    // (1) rotation factors of the CTA's tokens, all threads: [token][pair] (cos, sin) in the last two ring
    //     stages (the rows of a token's G heads share them); with few heads per KV head there are too many
    //     tokens for that space and every thread looks its own factors up instead
    float2* s_cs = reinterpret_cast<float2*>(ring + (PF_RING - 2) * TILE_BYTES);
    const float2* tab = reinterpret_cast<const float2*>(b.rope_tab);
    const int n_tok = r_hi - r_lo + 1;
    const bool cs_shared = (size_t)n_tok * HALF * sizeof(float2) <= (size_t)2 * TILE_BYTES;
    if (cs_shared) {
        constexpr int UN = 8;   // entries per thread in flight: positions first, then the table look-ups
        const int n_ent = n_tok * HALF;
        const int pw = b.rope_mode == 0 ? 1 : 3;
        for (int base = 0; base < n_ent; base += PF_THREADS * UN) {
            long long cpos[UN];
#pragma unroll
            for (int u = 0; u < UN; ++u) {
                const int i = base + u * PF_THREADS + threadIdx.x;
                if (i < n_ent) {
                    const int tk = i / HALF, pair = i % HALF;
                    const int axis = b.rope_mode == 0 ? 0 : (pair < b.sec_t ? 0 : (pair < b.sec_th ? 1 : 2));
                    cpos[u] = (long long)__ldg(q_pos + (p_row0 + r_lo + tk) * pw + axis) - shift;
                }
            }
#pragma unroll
            for (int u = 0; u < UN; ++u) {
                const int i = base + u * PF_THREADS + threadIdx.x;
                if (i < n_ent) {
                    // a token's factors are read back 64 bytes per thread at a 64-byte lane stride: the 16-byte
                    // chunks are XOR-swizzled so that eight such lanes hit eight different bank groups
                    const int tk = i / HALF, pair = i % HALF;
                    s_cs[tk * HALF + ((((pair >> 1) ^ (pair >> 4)) << 1) | (pair & 1))] =
                        svlm_rope_cs(tab, HALF, pair, cpos[u], b.theta[pair]);
                }
            }
        }
    }
    __syncthreads();
    // (2) rotation of the 256 rows, coalesced: a work item is (row, chunk c of 8 pairs) = the 16-byte chunk c of the
    //     row's low half with its partner chunk of the high half; consecutive threads take consecutive chunks of a
    //     row, so global loads and factor look-ups of a warp touch few lines and several items are in flight.
    if (warp < 8) {
        constexpr int CH = HALF / 8;               // chunks per half row
        constexpr int ITEMS = PF_ROWS * CH, PER = ITEMS / 256, UN = 4;
        static_assert(PER % UN == 0, "items per thread");
#pragma unroll 1
        for (int it0 = 0; it0 < PER; it0 += UN) {
            uint4 lo4[UN], hi4[UN];
            int row[UN], c8v[UN], tok[UN];
#pragma unroll
            for (int u = 0; u < UN; ++u) {         // all loads of the batch first
                const int item = (it0 + u) * 256 + threadIdx.x;
                row[u] = item / CH; c8v[u] = item % CH;
                const int mg = m0 + row[u];
                const bool live = mg < m_total;
                const int r = live ? mg / G : r_lo, h = live ? mg % G : 0;
                tok[u] = r;
                const uint4* src = reinterpret_cast<const uint4*>(Q + ((q_row0 + r) * q_heads + hk * G + h) * D);
                lo4[u] = live ? __ldg(src + c8v[u]) : make_uint4(0, 0, 0, 0);
                hi4[u] = live ? __ldg(src + CH + c8v[u]) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < UN; ++u) {
                const int c8 = c8v[u], g = row[u] >> 7, m = row[u] & 127;
                const float2* cs_row = s_cs + (size_t)(tok[u] - r_lo) * HALF;
                const int* qp = q_pos + (p_row0 + tok[u]) * (b.rope_mode == 0 ? 1 : 3);
                const unsigned* lw = reinterpret_cast<const unsigned*>(&lo4[u]);
                const unsigned* hw = reinterpret_cast<const unsigned*>(&hi4[u]);
                float2 cs8[8];
                if (cs_shared) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float4 v = *reinterpret_cast<const float4*>(cs_row + (((4 * c8 + j) ^ (c8 >> 1)) << 1));
                        cs8[2 * j] = make_float2(v.x, v.y);
                        cs8[2 * j + 1] = make_float2(v.z, v.w);
                    }
                } else {
#pragma unroll 1
                    for (int i = 0; i < 8; ++i) {      // direct look-ups (too many tokens for the shared table)
                        const int pair = c8 * 8 + i;
                        const int axis = b.rope_mode == 0 ? 0 : (pair < b.sec_t ? 0 : (pair < b.sec_th ? 1 : 2));
                        const float2 v = svlm_rope_cs(tab, HALF, pair, (long long)qp[b.rope_mode == 0 ? 0 : axis] - shift, b.theta[pair]);
#pragma unroll
                        for (int q = 0; q < 8; ++q) if (q == i) cs8[q] = v;
                    }
                }
                unsigned lo_o[4], hi_o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float xl[2] = {__uint_as_float(lw[j] << 16), __uint_as_float(lw[j] & 0xffff0000u)};
                    float xh[2] = {__uint_as_float(hw[j] << 16), __uint_as_float(hw[j] & 0xffff0000u)};
                    float ol[2], oh[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float2 cs = cs8[2 * j + e];
                        ol[e] = xl[e] * cs.x - xh[e] * cs.y;
                        oh[e] = xh[e] * cs.x + xl[e] * cs.y;
                    }
                    lo_o[j] = pack2(ol[0], ol[1]);
                    hi_o[j] = pack2(oh[0], oh[1]);
                }
                // element e of the row lives in block e/64, 16-byte chunk (e%64)/8, XOR-swizzled by row&7
                unsigned char* sQg = sQ + g * TILE_BYTES;
                const int e_lo = c8 * 8, e_hi = HALF + c8 * 8;
                unsigned char* dl = sQg + (e_lo / 64) * (128 * 128) + m * 128 + ((((e_lo % 64) / 8) ^ (m & 7)) << 4);
                unsigned char* dh = sQg + (e_hi / 64) * (128 * 128) + m * 128 + ((((e_hi % 64) / 8) ^ (m & 7)) << 4);
                *reinterpret_cast<uint4*>(dl) = make_uint4(lo_o[0], lo_o[1], lo_o[2], lo_o[3]);
                *reinterpret_cast<uint4*>(dh) = make_uint4(hi_o[0], hi_o[1], hi_o[2], hi_o[3]);
            }
        }
    }
    fence_proxy_async();   // the query tiles feed the tensor core, the borrowed ring stages get TMA writes next
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem = sh.tmem_base;
    // tile g: S (then P as bf16 pairs in its first 64 columns) at columns 128 g, O at 256 + 128 g

    if (warp == 8) {
        // ================= TMA producer: K(0) V(0) K(1) V(1) ... through one ring =================
        if (lane == 0) produce(0x7fffffff);
        __syncwarp();
    } else if (warp >= 9) {
        // ================= MMA issuers: warp 9 for tile A, warp 10 for tile B =================
        // Per tile the order is S(0) | PV(j) S(j+1) | ...: the tensor pipe executes one thread's instructions in
        // order, so S(j+1) overwrites the columns of P(j) only after PV(j) has read them.  Two issuing threads keep
        // the pipe fed while one of them sits in a wait.
        // The whole warp runs the loop (waits, descriptor arithmetic: warp-uniform values the compiler can keep in
        // uniform registers); one elected lane executes the tcgen05 instructions.
        if (warp - 9 < PF_ISSUERS) {
            const int g0 = warp - 9;
            const unsigned tmem = __shfl_sync(0xffffffffu, sh.tmem_base, 0);
            const bool leader = elect_one();
            constexpr unsigned IDESC_S = make_idesc(128, 128, 0);
            constexpr unsigned IDESC_O = make_idesc(128, D, 1);
            // descriptors: the 14-bit start-address field counts 16-byte units, so moving inside a tile is an
            // addition to the low word (all tile addresses stay below the field's range: shared memory is 228 KB)
            const unsigned long long dq = smem_desc(smem_u32(sQ), 16, 1024);                    // Q, K: K-major
            const unsigned long long dk = smem_desc(smem_u32(ring), 16, 1024);
            const unsigned long long dv = smem_desc(smem_u32(ring), 128 * 128, 1024);           // V: MN-major
            // every wait gives the same answer in all lanes, so the warp stays converged
            auto wait_bar = [&](void* bar, unsigned parity) {   // one lane polls, all lanes get the answer
                int r = 1;
                if (lane == 0) r = mbar_wait(bar, parity, abort_flag, wait_limit);
                return __shfl_sync(0xffffffffu, r, 0) != 0;
            };
            auto wait_item = [&](int n) { return wait_bar(&sh.full[n % PF_RING], (n / PF_RING) & 1); };
            auto issue_S = [&](int g, int j, bool release) {      // S_g = Q_g K(j)^T; K(j) is ring item 2j
                const int st = (2 * j) % PF_RING;
                const unsigned long long a0 = dq + (unsigned)(g * TILE_BYTES >> 4), b0 = dk + (unsigned)(st * TILE_BYTES >> 4);
                if (leader) {
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const unsigned off = ((ks / 4) * (128 * 128) + (ks % 4) * 32) >> 4;
                        tc_mma_ss(tmem + g * 128, a0 + off, b0 + off, IDESC_S, ks > 0);
                    }
                    tc_commit(&sh.s_full[g]);
                    if (release) tc_commit(&sh.empty[st]);
                }
                __syncwarp();
            };
            auto issue_PV = [&](int g, int j, bool release) {     // O_g += P_g V(j); V(j) is ring item 2j+1
                const int st = (2 * j + 1) % PF_RING;
                const unsigned long long b0 = dv + (unsigned)(st * TILE_BYTES >> 4);
                if (leader) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)      // 128 keys, 16 per MMA: A = 8 TMEM columns of bf16 pairs
                        tc_mma_ts(tmem + 256 + g * 128, tmem + g * 128 + ks * 8, b0 + (unsigned)(ks * 2048 >> 4), IDESC_O,
                                  (j > 0) || (ks > 0));
                    if (release) tc_commit(&sh.empty[st]);
                }
                __syncwarp();
            };
            // with one issuer the thread serves both tiles in turn and releases a page after tile B's use of it
            constexpr int NG = 3 - PF_ISSUERS;      // tiles per issuer: 1 or 2
            bool ok = true;
            if (n_proc > 0) {
                ok = wait_item(0);
                if (ok) {
                    tc_fence_after();
#pragma unroll
                    for (int i = 0; i < NG; ++i) issue_S(g0 + i, 0, i == NG - 1);
                }
            }
            for (int j = 0; j < n_proc && ok; ++j) {
                ok = wait_item(2 * j + 1);                                                   // V(j)
                if (ok && j + 1 < n_proc) ok = wait_item(2 * j + 2);                         // K(j+1)
#pragma unroll
                for (int i = 0; i < NG && ok; ++i) {
                    ok = wait_bar(&sh.p_full[g0 + i], j & 1);                                 // P(j)
                    if (!ok) break;
                    tc_fence_after();
                    issue_PV(g0 + i, j, i == NG - 1);
                    if (j + 1 < n_proc) issue_S(g0 + i, j + 1, i == NG - 1);
                }
            }
            if (ok && leader) {
                if (n_proc > 0) tc_commit(&sh.all_done);
                else mbar_arrive(&sh.all_done);   // nothing was issued: nothing to track
            }
        }
        __syncwarp();
    } else {
        // ================= softmax groups: one thread per row of tile g =================
        const int g = warp >> 2;
        const int m = threadIdx.x & 127;
        const int mg = m0 + g * 128 + m;
        const int r = min(mg / G, n_q - 1);
        const unsigned lane_base = (unsigned)((warp & 3) * 32) << 16;
        const unsigned tS = tmem + g * 128 + lane_base, tO = tmem + 256 + g * 128 + lane_base;
        const float c = 1.4426950408889634f * rsqrtf((float)D);
        const unsigned short* mrow = sh.minrow[g];
        float m_ref = -INFINITY, l = 0.f;
        int pi = 0, it = 0;
        bool ok = true;
        for (int j = 0; j < n_tiles && ok; ++j) {
            const unsigned t = sh.tile[j];
            if (t >> 15) continue;
            if (pi < p0 || pi >= p1) { ++pi; continue; }
            ++pi;
            const bool masked = (t >> 14) & 1;
            unsigned vlo = 0, vlen = SVLM_PAGE;
            if (masked) {
                // Column m's stream ordinal relative to the first query token (clamped), shared through
                // shared memory; it grows with the column, so the columns this row may see, valid ones with
                // ordinal <= the row's, form the interval [lo, bound) found by bisection.
                const SvlmTile tl = vw.tiles[j];
                unsigned short mr = 0xFFFF;
                if (m >= tl.lo && m < tl.hi) {
                    const long long rel = vw.slot_gid[tl.page * SVLM_PAGE + m] - gid_q0;
                    mr = rel <= 0 ? 0 : (rel > 0xFFF0ll ? 0xFFF0 : (unsigned short)rel);
                }
                asm volatile("bar.sync %0, 128;" ::"r"(1 + g));   // the previous masked page's readers are done
                sh.minrow[g][m] = mr;
                asm volatile("bar.sync %0, 128;" ::"r"(1 + g));
                int a = tl.lo, e = tl.hi;
                while (a < e) {
                    const int mid = (a + e) >> 1;
                    if ((unsigned)mrow[mid] <= (unsigned)r) a = mid + 1; else e = mid;
                }
                vlo = tl.lo;
                vlen = a - tl.lo;
            }
            ok = mbar_wait(&sh.s_full[g], it & 1, abort_flag, wait_limit);
            if (!ok) break;
            tc_fence_after();
            float rowsum, corr, m_new;
            if (masked) softmax_page<true>(tS, tO, D, vlo, vlen, c, m_ref, it > 0, rowsum, corr, m_new);
            else softmax_page<false>(tS, tO, D, vlo, vlen, c, m_ref, it > 0, rowsum, corr, m_new);
            tmem_wait_st();
            l = l * corr + rowsum;
            m_ref = m_new;
            tc_fence_before();
            mbar_arrive(&sh.p_full[g]);
            ++it;
        }
        if (ok) ok = mbar_wait(&sh.all_done, 0, abort_flag, wait_limit);
        tc_fence_after();

        // ---- hand-over between the two CTAs of the cluster, then the output ------------------------
        // CTA k of the pair finishes tile k.  Both warpgroups work on both steps, each on one half of the head
        // dimension (a warp reaches its TMEM lane quadrant in either tile): first tile 1-k's (O, m, l) goes to
        // the partner, then tile k's accumulator is merged with what the partner sent and written out.  The
        // exchange area is the K/V ring, idle once a CTA's MMAs have completed (cluster barrier #1 says so for
        // both); a row's (m, l) reaches the other warpgroup through the same area.
        float* xo = reinterpret_cast<float*>(ring);                      // [D/4 chunks][128 rows] float4
        float* xml = xo + (size_t)128 * D;                               // [128 rows][2]: the partner's (m, l)
        float2* lml = reinterpret_cast<float2*>(xml + 2 * 128);          // [2 tiles][128 rows]: this CTA's (m, l)
        const bool mine = n_proc > 0;                                    // this CTA processed pages
        lml[g * 128 + m] = make_float2(ok && mine ? m_ref : -INFINITY, ok && mine ? l : 0.f);
        cluster_sync_all();   // #1: neither CTA needs its ring any more; (m, l) of every row is visible
        const int gk = (int)rank, gs = gk ^ 1;                           // tile kept, tile sent
        constexpr int QH = D / 64;                                       // 32-column chunks of O per half
        {
            const unsigned tOs = tmem + 256 + gs * 128 + lane_base;
            const unsigned dst_o = map_to_rank(xo, rank ^ 1), dst_ml = map_to_rank(xml, rank ^ 1);
#pragma unroll 1
            for (int q4 = g * QH; q4 < (g + 1) * QH; ++q4) {
                float o[32];
                if (mine) { tmem_ld32(tOs + q4 * 32, o); tmem_wait_ld(); }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 v = mine ? make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3])
                                          : make_float4(0.f, 0.f, 0.f, 0.f);
                    st_cluster_v4(dst_o + (unsigned)(((q4 * 8 + i) * 128 + m) * 16), v);
                }
            }
            if (g == 0) st_cluster_v2(dst_ml + (unsigned)(m * 8), lml[gs * 128 + m]);
        }
        cluster_sync_all();   // #2: the partner's rows have arrived
        if (ok) {
            const unsigned tOk = tmem + 256 + gk * 128 + lane_base;
            const int mgk = m0 + gk * 128 + m;
            const int rk = min(mgk / G, n_q - 1);
            const float mb = xml[m * 2], lb = xml[m * 2 + 1];
            const float2 own = lml[gk * 128 + m];
            const float ma = own.x, la = own.y;
            const float M = fmaxf(ma, mb);
            const float fa = ma == -INFINITY ? 0.f : exp2f(ma - M), fb = mb == -INFINITY ? 0.f : exp2f(mb - M);
            const float L = la * fa + lb * fb;
            const float inv = L > 0.f ? 1.f / L : 0.f;
            const float ga = fa * inv, gb = fb * inv;
            const bool live = mgk < m_total;
            uint16_t* dst = out + ((q_row0 + rk) * q_heads + hk * G + (mgk % G)) * D;
#pragma unroll 1
            for (int q4 = g * QH; q4 < (g + 1) * QH; ++q4) {
                float o[32];
                if (mine) { tmem_ld32(tOk + q4 * 32, o); tmem_wait_ld(); }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 pb = *reinterpret_cast<const float4*>(xo + (size_t)((q4 * 8 + i) * 128 + m) * 4);
                    o[4 * i] = (ma > -INFINITY ? o[4 * i] * ga : 0.f) + (mb > -INFINITY ? pb.x * gb : 0.f);
                    o[4 * i + 1] = (ma > -INFINITY ? o[4 * i + 1] * ga : 0.f) + (mb > -INFINITY ? pb.y * gb : 0.f);
                    o[4 * i + 2] = (ma > -INFINITY ? o[4 * i + 2] * ga : 0.f) + (mb > -INFINITY ? pb.z * gb : 0.f);
                    o[4 * i + 3] = (ma > -INFINITY ? o[4 * i + 3] * ga : 0.f) + (mb > -INFINITY ? pb.w * gb : 0.f);
                }
                if (live) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        uint4 v;
                        v.x = pack2(o[8 * k], o[8 * k + 1]);
                        v.y = pack2(o[8 * k + 2], o[8 * k + 3]);
                        v.z = pack2(o[8 * k + 4], o[8 * k + 5]);
                        v.w = pack2(o[8 * k + 6], o[8 * k + 7]);
                        *reinterpret_cast<uint4*>(dst + q4 * 32 + 8 * k) = v;
                    }
                }
            }
        }
    }
    if (warp >= 8) {          // the producer and issuer warps take part in the two cluster barriers as well
        cluster_sync_all();
        cluster_sync_all();
    }

    // ---- teardown ------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (sh.abort_flag) {
        // Somebody gave up.  Copies already issued still land in this CTA's shared memory: give
        // every full-barrier a bounded chance to complete before the memory is released.
        if (threadIdx.x == 0) {
            for (int s = 0; s < PF_RING; ++s)
                for (unsigned p = 0; p < 2; ++p)
                    for (unsigned w = 0; w < (1u << 16) && !mbar_test(&sh.full[s], p); ++w) __nanosleep(32);
            atomicCAS(const_cast<int*>(&vw.ctrl->status), 0, -5);   // SVLM_ERR_TIMEOUT
        }
        __syncthreads();
    }
    if (warp == 8) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
    }
}

template <int D>
constexpr size_t prefill_smem() { return sizeof(PfShared) + 1024 + (size_t)(2 + PF_RING) * 128 * D * 2; }

template <int D>
cudaError_t launch(const SvlmAttendBatch& b, int layer0, int n_layers, const uint16_t* Q, const int* q_pos, int n_q,
                   int q_heads, uint16_t* out, cudaStream_t st) {
    cudaError_t e = svlm_allow_smem<prefill_kernel<D>>(prefill_smem<D>());
    if (e != cudaSuccess) return e;
    const int G = q_heads / b.kv_heads;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * ((n_q * G + PF_ROWS - 1) / PF_ROWS), b.kv_heads, b.n_caches * n_layers);
    cfg.blockDim = dim3(PF_THREADS);
    cfg.dynamicSmemBytes = prefill_smem<D>();
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;     // the two CTAs that share the pages of one row tile
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, prefill_kernel<D>, b, layer0, n_layers, Q, q_pos, n_q, q_heads, out);
    return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

bool svlm_prefill_supported(int n_pages, int group) { return n_pages <= PF_MAX_TILES && group >= 1; }

cudaError_t svlm_launch_prefill(const SvlmAttendBatch& b, int layer0, int n_layers, const void* Q, const int* q_pos,
                                int n_q, int q_heads, void* out, cudaStream_t st) {
    const cudaError_t e = b.head_dim == 128
        ? launch<128>(b, layer0, n_layers, (const uint16_t*)Q, q_pos, n_q, q_heads, (uint16_t*)out, st)
        : launch<64>(b, layer0, n_layers, (const uint16_t*)Q, q_pos, n_q, q_heads, (uint16_t*)out, st);
    svlm_count_launch();
    return e;
}
