// Split-KV decode attention (one query token per cache/layer attends over the whole retained cache;
// paper Section 3.3: per-token latency over a fixed-length context is the figure of merit), optionally
// fused with the append of that token's own key and value (one "decode step" of a layer).
//
// The step reads every stored key and value exactly once, so it is bound by HBM bandwidth.  Two kernels
// share the work split (grid = (splits, kv_heads, problems), about one CTA per SM; the G <= 8 query heads of
// a KV head ride in the N dimension of m16n8k16 MMAs, S^T = K Q^T and O^T += V^T P^T, so K and V are read
// once per group; rotation factors from a table; the new token of a fused step is patched into its
// shared-memory rows and written to the cache by the warp that owns its keys) and the combine (the six
// consumer warps merge through a bank-conflict-free buffer, a CTA's partial (o bf16, m, l) goes to scratch,
// the last CTA of a (cache, layer, KV head) to arrive merges all partials: arrival counter, nobody waits):
//
//   decode_stream_kernel   several problems per launch (batched streams, all layers of a token): a CTA walks
//       many 32-key sub-tiles; one producer thread streams them with TMA (128-byte swizzle) through a six-stage
//       ring, one stage per consumer warp, full/empty mbarriers with bounded waits.  Throughput kernel.
//
//   decode_layer_kernel    one problem per launch (one layer of one stream: the layer-sequential decoder).
//       At 19 MB per layer the data time is under 3 us and the launch is chained behind the previous layer's
//       (programmatic dependent launch): the next layer's kernel is resident while this one finishes, and
//       what a layer-step costs is the chain AFTER the query is known.  The kernel is arranged around that
//       chain.  A CTA's keys (about 270) are dealt out to the six consumer warps in 16-key units, three per
//       warp, and every warp loads its own units with cp.async into four private 4 KB slots: before the
//       dependency wait its three key units and its first value unit; the other two value units go into
//       the key slots as soon as the scores are computed and arrive (from L2, where a prefetch has put them)
//       while the softmax runs.  No producer thread, no barrier hand-offs, nothing to wait on but the
//       warp's own copies.  One pass: scores of 48 keys per warp in three independent MMA chains, one
//       softmax, P V unit by unit.
// Everything that depends on earlier kernels (query, new key/value, scratch) is read after the grid-dependency
// wait; the cache pages are not (the caller's contract, see the launcher).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "svlm_dev.h"
#include "svlm_launch.h"
#include "svlm_ptx.cuh"
#include "svlm_rope.cuh"

// Built with -DSVLM_DECODE_TRACE (the separate library the benchmark's decode-trace workload loads; never
// the product build), thread 0 of every CTA of decode_layer_kernel stamps %globaltimer at the stations
// of the chain into a device array: [launch][CTA][station], read back with svlm_debug_decode_trace_read.
#ifdef SVLM_DECODE_TRACE
#define SVLM_TR_LAUNCHES 64
#define SVLM_TR_CTAS 160
#define SVLM_TR_STATIONS 16
__device__ unsigned long long g_decode_trace[SVLM_TR_LAUNCHES][SVLM_TR_CTAS][SVLM_TR_STATIONS];
static int g_decode_trace_next = -1;
extern "C" void svlm_debug_decode_trace_start(void) { g_decode_trace_next = 0; }
extern "C" int svlm_debug_decode_trace_read(void* host) {
    return (int)cudaMemcpyFromSymbol(host, g_decode_trace, sizeof(g_decode_trace));
}
#ifndef SVLM_TRACE_MASK
#define SVLM_TRACE_MASK 0xFFFF   /* which stations are recorded (a stamp costs time: fewer stamps, truer totals) */
#endif
#define STAMP(i)                                                                                          \
    do {                                                                                                  \
        if (trace_idx >= 0 && ((SVLM_TRACE_MASK >> (i)) & 1)) {                                                                           \
            unsigned long long t_;                                                                        \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                        \
            g_decode_trace[trace_idx][blockIdx.y * gridDim.x + blockIdx.x][i] = t_;                       \
        }                                                                                                 \
    } while (0)
#define TRACE_PARAM , int trace_idx
#define TRACE_ARG , trace_idx
#else
#define STAMP(i) do { } while (0)
#define TRACE_PARAM
#define TRACE_ARG
#endif

namespace {

using namespace svlm_ptx;

constexpr int DEC_CWARPS = 6;                       // consumer warps
constexpr int DEC_THREADS = (DEC_CWARPS + 1) * 32;  // + one more warp: the producer of the streaming kernel; in
                                                    //   the per-layer kernel it only helps with the final merge
// Streaming kernel: one ring stage per consumer warp, so that a warp meets every phase of its stage's
// barriers in turn.  (With a stage shared between warps a waiter would skip phases, and a parity wait
// cannot tell the phase it wants from the one two earlier.)
constexpr int DEC_STAGES = DEC_CWARPS;
constexpr int SUB = 32;                             // keys per sub-tile of the streaming kernel
constexpr int DEC_MAX_TILES = 512;
// Per-layer kernel
constexpr int UNIT = 16;                            // keys per unit (one m16 MMA block)
constexpr int UPW = 3;                              // units per warp and round
constexpr int GROUP = DEC_CWARPS * UPW;             // units per round
constexpr int LAY_SLOTS = UPW + 1;                  // private slots per warp: the round's key units + one value unit
constexpr int MERGE_PAD = 4;                        // floats of padding per head row of the merge buffer
// The rotated query rows sit D + 8 elements apart in shared memory: the MMA fragment loads (lane = head * 4 + pair of
// dims) then hit 32 different banks; with rows D apart the eight heads of a load collide on four banks.
constexpr int QROW_PAD = 8;

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
__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Scratch layout per cache: arrival counters [layers*kv_heads] (zero between launches), then per
// (layer in launch, kv head): splits records { o[8][D] bf16, m[8] f32, l[8] f32 }.  The
// un-normalised partial outputs travel as bf16 (their error is of the size of the final rounding of
// the output), which lets the combining CTA stage every record in shared memory in one round trip.
template <int D>
__host__ __device__ constexpr int rec_bytes() { return 8 * D * 2 + 64; }
// Words in front of the records: the arrival counters [layers * kv_heads], rounded up so that the records start
// on a 16-byte boundary.
__host__ __device__ inline size_t ws_head_words(int layers, int kv_heads) {
    return ((size_t)layers * kv_heads + 3) & ~(size_t)3;
}

// The per-layer kernel's records live in an area of their own and carry a tag in every 64-bit word
// { payload, tag } (the payload: two bf16 partial outputs, or a head's maximum or sum as fp32): a reader that
// finds this launch's tag in a word has that word's payload, since an aligned 64-bit access is single-copy
// atomic.  No fence, no counter and no second round trip stand between a CTA's stores and the combining CTAs'
// loads.  Layout of the area: one epoch word per KV head (rounded up to 128 bytes), then per (KV head, split) a
// record { o[8][D] as 4 D words of 8 bytes, then per head (m, tag), (l, tag) }.  Nothing but tagged words is
// ever written to the record part, the tag of a launch is its KV head's epoch + 1 and the epoch goes up by one
// per launch, so a word left by an earlier launch never carries the current tag.
template <int D>
__host__ __device__ constexpr int ll_rec_bytes() { return 8 * D * 4 + 8 * 16; }
__host__ __device__ inline size_t ll_head_bytes(int kv_heads) { return ((size_t)kv_heads * 4 + 127) & ~(size_t)127; }
template <int D>
__host__ __device__ constexpr int partial_floats() { return rec_bytes<D>() / 4; }

__device__ __forceinline__ void st_tagged2(void* p, unsigned a, unsigned b, unsigned tag) {
    const unsigned long long hi = (unsigned long long)tag << 32;
    asm volatile("st.relaxed.gpu.global.v2.b64 [%0], {%1, %2};" ::"l"(p), "l"(hi | a), "l"(hi | b) : "memory");
}
__device__ __forceinline__ void ld_tagged2(const void* p, unsigned long long& a, unsigned long long& b) {
    asm volatile("ld.relaxed.gpu.global.v2.b64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "l"(p) : "memory");
}

// ---- the part both kernels share: from the consumer warps' accumulators to the output -----------------------

// Merge of the six consumer warps' partial results (o: this thread's MMA accumulator fragments of O^T, m and l:
// running maximum and sum of heads 2t, 2t+1) through `buf` and store of the CTA's record at `part`.  Called by
// the consumer warps only.  One slab [8 heads][D + 4] of fp32 per warp: with the padded row the 32 lanes of a
// store (4 head pairs x 8 dims) fall into 32 different banks.
// TAGGED: the record goes out in the per-layer kernel's tagged format (ll_rec_bytes).
template <int D, bool TAGGED, typename Stamp>
__device__ __forceinline__ void cta_merge_and_record(const float (&o)[D / 16][4], const float (&m)[2], const float (&l)[2],
                                                     float* buf, unsigned char* part, unsigned tag, Stamp stamp) {
    constexpr int MROW = D + MERGE_PAD, DBLK = D / 16;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
    float* s_o = buf;                                     // [warp][8 heads][MROW]
    float* s_m = s_o + DEC_CWARPS * 8 * MROW;             // [warp][8]
    float* s_l = s_m + DEC_CWARPS * 8;
    asm volatile("bar.sync 1, %0;" ::"n"(DEC_CWARPS * 32));   // every consumer warp is through with the buffer's old contents
    if (threadIdx.x == 0) stamp(7);
    {
        float* base = s_o + (size_t)warp * 8 * MROW;
#pragma unroll
        for (int db = 0; db < DBLK; ++db) {
            base[(2 * t) * MROW + db * 16 + g] = o[db][0];
            base[(2 * t + 1) * MROW + db * 16 + g] = o[db][1];
            base[(2 * t) * MROW + db * 16 + g + 8] = o[db][2];
            base[(2 * t + 1) * MROW + db * 16 + g + 8] = o[db][3];
        }
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
#pragma unroll 2
            for (int w = 0; w < DEC_CWARPS; ++w) {
                const float f = exp2f(s_m[w * 8 + h] - M);
                const float4 a = *reinterpret_cast<const float4*>(s_o + (size_t)w * 8 * MROW + h * MROW + d0);
                const float4 c = *reinterpret_cast<const float4*>(s_o + (size_t)w * 8 * MROW + h * MROW + d0 + 4);
                acc[0] += a.x * f; acc[1] += a.y * f; acc[2] += a.z * f; acc[3] += a.w * f;
                acc[4] += c.x * f; acc[5] += c.y * f; acc[6] += c.z * f; acc[7] += c.w * f;
            }
        uint4 pk;
        pk.x = pack_bf16(acc[0], acc[1]); pk.y = pack_bf16(acc[2], acc[3]);
        pk.z = pack_bf16(acc[4], acc[5]); pk.w = pack_bf16(acc[6], acc[7]);
        if constexpr (TAGGED) {
            st_tagged2(part + (size_t)(h * D + d0) * 4, pk.x, pk.y, tag);
            st_tagged2(part + (size_t)(h * D + d0) * 4 + 16, pk.z, pk.w, tag);
        } else {
            *reinterpret_cast<uint4*>(part + (size_t)(h * D + d0) * 2) = pk;
        }
    } else if (ct < D + 8) {
        const int h = ct - D;
        float M = -INFINITY, L = 0.f;
#pragma unroll
        for (int w = 0; w < DEC_CWARPS; ++w) M = fmaxf(M, s_m[w * 8 + h]);
        if (M > -INFINITY)
#pragma unroll
            for (int w = 0; w < DEC_CWARPS; ++w) L += s_l[w * 8 + h] * exp2f(s_m[w * 8 + h] - M);
        if constexpr (TAGGED) {
            st_tagged2(part + 8 * D * 4 + h * 16, __float_as_uint(M), __float_as_uint(L), tag);
        } else {
            float* ml = reinterpret_cast<float*>(part + 8 * D * 2);
            ml[h] = M;
            ml[8 + h] = L;
        }
    }
}

template <int D>
constexpr size_t merge_bytes() { return (size_t)DEC_CWARPS * 8 * (D + MERGE_PAD) * 4 + 2 * DEC_CWARPS * 8 * 4; }

// Counts this CTA as arrived; the last CTA of the (cache, layer, KV head) to arrive stages the splits'
// records in `buf` with independent 16-byte copies by every thread (one round trip to L2 for as many records as
// fit, normally all), then two threads per group of eight output elements merge them (even and odd records): first
// the maximum over the thread's records, then the weighted sums (loads in batches of four records), and the two
// halves meet through a shuffle.  Called by all DEC_THREADS threads after a __syncthreads() that follows the record's stores.
// A CTA that gave up (aborted) is counted too, so that the counter is back at zero when the launch ends, but
// does not combine.  stamp: trace hook (stations 8..11, 13).
template <int D, int BUF_BYTES, typename Stamp>
__device__ __forceinline__ void arrive_and_combine(int* s_last, unsigned* counter, int splits, const unsigned char* parts,
                                                   unsigned char* buf, int G, uint16_t* out_row0, bool aborted, Stamp stamp) {
    constexpr int REC = rec_bytes<D>();
    if (threadIdx.x == 0) {
        stamp(8);
        unsigned prev;
        asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(prev) : "l"(counter) : "memory");
        *s_last = (prev == (unsigned)splits - 1);
        if (*s_last) *counter = 0;   // ready for the next launch
        stamp(9);
        if (!*s_last) stamp(13);
    }
    __syncthreads();
    if (!*s_last || aborted) return;   // (after a time-out no output is produced; the status word says so)
    constexpr int PER_ROUND = BUF_BYTES / REC;
    const int pairs = G * (D / 8);                      // groups of eight output elements
    const bool two = pairs * 2 <= DEC_THREADS;          // otherwise one thread takes all records of its group
    const int grp = two ? threadIdx.x >> 1 : threadIdx.x, sub = two ? threadIdx.x & 1 : 0, stride = two ? 2 : 1;
    const bool owner = grp < pairs;
    const int h = owner ? grp / (D / 8) : 0, d0 = owner ? (grp % (D / 8)) * 8 : 0;
    float M = -INFINITY, L = 0.f;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int sp0 = 0; sp0 < splits; sp0 += PER_ROUND) {
        const int n = min(PER_ROUND, splits - sp0);
        __syncthreads();   // the buffer is free (first round: merge slabs; later: previous round read)
        {
            // asynchronous 16-byte copies straight into shared memory: no registers, all in flight at once
            const unsigned char* src = parts + (size_t)sp0 * REC;
            const int n16 = n * (REC / 16);
            for (int i = threadIdx.x; i < n16; i += DEC_THREADS) cp_async16(buf + (size_t)i * 16, src + (size_t)i * 16);
            cp_async_commit();
            cp_async_wait<0>();
        }
        __syncthreads();
        if (threadIdx.x == 0) stamp(10);
        // Loads are issued in batches of four records before anything uses them: shared-memory latency is paid
        // once per batch, not once per record.
        const unsigned char* ml = buf + 8 * D * 2 + h * 4;
        const unsigned char* ov = buf + (size_t)(h * D + d0) * 2;
        float bm = -INFINITY;
        for (int r0 = sub; r0 < n; r0 += 4 * stride) {
            float x[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int r = r0 + k * stride;
                x[k] = *reinterpret_cast<const float*>(ml + (size_t)(r < n ? r : sub) * REC);
            }
            bm = fmaxf(fmaxf(bm, fmaxf(x[0], x[1])), fmaxf(x[2], x[3]));   // (a repeated record changes nothing)
        }
        if (two) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 1));
        const float Mn = fmaxf(M, bm);
        if (Mn > -INFINITY) {
            const float resc = exp2f(M - Mn);   // M = -inf gives 0
            L *= resc;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] *= resc;
            for (int r0 = sub; r0 < n; r0 += 4 * stride) {
                float mr[4], lr[4];
                uint4 v[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int r = r0 + k * stride;
                    const size_t off = (size_t)(r < n ? r : sub) * REC;
                    mr[k] = r < n ? *reinterpret_cast<const float*>(ml + off) : -INFINITY;   // weight 0 past the end
                    lr[k] = *reinterpret_cast<const float*>(ml + off + 32);
                    v[k] = *reinterpret_cast<const uint4*>(ov + off);
                }
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float w = exp2f(mr[k] - Mn);
                    L += lr[k] * w;
                    acc[0] += __uint_as_float(v[k].x << 16) * w; acc[1] += __uint_as_float(v[k].x & 0xffff0000u) * w;
                    acc[2] += __uint_as_float(v[k].y << 16) * w; acc[3] += __uint_as_float(v[k].y & 0xffff0000u) * w;
                    acc[4] += __uint_as_float(v[k].z << 16) * w; acc[5] += __uint_as_float(v[k].z & 0xffff0000u) * w;
                    acc[6] += __uint_as_float(v[k].w << 16) * w; acc[7] += __uint_as_float(v[k].w & 0xffff0000u) * w;
                }
            }
            M = Mn;
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
        *reinterpret_cast<uint4*>(out_row0 + (size_t)h * D + d0) = pk;
    }
}

// The per-layer kernel's form of the same step.  One CTA pulling all the records of a KV head through its own
// port to L2 and merging them with code that runs once per launch (instruction fetch, not arithmetic, sets its
// pace) was the longest single piece of the layer-step, and the release fence plus the arrival atomic in front of
// it the next longest.  Here the first `shares` splits of a KV head split the output between them, at most eight
// groups of eight output elements each, and read their pieces of all the records in the tagged format (see
// ll_rec_bytes): a word that carries this launch's tag is that record's word.  Words that do not yet are read
// again, at most `wait_limit` times per thread; then the CTA records SVLM_ERR_TIMEOUT and writes whatever it has
// (limit 0: without a first try).  All CTAs of the launch are resident together (grid <= 2 CTAs per SM, and a
// programmatically launched successor only enters once every CTA here has passed its launch trigger), so the
// wait is for stragglers only.
//
// The loads are coalesced: eight lanes of a warp cover the (up to) eight groups of the CTA's share, which lie side
// by side in a record, the four lane groups of the 7 warps take 28 records at a time, two rounds in flight (one
// record per lane with the lanes a record apart was 2 us slower: 32 cache lines per load instruction).  The four
// record lanes meet through shuffles, the warps through `buf` (7 x 8 x 12 floats), and four threads per group
// write the result.  Split 0, which by then has seen every split's record and therefore knows that every CTA of
// the KV head has read the epoch, moves the epoch on for the next launch.  Called by all DEC_THREADS threads of the
// first `shares` splits after a __syncthreads() that follows their last use of `buf`.
// stamp: trace hook (stations 12, 15).
constexpr int DEC_WARPS = DEC_THREADS / 32;

__host__ __device__ inline int combine_shares(int groups, int splits) {
    const int want = (groups + DEC_WARPS - 1) / DEC_WARPS;
    return want < splits ? want : splits;
}

template <int D, typename Stamp>
__device__ __forceinline__ void combine_tagged(int share, int shares, int splits, const unsigned char* parts, unsigned tag,
                                               unsigned* epoch, float* buf, int G, uint16_t* out_row0, unsigned wait_limit,
                                               int* status, Stamp stamp) {
    constexpr int REC = ll_rec_bytes<D>();
    const int groups = G * (D / 8);                          // groups of eight output elements
    const int per = (groups + shares - 1) / shares;          // groups of one share
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gl = lane & 7, rl = lane >> 3;
    float* slab = buf + (size_t)(warp * 8 + gl) * 12;        // [warp][group of the round][M, L, acc[8], pad]
    bool timed_out = false;
#pragma unroll 1
    for (int g0 = 0; g0 < per; g0 += 8) {
        const int grp = share * per + g0 + gl;
        const bool valid = g0 + gl < per && grp < groups;
        const int h = valid ? grp / (D / 8) : 0, d0 = valid ? (grp % (D / 8)) * 8 : 0;
        const unsigned char* ml = parts + 8 * D * 4 + h * 16;
        const unsigned char* ov = parts + (size_t)(h * D + d0) * 4;
        float M = -INFINITY, L = 0.f;
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
        for (int r0 = warp * 4 + rl; r0 < splits; r0 += 2 * DEC_WARPS * 4) {
            unsigned long long w[2][6];                      // per record: o words 0..3, (m, tag), (l, tag)
            bool want[2];
#pragma unroll
            for (int k = 0; k < 2; ++k) want[k] = valid && r0 + k * DEC_WARPS * 4 < splits;
            for (unsigned polls = 0;; ++polls) {
                if (__builtin_expect(polls >= wait_limit, 0)) { timed_out = true; break; }
                bool ok = true;
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    if (!want[k]) continue;
                    const size_t off = (size_t)(r0 + k * DEC_WARPS * 4) * REC;
                    ld_tagged2(ov + off, w[k][0], w[k][1]);
                    ld_tagged2(ov + off + 16, w[k][2], w[k][3]);
                    ld_tagged2(ml + off, w[k][4], w[k][5]);
                }
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    if (!want[k]) continue;
#pragma unroll
                    for (int i = 0; i < 6; ++i) ok = ok && (unsigned)(w[k][i] >> 32) == tag;
                }
                if (ok) break;
            }
            float mr[2];
#pragma unroll
            for (int k = 0; k < 2; ++k) mr[k] = want[k] && !timed_out ? __uint_as_float((unsigned)w[k][4]) : -INFINITY;   // else weight 0
            const float Mn = fmaxf(M, fmaxf(mr[0], mr[1]));
            if (Mn > -INFINITY) {
                const float resc = exp2f(M - Mn);            // M = -inf gives 0
                L *= resc;
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] *= resc;
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    if (mr[k] == -INFINITY) continue;
                    const float wt = exp2f(mr[k] - Mn);
                    L += __uint_as_float((unsigned)w[k][5]) * wt;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const unsigned pr = (unsigned)w[k][i];
                        acc[2 * i] += __uint_as_float(pr << 16) * wt;
                        acc[2 * i + 1] += __uint_as_float(pr & 0xffff0000u) * wt;
                    }
                }
                M = Mn;
            }
        }
        if (threadIdx.x == 0) stamp(12);
        // the four record lanes of a group meet: common maximum first, then the sums
        const float Mw = fmaxf(fmaxf(M, __shfl_xor_sync(0xffffffffu, M, 8)),
                               fmaxf(__shfl_xor_sync(0xffffffffu, M, 16), __shfl_xor_sync(0xffffffffu, M, 24)));
        const float f = M > -INFINITY ? exp2f(M - Mw) : 0.f;
        L *= f;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] *= f;
#pragma unroll
        for (int sft = 8; sft < 32; sft <<= 1) {
            L += __shfl_xor_sync(0xffffffffu, L, sft);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], sft);
        }
        if (rl == 0) {
            *reinterpret_cast<float4*>(slab) = make_float4(Mw, L, acc[0], acc[1]);
            *reinterpret_cast<float4*>(slab + 4) = make_float4(acc[2], acc[3], acc[4], acc[5]);
            *reinterpret_cast<float2*>(slab + 8) = make_float2(acc[6], acc[7]);
        }
        __syncthreads();
        if (threadIdx.x == 0) stamp(15);
        // the warps' shares of a group meet: four threads per group, two output elements each
        if (threadIdx.x < 32) {
            const int fg = lane >> 2, e2 = lane & 3;
            const int fgrp = share * per + g0 + fg;
            const float* sl = buf + (size_t)fg * 12;
            float Ma = -INFINITY;
#pragma unroll
            for (int wp = 0; wp < DEC_WARPS; ++wp) Ma = fmaxf(Ma, sl[wp * 96]);
            float La = 0.f, a0 = 0.f, a1 = 0.f;
            if (Ma > -INFINITY)
#pragma unroll
                for (int wp = 0; wp < DEC_WARPS; ++wp) {
                    const float wt = exp2f(sl[wp * 96] - Ma);
                    const float2 a = *reinterpret_cast<const float2*>(sl + wp * 96 + 2 + 2 * e2);
                    La += sl[wp * 96 + 1] * wt;
                    a0 += a.x * wt;
                    a1 += a.y * wt;
                }
            if (g0 + fg < per && fgrp < groups) {
                const float inv = La > 0.f ? 1.f / La : 0.f;
                const int fh = fgrp / (D / 8), fd = (fgrp % (D / 8)) * 8 + 2 * e2;
                *reinterpret_cast<uint32_t*>(out_row0 + (size_t)fh * D + fd) = pack_bf16(a0 * inv, a1 * inv);
            }
        }
        if (g0 + 8 < per) __syncthreads();   // the slabs are read before the next round writes them
    }
    if (share == 0 && threadIdx.x == 0) __stcg(epoch, tag);
    if (__builtin_expect(timed_out, 0)) atomicCAS(status, 0, -5);   // SVLM_ERR_TIMEOUT
}

// =============================== streaming kernel (several problems per launch) ===============================

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
decode_stream_kernel(SvlmAttendBatch b, int layer0, int n_layers, const uint16_t* __restrict__ Q,
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
    uint16_t* s_new = s_q + 8 * (D + QROW_PAD);       // fused step: the new token's rotated key [D], then its value [D]

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
    const unsigned wait_limit = __ldcg(&vw.ctrl->wait_limit);
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
    unsigned char* ws_parts = reinterpret_cast<unsigned char*>(vw.ws + ws_head_words(b.layers, b.kv_heads));
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
                if (!mbar_wait(&sh.empty[st], ((it / DEC_STAGES) & 1) ^ 1, abort_flag, wait_limit)) break;
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
                s_q[h * (D + QROW_PAD) + pair] = __bfloat16_as_ushort(__float2bfloat16_rn(x * cs.x - y * cs.y));
                s_q[h * (D + QROW_PAD) + pair + HALF] = __bfloat16_as_ushort(__float2bfloat16_rn(y * cs.x + x * cs.y));
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
            qf[ks][0] = *reinterpret_cast<const unsigned*>(s_q + g * (D + QROW_PAD) + ks * 16 + 2 * t);
            qf[ks][1] = *reinterpret_cast<const unsigned*>(s_q + g * (D + QROW_PAD) + ks * 16 + 2 * t + 8);
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
            ok = mbar_wait(&sh.full[st], par, abort_flag, wait_limit);
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
        // the ring is free once all consumer warps are here (the merge waits for that)
        cta_merge_and_record<D, false>(o, m, l, reinterpret_cast<float*>(ring), part, 0u, [](int) {});
    }

    // ---- last CTA of this (cache, layer, kv head) combines the splits -----------------------------
    __syncthreads();
    const bool aborted = sh.abort_flag != 0;
    if (aborted && threadIdx.x == 0) {
        // Somebody gave up.  Copies already issued still land in this CTA's shared memory: give every
        // full barrier a bounded chance to complete before the memory is released.
        for (int s = 0; s < DEC_STAGES; ++s)
            for (unsigned p = 0; p < 2; ++p)
                for (unsigned w = 0; w < (1u << 12) && !mbar_test(&sh.full[s], p); ++w) __nanosleep(32);
        atomicCAS(const_cast<int*>(&vw.ctrl->status), 0, -5);   // SVLM_ERR_TIMEOUT
    }
    // The barrier above ordered every thread's partial-result stores before thread 0's release.
    arrive_and_combine<D, DEC_STAGES * STAGE_BYTES>(&sh.last, reinterpret_cast<unsigned*>(vw.ws) + li * b.kv_heads + hk, splits,
                                                    ws_parts + (size_t)(li * b.kv_heads + hk) * splits * REC, ring, G,
                                                    out + ((size_t)prob * q_heads + hk * G) * D, aborted, [](int) {});
}

template <int D>
constexpr size_t decode_stream_smem() {
    return sizeof(DecShared) + 1024 + (size_t)DEC_STAGES * 2 * SUB * D * 2 + 8 * (D + QROW_PAD) * 2 + 2 * D * 2;
}
static_assert(merge_bytes<128>() <= (size_t)DEC_STAGES * 2 * SUB * 128 * 2 && merge_bytes<64>() <= (size_t)DEC_STAGES * 2 * SUB * 64 * 2,
              "the merge slabs live in the ring");

// =============================== per-layer kernel (one problem per launch) ===============================

struct LayShared {
    int tag;                           // this launch's tag of the records' words
    int wait_limit;                    // times a combining thread may read a word again
    int pad[2];
    unsigned tile_pk[DEC_MAX_TILES];   // page | lo << 16 | hi << 24
};

// Position of a 16-byte chunk inside a unit's slot: 64-dim panels of [16 keys][128 B], chunks XOR-swizzled by
// the key's low three bits so that ldmatrix rows fall into different banks.
__device__ __forceinline__ int lay_off(int key, int chunk) {
    return (chunk >> 3) * (UNIT * 128) + key * 128 + (((chunk & 7) ^ (key & 7)) << 4);
}

template <int D>
__global__ void __launch_bounds__(DEC_THREADS, 2)
decode_layer_kernel(SvlmAttendBatch b, int layer, const uint16_t* __restrict__ Q, const int* __restrict__ q_pos, int q_heads,
                    uint16_t* __restrict__ out, int splits, const uint16_t* __restrict__ Knew,
                    const uint16_t* __restrict__ Vnew, int early_loads, unsigned char* __restrict__ records TRACE_PARAM) {
    if (threadIdx.x == 0) STAMP(0);                  // kernel entry
    constexpr int CH = D / 8;                        // 16-byte chunks per row
    constexpr int ITEM_BYTES = UNIT * D * 2;         // K or V of one unit
    constexpr int KSTEPS = D / 16;
    constexpr int DBLK = D / 16;
    constexpr int HALF = D / 2;
    constexpr int RING_BYTES = DEC_CWARPS * LAY_SLOTS * ITEM_BYTES;
    extern __shared__ unsigned char smem_raw[];
    LayShared& sh = *reinterpret_cast<LayShared*>(smem_raw);
    unsigned char* ring = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + sizeof(LayShared) + 127) & ~(uintptr_t)127);
    uint16_t* s_q = reinterpret_cast<uint16_t*>(ring + RING_BYTES);   // [8][D] bf16
    uint16_t* s_new = s_q + 8 * (D + QROW_PAD);       // fused step: the new token's rotated key [D], then its value [D]

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int split = blockIdx.x, hk = blockIdx.y;
    const SvlmAttendView& vw = b.view[0];
    const int G = q_heads / b.kv_heads;
    const bool consumer = warp < DEC_CWARPS;

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
    if (early_loads && warp == DEC_CWARPS && lane < 3) {
        // Bring the call's own small inputs towards L2 while the previous kernel still runs (a hint:
        // they are read for real only after the grid-dependency wait).
        const size_t qoff = (size_t)hk * G * D, koff = (size_t)hk * D;
        const void* p = lane == 0 ? (const void*)(Q + qoff) : lane == 1 ? (const void*)(Knew ? Knew + koff : Q + qoff)
                                                                        : (const void*)(Vnew ? Vnew + koff : Q + qoff);
        const int bytes = lane == 0 ? G * D * 2 : D * 2;
        for (int o = 0; o < bytes; o += 128)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(p) + o));
    }
    if (threadIdx.x == 0) sh.wait_limit = (int)min(__ldcg(&vw.ctrl->wait_limit), 0x7fffffffu);
    const long long shift = __ldcg(&vw.ctrl->shift_total);
    // the new token of a fused step: where it lives and whether it is still stored there
    int new_slot = -1;
    if (Knew && consumer) {
        const int s = __ldcg(vw.new_slot);
        if (__ldcg(&vw.ctrl->append_n) == 1 && __ldcg(vw.slot_gid + s) == __ldcg(&vw.ctrl->n_total) - 1) new_slot = s;
    }
    __syncthreads();
    if (threadIdx.x == 0) STAMP(1);                  // page list in shared memory

    // this CTA's run of units: eight nominal units per active page, dealt out evenly among the splits
    const int total_u = 8 * n_tiles;
    const int u0 = (int)((long long)split * total_u / splits), u1 = (int)((long long)(split + 1) * total_u / splits);
    const int n_units = u1 - u0;
    const int n_rounds = (n_units + GROUP - 1) / GROUP;
    const size_t head_row0 = ((size_t)layer * b.kv_heads + hk) * b.n_slots;
    constexpr int REC = ll_rec_bytes<D>();
    unsigned* epoch = reinterpret_cast<unsigned*>(records) + hk;
    unsigned char* ws_parts = records + ll_head_bytes(b.kv_heads) + (size_t)hk * splits * REC;   // this KV head's records
    unsigned char* part = ws_parts + (size_t)split * REC;                                       // 16-byte aligned

    if (consumer) {
        const uint16_t* Kh = vw.K + head_row0 * D;
        const uint16_t* Vh = vw.V + head_row0 * D;
        unsigned char* my = ring + warp * (LAY_SLOTS * ITEM_BYTES);   // this warp's four slots
        // This warp's units of round r are e = warp, warp + 6, warp + 12 of the round.  For unit j: the first
        // slot of the cache it covers (-1: no such unit, or no valid slot in it), the page's valid offsets.
        struct Units { int row[UPW], k0[UPW], lo[UPW], hi[UPW]; };
        auto get_units = [&](int r, Units& u) {
#pragma unroll
            for (int j = 0; j < UPW; ++j) {
                const int e = r * GROUP + warp + DEC_CWARPS * j;
                u.row[j] = -1; u.k0[j] = u.lo[j] = u.hi[j] = 0;
                if (e >= n_units) continue;
                const unsigned pk = sh.tile_pk[(u0 + e) >> 3];
                const int page = pk & 0xFFFF;
                u.lo[j] = (pk >> 16) & 0xFF; u.hi[j] = pk >> 24;
                u.k0[j] = ((u0 + e) & 7) * UNIT;
                if (u.k0[j] < u.hi[j] && u.k0[j] + UNIT > u.lo[j]) u.row[j] = page * SVLM_PAGE + u.k0[j];
            }
        };
        // all 32 lanes copy one unit (16 rows of D elements, contiguous in the cache) into a slot
        auto load_unit = [&](const uint16_t* base, int row, unsigned char* dst) {
            const uint16_t* src = base + (size_t)row * D;
#pragma unroll
            for (int i = lane; i < UNIT * CH; i += 32) cp_async16(dst + lay_off(i / CH, i % CH), src + (size_t)i * 8);
        };
        // front of a round: the key units (copy group 1) and the first value unit (copy group 2)
        auto issue_front = [&](const Units& u) {
#pragma unroll
            for (int j = 0; j < UPW; ++j)
                if (u.row[j] >= 0) load_unit(Kh, u.row[j], my + j * ITEM_BYTES);
            cp_async_commit();
            if (u.row[0] >= 0) load_unit(Vh, u.row[0], my + UPW * ITEM_BYTES);
            cp_async_commit();
        };
        Units u;
        // the value units that have to wait for a key slot go towards L2 meanwhile
        auto value_to_l2 = [&](int row) {
            for (int o = lane * 128; o < ITEM_BYTES; o += 32 * 128)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(Vh + (size_t)row * D) + o));
        };
        if (n_rounds > 0) {
            get_units(0, u);
            if (early_loads == 2) {
                // Reading ahead of a previous decode step there is time, and that kernel's short dependent loads
                // (query, partial results) queue behind whatever the whole grid has in flight: the warp asks
                // for one unit's worth at a time (keys of unit j with the values of unit j, copied or
                // prefetched) and lets it land before the next, a third of the burst's depth.
#pragma unroll
                for (int j = 0; j < UPW; ++j) {
                    if (u.row[j] >= 0) {
                        load_unit(Kh, u.row[j], my + j * ITEM_BYTES);
                        if (j == 0) load_unit(Vh, u.row[0], my + UPW * ITEM_BYTES);
                        else value_to_l2(u.row[j]);
                    }
                    cp_async_commit();
                    if (j + 1 < UPW) cp_async_wait<0>();
                }
                cp_async_commit();   // (empty: the round's "all but the latest group" then covers the last keys)
            } else {
                issue_front(u);
#pragma unroll
                for (int j = 1; j < UPW; ++j)
                    if (u.row[j] >= 0) value_to_l2(u.row[j]);
            }
        }
        if (threadIdx.x == 0) STAMP(2);              // the first round's copies are issued

        const float2* tab = reinterpret_cast<const float2*>(b.rope_tab);
        // ---- query rows: rotate at q_pos - shift_total, round to bf16, park in shared memory ----
        {
            const int pair = threadIdx.x & (HALF - 1);
            const int axis = b.rope_mode == 0 ? 0 : (pair < b.sec_t ? 0 : (pair < b.sec_th ? 1 : 2));
            // fused step: the query is the appended token, its position is already in the metadata, so the
            // rotation factors do not have to wait for the previous kernel; otherwise the position comes with the call
            long long cpos = 0;
            if (new_slot >= 0) {
                cpos = __ldcg(vw.slot_c + (size_t)axis * b.n_slots + new_slot);
            } else {
                if (early_loads) pdl_wait();
                cpos = (long long)q_pos[b.rope_mode == 0 ? 0 : axis] - shift;
            }
            const float2 cs = svlm_rope_cs(tab, HALF, pair, cpos, b.theta[pair]);
            if (new_slot >= 0 && early_loads) pdl_wait();
            if (threadIdx.x == 0) STAMP(3);          // the previous kernel has completed
            unsigned ep = 0;                         // the KV head's epoch (same round trip as the query)
            if (threadIdx.x == 0) ep = __ldcg(epoch);
            constexpr int HSTEP = (DEC_CWARPS * 32) / HALF, HN = (8 + HSTEP - 1) / HSTEP;   // heads per thread
            uint16_t qx[HN], qy[HN];
            // fused step: the new token's key and value rows come in with the query (same round trip); the key is
            // rotated with the query's factors (same token, same position) and both wait in shared memory for the
            // warp whose unit holds the token's slot
            const bool prep_new = new_slot >= 0 && threadIdx.x < HALF;
            uint16_t kx = 0, ky = 0, vx = 0, vy = 0;
            if (prep_new) {
                const size_t noff = (size_t)hk * D;
                kx = Knew[noff + pair]; ky = Knew[noff + pair + HALF];
                vx = Vnew[noff + pair]; vy = Vnew[noff + pair + HALF];
            }
#pragma unroll
            for (int k = 0; k < HN; ++k) {      // all loads first: one round trip
                const int h = threadIdx.x / HALF + k * HSTEP;
                const size_t off = (size_t)(hk * G + (h < G ? h : 0)) * D;   // n_q = 1
                qx[k] = Q[off + pair];
                qy[k] = Q[off + pair + HALF];
            }
#pragma unroll
            for (int k = 0; k < HN; ++k) {
                const int h = threadIdx.x / HALF + k * HSTEP;
                if (h >= 8) continue;
                const float x = h < G ? __bfloat162float(__ushort_as_bfloat16(qx[k])) : 0.f;
                const float y = h < G ? __bfloat162float(__ushort_as_bfloat16(qy[k])) : 0.f;
                s_q[h * (D + QROW_PAD) + pair] = __bfloat16_as_ushort(__float2bfloat16_rn(x * cs.x - y * cs.y));
                s_q[h * (D + QROW_PAD) + pair + HALF] = __bfloat16_as_ushort(__float2bfloat16_rn(y * cs.x + x * cs.y));
            }
            if (prep_new) {
                const float x = __bfloat162float(__ushort_as_bfloat16(kx)), y = __bfloat162float(__ushort_as_bfloat16(ky));
                s_new[pair] = __bfloat16_as_ushort(__float2bfloat16_rn(x * cs.x - y * cs.y));
                s_new[pair + HALF] = __bfloat16_as_ushort(__float2bfloat16_rn(y * cs.x + x * cs.y));
                s_new[D + pair] = vx;
                s_new[D + pair + HALF] = vy;
            }
            if (threadIdx.x == 0) sh.tag = (int)(ep + 1);
        }
        asm volatile("bar.sync 1, %0;" ::"n"(DEC_CWARPS * 32));   // consumer warps only
        if (threadIdx.x == 0) STAMP(4);              // rotated query in shared memory
        unsigned qf[KSTEPS][2];   // B fragments of Q^T: (d = ks*16 + 2t.., head g)
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            qf[ks][0] = *reinterpret_cast<const unsigned*>(s_q + g * (D + QROW_PAD) + ks * 16 + 2 * t);
            qf[ks][1] = *reinterpret_cast<const unsigned*>(s_q + g * (D + QROW_PAD) + ks * 16 + 2 * t + 8);
        }

        const float scale = 1.4426950408889634f * rsqrtf((float)D);
        float o[DBLK][4];
#pragma unroll
        for (int i = 0; i < DBLK; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
        float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};   // heads 2t, 2t+1 (l: this thread's share)
        const int lm_i = lane >> 3, lm_r = lane & 7;   // ldmatrix: which 8x8 matrix this lane addresses, and its row
        const int new_row16 = new_slot & ~15;          // first slot of the unit that holds the new token (fused step)

        for (int r = 0; r < n_rounds; ++r) {
            if (__builtin_expect(r > 0, 0)) {          // (larger caches only) the previous round is consumed: load the next
                __syncwarp();
                get_units(r, u);
                issue_front(u);
            }
            cp_async_wait<1>();                        // the key units have landed (the value unit may be in flight)
            __syncwarp();
            if (threadIdx.x == 32 && r == 0) STAMP(5);   // warp 1 has its keys
            // where the value units go: unit 0 has its own slot, units 1 and 2 take over the slots of key units 0 and 1
            unsigned char* const sv[UPW] = {my + UPW * ITEM_BYTES, my, my + ITEM_BYTES};
            int newj = -1;                             // the unit of this warp that holds the new token, if any
#pragma unroll
            for (int j = 0; j < UPW; ++j)
                if (new_slot >= 0 && u.row[j] == new_row16) newj = j;
            if (__builtin_expect(newj >= 0, 0)) {
                // fused append, key half: the rotated key goes into its shared-memory row and into the cache
                uint16_t* kdst = const_cast<uint16_t*>(Kh) + (size_t)new_slot * D;
                unsigned char* skw = my + newj * ITEM_BYTES;
#pragma unroll 1
                for (int e2 = lane; e2 < D; e2 += 32) {
                    const uint16_t kvl = s_new[e2];
                    kdst[e2] = kvl;
                    *reinterpret_cast<uint16_t*>(skw + lay_off(new_slot & 15, e2 >> 3) + (e2 & 7) * 2) = kvl;
                }
                __syncwarp();
            }
            // ---- S^T[48 keys x 8 heads] = K Q^T: three independent accumulation chains ----
            float s[UPW][4];
#pragma unroll
            for (int j = 0; j < UPW; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
            // (fragment loads in batches ahead of the MMAs that use them)
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ks += 2) {
                unsigned a[UPW][2][4];
#pragma unroll
                for (int j = 0; j < UPW; ++j)
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk) {
                        if (u.row[j] < 0) continue;    // warp-uniform
                        const int key = (lm_i & 1) * 8 + lm_r;
                        const int chunk = (ks + kk) * 2 + (lm_i >> 1);
                        ldmatrix_x4(a[j][kk][0], a[j][kk][1], a[j][kk][2], a[j][kk][3], my + j * ITEM_BYTES + lay_off(key, chunk));
                    }
#pragma unroll
                for (int kk = 0; kk < 2; ++kk)
#pragma unroll
                    for (int j = 0; j < UPW; ++j) {
                        if (u.row[j] < 0) continue;
                        mma_bf16(s[j], a[j][kk][0], a[j][kk][1], a[j][kk][2], a[j][kk][3], qf[ks + kk][0], qf[ks + kk][1]);
                    }
            }
            __syncwarp();                              // every lane has its key fragments: the key slots are free
#pragma unroll
            for (int j = 1; j < UPW; ++j)
                if (u.row[j] >= 0) load_unit(Vh, u.row[j], sv[j]);
            cp_async_commit();                         // copy group 3 (possibly empty)
            // scale, mask slots outside [lo, hi), column (head) maxima over the warp's keys
            float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int j = 0; j < UPW; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int key = u.k0[j] + g + (e >> 1) * 8;
                    const bool in = u.row[j] >= 0 && key >= u.lo[j] && key < u.hi[j];
                    s[j][e] = in ? s[j][e] * scale : -INFINITY;
                    mx[e & 1] = fmaxf(mx[e & 1], s[j][e]);
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
            unsigned pb[UPW][2];   // P^T as B fragments, per unit: [k halves]
#pragma unroll
            for (int j = 0; j < UPW; ++j) {
                float p[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    p[e] = exp2f(s[j][e] - mu[e & 1]);
                    l[e & 1] += p[e];
                }
                pb[j][0] = movmatrix_trans(pack_bf16(p[0], p[1]));
                pb[j][1] = movmatrix_trans(pack_bf16(p[2], p[3]));
            }
            if (threadIdx.x == 32 && r == 0) STAMP(14);  // warp 1: scores and softmax done
            if (__builtin_expect(r > 0, 0)) {
#pragma unroll
                for (int db = 0; db < DBLK; ++db) {
                    o[db][0] *= corr[0]; o[db][2] *= corr[0];
                    o[db][1] *= corr[1]; o[db][3] *= corr[1];
                }
            }
            // ---- O^T[D x 8 heads] += V^T P^T, unit by unit as the values arrive ----
#pragma unroll
            for (int j = 0; j < UPW; ++j) {
                if (j == 0) cp_async_wait<1>();        // the first value unit (copied before the scores)
                if (j == 1) cp_async_wait<0>();        // the two that followed the scores
                if (j < 2) __syncwarp();
                if (u.row[j] < 0) continue;
                if (__builtin_expect(newj == j, 0)) {  // fused append, value half
                    uint16_t* vdst = const_cast<uint16_t*>(Vh) + (size_t)new_slot * D;
#pragma unroll 1
                    for (int e2 = lane; e2 < D; e2 += 32) {
                        const uint16_t vvl = s_new[D + e2];
                        vdst[e2] = vvl;
                        *reinterpret_cast<uint16_t*>(sv[j] + lay_off(new_slot & 15, e2 >> 3) + (e2 & 7) * 2) = vvl;
                    }
                    __syncwarp();
                }
#pragma unroll
                for (int db = 0; db < DBLK; db += 4) {
                    unsigned a[4][4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int key = (lm_i >> 1) * 8 + lm_r;
                        const int chunk = (db + q) * 2 + (lm_i & 1);
                        ldmatrix_x4_trans(a[q][0], a[q][1], a[q][2], a[q][3], sv[j] + lay_off(key, chunk));
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) mma_bf16(o[db + q], a[q][0], a[q][1], a[q][2], a[q][3], pb[j][0], pb[j][1]);
                }
            }
        }
        if (threadIdx.x == 32) STAMP(6);             // warp 1 through with its units
        // l: sum the shares of the 8 lane groups that hold the same heads
#pragma unroll
        for (int sft = 4; sft < 32; sft <<= 1) {
            l[0] += __shfl_xor_sync(0xffffffffu, l[0], sft);
            l[1] += __shfl_xor_sync(0xffffffffu, l[1], sft);
        }
        // the slots are free once all consumer warps are here (the merge waits for that)
#ifdef SVLM_DECODE_TRACE
        auto stamp7 = [&](int i) { STAMP(i); };
#else
        auto stamp7 = [](int) {};
#endif
        cta_merge_and_record<D, true>(o, m, l, reinterpret_cast<float*>(ring), part, (unsigned)sh.tag, stamp7);
    }

    // ---- the first splits of this KV head combine all the splits' records -----------------------------
    __syncthreads();                                  // the merge slabs in `ring` are read
    if (threadIdx.x == 0) STAMP(8);                   // the CTA's record is on its way
    const int shares = combine_shares(G * (D / 8), splits);
    if (split >= shares) {
        if (threadIdx.x == 0) STAMP(13);
        return;
    }
#ifdef SVLM_DECODE_TRACE
    auto stamp = [&](int i) { STAMP(i); };
#else
    auto stamp = [](int) {};
#endif
    combine_tagged<D>(split, shares, splits, ws_parts, (unsigned)sh.tag, epoch, reinterpret_cast<float*>(ring), G,
                      out + (size_t)hk * G * D, (unsigned)sh.wait_limit, const_cast<int*>(&vw.ctrl->status), stamp);
#ifdef SVLM_DECODE_TRACE
    __syncthreads();
    if (threadIdx.x == 0) { STAMP(11); STAMP(13); }   // output written; leaving
#endif
}

template <int D>
constexpr size_t decode_layer_smem() {
    return sizeof(LayShared) + 128 + (size_t)DEC_CWARPS * LAY_SLOTS * UNIT * D * 2 + 8 * (D + QROW_PAD) * 2 + 2 * D * 2;
}
static_assert(merge_bytes<128>() <= (size_t)DEC_CWARPS * LAY_SLOTS * UNIT * 128 * 2 && merge_bytes<64>() <= (size_t)DEC_CWARPS * LAY_SLOTS * UNIT * 64 * 2,
              "the merge slabs live in the warps' slots");

}  // namespace

// Scratch floats needed per cache for `splits` splits (all layers at once is the largest launch).
size_t svlm_decode_ws_floats(int layers, int kv_heads, int head_dim, int splits) {
    const size_t pf = head_dim == 128 ? partial_floats<128>() : partial_floats<64>();
    return ws_head_words(layers, kv_heads) + (size_t)layers * kv_heads * splits * pf;
}

// Bytes of the per-layer kernel's area of tagged records (zero-filled at allocation, never written by anything else).
size_t svlm_decode_tagged_bytes(int kv_heads, int head_dim, int splits) {
    return ll_head_bytes(kv_heads) + (size_t)kv_heads * splits * (head_dim == 128 ? ll_rec_bytes<128>() : ll_rec_bytes<64>());
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
                               void* tagged, cudaStream_t st) {
    const int problems = b.n_caches * n_layers;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(splits, b.kv_heads, problems);
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
    if (problems == 1 && tagged) {
#ifdef SVLM_DECODE_TRACE
        int trace_idx = -1;
        if (g_decode_trace_next >= 0 && g_decode_trace_next < SVLM_TR_LAUNCHES && splits * b.kv_heads <= SVLM_TR_CTAS)
            trace_idx = g_decode_trace_next++;
#endif
        if (b.head_dim == 128) {
            e = svlm_allow_smem<decode_layer_kernel<128>>(decode_layer_smem<128>());
            if (e != cudaSuccess) return e;
            cfg.dynamicSmemBytes = decode_layer_smem<128>();
            e = cudaLaunchKernelEx(&cfg, decode_layer_kernel<128>, b, layer0, Qp, q_pos, q_heads, Op, splits, Kn, Vn,
                                   early_loads, (unsigned char*)tagged TRACE_ARG);
        } else {
            e = svlm_allow_smem<decode_layer_kernel<64>>(decode_layer_smem<64>());
            if (e != cudaSuccess) return e;
            cfg.dynamicSmemBytes = decode_layer_smem<64>();
            e = cudaLaunchKernelEx(&cfg, decode_layer_kernel<64>, b, layer0, Qp, q_pos, q_heads, Op, splits, Kn, Vn,
                                   early_loads, (unsigned char*)tagged TRACE_ARG);
        }
    } else if (b.head_dim == 128) {
        e = svlm_allow_smem<decode_stream_kernel<128>>(decode_stream_smem<128>());
        if (e != cudaSuccess) return e;
        cfg.dynamicSmemBytes = decode_stream_smem<128>();
        e = cudaLaunchKernelEx(&cfg, decode_stream_kernel<128>, b, layer0, n_layers, Qp, q_pos, q_heads, Op, splits, Kn, Vn,
                               early_loads);
    } else {
        e = svlm_allow_smem<decode_stream_kernel<64>>(decode_stream_smem<64>());
        if (e != cudaSuccess) return e;
        cfg.dynamicSmemBytes = decode_stream_smem<64>();
        e = cudaLaunchKernelEx(&cfg, decode_stream_kernel<64>, b, layer0, n_layers, Qp, q_pos, q_heads, Op, splits, Kn, Vn,
                               early_loads);
    }
    svlm_count_launch();
    return e != cudaSuccess ? e : cudaGetLastError();
}
