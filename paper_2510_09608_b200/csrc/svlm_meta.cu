// Metadata kernels: token bookkeeping on append, and the keep-mask / prefix-scan / re-index step
// of eviction (paper Section 2.1, "Streaming-aware KV Cache" and "Contiguous RoPE").  Integer work
// only; one CTA each (a few thousand records), results must be bit-exact.
#include <cuda_runtime.h>
#include "svlm_dev.h"
#include "svlm_launch.h"

namespace {

constexpr int META_THREADS = 1024;
constexpr int META_WARPS = META_THREADS / 32;

// Block-wide exclusive scans over one value per thread.  `carry` is the running value over all
// earlier rounds; on return every thread holds the exclusive result including the carry, and carry
// has been advanced by this round's total.  All threads of the block must call.
__device__ int block_excl_sum(int v, int& carry, int* warp_buf) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) warp_buf[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int w = warp_buf[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += t;
        }
        warp_buf[lane] = w;   // inclusive over warps
    }
    __syncthreads();
    const int before = (warp ? warp_buf[warp - 1] : 0);
    const int total = warp_buf[META_WARPS - 1];
    const int res = carry + before + inc - v;
    __syncthreads();
    carry += total;
    return res;
}

__device__ long long block_excl_sum64(long long v, long long& carry, long long* warp_buf) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    long long inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        long long t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) warp_buf[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        long long w = warp_buf[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            long long t = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += t;
        }
        warp_buf[lane] = w;
    }
    __syncthreads();
    const long long before = (warp ? warp_buf[warp - 1] : 0);
    const long long total = warp_buf[META_WARPS - 1];
    const long long res = carry + before + inc - v;
    __syncthreads();
    carry += total;
    return res;
}

// Exclusive prefix maximum (carry = maximum over everything earlier).
__device__ long long block_excl_max64(long long v, long long& carry, long long* warp_buf) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long NEG = -(1ll << 62);
    long long inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        long long t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc = max(inc, t);
    }
    long long exc = __shfl_up_sync(0xffffffffu, inc, 1);
    if (lane == 0) exc = NEG;
    if (lane == 31) warp_buf[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        long long w = warp_buf[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            long long t = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w = max(w, t);
        }
        warp_buf[lane] = w;
    }
    __syncthreads();
    const long long before = (warp ? warp_buf[warp - 1] : NEG);
    const long long total = warp_buf[META_WARPS - 1];
    const long long res = max(carry, max(before, exc));
    __syncthreads();
    carry = max(carry, total);
    return res;
}

__device__ __forceinline__ int ring_slot(const SvlmCacheDev& cd, int type, long long u) {
    const int page = cd.page_table[type][(int)(u / SVLM_PAGE) & (cd.pt_size - 1)];
    return page * SVLM_PAGE + (int)(u % SVLM_PAGE);
}

__device__ __forceinline__ long long ceil_page(long long x) { return (x + SVLM_PAGE - 1) / SVLM_PAGE; }

// Rebuild the list of active pages (sink pages, then the text ring, then the vision ring).
// Called by all threads after the slot metadata of this kernel has been written and synchronised.
__device__ void rebuild_tiles(const SvlmCacheDev& cd, int sink_fill, const long long ring_lo[2],
                              const long long ring_n[2]) {
    const int n_sink_tiles = (sink_fill + SVLM_PAGE - 1) / SVLM_PAGE;
    int cnt[2];
    long long first[2];
    for (int t = 0; t < 2; ++t) {
        first[t] = ring_lo[t] / SVLM_PAGE;
        cnt[t] = ring_n[t] > ring_lo[t] ? (int)((ring_n[t] - 1) / SVLM_PAGE - first[t] + 1) : 0;
    }
    const int total = n_sink_tiles + cnt[0] + cnt[1];
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
        SvlmTile tl;
        if (i < n_sink_tiles) {
            tl.page = i;
            tl.lo = 0;
            tl.hi = min(SVLM_PAGE, sink_fill - i * SVLM_PAGE);
        } else {
            const int t = (i - n_sink_tiles < cnt[0]) ? 0 : 1;
            const long long k = first[t] + (i - n_sink_tiles - (t ? cnt[0] : 0));
            tl.page = cd.page_table[t][(int)k & (cd.pt_size - 1)];
            tl.lo = (int)max(0ll, ring_lo[t] - k * SVLM_PAGE);
            tl.hi = (int)min((long long)SVLM_PAGE, ring_n[t] - k * SVLM_PAGE);
        }
        tl.pad = 0;
        tl.min_gid = cd.slot_gid[tl.page * SVLM_PAGE + tl.lo];
        tl.max_gid = cd.slot_gid[tl.page * SVLM_PAGE + tl.hi - 1];
        cd.tiles[i] = tl;
    }
    if (threadIdx.x == 0) cd.ctrl->n_tiles = total;
}

// ---------------------------------------------------------------------------------------------
// Append of ONE token (every decode step): the same bookkeeping as the general kernel below without its
// block-wide scans, and with the list of active pages edited instead of rebuilt: a single token changes
// one entry (the last page of its ring, or of the sinks, grows by one slot) or adds one (a page opens),
// which shifts the entries behind it.  The old entries are fetched while the control block is still on
// its way, so the kernel is two dependent round trips (control block, then page table or free stack)
// instead of six.  Returns false, having done nothing, when the list is longer than the block.
__device__ __forceinline__ bool append_one_body(const SvlmCacheDev& cd, const unsigned char* types, const int* pos) {
    __shared__ int s_state;       // 0: go on; 1: append dropped (capacity)
    SvlmCtrl* ctrl = cd.ctrl;
    const int tid = threadIdx.x;
    SvlmTile old;                 // entry `tid` of the present list (garbage beyond its end; never used then)
    if (tid < cd.n_pages) old = cd.tiles[tid];
    const int n_tiles0 = ctrl->n_tiles;
    if (n_tiles0 > (int)blockDim.x) return false;          // uniform: every thread reads the same word
    const long long n_total0 = ctrl->n_total;
    const int ty = types[0] ? 1 : 0;
    const long long ord = ctrl->n_type[ty];
    const long long cursor0 = ctrl->cursor;
    const long long shift = cd.contiguous ? ctrl->shift_total : 0;
    const long long ring_n0[2] = {ctrl->ring_n[0], ctrl->ring_n[1]};
    const long long ring_lo0[2] = {ctrl->ring_lo[0], ctrl->ring_lo[1]};
    const int sink_fill0 = ctrl->sink_fill;
    const int n_stored0 = ctrl->n_stored;
    const int free_top0 = ctrl->free_top;
    long long p[3];
    if (cd.rope_mode == 0) { p[0] = p[1] = p[2] = pos[0]; }
    else { p[0] = pos[0]; p[1] = pos[1]; p[2] = pos[2]; }

    const long long gid = n_total0;
    const bool is_sink = cd.sink_any ? (gid < cd.n_sink) : (ty == 0 && ord < cd.n_sink);
    const long long u = ring_n0[ty];                       // the token's ring ordinal if it is not a sink
    const bool new_page = !is_sink && (u % SVLM_PAGE) == 0;
    // the list as it is: sink pages, text ring pages, vision ring pages
    const int ns0 = (sink_fill0 + SVLM_PAGE - 1) / SVLM_PAGE;
    int cnt0[2];
    for (int t = 0; t < 2; ++t)
        cnt0[t] = ring_n0[t] > ring_lo0[t] ? (int)((ring_n0[t] - 1) / SVLM_PAGE - ring_lo0[t] / SVLM_PAGE + 1) : 0;
    // the entry the token lands in: position in the OLD list if it exists there, else where it is inserted
    bool adds;              // a new entry appears
    int at;                 // old index of the entry that grows, or new index of the entry that appears
    if (is_sink) {
        adds = (sink_fill0 % SVLM_PAGE) == 0;
        at = adds ? ns0 : ns0 - 1;
    } else {
        const int cnt1 = (int)(u / SVLM_PAGE - ring_lo0[ty] / SVLM_PAGE + 1);
        adds = cnt1 != cnt0[ty];
        at = ns0 + (ty ? cnt0[0] : 0) + (adds ? cnt0[ty] : cnt0[ty] - 1);
    }
    if (tid == 0) {
        const bool ok = (n_stored0 + 1 <= cd.capacity) && (!new_page || free_top0 >= 1) &&
                        (!is_sink || sink_fill0 + 1 <= cd.n_sink_pages * SVLM_PAGE);
        s_state = ok ? 0 : 1;
        if (!ok) {
            ctrl->append_n = 0;
            if (ctrl->status == 0) ctrl->status = -2;   // SVLM_ERR_CAPACITY
        }
    }
    __syncthreads();                                    // also: every old entry is in registers
    if (s_state) return true;

    // entries behind an inserted one move up by one; the one that grows is rewritten by its owner
    if (tid < n_tiles0) {
        if (adds && tid >= at) cd.tiles[tid + 1] = old;
        if (!adds && tid == at) {
            old.hi += 1;
            old.max_gid = gid;
            cd.tiles[tid] = old;
        }
    }
    if (tid == 0) {
        int slot, page;
        if (is_sink) {
            slot = (int)(cd.sink_any ? gid : ord);
            page = slot / SVLM_PAGE;
        } else {
            const int pt = (int)(u / SVLM_PAGE) & (cd.pt_size - 1);
            if (new_page) {
                page = cd.free_stack[free_top0 - 1];
                cd.page_table[ty][pt] = page;
                ctrl->free_top = free_top0 - 1;
            } else {
                page = cd.page_table[ty][pt];
            }
            slot = page * SVLM_PAGE + (int)(u % SVLM_PAGE);
        }
        if (adds) {
            SvlmTile tl;
            tl.page = page;
            tl.lo = slot % SVLM_PAGE;
            tl.hi = tl.lo + 1;
            tl.pad = 0;
            tl.min_gid = tl.max_gid = gid;
            cd.tiles[at] = tl;
            ctrl->n_tiles = n_tiles0 + 1;
        }
        const long long top = max(p[0], max(p[1], p[2])) + 1;
        cd.slot_gid[slot] = gid;
        cd.slot_type[slot] = (unsigned char)ty;
        cd.slot_a[slot] = (int)max(0ll, top - cursor0);
        cd.slot_delta[slot] = 0;
        cd.new_slot[0] = slot;
        for (int k = 0; k < 3; ++k) {
            const int c = (int)(p[k] - shift);
            cd.slot_c[k * cd.n_slots + slot] = c;
            cd.new_c[k] = c;
        }
        ctrl->n_total = n_total0 + 1;
        ctrl->n_type[ty] = ord + 1;
        ctrl->cursor = max(cursor0, top);
        if (is_sink) {
            ctrl->sink_cnt[ty] += 1;
            ctrl->sink_fill = sink_fill0 + 1;
        } else {
            ctrl->ring_n[ty] = u + 1;
        }
        ctrl->n_stored = n_stored0 + 1;
        ctrl->append_n = 1;
    }
    return true;
}

// ---------------------------------------------------------------------------------------------
// Append: stream ordinal, per-type ordinal, cursor advance a = max(0, max(p)+1 - cursor),
// contiguous position c = p - shift_total, and the storage slot of each of the n new tokens.
__device__ __forceinline__ void append_meta_body(const SvlmCacheDev& cd, const unsigned char* types, const int* pos,
                                                 int n) {
    if (n == 1 && append_one_body(cd, types, pos)) return;
    __shared__ int wbuf[META_WARPS];
    __shared__ long long wbuf64[META_WARPS];
    __shared__ int s_cnt[3];     // text tokens; sink tokens of type TEXT / VISION in this append
    __shared__ int s_ok;
    SvlmCtrl* ctrl = cd.ctrl;
    const int tid = threadIdx.x;
    if (tid < 3) s_cnt[tid] = 0;
    __syncthreads();

    const long long n_total0 = ctrl->n_total;
    const long long nt0[2] = {ctrl->n_type[0], ctrl->n_type[1]};
    const long long cursor0 = ctrl->cursor;
    const long long shift = cd.contiguous ? ctrl->shift_total : 0;
    const long long ring_n0[2] = {ctrl->ring_n[0], ctrl->ring_n[1]};
    const long long ring_lo0[2] = {ctrl->ring_lo[0], ctrl->ring_lo[1]};
    const int sink_cnt0[2] = {ctrl->sink_cnt[0], ctrl->sink_cnt[1]};
    const int sink_fill0 = ctrl->sink_fill;
    const int n_stored0 = ctrl->n_stored;
    const int free_top0 = ctrl->free_top;

    // pass 0: totals
    {
        int text = 0, sink_text = 0, sink_vis = 0;
        const long long any_limit = (long long)cd.n_sink - n_total0;   // tokens i < any_limit are sinks (any-type policy)
        for (int i = tid; i < n; i += META_THREADS) {
            const int ty = types[i] ? 1 : 0;
            text += (ty == 0);
            if (cd.sink_any && i < any_limit) { sink_text += (ty == 0); sink_vis += (ty == 1); }
        }
        atomicAdd(&s_cnt[0], text);
        atomicAdd(&s_cnt[1], sink_text);
        atomicAdd(&s_cnt[2], sink_vis);
    }
    __syncthreads();
    const int n_text_new = s_cnt[0];
    int sink_new[2];
    if (cd.sink_any) {
        sink_new[0] = s_cnt[1];
        sink_new[1] = s_cnt[2];
    } else {   // the first n_sink text ordinals are the sinks
        long long room = (long long)cd.n_sink - nt0[0];
        sink_new[0] = (int)max(0ll, min(room, (long long)n_text_new));
        sink_new[1] = 0;
    }
    const int new_by_type[2] = {n_text_new, n - n_text_new};
    long long ring_n1[2];
    int pages_needed = 0;
    for (int t = 0; t < 2; ++t) {
        ring_n1[t] = ring_n0[t] + new_by_type[t] - sink_new[t];
        pages_needed += (int)(ceil_page(ring_n1[t]) - ceil_page(ring_n0[t]));
    }
    if (tid == 0) {
        const bool ok = (n_stored0 + n <= cd.capacity) && (pages_needed <= free_top0) &&
                        (sink_fill0 + sink_new[0] + sink_new[1] <= cd.n_sink_pages * SVLM_PAGE);
        s_ok = ok;
        if (!ok) {
            ctrl->append_n = 0;
            if (ctrl->status == 0) ctrl->status = -2;   // SVLM_ERR_CAPACITY
        } else {   // take pages for the ring ordinals this append opens
            int top = free_top0;
            for (int t = 0; t < 2; ++t)
                for (long long k = ceil_page(ring_n0[t]); k < ceil_page(ring_n1[t]); ++k)
                    cd.page_table[t][(int)k & (cd.pt_size - 1)] = cd.free_stack[--top];
            ctrl->free_top = top;
        }
    }
    __syncthreads();
    if (!s_ok) return;

    // pass 1: per-token scans, in rounds of one token per thread
    int text_carry = 0;
    long long top_carry = cursor0;
    const int sink_final[2] = {sink_cnt0[0] + sink_new[0], sink_cnt0[1] + sink_new[1]};
    for (int base = 0; base < n; base += META_THREADS) {
        const int i = base + tid;
        const bool live = i < n;
        const int ty = live ? (types[i] ? 1 : 0) : 1;
        long long p[3] = {0, 0, 0};
        if (live) {
            if (cd.rope_mode == 0) { p[0] = p[1] = p[2] = pos[i]; }
            else { p[0] = pos[3 * i]; p[1] = pos[3 * i + 1]; p[2] = pos[3 * i + 2]; }
        }
        const long long top = live ? max(p[0], max(p[1], p[2])) + 1 : -(1ll << 62);
        const int text_before = block_excl_sum(live && ty == 0, text_carry, wbuf);
        const long long cur_before = block_excl_max64(top, top_carry, wbuf64);
        if (!live) continue;
        const long long gid = n_total0 + i;
        const long long ord = nt0[ty] + (ty == 0 ? text_before : i - text_before);
        const long long a = max(0ll, top - cur_before);
        const bool is_sink = cd.sink_any ? (gid < cd.n_sink) : (ty == 0 && ord < cd.n_sink);
        int slot;
        if (is_sink) slot = (int)(cd.sink_any ? gid : ord);
        else slot = ring_slot(cd, ty, ord - sink_final[ty]);
        cd.slot_gid[slot] = gid;
        cd.slot_type[slot] = (unsigned char)ty;
        cd.slot_a[slot] = (int)a;
        cd.slot_delta[slot] = 0;
        cd.new_slot[i] = slot;
        for (int k = 0; k < 3; ++k) {
            const int c = (int)(p[k] - shift);
            cd.slot_c[k * cd.n_slots + slot] = c;
            cd.new_c[3 * i + k] = c;
        }
    }
    __syncthreads();
    const int sink_fill1 = sink_fill0 + sink_new[0] + sink_new[1];
    rebuild_tiles(cd, sink_fill1, ring_lo0, ring_n1);
    if (tid == 0) {
        ctrl->n_total = n_total0 + n;
        ctrl->n_type[0] = nt0[0] + new_by_type[0];
        ctrl->n_type[1] = nt0[1] + new_by_type[1];
        ctrl->cursor = top_carry;
        ctrl->ring_n[0] = ring_n1[0];
        ctrl->ring_n[1] = ring_n1[1];
        ctrl->sink_cnt[0] = sink_final[0];
        ctrl->sink_cnt[1] = sink_final[1];
        ctrl->sink_fill = sink_fill1;
        ctrl->n_stored = n_stored0 + n;
        ctrl->append_n = n;
    }
}

// Number of entries of the sorted list g[0..n) that are smaller than key.
__device__ __forceinline__ int count_below(const long long* g, int n, long long key) {
    int lo = 0, hi = n;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (g[mid] < key) lo = mid + 1; else hi = mid;
    }
    return lo;
}

constexpr int EV_SMEM = 2048;   // evicted tokens of one call whose lists also fit in shared memory
constexpr int KEPT_BATCH = 2;   // retained tokens a thread handles per round (loads of a round are issued together)
constexpr int EV_CLUSTER = 8;   // CTAs (one thread-block cluster) that share the retained tokens of one cache

__device__ __forceinline__ unsigned cluster_ctarank() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// All threads of all CTAs of the cluster; orders their global-memory accesses before and after it.
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// ---------------------------------------------------------------------------------------------
// Evict: keep-mask (a suffix of each ring plus the sinks), prefix sums of the evicted tokens'
// cursor advances, and the left-shift E(i) of every retained token i: the advances of all evicted
// tokens that precede it in the stream.
//
// The kernel is a chain of dependent round trips to L2 (page table -> slot -> ordinal -> search ->
// position), so every stage issues the loads of all its items before it uses any of them, and the
// lists that the searches walk sit in shared memory when they fit.  A cluster of EV_CLUSTER CTAs
// serves one cache: every CTA builds the (short) evicted lists for itself, the retained tokens are
// dealt out among the CTAs, and CTA 0 alone changes what the others read (after the cluster barrier)
// and keeps the books.
__device__ __forceinline__ void evict_meta_body(const SvlmCacheDev& cd) {
    const unsigned crank = cluster_ctarank();
    __shared__ long long wbuf64[2][META_WARPS];
    __shared__ long long s_gid[EV_SMEM];       // ordinals of the evicted tokens: text ring, then vision ring
    __shared__ long long s_pref[EV_SMEM + 2];  // exclusive prefix sums of their advances (n+1 entries per ring)
    __shared__ int s_moved;
    SvlmCtrl* ctrl = cd.ctrl;
    const int tid = threadIdx.x;
    if (tid == 0) s_moved = 0;

    const long long ring_n[2] = {ctrl->ring_n[0], ctrl->ring_n[1]};
    const long long lo0[2] = {ctrl->ring_lo[0], ctrl->ring_lo[1]};
    const int sink_fill = ctrl->sink_fill;
    const int free_top0 = ctrl->free_top;
    const int win[2] = {cd.text_window, cd.vision_window};
    long long lo1[2];
    int n_ev[2];
    for (int t = 0; t < 2; ++t) {
        lo1[t] = min(ring_n[t], max(lo0[t], ring_n[t] - (long long)win[t]));
        n_ev[t] = (int)(lo1[t] - lo0[t]);
    }
    if (crank == 0 && threadIdx.x == 0) ctrl->evict_moved = 0;
    const bool in_smem = n_ev[0] + n_ev[1] <= EV_SMEM;
    // where the searches read the lists of ring t
    const long long* gid_list[2] = {in_smem ? s_gid : cd.ev_gid[0], in_smem ? s_gid + n_ev[0] : cd.ev_gid[1]};
    const long long* pref_list[2] = {in_smem ? s_pref : cd.ev_pref[0], in_smem ? s_pref + n_ev[0] + 1 : cd.ev_pref[1]};
    __syncthreads();

    // evicted tokens of both rings in ordinal (= stream) order, with exclusive prefix sums of a
    long long freed[2] = {0, 0};
    for (int base = 0; base < max(n_ev[0], n_ev[1]); base += META_THREADS) {
        const int i = base + tid;
        int slot[2] = {-1, -1};
        long long a[2] = {0, 0}, g[2] = {0, 0};
#pragma unroll
        for (int t = 0; t < 2; ++t)
            if (i < n_ev[t]) slot[t] = ring_slot(cd, t, lo0[t] + i);
#pragma unroll
        for (int t = 0; t < 2; ++t)
            if (slot[t] >= 0) {
                a[t] = cd.contiguous ? cd.slot_a[slot[t]] : 0;
                g[t] = cd.slot_gid[slot[t]];
            }
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            if (base >= n_ev[t]) continue;            // uniform over the block
            const long long ex = block_excl_sum64(a[t], freed[t], wbuf64[t]);
            if (slot[t] >= 0) {
                if (in_smem) {
                    s_gid[(t ? n_ev[0] : 0) + i] = g[t];
                    s_pref[(t ? n_ev[0] + 1 : 0) + i] = ex;
                } else {   // every CTA writes the same values
                    cd.ev_gid[t][i] = g[t];
                    cd.ev_pref[t][i] = ex;
                }
            }
        }
    }
    if (tid == 0)
        for (int t = 0; t < 2; ++t) {
            if (in_smem) s_pref[(t ? n_ev[0] + 1 : 0) + n_ev[t]] = freed[t];
            else cd.ev_pref[t][n_ev[t]] = freed[t];
        }
    __syncthreads();
    cluster_barrier();   // every CTA has read the control block and the evicted slots' metadata
    if (crank == 0) {    // now the evicted slots can be marked empty
        for (int t = 0; t < 2; ++t)
            for (int i = tid; i < n_ev[t]; i += META_THREADS) {
                const int slot = ring_slot(cd, t, lo0[t] + i);
                cd.slot_gid[slot] = -1;
                cd.slot_delta[slot] = 0;
            }
    }

    // retained tokens: sinks, then the kept suffix of each ring; CTA r takes every EV_CLUSTER-th block of them
    const long long kept_ring[2] = {ring_n[0] - lo1[0], ring_n[1] - lo1[1]};
    const long long n_kept = sink_fill + kept_ring[0] + kept_ring[1];
    int moved = 0;
    for (long long base = (long long)crank * KEPT_BATCH * META_THREADS; base < n_kept;
         base += (long long)EV_CLUSTER * KEPT_BATCH * META_THREADS) {
        int slot[KEPT_BATCH];
        long long g[KEPT_BATCH];
        int E[KEPT_BATCH], c[KEPT_BATCH][3];
#pragma unroll
        for (int u = 0; u < KEPT_BATCH; ++u) {
            const long long i = base + (long long)u * META_THREADS + tid;
            if (i >= n_kept) slot[u] = -1;
            else if (i < sink_fill) slot[u] = (int)i;
            else if (i < sink_fill + kept_ring[0]) slot[u] = ring_slot(cd, 0, lo1[0] + (i - sink_fill));
            else slot[u] = ring_slot(cd, 1, lo1[1] + (i - sink_fill - kept_ring[0]));
        }
#pragma unroll
        for (int u = 0; u < KEPT_BATCH; ++u) {
            g[u] = slot[u] >= 0 ? cd.slot_gid[slot[u]] : 0;
#pragma unroll
            for (int k = 0; k < 3; ++k) c[u][k] = slot[u] >= 0 ? cd.slot_c[k * cd.n_slots + slot[u]] : 0;
        }
#pragma unroll
        for (int u = 0; u < KEPT_BATCH; ++u) {
            long long e = 0;
            if (slot[u] >= 0)
                for (int t = 0; t < 2; ++t)
                    if (n_ev[t]) e += pref_list[t][count_below(gid_list[t], n_ev[t], g[u])];
            E[u] = (int)e;
        }
#pragma unroll
        for (int u = 0; u < KEPT_BATCH; ++u) {
            if (slot[u] < 0) continue;
            cd.slot_delta[slot[u]] = E[u];
            if (E[u]) {
                moved = 1;
#pragma unroll
                for (int k = 0; k < 3; ++k) cd.slot_c[k * cd.n_slots + slot[u]] = c[u][k] - E[u];
            }
        }
    }
    if (moved) s_moved = 1;
    __syncthreads();
    if (tid == 0 && s_moved) atomicOr(&ctrl->evict_moved, 1);
    if (crank != 0) return;

    // release the pages that fell wholly below the new low-water mark (text ring's first, in ring order)
    {
        long long first[2], cnt[2];
        for (int t = 0; t < 2; ++t) {
            first[t] = lo0[t] / SVLM_PAGE;
            cnt[t] = max(0ll, min(lo1[t] / SVLM_PAGE, ceil_page(ring_n[t])) - first[t]);
        }
        for (long long i = tid; i < cnt[0] + cnt[1]; i += META_THREADS) {
            const int t = i < cnt[0] ? 0 : 1;
            const long long k = first[t] + (t ? i - cnt[0] : i);
            cd.free_stack[free_top0 + i] = cd.page_table[t][(int)k & (cd.pt_size - 1)];
        }
        if (tid == 0) ctrl->free_top = free_top0 + (int)(cnt[0] + cnt[1]);
    }
    __syncthreads();
    rebuild_tiles(cd, sink_fill, lo1, ring_n);
    if (tid == 0) {
        ctrl->ring_lo[0] = lo1[0];
        ctrl->ring_lo[1] = lo1[1];
        ctrl->shift_total += freed[0] + freed[1];
        ctrl->n_stored = (int)n_kept;
    }
}

__global__ void __launch_bounds__(META_THREADS) append_meta_kernel(SvlmCacheDev cd, const unsigned char* types,
                                                                   const int* pos, int n) {
    append_meta_body(cd, types, pos, n);
}

__global__ void __launch_bounds__(META_THREADS) evict_meta_kernel(SvlmCacheDev cd) { evict_meta_body(cd); }

// Batched forms: block i serves cache i, whose descriptor it first copies from device memory into
// shared memory.  types is [n_caches][n], pos [n_caches][n] (1D) or [n_caches][n][3].
__global__ void __launch_bounds__(META_THREADS) append_meta_batch_kernel(SvlmCacheList list, const unsigned char* types,
                                                                         const int* pos, int n) {
    __shared__ SvlmCacheDev s_cd;
    svlm_load_desc(&s_cd, list.cd[blockIdx.x]);
    append_meta_body(s_cd, types + (size_t)blockIdx.x * n, pos + (size_t)blockIdx.x * n * (s_cd.rope_mode == 0 ? 1 : 3), n);
}

__global__ void __launch_bounds__(META_THREADS) evict_meta_batch_kernel(SvlmCacheList list) {
    __shared__ SvlmCacheDev s_cd;
    svlm_load_desc(&s_cd, list.cd[blockIdx.x / EV_CLUSTER]);
    evict_meta_body(s_cd);
}

// Launch `clusters` clusters of EV_CLUSTER CTAs.
template <typename... Args>
void launch_evict_meta(void (*kernel)(Args...), int clusters, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(EV_CLUSTER * clusters);
    cfg.blockDim = dim3(META_THREADS);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = EV_CLUSTER;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, args...);
}

}  // namespace

void svlm_launch_append_meta_batch(const SvlmCacheList& list, const unsigned char* types, const int* pos, int n,
                                   cudaStream_t st) {
    append_meta_batch_kernel<<<list.n, META_THREADS, 0, st>>>(list, types, pos, n);
    svlm_count_launch();
}

void svlm_launch_evict_meta_batch(const SvlmCacheList& list, cudaStream_t st) {
    launch_evict_meta(evict_meta_batch_kernel, list.n, st, list);
    svlm_count_launch();
}

void svlm_launch_append_meta(const SvlmCacheDev& cd, const unsigned char* types, const int* pos, int n,
                             cudaStream_t st) {
    append_meta_kernel<<<1, META_THREADS, 0, st>>>(cd, types, pos, n);
    svlm_count_launch();
}

void svlm_launch_evict_meta(const SvlmCacheDev& cd, cudaStream_t st) {
    launch_evict_meta(evict_meta_kernel, 1, st, cd);
    svlm_count_launch();
}
