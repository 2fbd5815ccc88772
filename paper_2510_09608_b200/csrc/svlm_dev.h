// Device-side data layout of one stream's cache, shared by the host runtime and the kernels.
//
// Storage is PAGED AND KEYED BY TOKEN TYPE.  A page is 128 consecutive slots of every
// [layer][kv_head] slab, i.e. exactly one key/value tile of the attention kernels.
//   * sink pages   [0, n_sink_pages): sink tokens in arrival order, never released;
//   * pool pages   the rest; each is owned by the TEXT ring or the VISION ring of the stream.
// Inside a ring a token's place is a pure function of its ring ordinal u (its per-type ordinal
// minus the sinks of that type): page-table entry u/128, offset u%128.  The retention rule of the
// paper ("Streaming-aware KV Cache", Section 2.1) keeps a suffix of each ring, so eviction is an
// advance of the ring's low-water mark plus the release of pages that fell below it: values never
// move, and keys are re-rotated in place (the position left-shift of the "Contiguous RoPE"
// paragraph).  Attention is invariant to storage order; the causal rule inside a new chunk uses
// the per-slot stream ordinal.
#pragma once
#include <stdint.h>

#define SVLM_PAGE 128
#define SVLM_MAX_HALF 64   // head_dim/2 <= 64
#define SVLM_MAX_BATCH 32

struct SvlmCtrl {            // one per cache, device memory; only meta kernels write it
    long long n_total;       // tokens ever appended = next stream ordinal (gid)
    long long n_type[2];     // per-type ordinals issued so far (TEXT, VISION)
    long long cursor;        // native position cursor (max native index + 1 seen so far)
    long long shift_total;   // sum of all left-shifts applied so far
    long long ring_n[2];     // ring ordinals issued so far per type
    long long ring_lo[2];    // lowest retained ring ordinal per type
    int sink_cnt[2];         // tokens of each type living in the sink pages
    int sink_fill;           // slots used in the sink pages
    int n_stored;            // tokens currently stored
    int free_top;            // free-page stack height
    int n_tiles;             // entries of the tile list
    int status;              // sticky svlm_status
    int append_n;            // tokens staged by the latest metadata append (0 if it was dropped)
    int evict_moved;         // 1 if the latest evict shifted any retained token
    unsigned wait_limit;     // polls a bounded device-side wait makes before it gives up (set at creation)
};

struct SvlmTile {            // one active page as the attention kernels see it
    int page;                // physical page: slots [page*128, page*128+128)
    int lo, hi;              // valid offsets [lo, hi)
    int pad;
    long long min_gid;       // stream ordinal of slot lo
    long long max_gid;       // stream ordinal of slot hi-1 (ordinals grow with the offset inside a page)
};

struct SvlmCacheDev {        // passed by value to kernels
    int layers, kv_heads, head_dim;
    int n_sink, vision_window, text_window, capacity;
    int n_pages, n_sink_pages, n_slots, pt_size;   // pt_size: power of two > n_pages
    int rope_mode, sink_any, contiguous;
    int sec_t, sec_th;       // pairs [0,sec_t) use t, [sec_t,sec_th) use h, the rest w
    SvlmCtrl* ctrl;
    int* free_stack;         // [n_pages]
    int* page_table[2];      // [pt_size] per type: ring page index -> physical page
    long long* slot_gid;     // [n_slots]
    int* slot_c;             // [3][n_slots] contiguous position per axis
    int* slot_a;             // [n_slots] native cursor advance of the token
    int* slot_delta;         // [n_slots] left-shift applied by the latest evict
    unsigned char* slot_type;// [n_slots]
    SvlmTile* tiles;         // [n_pages]
    int* new_slot;           // [capacity] slots of the latest append
    int* new_c;              // [capacity][3] positions of the latest append
    long long* ev_gid[2];    // [capacity] evict scratch: ordinals of evicted ring tokens
    long long* ev_pref[2];   // [capacity+1] exclusive prefix of their cursor advances
    uint16_t* K;             // [layers][kv_heads][n_slots][head_dim] bf16, rotated at slot_c
    uint16_t* V;             // same shape, as appended
    float* ws;               // split-KV partials
    void* tmaps;             // TMA descriptors (device memory, 4 x 128 bytes): K, V slabs with a 128-row box
                             // (chunk prefill), then K, V with a 32-row box (batched decode)
    float* rope_tab;         // [3][256][head_dim/2] (cos, sin) pairs, see svlm_rope.cuh
    double theta[SVLM_MAX_HALF];   // base^(-2i/head_dim)
};

struct SvlmCacheList {       // kernel parameter of the batched metadata and re-rotation kernels
    int n;
    const SvlmCacheDev* cd[SVLM_MAX_BATCH];   // the caches' descriptors, copies in device memory
};

#ifdef __CUDACC__
// All threads of the block copy a descriptor from device memory to shared memory and synchronise.
__device__ __forceinline__ void svlm_load_desc(SvlmCacheDev* dst, const SvlmCacheDev* src) {
    static_assert(sizeof(SvlmCacheDev) % 4 == 0, "descriptor is copied in 32-bit words");
    for (int i = threadIdx.x; i < (int)(sizeof(SvlmCacheDev) / 4); i += blockDim.x)
        reinterpret_cast<int*>(dst)[i] = reinterpret_cast<const int*>(src)[i];
    __syncthreads();
}
#endif

struct SvlmAttendView {      // what attention needs from one cache
    const uint16_t* K;
    const uint16_t* V;
    const SvlmCtrl* ctrl;
    const SvlmTile* tiles;
    const long long* slot_gid;
    float* ws;
    const void* tmaps;       // four 128-byte TMA descriptors in device memory (see SvlmCacheDev)
    const int* new_slot;     // slots of the latest append
    const int* slot_c;       // [3][n_slots] current positions
};

struct SvlmAttendBatch {     // kernel parameter: up to 32 caches share one launch
    int n_caches;
    int layers, kv_heads, head_dim, n_slots;
    int rope_mode, sec_t, sec_th;
    SvlmAttendView view[SVLM_MAX_BATCH];
    int q_varlen;            // chunk prefill only: the caches bring different numbers of query rows,
    int q_off[SVLM_MAX_BATCH];   //   cache i's rows start at row q_off[i] of Q, q_pos and out
    int q_cnt[SVLM_MAX_BATCH];   //   and there are q_cnt[i] of them
    const float* rope_tab;   // rotation table of the first cache (all caches of a batch share the geometry)
    double theta[SVLM_MAX_HALF];
};
