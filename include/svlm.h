/*
 * svlm - the per-chunk KV-cache step of StreamingVLM-style streaming inference, for NVIDIA B200.
 *
 * One svlm_cache is the KV cache of one video stream.  Per one-second chunk the caller
 *   1. appends the chunk's tokens (vision then text) with their native positions,
 *   2. evicts (type-aware retention, left-shift of the retained positions, re-rotation of the
 *      retained keys),
 *   3. attends with the chunk's queries over the retained cache (chunk prefill),
 *   4. and for every generated token appends one text token and attends with one query (decode).
 *
 * The operations follow Section 2.1 of the paper: the "Streaming-aware KV Cache" paragraph defines
 * what is retained, the "Contiguous RoPE" paragraph defines the position re-indexing (1D and 3D).
 *
 * Conventions for every entry point
 *   - returns SVLM_OK (0) or a negative svlm_status; never throws, never aborts the process;
 *   - tensor arguments are DEVICE pointers owned by the caller unless the name ends in _host; the
 *     library reads or writes them in the stream order of the cache's CUDA stream and keeps no
 *     reference after the enqueued work has finished;
 *   - work is enqueued on the cache's stream and the call returns without synchronising, except
 *     svlm_cache_query, svlm_cache_status and the *_host variants' final copy where stated;
 *   - conditions only the device can see (a type mix that overflows the capacity) set a sticky
 *     status word that svlm_cache_status returns; the offending append is dropped as a whole;
 *   - bf16 means the 16-bit brain-float bit pattern; Q/K are passed UN-rotated.
 */
#ifndef SVLM_H
#define SVLM_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct svlm_cache svlm_cache; /* opaque; one per stream */

enum svlm_token_type { SVLM_TEXT = 0, SVLM_VISION = 1 };
enum svlm_rope_mode { SVLM_ROPE_1D = 0, SVLM_ROPE_MROPE = 1 };
enum svlm_status {
    SVLM_OK = 0,
    SVLM_ERR_ARG = -1,      /* bad argument */
    SVLM_ERR_CAPACITY = -2, /* append would exceed the capacity given at creation */
    SVLM_ERR_ORDER = -3,    /* call sequence invalid (e.g. more queries than tokens appended) */
    SVLM_ERR_CUDA = -4,     /* a CUDA runtime or driver call failed */
    SVLM_ERR_TIMEOUT = -5,  /* a bounded device-side wait ran out */
    SVLM_ERR_NOMEM = -6,    /* device or host allocation failed */
    SVLM_ERR_TOO_LARGE = -7 /* problem exceeds the fixed scratch of svlm_attend_decode_noalloc */
};

/*
 * Create the cache of one stream (paper Section 2.1, "Streaming-aware KV Cache": T_sink, V_window,
 * T_window).  n_sink, vision_window and text_window are token counts (a 16 s vision window of
 * 512 tokens/s is 8192).  capacity is the largest number of tokens that is ever stored at once,
 * i.e. retained tokens plus everything appended before the next svlm_cache_evict.
 * head_dim is 64 or 128.  Allocates device memory for `layers` K and V slabs
 * ([layers][kv_heads][pages*128][head_dim] bf16, pages*128 >= capacity), per-token metadata and
 * split-KV scratch; the current CUDA device at the time of the call owns the cache.
 * Defaults: 1D RoPE with base 10000, sinks are text tokens, contiguous positions, legacy stream 0.
 */
int svlm_cache_create(svlm_cache** out, int layers, int kv_heads, int head_dim, int n_sink, int vision_window,
                      int text_window, int capacity);

/* Frees everything the cache owns after synchronising its stream.  Null is ignored. */
void svlm_cache_destroy(svlm_cache* c);

/*
 * Rotary embedding geometry.  Pair (i, i + head_dim/2) rotates by position * base^(-2i/head_dim).
 * SVLM_ROPE_1D: one position per token.  SVLM_ROPE_MROPE (3D positions of the Qwen-VL family,
 * "Contiguous RoPE" paragraph): positions are (t,h,w) and sections[3] gives how many consecutive
 * pairs use t, then h, then w; the three must sum to head_dim/2.  sections is ignored in 1D mode.
 * Must be called before the first append.
 */
int svlm_cache_set_rope(svlm_cache* c, int mode, double base, const int sections[3]);

/*
 * Policy variants (defaults 0, 1).  sink_any_type != 0: the sinks are the first n_sink tokens of
 * the stream whatever their type, instead of the first n_sink text tokens.  contiguous == 0:
 * native RoPE, positions are never shifted (the paper's Table 4 ablation); eviction then only
 * frees storage.  Must be called before the first append.
 */
int svlm_cache_set_policy(svlm_cache* c, int sink_any_type, int contiguous);

/* CUDA stream (a cudaStream_t) on which all later work of this cache is enqueued. */
int svlm_cache_set_stream(svlm_cache* c, void* cuda_stream);

/*
 * Append n tokens in stream order.
 *   layer       -1: K and V are [layers][n][kv_heads][head_dim] and all layers are written;
 *               l >= 0: K and V are [n][kv_heads][head_dim] for that layer only.
 *   token_type  uint8 [n], SVLM_TEXT or SVLM_VISION    (read when layer is -1 or 0)
 *   pos         int32 native positions, [n] in 1D mode or [n][3] = (t,h,w)   (read when layer is -1 or 0)
 * The per-token metadata (stream ordinal, per-type ordinal, contiguous position = native position
 * minus everything shifted so far, storage slot) is taken once per token, by the call with layer
 * -1 or 0; calls for layers 1..layers-1 of the same tokens must follow with the same n and may pass
 * null token_type/pos.  K is stored rotated at the token's contiguous position, V as is.
 * Errors: SVLM_ERR_ARG; SVLM_ERR_CAPACITY when the host can already tell that n does not fit;
 * otherwise an overflow is detected on the device, the append is dropped and the sticky status set.
 */
int svlm_cache_append(svlm_cache* c, int layer, const void* K, const void* V, const uint8_t* token_type,
                      const int32_t* pos, int n);

/*
 * The step on the input side of the path, fused with svlm_cache_append: the Q/K/V projection of one layer for
 * the n new tokens, whose epilogue stores keys (rotated at each token's contiguous position, "Contiguous
 * RoPE" paragraph) and values straight into the tokens' cache slots and hands the queries back:
 *   [Q | K | V] = X W^T      X bf16 [n][hidden], W bf16 [(q_heads + 2 kv_heads) * head_dim][hidden], rows ordered
 *                            query heads, key heads, value heads; fp32 accumulation
 *   Q_out  bf16 [n][q_heads][head_dim], un-rotated (what svlm_attend expects)
 * token_type / pos as for svlm_cache_append: read by the call with layer 0, which takes the metadata;
 * calls for layers 1.. of the same tokens follow with the same n (layer-sequential use, layer >= 0 only).
 * Results equal svlm_cache_append with K, V = the projection's outputs, except that a key is rounded to
 * bf16 once, after its rotation, instead of before and after.
 * Requires head_dim 128, hidden a multiple of 64, X, W and Q_out 16-byte aligned.
 * Errors: SVLM_ERR_ARG, SVLM_ERR_CAPACITY, SVLM_ERR_ORDER as svlm_cache_append.
 */
int svlm_qkv_append(svlm_cache* c, int layer, const void* X, const void* W, int hidden, int q_heads,
                    const uint8_t* token_type, const int32_t* pos, int n, void* Q_out);

/*
 * The step on the output side of the path: the projection that consumes the attention output,
 *   Y = A Wo^T      A bf16 [n][in_dim] (svlm_attend's out viewed as [n][q_heads * head_dim]), Wo bf16 [out_dim][in_dim],
 *                   Y bf16 [n][out_dim]; fp32 accumulation, the same tensor-core kernel as svlm_qkv_append.
 * Up to 16 rows (decode) take a bandwidth kernel that reads Wo once instead.  The same call serves the input
 * side of a decode step: [q | k | v] = svlm_out_proj(x, W_qkv) is laid out as svlm_decode_step's Q, K and V.
 * Enqueued on the cache's stream (the cache is otherwise untouched).  in_dim a multiple of 64, out_dim a
 * multiple of 128, pointers 16-byte aligned.  Errors: SVLM_ERR_ARG.
 * Wo holds weights: with n <= 16 the kernel starts reading it while the work enqueued just before it on the
 * stream may still be running (only A waits for that work), so Wo must be complete in device memory before
 * that work starts; a kernel enqueued directly before this call must not be the one that writes Wo.
 */
int svlm_out_proj(svlm_cache* c, const void* A, const void* Wo, int in_dim, int out_dim, int n, void* Y);

/*
 * Evict, compact and re-index, all layers at once ("Streaming-aware KV Cache" and "Contiguous
 * RoPE" paragraphs).  Keeps the n_sink sink tokens, the last text_window text tokens and the last
 * vision_window vision tokens; every retained token's position moves left by the native position
 * span of the evicted tokens before it, and its stored key is re-rotated by that amount; storage of
 * evicted tokens is released.  Values never move.
 */
int svlm_cache_evict(svlm_cache* c);

/*
 * Grouped-query attention of the LAST n_q appended tokens over the stored tokens of one layer.
 *   layer    l >= 0: Q and out are [n_q][q_heads][head_dim] bf16;
 *            -1: all layers in one launch, Q and out are [layers][n_q][q_heads][head_dim].
 *   q_pos    int32 native positions of the queries ([n_q] or [n_q][3])
 * Query row r is the token with stream ordinal (tokens appended so far) - n_q + r; it is rotated at
 * q_pos minus the total shift and sees every stored token whose ordinal does not exceed its own
 * (retained history fully, the new chunk causally).  Query head h reads KV head
 * h / (q_heads / kv_heads).  Scores are scaled by 1/sqrt(head_dim); a row that sees nothing yields
 * zeros.  n_q == 1 takes the split-KV decode path, n_q >= 2 the chunk-prefill path; shapes neither of
 * them is built for (more than 8 query heads per KV head at n_q == 1; a cache of more than 512 pages of 128
 * slots, i.e. a capacity beyond roughly 65,000 tokens) take a slower general kernel with the same result.
 * Errors: SVLM_ERR_ARG (q_heads not a multiple of kv_heads, n_q < 1, null pointers),
 * SVLM_ERR_ORDER (n_q exceeds the tokens appended so far).
 */
int svlm_attend(svlm_cache* c, int layer, const void* Q, const int32_t* q_pos, int n_q, int q_heads, void* out);

/*
 * One decode step of one layer in a single launch: append ONE token (the token just generated; paper
 * Section 2.1 keeps past outputs as previous text) and attend with that token's query, i.e.
 * svlm_cache_append(c, layer, K, V, token_type, pos, 1) followed by
 * svlm_attend(c, layer, Q, pos, 1, q_heads, out), with identical results (paper Section 3.3: the
 * per-token latency of this step over the fixed-length cache is the efficiency figure).
 *   K, V        bf16 [kv_heads][head_dim], un-rotated     Q, out   bf16 [q_heads][head_dim]
 *   token_type  uint8 [1], pos int32 [1] or [3]: the metadata is taken by the call with layer 0;
 *               calls for layers 1.. of the same token follow and may pass null token_type (pos is
 *               still needed: it is the query's position).
 * layer -1 takes all layers of the token in ONE launch, for callers that hold every layer's inputs at once (an
 * attention-only stack, a benchmark): K, V are [layers][kv_heads][head_dim], Q and out [layers][q_heads][head_dim].
 * At most 8 query heads per KV head and at most 512 cache pages (a capacity up to roughly 65,000 tokens;
 * beyond that SVLM_ERR_ARG: use svlm_cache_append + svlm_attend).  Consecutive calls for different layers of the same token
 * overlap on the GPU (the next layer's cache pages are fetched while the previous layer finishes);
 * K, V, Q and everything else produced by earlier work in the stream are read only after that work
 * has completed.
 * Errors: SVLM_ERR_ARG, SVLM_ERR_ORDER (layer > 0 without a preceding one-token append).
 */
int svlm_decode_step(svlm_cache* c, int layer, const void* K, const void* V, const uint8_t* token_type,
                     const int32_t* pos, const void* Q, int q_heads, void* out);

/*
 * The same for n_caches independent streams in one launch (layer >= 0 only).  All caches must
 * share geometry, RoPE settings, device and stream (the first cache's stream is used).
 * Q and out are [n_caches][n_q][q_heads][head_dim]; q_pos is [n_caches][n_q] or [n_caches][n_q][3].
 * n_caches <= 32.
 */
int svlm_attend_batched(svlm_cache* const* caches, int n_caches, int layer, const void* Q, const int32_t* q_pos,
                        int n_q, int q_heads, void* out);

/*
 * svlm_attend_batched for streams whose new chunks differ in length (each second's text burst varies):
 * cache i attends with its last n_q[i] appended tokens, n_q a HOST array of n_caches counts >= 1.
 * Q, out are [sum n_q][q_heads][head_dim], q_pos [sum n_q] or [sum n_q][3]: the caches' rows one after
 * another in the order of `caches`.  One chunk-prefill launch serves all caches (also rows-of-one
 * caches: the split-KV decode path is not taken here).  layer >= 0 only.
 * Errors: as svlm_attend_batched; SVLM_ERR_ARG for a repeated cache or a count below 1.
 */
int svlm_attend_batched_varlen(svlm_cache* const* caches, int n_caches, int layer, const void* Q, const int32_t* q_pos,
                               const int32_t* n_q, int q_heads, void* out);

/*
 * Batched forms for independent streams that advance in lock step (one generated token per stream per
 * step, as in batched serving; the paper's policy is per stream, so each cache behaves exactly as under
 * the single-cache calls).  Same requirements on the caches as svlm_attend_batched; a cache may appear
 * only once.
 *
 * svlm_decode_step_batched = svlm_decode_step on every cache, one metadata launch (layer 0) and one
 * attention launch for all of them:
 *   K, V        bf16 [n_caches][kv_heads][head_dim]      Q, out   bf16 [n_caches][q_heads][head_dim]
 *   token_type  uint8 [n_caches]      pos   int32 [n_caches] or [n_caches][3]
 * svlm_cache_evict_batched = svlm_cache_evict on every cache, one metadata launch and one re-rotation
 * launch for all of them.
 * Errors: as the single-cache calls; SVLM_ERR_ARG also for mismatched or repeated caches.
 */
int svlm_decode_step_batched(svlm_cache* const* caches, int n_caches, int layer, const void* K, const void* V,
                             const uint8_t* token_type, const int32_t* pos, const void* Q, int q_heads, void* out);
int svlm_cache_evict_batched(svlm_cache* const* caches, int n_caches);

/*
 * Host-buffer variants: the same operations with K, V, token_type, pos / Q, q_pos, out in HOST
 * memory (pinned memory makes the copies asynchronous).  The library stages them through device
 * buffers it owns (grown on demand, which synchronises once).  svlm_attend_host returns after the
 * result has arrived in out_host (it synchronises the stream).  For all layers of a chunk (layer -1, n_q >= 2)
 * svlm_attend_host runs the layers as a pipeline on two copy streams of its own beside the cache's stream, so
 * that one layer's copies hide behind another layer's attention; pinned host buffers are needed for that.
 */
int svlm_cache_append_host(svlm_cache* c, int layer, const void* K_host, const void* V_host,
                           const uint8_t* token_type_host, const int32_t* pos_host, int n);
int svlm_attend_host(svlm_cache* c, int layer, const void* Q_host, const int32_t* q_pos_host, int n_q, int q_heads,
                     void* out_host);
/*
 * svlm_decode_step with host buffers (layer -1: all layers of the token in one launch); returns with out_host
 * filled.  The step's inputs are a few KB: they are gathered in a page-locked buffer of the library and go up in
 * one copy.  For layer -1, when every buffer is itself page-locked and mapped (as pinned allocations are under
 * unified addressing) and 16-byte aligned, nothing is copied at all: the kernels read the inputs and write the
 * output where they are.
 */
int svlm_decode_step_host(svlm_cache* c, int layer, const void* K_host, const void* V_host, const uint8_t* token_type_host,
                          const int32_t* pos_host, const void* Q_host, int q_heads, void* out_host);

/*
 * Decode attention (one query token, as svlm_attend with n_q == 1 and layer >= 0) for callers that
 * cannot allocate device memory when they attend.  (The paper has no counterpart: this is a
 * deployment convenience of the library.)
 * Some hosts of this library may not call the CUDA allocator once they are running: a server that has
 * given every free byte of the GPU to its own memory pool, a real-time loop that cannot afford the
 * allocator's device-wide lock, code that runs where allocation calls are forbidden.  svlm_attend
 * keeps its split-KV partial results in scratch memory that svlm_cache_create allocated; this entry
 * point uses a fixed array of SVLM_NOALLOC_SCRATCH_BYTES that is part of the library image instead,
 * and calls neither cudaMalloc nor cudaFree nor anything else that allocates.
 *   Q, q_pos, out   as for svlm_attend with n_q == 1: bf16 [q_heads][head_dim], int32 [1] or [3],
 *                   bf16 [q_heads][head_dim]; device pointers owned by the caller
 *   q_heads         a multiple of kv_heads, at most 8 query heads per KV head
 * Limits and rules
 *   - the array is resident on every GPU that loads the library, for the life of the process;
 *   - kv_heads x (number of KV splits: about one CTA per SM over the KV heads) x (16*head_dim + 64)
 *     bytes plus one counter per (layer, kv_head) must fit in it, otherwise SVLM_ERR_TOO_LARGE is
 *     returned and nothing runs (28 layers x 4 KV heads x head_dim 128 needs about 0.31 MB);
 *   - the cache has at most 512 pages (capacity up to roughly 65,000 tokens), otherwise SVLM_ERR_TOO_LARGE;
 *   - all calls on one GPU share the array and it keeps the previous call's contents; the call
 *     clears what has to start at zero, on the cache's stream, before its kernel.  Calls whose
 *     kernels can overlap on the GPU (different streams, different caches) race on it: order them;
 *   - the first call on each GPU looks up the array's device address, which can load the library's
 *     code on that GPU: make that first call before starting any stream capture.
 * Errors: SVLM_ERR_ARG, SVLM_ERR_ORDER (nothing appended yet), SVLM_ERR_TOO_LARGE, SVLM_ERR_CUDA.
 * The result agrees with svlm_attend's for the same state and inputs to within the rounding of the bf16
 * partial results (the streaming split-KV kernel computes it; svlm_attend serves one layer of one
 * cache with a kernel that keeps its partial results in a cache-owned area).
 */
#define SVLM_NOALLOC_SCRATCH_BYTES (512u << 10)
int svlm_attend_decode_noalloc(svlm_cache* c, int layer, const void* Q, const int32_t* q_pos, int q_heads, void* out);

/*
 * Read back the stored tokens in stream order (HOST output buffers, each may be null; sized for
 * `capacity` entries): stream ordinals, contiguous positions [n][3] (1D mode repeats the index),
 * types.  n_kept and shift_total (sum of all left-shifts so far) are single values.
 * Synchronises the cache's stream.
 */
int svlm_cache_query(svlm_cache* c, int64_t* n_kept, int64_t* gids, int32_t* pos, uint8_t* types, int64_t* shift_total);

/*
 * Copy the stored keys (as stored: rotated at the current positions) and values of one layer for
 * the tokens svlm_cache_query lists, in that order, into HOST buffers [n_kept][kv_heads][head_dim]
 * bf16 (either may be null).  Synchronises.  For tests and debugging.
 */
int svlm_cache_read_kv(svlm_cache* c, int layer, void* K_host, void* V_host);

/* Sticky device-side status (SVLM_OK if nothing went wrong).  Synchronises the cache's stream. */
int svlm_cache_status(svlm_cache* c);

/*
 * Debugging aid: the number of polls a bounded device-side wait of this cache's kernels makes before it
 * gives up (every wait inside the kernels is bounded; one that runs out makes its thread block record
 * SVLM_ERR_TIMEOUT in the sticky status, wait for its copies in flight, release what it holds and return).
 * The default, 2^20 polls, is seconds; 0 makes every wait give up at once, which is how the tests walk
 * the give-up paths without anything actually hanging.  The results of calls that timed out are
 * undefined; the cache's metadata and stored K/V are not touched by the attention kernels and stay valid,
 * but the sticky status stays set for the life of the cache.  Synchronises the cache's stream.
 */
int svlm_debug_set_wait_limit(svlm_cache* c, unsigned polls);

/* Number of kernels this library has launched in this process (all caches). */
int64_t svlm_launch_count(void);

/* Static description of a status code. */
const char* svlm_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* SVLM_H */
