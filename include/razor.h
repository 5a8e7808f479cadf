/*
 * razor.h - C ABI of the B200 (sm_100a) RazorAttention hot path.
 *
 * RazorAttention (arXiv 2407.15891) keeps the whole KV cache only for "retrieval" heads.  Every
 * other head keeps its first N0 attention-sink tokens and its most recent L tokens (Algorithm 1)
 * and folds all dropped tokens into one compensation token, the mean of the dropped
 * keys and values (Eq. 4).  At decode time that token enters the softmax with weight N_d, the
 * number of dropped tokens (Eq. 5); retrieval heads use ordinary attention (Algorithm 1).
 *
 * This library builds that head-heterogeneous cache at the end of prefill (razor_compress), adds
 * decode tokens to it (razor_append) and runs decode attention over it (razor_decode_attention).
 *
 * Conventions
 *   - Every function returns RAZOR_OK (0) or a negative razor_status code.  Nothing throws, aborts
 *     or traps on the device.
 *   - "device" pointers are CUDA device memory of the current device; "host" pointers are ordinary
 *     host memory, read before the call returns.
 *   - The caller owns every device buffer: dense K/V, queries, outputs, the page pool and the
 *     workspace.  The library never allocates device memory; it owns only the host-side handle
 *     (and a small pinned host staging area), released by razor_cache_destroy.
 *   - Work is enqueued on the CUDA stream passed as `stream` (a cudaStream_t cast to void*; NULL is
 *     the default stream) and is asynchronous with respect to the host.  All calls on one cache
 *     must be stream-ordered with respect to each other (they share scratch buffers).
 *   - Storage dtype of K, V and q is config.dtype; compensation sums/means and outputs are fp32.
 *   - The library never applies rotary embeddings: K and q arrive after the rotary transformation,
 *     as the paper's cache does (Section 3.2, text below Eq. 4).
 */
#ifndef RAZOR_H_
#define RAZOR_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define RAZOR_API __attribute__((visibility("default")))
#else
#define RAZOR_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RAZOR_OK = 0,
  RAZOR_E_INVALID_ARG = -1,     /* a size, index or flag is out of range */
  RAZOR_E_NULL_PTR = -2,        /* a required pointer is NULL */
  RAZOR_E_UNSUPPORTED_DIM = -3, /* head_dim / dtype / group size / page size not supported */
  RAZOR_E_POOL_TOO_SMALL = -4,  /* page pool or workspace smaller than razor_query_bytes reports */
  RAZOR_E_CAPACITY = -5,        /* append beyond max_new_tokens, or context beyond max_ctx_len */
  RAZOR_E_NOT_COMPRESSED = -6,  /* append/decode/export on a layer (or sequence) not yet compressed */
  RAZOR_E_CUDA = -7,            /* a CUDA runtime call failed; razor_last_cuda_error() has the code */
  RAZOR_E_MISALIGNED = -8       /* a device pointer or stride breaks the 16-byte alignment rule */
} razor_status;

enum { RAZOR_F32 = 0, RAZOR_BF16 = 1 };

typedef struct razor_cache razor_cache_t; /* opaque host object */

typedef struct {
  int32_t batch;            /* B: sequences                                                        */
  int32_t n_layers;         /* L                                                                   */
  int32_t n_q_heads;        /* Hq; must be a multiple of n_kv_heads; group = Hq/Hkv in {1,2,4,8}   */
  int32_t n_kv_heads;       /* Hkv                                                                 */
  int32_t head_dim;         /* D: 64 or 128                                                        */
  int32_t dtype;            /* RAZOR_F32 or RAZOR_BF16: storage of K, V and q                      */
  int32_t page_tokens;      /* tokens per page; must be 16                                         */
  int32_t n_sink;           /* N0 of Algorithm 1 (Table 2: 4); >= 0                                */
  int32_t max_ctx_len;      /* largest context length any sequence has at compression time        */
  int32_t max_new_tokens;   /* append capacity per sequence after compression                      */
  int32_t use_compensation; /* 1: Eq. 5.  0: plain truncation (sinks + window only, Table 1 scheme) */
  int32_t page_shuffle_seed;/* 0: pages of a head are consecutive.  != 0: page ids are permuted
                               (exercises the page indirection the way a serving allocator would)  */
  float sm_scale;           /* multiplies every logit, the compensation logit included; 0 means
                               1/sqrt(head_dim).  Eq. 3 and Eq. 5 print no scale: that is 1.0f     */
} razor_config_t;

/*
 * Sizes of the two caller-owned device buffers (Algorithm 1 fixes how many tokens each
 * head keeps).  ctx_len[B], window[B]: host; head_is_retrieval[L*Hkv]: host, 1 = the KV head keeps
 * every token (for grouped-query models the caller ORs the flags of the group's query heads,
 * Section 4.1).  pool_bytes covers every layer compressed once, with room for max_new_tokens
 * appends; workspace_bytes depends on the config only.  Both are multiples of 256.
 */
RAZOR_API int razor_query_bytes(const razor_config_t* cfg, const int32_t* ctx_len, const int32_t* window,
                      const uint8_t* head_is_retrieval, size_t* pool_bytes, size_t* workspace_bytes);

/*
 * Create a cache over caller-owned device memory.  pool_dev and workspace_dev must be 256-byte
 * aligned and stay valid until razor_cache_destroy.  The workspace is cleared on `stream`.
 * Errors: NULL_PTR, INVALID_ARG, UNSUPPORTED_DIM, MISALIGNED, POOL_TOO_SMALL (workspace), CUDA.
 */
RAZOR_API int razor_cache_create(razor_cache_t** out, const razor_config_t* cfg, void* pool_dev, size_t pool_bytes,
                       void* workspace_dev, size_t workspace_bytes, void* stream);

/*
 * Prefill-end compression of one layer (Algorithm 1, Eq. 4).
 *   K, V     device, [B, Hkv, N, D] with element strides stride_b / stride_h / stride_n (innermost
 *            dimension contiguous); rows at or beyond ctx_len[b] are never read.  Base pointers
 *            16-byte aligned, strides multiples of 16 bytes.
 *   ctx_len  host [B]: tokens of each sequence (0 <= ctx_len[b] <= max_ctx_len)
 *   head_is_retrieval  host [Hkv] for this layer
 *   n_sink   must equal config.n_sink
 *   window   host [B]: recent-window length L_h of each sequence (>= 0); the caller evaluates
 *            max(S0, N/C) of Algorithm 1
 * A retrieval head, and any head with ctx_len <= n_sink + window, keeps positions [0, N).  Any
 * other head keeps [0, n_sink) and [N - window, N); positions [n_sink, N - window) are summed in
 * fp32 into its compensation sums, and the means and the count N_d are stored.  Kept rows are
 * copied bit for bit into the page pool in ascending position order.  Compressing a layer again
 * reuses its pages when the new plan fits in them.
 * Errors: NULL_PTR, INVALID_ARG, MISALIGNED, CAPACITY (ctx_len > max_ctx_len), POOL_TOO_SMALL, CUDA.
 */
RAZOR_API int razor_compress(razor_cache_t* cache, int32_t layer, const void* K, const void* V, int64_t stride_b,
                   int64_t stride_h, int64_t stride_n, const int32_t* ctx_len,
                   const uint8_t* head_is_retrieval, int32_t n_sink, const int32_t* window, void* stream);

/*
 * The same for ONE sequence b of the batch (serving admission: sequences arrive one at a time and
 * their dense K/V need not coexist).  K, V device [Hkv, N, D] with strides stride_h / stride_n.
 * head_is_retrieval must be the same for every sequence of a layer.
 */
RAZOR_API int razor_compress_seq(razor_cache_t* cache, int32_t layer, int32_t b, const void* K, const void* V,
                       int64_t stride_h, int64_t stride_n, int32_t ctx_len, const uint8_t* head_is_retrieval,
                       int32_t n_sink, int32_t window, void* stream);

/*
 * Add one decode token per sequence to a compressed layer.  k_new, v_new: device [B, Hkv, D],
 * contiguous.  Retrieval heads, and heads whose window is not yet full, store the row in the next
 * slot.  A head with a full window first folds its oldest recent token into the compensation sums
 * (count + 1, means recomputed: Eq. 4 over all tokens dropped so far), then stores the new row in
 * that slot; the window length stays what it was at compression (the paper does not say how the
 * cache grows while decoding).  Hence t appends leave exactly the state that compressing the
 * (N + t)-token context with the same window would.
 * Ordering: the kernel is launched so that it may start while the kernel before it on the stream is
 * still finishing.  In that early phase it reads only the library's own state of this layer (written
 * by earlier razor calls on the same stream).  k_new and v_new are read, and everything is written,
 * only after the preceding kernel has completed and its writes are visible, so the kernel that produces
 * k_new / v_new may be the one directly before this call.  None of the caller's memory is ever read
 * before the preceding kernel has finished; the same holds for q of razor_decode_attention.
 * Errors: NULL_PTR, INVALID_ARG, NOT_COMPRESSED, CAPACITY (more than max_new_tokens appends), CUDA.
 */
RAZOR_API int razor_append(razor_cache_t* cache, int32_t layer, const void* k_new, const void* v_new, void* stream);

/*
 * Decode attention of one query token per sequence over the compressed layer (Eq. 5; Algorithm 1).
 * q: device [B, Hq, D] contiguous, config.dtype.  out: device [B, Hq, D] fp32.
 * Query head j reads KV head j / group.  For a head with N_d > 0 dropped tokens
 *   out = (N_d e^{s_c} v_hat + sum_kept e^{s_n} v_n) / (N_d e^{s_c} + sum_kept e^{s_n}),
 *   s_n = sm_scale q.k_n,  s_c = sm_scale q.k_hat;
 * other heads get softmax attention over all their tokens.  A sequence with no tokens gives zeros
 * (both sums are empty).
 * Call razor_append first when the query token should attend to itself.
 * Errors: NULL_PTR, INVALID_ARG, NOT_COMPRESSED, CUDA.
 */
RAZOR_API int razor_decode_attention(razor_cache_t* cache, int32_t layer, const void* q, float* out, void* stream);

/*
 * One decode step of a layer in a single launch: razor_append(k_new, v_new) followed by
 * razor_decode_attention(q, out), with the same arguments, the same result for `out` and the same cache
 * state afterwards (Algorithm 1 + Eq. 4 for the new token, Eq. 5 for the attention).  The streaming kernel
 * itself stores the new rows: the part of a head that holds the row's page puts the row into its copy of
 * the page and into the pool, folds the evicted row into the compensation sums when the window is full,
 * and the head states advance when the last CTA has finished.  This removes the append kernel, and the
 * wait for it, from every decode step.  k_new, v_new and q are read only after the kernel before this call
 * on the stream has completed.
 * Errors: as razor_append and razor_decode_attention.
 */
RAZOR_API int razor_decode_step(razor_cache_t* cache, int32_t layer, const void* k_new, const void* v_new,
                                const void* q, float* out, void* stream);

/*
 * A round of several new tokens per sequence (a second prompt chunk, a speculative-decoding verify
 * step).  The paper runs Algorithm 1 once on the prompt and says nothing about such rounds; the
 * reading taken extends the single-token rule.
 *   razor_append_many             adds n_tokens tokens per sequence, k_new, v_new device
 *                                 [B, n_tokens, Hkv, D] contiguous: exactly what n_tokens razor_append
 *                                 calls would leave (window fixed, evicted tokens folded into Eq. 4).
 *                                 Any length up to the remaining max_new_tokens; runs of 8 tokens or more
 *                                 are appended in parallel over the tokens.  This is also how a chunked
 *                                 prefill hands its K/V over without a dense cache of the whole context:
 *                                 razor_compress with ctx_len 0 (K, V may be NULL) fixes the layer's windows
 *                                 and retrieval set, then each chunk is appended; the result is the cache
 *                                 that one razor_compress of the whole context would build.
 *   razor_decode_attention_multi  q device [B, n_tokens, Hq, D], out device fp32 [B, n_tokens, Hq, D]:
 *                                 query t is the token at position (tokens seen) - n_tokens + t and
 *                                 attends to the kept tokens at positions <= its own (Section 3.1:
 *                                 n <= m) plus the compensation token with its count N_d (Eq. 5).
 *                                 n_tokens = 1 is razor_decode_attention.
 * Limits of the multi-token call: bf16; at least n_tokens tokens cached; every head that has dropped
 * tokens must have a window >= n_tokens (otherwise its mean would hold tokens that come after a query).
 * A round of at most 8 query rows per KV head (query heads of the group x query tokens) is one launch of
 * the streaming kernel on a tile of 2, 4 or 8 rows (matrix instructions).  A longer round runs on the
 * query-tiled tensor-core kernel (128 rows per tile; the threshold is RAZOR_OPT_ROUND_TILED_MIN_ROWS; with
 * ALiBi it adds Eq. 1's distance penalty to every score) - except in an ALiBi cache that keeps sink tokens,
 * or below the threshold: there it runs as several launches of the streaming kernel, block by block, each
 * streaming the cache once and masking the round's tokens that come after its block.
 * Errors: NULL_PTR, INVALID_ARG, UNSUPPORTED_DIM, NOT_COMPRESSED, CAPACITY (append), MISALIGNED, CUDA.
 */
RAZOR_API int razor_append_many(razor_cache_t* cache, int32_t layer, const void* k_new, const void* v_new,
                      int32_t n_tokens, void* stream);

/*
 * Host only: what a run of n_tokens appends does to ONE head whose state is (len, n_drop, ring_head,
 * window; window < 0: the head keeps everything), in closed form - the rule the parallel append kernel
 * and the library's host mirror apply.  slot[a] (host, [n_tokens] or NULL): physical slot token a ends up
 * in, -1 when the run itself evicts it again (it is then folded into the compensation sums directly);
 * evicts_old[a] (host or NULL): 1 when that slot held a token from before the run, which is folded into
 * the sums first.  The state after the run goes to the three out-pointers (each may be NULL).
 * Errors: INVALID_ARG (a state no sequence of appends can produce).
 */
RAZOR_API int razor_append_plan(int32_t len, int32_t n_drop, int32_t ring_head, int32_t window, int32_t n_sink,
                                int32_t n_tokens, int32_t* slot, uint8_t* evicts_old, int32_t* len_after,
                                int32_t* n_drop_after, int32_t* ring_head_after);
RAZOR_API int razor_decode_attention_multi(razor_cache_t* cache, int32_t layer, const void* q, float* out,
                                 int32_t n_tokens, void* stream);

/*
 * Read back the compressed state of one (layer, sequence, KV head) in LOGICAL order (ascending
 * original position), whatever the physical slot order is.  Device outputs, any of which may be
 * NULL: kept_pos int32[n_kept]; K, V [n_kept, D] in config.dtype; comp_mean_k/v and comp_sum_k/v
 * fp32[D].  Host outputs (may be NULL): n_kept, n_drop.  n_kept is known on the host without a
 * device read, so call once with NULL device pointers to size the buffers.  Snapshot and parity probe.
 */
RAZOR_API int razor_cache_export(razor_cache_t* cache, int32_t layer, int32_t b, int32_t kv_head, int32_t* kept_pos,
                       void* K, void* V, float* comp_mean_k, float* comp_mean_v, float* comp_sum_k,
                       float* comp_sum_v, int32_t* n_kept, int32_t* n_drop, void* stream);

/* Host-side accounting of one layer: bytes of kept K+V rows and of the dense cache they stand for. */
RAZOR_API int razor_cache_stats(const razor_cache_t* cache, int32_t layer, size_t* kept_bytes, size_t* dense_bytes);

/*
 * The decode work schedule (host only; no device is touched).  The page streams of all (sequence,
 * KV head) pairs are laid end to end, longest first.  The first static_percent of the pages is cut
 * into one equal span per CTA (a span that crosses a head boundary becomes several work items, one
 * per head); the rest is cut into tail items which the CTAs pull one by one when their span is done.
 * Tail items shrink along the stream: each is 1 / tail_items_per_cta of an equal share of the tail
 * still left, but at least min_chunk_pages (and never across a head boundary).  A job is what a CTA
 * pulls: a span or one tail item.
 *   razor_schedule_plan   plans for given stream lengths: tokens host int32[n_heads] (tokens stored
 *                         per head), n_ctas >= 1 (the SM count), 0 <= static_percent <= 100,
 *                         tail_items_per_cta >= 1, min_chunk_pages >= 1 (smallest span / tail item).
 *   razor_schedule_query  the plan the next razor_decode_attention of `layer` would use.
 *   razor_schedule_combine_heads  which heads of that plan are left to the combine kernel (none: the decode
 *                         step is one launch).  A head cut into several parts leaves one partial softmax
 *                         record per part (Eq. 5 regrouped).  The streaming kernel folds the records of a head
 *                         in few parts itself - the part written last does it; the others are folded by a
 *                         small kernel launched behind it.  heads: host int32[max_heads] receiving their
 *                         indices b*Hkv + kv_head, may be NULL; n_heads receives the count.
 * items: host int32[max_items][5] = {head index b*Hkv + kv_head, first_page, end_page (-1: to the
 * end of the stream), parts_of_this_head, job}, in job order, may be NULL; n_items receives the
 * count, n_spans (may be NULL) how many of the jobs are spans.  A page is 16 tokens.
 * Errors: NULL_PTR, INVALID_ARG (also when max_items is too small), NOT_COMPRESSED.
 */
RAZOR_API int razor_schedule_plan(const int32_t* tokens, int32_t n_heads, int32_t n_ctas, int32_t static_percent,
                        int32_t tail_items_per_cta, int32_t min_chunk_pages, int32_t* items, int32_t max_items,
                        int32_t* n_items, int32_t* n_spans);
RAZOR_API int razor_schedule_query(razor_cache_t* cache, int32_t layer, int32_t* items, int32_t max_items,
                         int32_t* n_items);
RAZOR_API int razor_schedule_combine_heads(razor_cache_t* cache, int32_t layer, int32_t* heads, int32_t max_heads,
                                 int32_t* n_heads);

/*
 * Decode tuning knobs; the defaults suit long-context caches on a B200.  A change takes effect at the
 * next razor_decode_attention.  Errors: NULL_PTR, INVALID_ARG (unknown option or value out of range).
 */
enum {
  RAZOR_OPT_DECODE_TAIL_ITEMS_PER_SM = 1, /* a tail item is 1/k of an SM's share of the remaining tail
                                             (k = 1..1024; default 3)                                      */
  RAZOR_OPT_DECODE_MIN_CHUNK_PAGES = 2, /* smallest span or tail item in pages (default 32)               */
  RAZOR_OPT_DECODE_RING_KB = 3,         /* shared-memory page ring per CTA in KiB; 0 = as large as fits   */
  RAZOR_OPT_DECODE_CONSUMER_WARPS = 4,  /* streaming warps per CTA: 0 = default; 4, 8, 12 or 16; a value
                                           the head shape has no kernel for falls back to the default     */
  RAZOR_OPT_DECODE_TENSOR_CORES = 5,    /* bf16 heads: 0 = matrix instructions from group 4 up (default),
                                           1 = for every group size (a single head fills one row of the
                                           tile), 2 = never                                               */
  RAZOR_OPT_DECODE_STATIC_PERCENT = 6,  /* share of the pages handed out as per-CTA spans (0..100;
                                           default 80); 0 makes every job a tail item                     */
  RAZOR_OPT_DECODE_EARLY_PREFETCH = 7,  /* most pages (0..64; default 12) a CTA copies from the start of its span
                                           into shared memory before the kernel waits for the launch before it
                                           on the stream - only pages that no kernel still in flight can be
                                           writing (the host knows which page a preceding razor_append
                                           touched); 0: every copy waits                                   */
  RAZOR_OPT_ROUND_TILED_MIN_ROWS = 8    /* razor_decode_attention_multi: rounds with at least this many query
                                           rows per KV head (query heads of the group x new tokens; default 9,
                                           i.e. more than one launch of the streaming kernel takes) run on the
                                           query-tiled tensor-core kernel, shorter ones block by block on the
                                           streaming kernel                                                    */
};
RAZOR_API int razor_cache_set_option(razor_cache_t* cache, int32_t option, int32_t value);

/*
 * Device-side health of the cache's kernels.  Every wait inside the decode kernel is bounded; a wait
 * that runs out makes the kernel stop early and set a bit of a sticky status word instead of hanging.
 * This call synchronises `stream`, stores the word in *status (0 = healthy) and, when it is non-zero,
 * clears it together with the kernel's work counters so that the cache can be used again; outputs of
 * the affected launch are undefined.  Bits: 1 producer wait, 2 consumer wait, 4 reducer wait, 8 copies
 * still in flight at exit, 16 the self-test below, 32 an early-prefetch count that did not match the
 * device's lengths.  Errors: NULL_PTR, CUDA.
 */
RAZOR_API int razor_cache_device_status(razor_cache_t* cache, int32_t* status, void* stream);

/*
 * ALiBi models (Section 3.1).  Their head h scores a key at distance m - n with q.k - l_h (m - n)
 * (Eq. 1) and keeps only its most recent L_h tokens, L_h being the head's vision scope (Theorem 1;
 * computing it needs the model's weights, so it is an input here).
 *   razor_cache_set_alibi         slopes host fp32 [L * Hq], l_h >= 0 of every query head; from the next
 *                                 decode call on, every logit gets - l_h * (query position - key
 *                                 position); sm_scale multiplies q.k only.  NULL switches it off.
 *                                 Needs config.use_compensation = 0 (a mean of dropped tokens has no
 *                                 position; the paper uses none for ALiBi heads); n_sink = 0 gives the
 *                                 paper's recent-tokens-only cache.  The query of a decode step is the
 *                                 newest cached token (append first); in a multi-token round query t
 *                                 sits at its own position.
 *   razor_cache_set_head_windows  window_h host int32 [Hkv] for one layer: from the next razor_compress
 *                                 of that layer on, KV head g keeps min(window[b], window_h[g]) recent
 *                                 tokens (heads flagged in head_is_retrieval still keep everything).
 *                                 NULL removes the caps.  Pool sizing stays razor_query_bytes' with
 *                                 window[b] (an upper bound).
 * Errors: NULL_PTR, INVALID_ARG, CUDA.
 */
RAZOR_API int razor_cache_set_alibi(razor_cache_t* cache, const float* slopes, void* stream);
RAZOR_API int razor_cache_set_head_windows(razor_cache_t* cache, int32_t layer, const int32_t* window_h);

/*
 * Retrieval-head identification, the arithmetic of Section 3.3.  The model is run (by the caller) on
 * `period` random tokens repeated several times; for one layer's heads this call takes their
 * post-rotary queries and keys on that input and returns, per head, the echo score (causal-softmax
 * attention weight on the earlier copies of the current token, positions m - j*period) and the
 * induction score (weight on the tokens right after those, m - j*period + 1), each summed over j and
 * averaged over the queries m >= period.
 *   Q, K       device bf16 [n_heads, n_tokens, head_dim] contiguous (a grouped-query model passes each
 *              query head with its KV head's keys); head_dim 64 or 128; 2 <= period < n_tokens
 *   sm_scale   multiplies q.k; 0 means 1/sqrt(head_dim)
 *   echo, induction   device fp32 [n_heads]
 *   scratch    device, 16-byte aligned, razor_head_scores_scratch_bytes(n_heads, n_tokens) bytes,
 *              caller-owned; its content on entry does not matter
 * The kernel's internal waits are bounded in time; should one ever run out, every score of the call is
 * NaN (nothing else is touched, the context stays usable).
 * razor_select_retrieval_heads (host only) then marks the top frac_induction of the heads by
 * induction score and the top frac_echo by echo score (Table 2: 0.14 and 0.01; counts rounded to the
 * nearest integer, at least one each, ties to the lower index): mask[h] = 1 for a retrieval head.
 * Errors: NULL_PTR, INVALID_ARG, UNSUPPORTED_DIM, MISALIGNED, POOL_TOO_SMALL (scratch), CUDA.
 */
RAZOR_API int razor_head_scores_scratch_bytes(int32_t n_heads, int32_t n_tokens, size_t* bytes);
RAZOR_API int razor_head_scores(const void* Q, const void* K, int32_t n_heads, int32_t n_tokens, int32_t head_dim,
                      int32_t dtype, int32_t period, float sm_scale, float* echo, float* induction, void* scratch,
                      size_t scratch_bytes, void* stream);
RAZOR_API int razor_select_retrieval_heads(const float* echo, const float* induction, int32_t n_heads,
                                 float frac_induction, float frac_echo, uint8_t* mask);

/*
 * Self-test of the bounded waits.  Enqueues a one-warp kernel that waits, with the decode kernel's own
 * wait routine and a limit of limit_ns (1 us .. 1 s), on a barrier nothing ever arrives on.  The wait
 * has to give up by itself; razor_cache_device_status then reports bit 16 (and clears it), and the
 * cache stays usable.  Nothing faults, traps or spins without bound.
 * Errors: NULL_PTR, INVALID_ARG, CUDA.
 */
RAZOR_API int razor_cache_wait_selftest(razor_cache_t* cache, int64_t limit_ns, void* stream);

/*
 * The compensation token of the KV heads of ONE sequence without a cache, a pool or a workspace.
 * (The paper has no counterpart to this call; it computes the same means as Eq. 4.)
 *
 * For callers that cannot allocate device memory: a plugin inside an application that owns the
 * allocator and passes in only input and output tensors, code running while a stream is being
 * captured, a process whose memory was fixed at start-up.  They cannot set up razor_cache_create's
 * buffers, yet the means of the dropped rows need a cross-block reduction and so some scratch.  Here
 * that scratch is a fixed 2 MiB array inside the library itself (each GPU that loads the library
 * holds it until the process ends); the call allocates nothing and frees nothing.
 *
 *   K, V       device, [n_kv_heads, >= ctx_len, head_dim] with element strides stride_h / stride_n,
 *              16-byte aligned like razor_compress's inputs; dtype RAZOR_F32 or RAZOR_BF16
 *   mean_k/v   device fp32 [n_kv_heads, head_dim]: means over rows [n_sink, ctx_len - window);
 *              zeros when ctx_len <= n_sink + window
 *   n_drop     host, may be NULL: number of rows averaged
 * Limits: n_kv_heads <= 64 (RAZOR_E_CAPACITY beyond that: split the heads over several calls),
 * head_dim 64 or 128.
 * The first call on a device looks up the array's device address; make that call outside any stream
 * capture.  All calls on a device share the array, so two calls whose kernels could run at the same
 * time (different streams, no ordering between them) corrupt each other: keep them stream-ordered.
 * Nothing in the array needs clearing between calls.
 * Errors: NULL_PTR, INVALID_ARG, CAPACITY, UNSUPPORTED_DIM, MISALIGNED, CUDA.
 */
RAZOR_API int razor_compensation_mean_static(const void* K, const void* V, int64_t stride_h, int64_t stride_n,
                                   int32_t n_kv_heads, int32_t head_dim, int32_t dtype, int32_t ctx_len,
                                   int32_t n_sink, int32_t window, float* mean_k, float* mean_v, int32_t* n_drop,
                                   void* stream);

/* Forget every compressed layer and give all pages back (the handle and buffers stay usable). */
RAZOR_API int razor_cache_reset(razor_cache_t* cache);

/* Free the host-side handle.  Device buffers belong to the caller. */
RAZOR_API int razor_cache_destroy(razor_cache_t* cache);

/* Text for a status code; never NULL. */
RAZOR_API const char* razor_status_string(int status);

/* cudaError_t value of the last failed CUDA call seen by this library in this thread (0 if none). */
RAZOR_API int razor_last_cuda_error(void);

/* Library version, "major.minor". */
RAZOR_API const char* razor_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RAZOR_H_ */
