// Internal declarations shared by the host side (razor_api.cu, razor_schedule.cpp) and the kernels.
// Nothing here is part of the public ABI (that is include/razor.h).
#ifndef RAZOR_INTERNAL_H_
#define RAZOR_INTERNAL_H_

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "razor.h"

namespace razor {

constexpr int kPageTokens = 16;        // tokens per page
constexpr int kMaxGroup = 8;           // query heads per KV head
// A head cut into few parts is finished inside the streaming kernel: whichever of its parts is written last (an
// atomic ticket, nobody waits) folds the head's partial records, in part order.  "Few" is at most
// kMergeInKernelMaxRows record rows in all (parts x query rows of the KV head's tile), never more than
// kMergeInKernelMaxParts parts: one warp folds them in about a microsecond.  Heads in more parts are left to the
// combine kernel that follows.
constexpr int kMergeInKernelMaxParts = 16;
constexpr int kMergeInKernelMaxRows = 16;
inline int merge_in_kernel_max_parts(int rows) { return rows >= kMergeInKernelMaxRows ? 1 : kMergeInKernelMaxRows / rows; }
constexpr int kCompressMaxSlices = 512;    // row slices per (sequence, KV head) in the compression kernel
constexpr int kCompressSliceBudget = 8192; // slice sums a call may produce beyond one per head (sizes the scratch)

// Device-resident state of one (layer, sequence, KV head).  window < 0 marks a head that keeps every
// token (retrieval head).  Physical slots: [0, n_sink) sinks, then the recent window as a ring whose
// oldest element sits at ring index ring_head (Algorithm 1 keeps sinks + recent tokens).
struct HeadState {
  int32_t len;        // tokens stored (physical slots in use)
  int32_t n_drop;     // N_d of Eq. 4: tokens folded into the compensation sums so far
  int32_t ring_head;  // ring index of the oldest recent token
  int32_t window;     // recent-window length; < 0: keeps everything
};

// A run of n_tok appended tokens, decided per token in closed form (what n_tok single appends do one after
// the other).  With cap = N0 + W: the first f tokens still fit (all of them for a head that keeps everything),
// the other E = n_tok - f each evict the oldest recent token.  Token a < f goes to slot len + a and is overwritten
// again within the run when its ring index len + a - N0 is below E (the ring starts at index 0 while it fills);
// evicting token j = a - f goes to ring index (ring_head + j) mod W and stays iff j >= E - W.  A token that stays
// in a ring slot which held a token from before the run (ring index below the old ring fill) evicts that old
// row: it has to be added to the compensation sums before it is overwritten.  A token that does not stay is
// added to the sums itself.
struct AppendFate {
  int32_t slot;     // physical slot the token ends up in, -1 when it does not stay
  bool evicts_old;  // the slot held a token from before the run
};
#if defined(__CUDACC__)
#define RAZOR_HD __host__ __device__
#else
#define RAZOR_HD
#endif
RAZOR_HD inline int append_run_fits(const HeadState& st, int n_sink, int n_tok) {
  if (st.window < 0) return n_tok;
  const int room = n_sink + st.window - st.len;
  return room <= 0 ? 0 : (room < n_tok ? room : n_tok);
}
RAZOR_HD inline AppendFate append_fate(const HeadState& st, int n_sink, int n_tok, int a) {
  const int f = append_run_fits(st, n_sink, n_tok), E = n_tok - f, W = st.window;
  AppendFate r{-1, false};
  if (a < f) {
    const int slot = st.len + a;
    if (W < 0 || slot < n_sink || slot - n_sink >= E) r.slot = slot;
  } else {
    const int j = a - f;
    if (j >= E - W) {   // never when W == 0
      const int ring = (int)(((long long)st.ring_head + j) % W);
      const int ring_fill = st.len > n_sink ? st.len - n_sink : 0;   // ring tokens from before the run
      r.slot = n_sink + ring;
      r.evicts_old = ring < ring_fill;
    }
  }
  return r;
}
RAZOR_HD inline HeadState state_after_run(const HeadState& st, int n_sink, int n_tok) {
  const int f = append_run_fits(st, n_sink, n_tok), E = n_tok - f;
  HeadState nx = st;
  nx.len = st.len + f;
  nx.n_drop = st.n_drop + E;
  nx.ring_head = st.window > 0 ? (int)(((long long)st.ring_head + E) % st.window) : 0;
  return nx;
}

// One decode work item: pages [page_begin, page_end) of one head's token stream, streamed by one CTA.
// page_end < 0 means "to the end of the stream as it is now" (the last part of a head grows with
// appends).  A head cut into n_parts > 1 items owns n_parts partial records starting at rec_base, which
// the combine kernel merges; a head in one part writes its output directly.
struct WorkItem {
  int32_t head;       // b * Hkv + kv_head
  int32_t page_begin;
  int32_t page_end;
  int32_t part_idx;   // index of this part within its head
  int32_t n_parts;    // parts of this head
  int32_t rec_base;
  int32_t merge_here;   // 1: the head's parts are folded by the streaming kernel itself (its last part to arrive)
  int32_t pad1;
};

// A head whose stream was cut into several parts: one entry of the combine kernel's work list.
struct MultiHead {
  int32_t head;       // b * Hkv + kv_head
  int32_t rec_base;
  int32_t n_parts;
  int32_t pad;
};

// One sequence handed to the compression kernel.
struct SeqDesc {
  const void* K;
  const void* V;
  int64_t stride_h;   // elements
  int64_t stride_n;   // elements
  int32_t n_ctx;
  int32_t window;
  int32_t b;
  int32_t pad;
};

// One (sequence, KV head) of a compression call, as planned on the host: the head's state after the
// call and the run of consecutive pool pages that backs its page-table row.  n_pages = 0 leaves the row
// alone (the host has written it itself, e.g. in a permuted order).
struct HeadPlan {
  int32_t head;        // b * Hkv + kv_head
  int32_t first_page;
  int32_t n_pages;
  int32_t len, n_drop, window;   // HeadState after compression (ring_head = 0)
};

// Bits of the device status word (razor_cache_device_status).
enum : int32_t {
  kStatusProducerTimeout = 1,   // the copy-issuing warp gave up waiting for a free ring stage or item slot
  kStatusConsumerTimeout = 2,   // a streaming warp gave up waiting for a page or an item
  kStatusReducerTimeout = 4,    // the merging warp gave up waiting for the streaming warps' states
  kStatusDrainTimeout = 8,      // copies were still in flight when the abort path stopped waiting for them
  kStatusSelfTest = 16,         // razor_cache_wait_selftest: the deliberately unanswered wait gave up, as it must
  kStatusEarlyMismatch = 32     // a CTA was told to prefetch more pages than its first work item turned out to have
};

struct RoundItem;
struct RoundUnit;
// Pointers into the caller's workspace, plus the dimensions the kernels need.
struct DeviceView {
  uint8_t* pool;            // pages: [page][K rows | V rows][16][D]
  HeadState* state;         // [L][B*Hkv]
  float* comp_sum;          // [L][B*Hkv][2][D]  (K sums then V sums)
  float* comp_mean;         // [L][B*Hkv][2][D]
  float* ring_sum;          // [L][B*Hkv][2][D]  sum of the K and V rows now in the recent window, valid when ring_valid says so
  int32_t* ring_valid;      // [L][B*Hkv]        1: ring_sum is up to date (only the bulk append keeps it so)
  int32_t* page_table;      // [L][B*Hkv][max_pages]
  WorkItem* items;          // [L][max_items]
  int32_t* jobs;            // [L][max_items + 1]  first item of every job (a span or one tail item), then n_items
  MultiHead* multi;         // [L][B*Hkv]          heads in several parts (combine kernel's work list)
  float2* rec_ml;           // [max_items][G]      running max (log2 domain) and denominator of a partial
  float* rec_o;             // [max_items][G][D]   un-normalised numerator of a partial
  int32_t* queue;           // [4]: next item, CTAs done, spare, spare (zero at rest)
  int32_t* tickets;         // [B*Hkv]: parts of the head written so far in the running decode launch (zero at rest)
  int32_t* status;          // [1]: kStatus* bits, sticky until razor_cache_device_status clears them
  float* compress_scratch;  // [kCompressSliceBudget + B*Hkv][2][D]: slice s of head h of a call at h_in_call * n_slices + s
  HeadPlan* plan;           // [B*Hkv]  heads of the compression call in flight
  SeqDesc* seq_desc;        // [B]      directly behind plan[]: both arrive in one copy
  float* alibi_slopes;      // [L][Hq]  ALiBi slopes l_h times log2(e); read only when alibi != 0
  RoundItem* round_items;   // [kRoundMaxItems]  work list of the round kernel's launch in flight
  RoundUnit* round_units;   // [kRoundMaxUnits]  its units in several parts
  int32_t alibi;            // 1: logits get - l_h (m - n) (Eq. 1), from razor_cache_set_alibi
  int32_t n_heads;          // B*Hkv
  int32_t n_kv_heads;
  int32_t max_pages;        // page-table row length
  int32_t max_items;
  int32_t head_dim;
  int32_t n_sink;
  int32_t group;
  int32_t use_comp;
  size_t page_bytes;
  float scale_log2;         // sm_scale * log2(e)
};

// Decode launch tuning (razor_cache_set_option).
struct DecodeTuning {
  int32_t tail_items_per_sm;  // small items per SM that the dynamic tail of the schedule is cut into
  int32_t static_pct;         // percent of the pages handed out as one equal span per CTA
  int32_t min_chunk_pages;    // smallest span / tail item
  int32_t ring_kb;          // shared-memory page ring per CTA, KiB (0: as large as fits)
  int32_t consumer_warps;   // 0: default for the group size
  int32_t tensor_cores;     // grouped bf16 heads: 0 auto (group >= 4), 1 on (group >= 2), 2 off
  int32_t early_prefetch;   // most pages a span CTA copies ahead of the launch dependency (0: none)
};

// Records the code razor_last_cuda_error() reports (per thread) and clears the runtime's sticky-free error state.
// Every entry point that returns RAZOR_E_CUDA goes through it, whichever source file it lives in.
void note_cuda_error(cudaError_t e);

// Kernel launchers (defined in the .cu files).  Each returns the cudaError_t of the launch.
// n_plan: entries of dv.plan to apply (state and page-table rows) before the rows are streamed.
cudaError_t launch_compress(const DeviceView& dv, int dtype, int layer, int n_seqs, int n_slices, int n_plan,
                            cudaStream_t stream);
// early_reads: the last kernel the library launched that WROTE this layer's pages, state or sums is not the one
// directly before this append in the stream, so the append may read before it waits for that kernel.
cudaError_t launch_append(const DeviceView& dv, int dtype, int layer, const void* k_new, const void* v_new,
                          int early_reads, cudaStream_t stream);
// n_slices > 0: the run is long, use the kernel that is parallel over the tokens with that many slices per
// head (n_heads * n_slices slice sums must fit the compression scratch); 0: one warp per head, token by token.
cudaError_t launch_append_many(const DeviceView& dv, int dtype, int layer, const void* k_new, const void* v_new,
                               int n_tok, int n_slices, cudaStream_t stream);
// What a decode launch pulls from the queue: n_jobs jobs, the first n_spans of them spans (item
// ranges jobs[j]..jobs[j+1]), the others single items starting at tail_first.
constexpr int kEarlyCtas = 160;   // CTAs that can be told how far to prefetch ahead of the launch dependency
struct DecodeJobs {
  int32_t n_items, n_jobs, n_spans, tail_first;
  int32_t n_multi;   // heads in several parts
  int32_t n_tok;     // query tokens per sequence in this launch (1 for a decode step)
  // A round longer than one launch can take is run block by block: q and out point at the block's first
  // token, tok_stride is the round's length (tokens per sequence in q and out), q_after the number of
  // tokens of the round that come after the block (they are cached already, and masked).
  int32_t tok_stride;
  int32_t q_after;
  // 1: no kernel that can still be in flight when this launch starts writes this layer's head states, so a CTA
  // may load the state of its first work item ahead of the launch dependency (the host tracks the writers)
  int32_t state_stable;
  // early[i]: how many of the first pages of CTA i's span (pages of the span's first work item, in order) may
  // be copied into the ring BEFORE the kernel waits for the launch it depends on.  The host knows every head's
  // length and which page the preceding append (if any) wrote, so it can name pages that nothing in flight
  // writes.  0: none.  Only the first kEarlyCtas CTAs take part.
  uint8_t early[kEarlyCtas];
  // Not NULL: the launch first adds one token per sequence (k_new, v_new device [B, Hkv, D]) exactly as the
  // append kernel would, and attends over the cache with that token in it.
  const void* k_new;
  const void* v_new;
};
cudaError_t launch_decode(const DeviceView& dv, int dtype, int layer, const DecodeJobs& jobs, const void* q,
                          float* out, int n_sms, const DecodeTuning& tune, cudaStream_t stream);
// ---- rounds of many query tokens (razor_round.cu): the query rows of a KV head (query tokens x query heads of
// the group) are tiled kRoundTileRows at a time and the head's slot stream is walked in blocks of kRoundBlockTokens.
constexpr int kRoundTileRows = 128;
constexpr int kRoundBlockTokens = 128;
constexpr int kRoundMaxItems = 8192;
constexpr int kRoundMaxUnits = 4096;
struct RoundItem {
  int32_t head;        // b * Hkv + kv_head
  int32_t q_tile;      // rows [q_tile * 128, + 128) of the head's query rows
  int32_t blk_begin;   // 128-token blocks [blk_begin, blk_end) of the head's slots
  int32_t blk_end;
  int32_t part_idx;    // index of this part within its (head, q_tile) unit
  int32_t n_parts;
  int32_t rec_base;    // first record row of the unit (each part owns kRoundTileRows rows)
  int32_t pad;
};
struct RoundUnit {     // a (head, q_tile) cut into several parts: one entry of the merge kernel's work list
  int32_t head, q_tile, rec_base, n_parts;
};
struct RoundJobs {
  int32_t n_items, n_units, n_tok, pad;
};
cudaError_t launch_round(const DeviceView& dv, long long pool_pages, int layer, const RoundJobs& jb, const void* q,
                         float* out, int n_sms, cudaStream_t stream);
cudaError_t launch_wait_selftest(const DeviceView& dv, unsigned long long limit_ns, cudaStream_t stream);
cudaError_t launch_export(const DeviceView& dv, int dtype, int layer, int head, int32_t* kept_pos, void* K, void* V,
                          float* mean_k, float* mean_v, float* sum_k, float* sum_v, cudaStream_t stream);

// Host-only schedule builder (razor_schedule.cpp).
struct SchedParams {
  int n_ctas;              // CTAs of the launch (one per SM)
  int static_pct;          // 0..100
  int tail_items_per_cta;  // >= 1
  int min_chunk_pages;     // >= 1
  int merge_max_parts;     // heads in at most this many parts are folded inside the streaming kernel
};
struct SchedInfo {
  int n_items, n_jobs, n_spans;   // the first n_spans jobs are spans
  int span_pages, chunk_pages;    // size of a span, largest tail item
  int n_multi;                    // entries written to multi[]
};
// pages[h] = pages of head h's token stream now.  Writes the work items in job order to out[] and the
// first item of each job to jobs[] (n_jobs + 1 entries); lays out the partial records of the heads cut
// into several parts and lists those heads in multi[] (at most n_heads entries).  Returns the number of
// items (<= max_items), or -1 when they would not fit.
int build_schedule(const int32_t* pages, int n_heads, const SchedParams& sp, int max_items, WorkItem* out,
                   int32_t* jobs, MultiHead* multi, SchedInfo* info);

}  // namespace razor
#endif
