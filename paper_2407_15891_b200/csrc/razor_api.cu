// Host side of the C ABI declared in include/razor.h: argument checks, the per-head plan
// (Algorithm 1: how many tokens each head keeps), page allocation, host mirrors of the
// per-head lengths (they are deterministic, so no device->host read is ever needed), the cached
// decode schedule, and the kernel launches.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "razor_internal.h"

using namespace razor;

namespace {

thread_local int g_last_cuda_error = 0;

#define RZ_CUDA(call)                          \
  do {                                         \
    cudaError_t e__ = (call);                  \
    if (e__ != cudaSuccess) {                  \
      razor::note_cuda_error(e__);             \
      return RAZOR_E_CUDA;                     \
    }                                          \
  } while (0)

constexpr int kItemBudget = 16384;     // upper bound on split parts beyond one per head
constexpr size_t kAlign = 256;

inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }
inline int ceil_div(long long a, long long b) { return (int)((a + b - 1) / b); }

struct Layout {
  size_t state, comp_sum, comp_mean, ring_sum, ring_valid, page_table, items, jobs, multi, rec_ml, rec_o, queue, tickets, scratch, plan, slopes, round_items, round_units, total;
  int max_pages, max_items;
};

int check_config(const razor_config_t* c) {
  if (!c) return RAZOR_E_NULL_PTR;
  if (c->batch < 1 || c->n_layers < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1) return RAZOR_E_INVALID_ARG;
  if (c->n_q_heads % c->n_kv_heads) return RAZOR_E_INVALID_ARG;
  const int g = c->n_q_heads / c->n_kv_heads;
  if (g != 1 && g != 2 && g != 4 && g != 8) return RAZOR_E_UNSUPPORTED_DIM;
  if (c->head_dim != 64 && c->head_dim != 128) return RAZOR_E_UNSUPPORTED_DIM;
  if (c->dtype != RAZOR_F32 && c->dtype != RAZOR_BF16) return RAZOR_E_UNSUPPORTED_DIM;
  if (c->page_tokens != kPageTokens) return RAZOR_E_UNSUPPORTED_DIM;
  if (c->n_sink < 0 || c->max_ctx_len < 0 || c->max_new_tokens < 0) return RAZOR_E_INVALID_ARG;
  if ((long long)c->max_ctx_len + c->max_new_tokens > (1LL << 30)) return RAZOR_E_INVALID_ARG;
  if ((long long)c->batch * c->n_kv_heads > (1 << 20)) return RAZOR_E_INVALID_ARG;
  if (!(c->sm_scale >= 0.f) || std::isinf(c->sm_scale)) return RAZOR_E_INVALID_ARG;
  return RAZOR_OK;
}

inline size_t esz(const razor_config_t& c) { return c.dtype == RAZOR_BF16 ? 2 : 4; }
inline size_t row_bytes(const razor_config_t& c) { return (size_t)c.head_dim * esz(c); }
inline size_t page_bytes(const razor_config_t& c) { return 2 * (size_t)kPageTokens * row_bytes(c); }

Layout make_layout(const razor_config_t& c) {
  Layout l;
  const size_t nh = (size_t)c.batch * c.n_kv_heads, L = c.n_layers, D = c.head_dim;
  const int g = c.n_q_heads / c.n_kv_heads;
  l.max_pages = std::max(1, ceil_div((long long)c.max_ctx_len + c.max_new_tokens, kPageTokens));
  l.max_items = (int)nh + kItemBudget;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  l.state = take(L * nh * sizeof(HeadState));
  l.comp_sum = take(L * nh * 2 * D * sizeof(float));
  l.comp_mean = take(L * nh * 2 * D * sizeof(float));
  l.ring_sum = take(L * nh * 2 * D * sizeof(float));
  l.ring_valid = take(L * nh * sizeof(int32_t));
  l.page_table = take(L * nh * (size_t)l.max_pages * sizeof(int32_t));
  l.items = take(L * (size_t)l.max_items * sizeof(WorkItem));
  l.jobs = take(L * ((size_t)l.max_items + 1) * sizeof(int32_t));
  l.multi = take(L * nh * sizeof(MultiHead));
  // a partial record holds up to kMaxGroup rows: query heads of the group x query tokens of a round
  l.rec_ml = take((size_t)l.max_items * kMaxGroup * sizeof(float2));
  l.rec_o = take((size_t)l.max_items * kMaxGroup * D * sizeof(float));
  (void)g;
  l.queue = take(8 * sizeof(int32_t));   // queue[0..3], then the status word
  l.tickets = take(nh * sizeof(int32_t));
  l.scratch = take(((size_t)kCompressSliceBudget + nh) * 2 * D * sizeof(float));
  l.plan = take(nh * sizeof(HeadPlan) + (size_t)c.batch * sizeof(SeqDesc));   // plan[], then seq_desc[]
  l.slopes = take(L * (size_t)c.n_q_heads * sizeof(float));
  l.round_items = take((size_t)kRoundMaxItems * sizeof(RoundItem));
  l.round_units = take((size_t)kRoundMaxUnits * sizeof(RoundUnit));
  l.total = off;
  return l;
}

// Tokens a head can ever hold (Algorithm 1 plus room for appended decode tokens).
inline long long head_capacity_tokens(const razor_config_t& c, int n_ctx, int window, bool retrieval) {
  const long long grown = (long long)n_ctx + c.max_new_tokens;
  return retrieval ? grown : std::min(grown, (long long)c.n_sink + window);
}

constexpr int kPlanSlots = 16;   // compression plans that may be on their way to the device at once
constexpr int kRoundSlots = 8;   // work lists of the round kernel that may be on their way to the device at once
constexpr size_t kRoundSlotBytes = (size_t)kRoundMaxItems * sizeof(RoundItem) + (size_t)kRoundMaxUnits * sizeof(RoundUnit);

struct LayerHost {
  bool any = false;
  int n_done = 0;
  std::vector<uint8_t> retr;        // [Hkv]
  std::vector<int32_t> head_window; // [Hkv] per-head cap on the recent window (razor_cache_set_head_windows); empty: none
  std::vector<uint8_t> seq_done;    // [B]
  std::vector<HeadState> hs;        // [B*Hkv] mirror of the device state
  std::vector<long long> region_start, region_count;   // pages owned by (layer, b)
  int appended = 0;
  // decode schedule
  bool sched_valid = false;
  int n_items = 0, n_jobs = 0, n_spans = 0, n_multi = 0, chunk_pages = 0, growth_tokens = 0, sched_rows = 0;
  WorkItem* items = nullptr;        // pinned host, [max_items]
  int32_t* jobs = nullptr;          // pinned host, [max_items + 1]
  MultiHead* multi = nullptr;       // pinned host, [B*Hkv]
  cudaEvent_t upload_done = nullptr;
};

uint64_t mix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

}  // namespace

void razor::note_cuda_error(cudaError_t e) {
  g_last_cuda_error = (int)e;
  (void)cudaGetLastError();
}

struct razor_cache {
  razor_config_t cfg;
  Layout lay;
  DeviceView dv;
  long long pool_pages = 0, next_page = 0;
  int n_sms = 148;
  DecodeTuning tune{3, 80, 32, 0, 0, 0, 12};
  int round_tiled_min_rows = 9;   // rounds with at least this many query rows per KV head run on the query-tiled kernel
  std::vector<LayerHost> layers;
  WorkItem* pinned_items = nullptr;   // [L][max_items]
  int32_t* pinned_jobs = nullptr;     // [L][max_items + 1]
  MultiHead* pinned_multi = nullptr;  // [L][B*Hkv]
  // Compression plan staging: a ring of images of the device's plan region (HeadPlan[B*Hkv], then SeqDesc[B]),
  // so that a run of compression calls does not wait for each upload before preparing the next.
  uint8_t* pinned_plan = nullptr;     // [kPlanSlots][plan_bytes]
  size_t plan_bytes = 0;
  cudaEvent_t plan_done[kPlanSlots] = {};
  int plan_next = 0;
  // Work list of the round kernel (razor_decode_attention_multi on long rounds): pinned staging, one upload in flight.
  // kRoundSlots staging areas used in turn (RoundItem[kRoundMaxItems], then RoundUnit[kRoundMaxUnits] each), so that
  // the host waits for an upload only when it comes round to that upload's area again and can otherwise run ahead
  uint8_t* pinned_round = nullptr;
  cudaEvent_t round_done[kRoundSlots] = {};
  int round_slot = 0;
  // Layer whose pages, state or sums the last kernel launched for this cache wrote (-1: it wrote none, a decode).
  // An append of another layer may read before it waits for that kernel.
  int last_writer_layer = -1;
  // Kernels launched since the last decode launch that write a layer: (layer, kind).  A decode kernel waits for
  // everything before it and only then lets its successors start, so these are the only library kernels that
  // can still be in flight while the NEXT decode kernel runs the part that precedes its own dependency wait.
  enum { kWriteOneToken = 1, kWriteBulk = 2 };
  std::vector<std::pair<int, int>> writes_since_decode;
  bool writes_overflow = false;
  void note_write(int layer, int kind) {
    last_writer_layer = layer;
    if (writes_since_decode.size() < 256) writes_since_decode.emplace_back(layer, kind);
    else writes_overflow = true;
  }
};

extern "C" {

const char* razor_version(void) { return "0.1"; }

int razor_last_cuda_error(void) { return g_last_cuda_error; }

const char* razor_status_string(int s) {
  switch (s) {
    case RAZOR_OK: return "ok";
    case RAZOR_E_INVALID_ARG: return "invalid argument";
    case RAZOR_E_NULL_PTR: return "null pointer";
    case RAZOR_E_UNSUPPORTED_DIM: return "unsupported head_dim, dtype, group size or page size";
    case RAZOR_E_POOL_TOO_SMALL: return "page pool or workspace too small";
    case RAZOR_E_CAPACITY: return "capacity exceeded (max_new_tokens or max_ctx_len)";
    case RAZOR_E_NOT_COMPRESSED: return "layer or sequence not compressed yet";
    case RAZOR_E_CUDA: return "CUDA runtime error (see razor_last_cuda_error)";
    case RAZOR_E_MISALIGNED: return "pointer or stride not 16-byte aligned";
    default: return "unknown status";
  }
}

int razor_query_bytes(const razor_config_t* cfg, const int32_t* ctx_len, const int32_t* window,
                      const uint8_t* head_is_retrieval, size_t* pool_bytes, size_t* workspace_bytes) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!ctx_len || !window || !head_is_retrieval) return RAZOR_E_NULL_PTR;
  if (!pool_bytes && !workspace_bytes) return RAZOR_E_NULL_PTR;
  unsigned long long pages = 0;
  for (int b = 0; b < cfg->batch; ++b) {
    if (ctx_len[b] < 0 || window[b] < 0) return RAZOR_E_INVALID_ARG;
    if (ctx_len[b] > cfg->max_ctx_len) return RAZOR_E_CAPACITY;
    for (int l = 0; l < cfg->n_layers; ++l)
      for (int g = 0; g < cfg->n_kv_heads; ++g)
        pages += ceil_div(head_capacity_tokens(*cfg, ctx_len[b], window[b],
                                               head_is_retrieval[(size_t)l * cfg->n_kv_heads + g] != 0),
                          kPageTokens);
  }
  if (pool_bytes) *pool_bytes = align_up(std::max<size_t>(1, pages) * page_bytes(*cfg));
  if (workspace_bytes) *workspace_bytes = make_layout(*cfg).total;
  return RAZOR_OK;
}

int razor_cache_create(razor_cache_t** out, const razor_config_t* cfg, void* pool_dev, size_t pool_bytes,
                       void* workspace_dev, size_t workspace_bytes, void* stream) {
  if (!out) return RAZOR_E_NULL_PTR;
  *out = nullptr;
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!pool_dev || !workspace_dev) return RAZOR_E_NULL_PTR;
  if (((uintptr_t)pool_dev | (uintptr_t)workspace_dev) & (kAlign - 1)) return RAZOR_E_MISALIGNED;
  const Layout lay = make_layout(*cfg);
  if (workspace_bytes < lay.total) return RAZOR_E_POOL_TOO_SMALL;
  if (pool_bytes < page_bytes(*cfg)) return RAZOR_E_POOL_TOO_SMALL;

  int dev = 0, sms = 0;
  RZ_CUDA(cudaGetDevice(&dev));
  RZ_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));

  razor_cache* c = new (std::nothrow) razor_cache();
  if (!c) return RAZOR_E_INVALID_ARG;
  c->cfg = *cfg;
  if (c->cfg.sm_scale == 0.f) c->cfg.sm_scale = 1.0f / std::sqrt((float)cfg->head_dim);
  c->lay = lay;
  c->n_sms = sms;
  c->pool_pages = (long long)(pool_bytes / page_bytes(*cfg));
  uint8_t* ws = (uint8_t*)workspace_dev;
  DeviceView& dv = c->dv;
  dv.pool = (uint8_t*)pool_dev;
  dv.state = (HeadState*)(ws + lay.state);
  dv.comp_sum = (float*)(ws + lay.comp_sum);
  dv.comp_mean = (float*)(ws + lay.comp_mean);
  dv.ring_sum = (float*)(ws + lay.ring_sum);
  dv.ring_valid = (int32_t*)(ws + lay.ring_valid);
  dv.page_table = (int32_t*)(ws + lay.page_table);
  dv.items = (WorkItem*)(ws + lay.items);
  dv.jobs = (int32_t*)(ws + lay.jobs);
  dv.rec_ml = (float2*)(ws + lay.rec_ml);
  dv.rec_o = (float*)(ws + lay.rec_o);
  dv.multi = (MultiHead*)(ws + lay.multi);
  dv.queue = (int32_t*)(ws + lay.queue);
  dv.status = dv.queue + 4;
  dv.tickets = (int32_t*)(ws + lay.tickets);
  dv.compress_scratch = (float*)(ws + lay.scratch);
  dv.plan = (HeadPlan*)(ws + lay.plan);
  dv.seq_desc = (SeqDesc*)(ws + lay.plan + (size_t)cfg->batch * cfg->n_kv_heads * sizeof(HeadPlan));
  dv.alibi_slopes = (float*)(ws + lay.slopes);
  dv.round_items = (RoundItem*)(ws + lay.round_items);
  dv.round_units = (RoundUnit*)(ws + lay.round_units);
  dv.alibi = 0;
  dv.n_heads = cfg->batch * cfg->n_kv_heads;
  dv.n_kv_heads = cfg->n_kv_heads;
  dv.max_pages = lay.max_pages;
  dv.max_items = lay.max_items;
  dv.head_dim = cfg->head_dim;
  dv.n_sink = cfg->n_sink;
  dv.group = cfg->n_q_heads / cfg->n_kv_heads;
  dv.use_comp = cfg->use_compensation ? 1 : 0;
  dv.page_bytes = page_bytes(*cfg);
  dv.scale_log2 = c->cfg.sm_scale * 1.4426950408889634f;

  cudaError_t e = cudaMemsetAsync(workspace_dev, 0, lay.total, (cudaStream_t)stream);
  if (e == cudaSuccess)
    e = cudaHostAlloc((void**)&c->pinned_items, (size_t)cfg->n_layers * lay.max_items * sizeof(WorkItem),
                      cudaHostAllocDefault);
  if (e == cudaSuccess)
    e = cudaHostAlloc((void**)&c->pinned_jobs, (size_t)cfg->n_layers * (lay.max_items + 1) * sizeof(int32_t),
                      cudaHostAllocDefault);
  if (e == cudaSuccess)
    e = cudaHostAlloc((void**)&c->pinned_multi, (size_t)cfg->n_layers * dv.n_heads * sizeof(MultiHead),
                      cudaHostAllocDefault);
  c->plan_bytes = (size_t)dv.n_heads * sizeof(HeadPlan) + (size_t)cfg->batch * sizeof(SeqDesc);
  if (e == cudaSuccess)
    e = cudaHostAlloc((void**)&c->pinned_plan, (size_t)kPlanSlots * c->plan_bytes, cudaHostAllocDefault);
  if (e == cudaSuccess)
    e = cudaHostAlloc((void**)&c->pinned_round, (size_t)kRoundSlots * kRoundSlotBytes, cudaHostAllocDefault);
  if (e != cudaSuccess) {
    note_cuda_error(e);
    if (c->pinned_items) cudaFreeHost(c->pinned_items);
    if (c->pinned_jobs) cudaFreeHost(c->pinned_jobs);
    if (c->pinned_multi) cudaFreeHost(c->pinned_multi);
    if (c->pinned_plan) cudaFreeHost(c->pinned_plan);
    if (c->pinned_round) cudaFreeHost(c->pinned_round);
    delete c;
    return RAZOR_E_CUDA;
  }
  c->layers.resize(cfg->n_layers);
  for (int l = 0; l < cfg->n_layers; ++l) {
    LayerHost& L = c->layers[l];
    L.retr.assign(cfg->n_kv_heads, 0);
    L.seq_done.assign(cfg->batch, 0);
    L.hs.assign((size_t)dv.n_heads, HeadState{0, 0, 0, 0});
    L.region_start.assign(cfg->batch, 0);
    L.region_count.assign(cfg->batch, 0);
    L.items = c->pinned_items + (size_t)l * lay.max_items;
    L.jobs = c->pinned_jobs + (size_t)l * (lay.max_items + 1);
    L.multi = c->pinned_multi + (size_t)l * dv.n_heads;
  }
  *out = c;
  return RAZOR_OK;
}

int razor_cache_reset(razor_cache_t* c) {
  if (!c) return RAZOR_E_NULL_PTR;
  c->next_page = 0;
  for (LayerHost& L : c->layers) {
    L.any = false;
    L.n_done = 0;
    L.appended = 0;
    L.sched_valid = false;
    std::fill(L.seq_done.begin(), L.seq_done.end(), 0);
    std::fill(L.region_count.begin(), L.region_count.end(), 0);
    std::fill(L.hs.begin(), L.hs.end(), HeadState{0, 0, 0, 0});
  }
  return RAZOR_OK;
}

int razor_cache_destroy(razor_cache_t* c) {
  if (!c) return RAZOR_E_NULL_PTR;
  for (LayerHost& L : c->layers) {
    if (L.upload_done) cudaEventDestroy(L.upload_done);
  }
  if (c->pinned_items) cudaFreeHost(c->pinned_items);
  if (c->pinned_jobs) cudaFreeHost(c->pinned_jobs);
  if (c->pinned_multi) cudaFreeHost(c->pinned_multi);
  if (c->pinned_plan) cudaFreeHost(c->pinned_plan);
  if (c->pinned_round) cudaFreeHost(c->pinned_round);
  for (cudaEvent_t ev : c->round_done)
    if (ev) cudaEventDestroy(ev);
  for (cudaEvent_t ev : c->plan_done)
    if (ev) cudaEventDestroy(ev);
  delete c;
  return RAZOR_OK;
}

}  // extern "C"

namespace {

constexpr int kAppendChunkMin = 8;   // razor_append_many: runs this long are appended in parallel over the tokens
                                     // (shorter ones token by token in one kernel: about 2 us per token)

struct SeqIn {
  int b;
  const void* K;
  const void* V;
  int64_t stride_h, stride_n;
  int n_ctx, window;
};

int ensure_schedule(razor_cache* c, int layer, cudaStream_t stream, bool upload, int rows);

// Shared body of razor_compress / razor_compress_seq: the plan (C0), page allocation, uploads, launch.
int compress_impl(razor_cache* c, int layer, const std::vector<SeqIn>& seqs, const uint8_t* retr, int n_sink,
                  cudaStream_t stream) {
  const razor_config_t& cfg = c->cfg;
  if (layer < 0 || layer >= cfg.n_layers) return RAZOR_E_INVALID_ARG;
  if (n_sink != cfg.n_sink) return RAZOR_E_INVALID_ARG;
  LayerHost& L = c->layers[layer];
  const int H = cfg.n_kv_heads;
  const size_t es = esz(cfg);
  std::vector<uint8_t> flags(H);
  for (int g = 0; g < H; ++g) flags[g] = retr[g] ? 1 : 0;

  // The retrieval set belongs to the layer: sequences compressed one at a time must agree on it.
  bool others_done = false;
  {
    std::vector<uint8_t> in_call(cfg.batch, 0);
    for (const SeqIn& s : seqs) in_call[s.b] = 1;
    for (int b = 0; b < cfg.batch; ++b) others_done |= (L.seq_done[b] && !in_call[b]);
  }
  if (others_done && std::memcmp(flags.data(), L.retr.data(), H) != 0) return RAZOR_E_INVALID_ARG;

  int n_max = 0;
  for (const SeqIn& s : seqs) {
    if (s.b < 0 || s.b >= cfg.batch) return RAZOR_E_INVALID_ARG;
    if (s.n_ctx < 0 || s.window < 0) return RAZOR_E_INVALID_ARG;
    if (s.n_ctx > cfg.max_ctx_len) return RAZOR_E_CAPACITY;
    if (s.n_ctx > 0) {
      if (!s.K || !s.V) return RAZOR_E_NULL_PTR;
      if (((uintptr_t)s.K | (uintptr_t)s.V) & 15) return RAZOR_E_MISALIGNED;
      if (((s.stride_h * (int64_t)es) | (s.stride_n * (int64_t)es)) & 15) return RAZOR_E_MISALIGNED;
      if (s.stride_n < cfg.head_dim || s.stride_h < 0) return RAZOR_E_INVALID_ARG;
    }
    n_max = std::max(n_max, s.n_ctx);
  }

  // A head's recent window: the sequence's, capped by the head's own when per-head windows are set
  // (ALiBi heads each have their own vision scope, Section 3.1).
  auto eff_window = [&](int seq_window, int g) {
    return L.head_window.empty() ? seq_window : std::min(seq_window, L.head_window[g]);
  };
  // Page plan per sequence; allocate (or reuse) the sequence's region, all-or-nothing.
  std::vector<long long> need(seqs.size());
  long long next = c->next_page;
  std::vector<long long> new_start(seqs.size(), -1);
  for (size_t i = 0; i < seqs.size(); ++i) {
    long long pages = 0;
    for (int g = 0; g < H; ++g)
      pages += ceil_div(head_capacity_tokens(cfg, seqs[i].n_ctx, eff_window(seqs[i].window, g), flags[g] != 0),
                        kPageTokens);
    need[i] = pages;
    if (pages > L.region_count[seqs[i].b]) {
      if (next + pages > c->pool_pages) return RAZOR_E_POOL_TOO_SMALL;
      new_start[i] = next;
      next += pages;
    }
  }
  // Nothing of the host mirror (page cursor, regions, head states, "compressed" marks) is touched until every
  // CUDA call of this function has succeeded: after a failure the layer is left as it was, so a later call
  // cannot run on lengths the device never received.
  std::vector<HeadState> new_hs(seqs.size() * (size_t)H);
  std::vector<long long> region_start(seqs.size());
  // Once something has been enqueued the device copy of these sequences may have changed (page-table rows, the
  // plan): after a failure from there on they count as not compressed until a compression of them succeeds.
  auto fail_enqueued = [&](cudaError_t e) {
    for (const SeqIn& s : seqs)
      if (L.seq_done[s.b]) { L.seq_done[s.b] = 0; L.n_done -= 1; }
    L.sched_valid = false;
    note_cuda_error(e);
    return (int)RAZOR_E_CUDA;
  };
  cudaError_t ce;

  // The plan goes to the device in one copy from pinned memory: per head its state after the call and the
  // run of pool pages behind its page-table row (compress_plan_kernel writes both), then the sequences.
  const int slot = c->plan_next;
  if (c->plan_done[slot]) RZ_CUDA(cudaEventSynchronize(c->plan_done[slot]));   // its last upload has left the slot
  uint8_t* staging = c->pinned_plan + (size_t)slot * c->plan_bytes;
  HeadPlan* plan = (HeadPlan*)staging;
  SeqDesc* descs = (SeqDesc*)(staging + (size_t)c->dv.n_heads * sizeof(HeadPlan));
  int n_plan = 0;
  std::vector<int32_t> rows;   // only for permuted page ids
  for (size_t i = 0; i < seqs.size(); ++i) {
    const SeqIn& s = seqs[i];
    region_start[i] = new_start[i] >= 0 ? new_start[i] : L.region_start[s.b];
    const bool shuffled = cfg.page_shuffle_seed != 0;
    std::vector<int32_t> ids;
    if (shuffled) {   // page ids of the region, permuted: the rows are written from the host
      ids.resize((size_t)need[i]);
      for (long long k = 0; k < need[i]; ++k) ids[(size_t)k] = (int32_t)(region_start[i] + k);
      uint64_t st = mix64((uint64_t)cfg.page_shuffle_seed * 1315423911ull + (uint64_t)layer * 2654435761ull + s.b);
      for (long long k = need[i] - 1; k > 0; --k) {
        st = mix64(st);
        std::swap(ids[(size_t)k], ids[(size_t)(st % (uint64_t)(k + 1))]);
      }
      rows.assign((size_t)H * c->lay.max_pages, 0);
    }
    long long cursor = 0;
    for (int g = 0; g < H; ++g) {
      const bool r = flags[g] != 0;
      const int wg = eff_window(s.window, g);
      const int cap_pages = ceil_div(head_capacity_tokens(cfg, s.n_ctx, wg, r), kPageTokens);
      const bool keep_all = r || s.n_ctx <= cfg.n_sink + wg;
      HeadState h;
      h.len = keep_all ? s.n_ctx : cfg.n_sink + wg;
      h.n_drop = keep_all ? 0 : s.n_ctx - cfg.n_sink - wg;
      h.ring_head = 0;
      h.window = r ? -1 : wg;
      new_hs[i * (size_t)H + g] = h;
      HeadPlan& pl = plan[n_plan++];
      pl.head = s.b * H + g;
      pl.first_page = (int32_t)(region_start[i] + cursor);
      pl.n_pages = shuffled ? 0 : cap_pages;
      pl.len = h.len;
      pl.n_drop = h.n_drop;
      pl.window = h.window;
      if (shuffled)
        for (int k = 0; k < cap_pages; ++k) rows[(size_t)g * c->lay.max_pages + k] = ids[(size_t)(cursor + k)];
      cursor += cap_pages;
    }
    if (shuffled) {
      const size_t head0 = (size_t)layer * c->dv.n_heads + (size_t)s.b * H;
      ce = cudaMemcpyAsync(c->dv.page_table + head0 * c->lay.max_pages, rows.data(), rows.size() * sizeof(int32_t),
                           cudaMemcpyHostToDevice, stream);   // pageable source: staged before the call returns
      if (ce != cudaSuccess) return fail_enqueued(ce);
    }
    SeqDesc d;
    d.K = s.K; d.V = s.V; d.stride_h = s.stride_h; d.stride_n = s.stride_n;
    d.n_ctx = s.n_ctx; d.window = s.window; d.b = s.b; d.pad = 0;
    descs[i] = d;
  }
  // one copy covers plan[0 .. n_plan) and, behind the full plan array, the sequence descriptors
  if (!c->plan_done[slot] &&
      (ce = cudaEventCreateWithFlags(&c->plan_done[slot], cudaEventDisableTiming)) != cudaSuccess)
    return fail_enqueued(ce);
  if ((ce = cudaMemcpyAsync(c->dv.plan, staging, c->plan_bytes, cudaMemcpyHostToDevice, stream)) != cudaSuccess)
    return fail_enqueued(ce);
  c->plan_next = (slot + 1) % kPlanSlots;   // the slot is in use from here on, whatever happens next
  if ((ce = cudaEventRecord(c->plan_done[slot], stream)) != cudaSuccess) return fail_enqueued(ce);

  // Slices per head: about 48 CTAs per SM in all (sixteen rounds of the three a SM holds: short CTAs keep the
  // end of the grid even, whichever heads come last), slices no shorter than 512 rows where the context allows
  // (a CTA that streams less pays more for its start than it evens out) and never shorter than 64, and no more
  // slice sums than the scratch has room for.
  const long long heads_in_call = (long long)seqs.size() * H;
  const long long room = ((long long)kCompressSliceBudget + c->dv.n_heads) / heads_in_call;
  long long slices = ceil_div((long long)c->n_sms * 48, heads_in_call);
  const long long by_rows = n_max >= 8 * 512 ? n_max / 512 : std::max(1, n_max / 64);
  slices = std::max(1LL, std::min({slices, (long long)kCompressMaxSlices, room, by_rows}));
  c->note_write(layer, razor_cache::kWriteBulk);
  ce = launch_compress(c->dv, cfg.dtype, layer, (int)seqs.size(), (int)slices, n_plan, stream);
  if (ce != cudaSuccess) return fail_enqueued(ce);
  // ---- commit
  c->next_page = next;
  for (size_t i = 0; i < seqs.size(); ++i) {
    const int b = seqs[i].b;
    if (new_start[i] >= 0) {
      L.region_start[b] = new_start[i];
      L.region_count[b] = need[i];
    }
    for (int g = 0; g < H; ++g) L.hs[(size_t)b * H + g] = new_hs[i * (size_t)H + g];
    if (!L.seq_done[b]) { L.seq_done[b] = 1; L.n_done += 1; }
  }
  L.retr = flags;
  L.any = true;
  L.appended = 0;
  L.sched_valid = false;
  // With the layer complete, its decode schedule is planned and sent to the device here, behind the compression
  // kernels, rather than in front of the layer's first decode launch, where the copies would sit between two
  // kernels that otherwise overlap.  (A failure here is not an error of the compression: the decode call plans again.)
  if (L.n_done == cfg.batch) (void)ensure_schedule(c, layer, stream, true, cfg.n_q_heads / cfg.n_kv_heads);
  return RAZOR_OK;
}

int ensure_schedule(razor_cache* c, int layer, cudaStream_t stream, bool upload, int rows) {
  LayerHost& L = c->layers[layer];
  // (which heads the streaming kernel folds itself depends on the rows of a KV head's tile in this launch)
  const bool stale = !L.sched_valid || L.sched_rows != rows || (long long)L.growth_tokens * 4 >= (long long)L.chunk_pages * kPageTokens;
  if (!stale) return RAZOR_OK;
  const int nh = c->dv.n_heads;
  std::vector<int32_t> pages(nh);
  for (int h = 0; h < nh; ++h) pages[h] = ceil_div(L.hs[h].len, kPageTokens);
  if (L.upload_done) RZ_CUDA(cudaEventSynchronize(L.upload_done));   // previous upload has left the staging area
  const SchedParams sp{c->n_sms, c->tune.static_pct, c->tune.tail_items_per_sm, c->tune.min_chunk_pages,
                       std::min((int)kMergeInKernelMaxParts, merge_in_kernel_max_parts(rows))};
  SchedInfo info{};
  const int n = build_schedule(pages.data(), nh, sp, c->lay.max_items, L.items, L.jobs, L.multi, &info);
  L.sched_rows = rows;
  if (n < 0) return RAZOR_E_INVALID_ARG;
  L.n_items = n;
  L.n_jobs = info.n_jobs;
  L.n_spans = info.n_spans;
  L.n_multi = info.n_multi;
  L.chunk_pages = info.chunk_pages;
  L.growth_tokens = 0;
  if (upload) {
    if (!L.upload_done) RZ_CUDA(cudaEventCreateWithFlags(&L.upload_done, cudaEventDisableTiming));
    RZ_CUDA(cudaMemcpyAsync(c->dv.items + (size_t)layer * c->lay.max_items, L.items, (size_t)n * sizeof(WorkItem),
                            cudaMemcpyHostToDevice, stream));
    RZ_CUDA(cudaMemcpyAsync(c->dv.jobs + (size_t)layer * (c->lay.max_items + 1), L.jobs,
                            (size_t)(L.n_jobs + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, stream));
    if (L.n_multi)
      RZ_CUDA(cudaMemcpyAsync(c->dv.multi + (size_t)layer * nh, L.multi, (size_t)L.n_multi * sizeof(MultiHead),
                              cudaMemcpyHostToDevice, stream));
    RZ_CUDA(cudaEventRecord(L.upload_done, stream));
    L.sched_valid = true;
  } else {
    L.sched_valid = false;   // the device copy no longer matches; the next decode uploads again
  }
  return RAZOR_OK;
}

inline int layer_ready(const razor_cache* c, int layer) {
  if (layer < 0 || layer >= c->cfg.n_layers) return RAZOR_E_INVALID_ARG;
  const LayerHost& L = c->layers[layer];
  if (!L.any || L.n_done != c->cfg.batch) return RAZOR_E_NOT_COMPRESSED;
  return RAZOR_OK;
}

int emit_items(const WorkItem* w, int n, const int32_t* jobs, int n_jobs, int32_t* items, int32_t max_items,
               int32_t* n_items) {
  *n_items = n;
  if (!items) return RAZOR_OK;
  if (max_items < n) return RAZOR_E_INVALID_ARG;
  int job = 0;
  for (int i = 0; i < n; ++i) {
    while (job + 1 < n_jobs && jobs[job + 1] <= i) ++job;
    items[5 * i + 0] = w[i].head;
    items[5 * i + 1] = w[i].page_begin;
    items[5 * i + 2] = w[i].page_end;
    items[5 * i + 3] = w[i].n_parts;
    items[5 * i + 4] = job;
  }
  return RAZOR_OK;
}

}  // namespace

extern "C" {

int razor_compress(razor_cache_t* c, int32_t layer, const void* K, const void* V, int64_t stride_b, int64_t stride_h,
                   int64_t stride_n, const int32_t* ctx_len, const uint8_t* head_is_retrieval, int32_t n_sink,
                   const int32_t* window, void* stream) {
  if (!c || !ctx_len || !head_is_retrieval || !window) return RAZOR_E_NULL_PTR;
  const size_t es = esz(c->cfg);
  if ((stride_b * (int64_t)es) & 15) return RAZOR_E_MISALIGNED;
  if (stride_b < 0) return RAZOR_E_INVALID_ARG;
  std::vector<SeqIn> seqs(c->cfg.batch);
  for (int b = 0; b < c->cfg.batch; ++b) {
    SeqIn s;
    s.b = b;
    s.K = K ? (const char*)K + (size_t)b * stride_b * es : nullptr;
    s.V = V ? (const char*)V + (size_t)b * stride_b * es : nullptr;
    s.stride_h = stride_h;
    s.stride_n = stride_n;
    s.n_ctx = ctx_len[b];
    s.window = window[b];
    seqs[b] = s;
  }
  return compress_impl(c, layer, seqs, head_is_retrieval, n_sink, (cudaStream_t)stream);
}

int razor_compress_seq(razor_cache_t* c, int32_t layer, int32_t b, const void* K, const void* V, int64_t stride_h,
                       int64_t stride_n, int32_t ctx_len, const uint8_t* head_is_retrieval, int32_t n_sink,
                       int32_t window, void* stream) {
  if (!c || !head_is_retrieval) return RAZOR_E_NULL_PTR;
  std::vector<SeqIn> seqs(1);
  seqs[0] = SeqIn{b, K, V, stride_h, stride_n, ctx_len, window};
  return compress_impl(c, layer, seqs, head_is_retrieval, n_sink, (cudaStream_t)stream);
}

int razor_append(razor_cache_t* c, int32_t layer, const void* k_new, const void* v_new, void* stream) {
  if (!c || !k_new || !v_new) return RAZOR_E_NULL_PTR;
  int rc = layer_ready(c, layer);
  if (rc) return rc;
  if (((uintptr_t)k_new | (uintptr_t)v_new) & 15) return RAZOR_E_MISALIGNED;
  LayerHost& L = c->layers[layer];
  if (L.appended >= c->cfg.max_new_tokens) return RAZOR_E_CAPACITY;
  const int early_reads = c->last_writer_layer != layer;
  RZ_CUDA(launch_append(c->dv, c->cfg.dtype, layer, k_new, v_new, early_reads, (cudaStream_t)stream));
  c->note_write(layer, razor_cache::kWriteOneToken);
  // Host mirror of the kernel's state update.
  const int n_sink = c->cfg.n_sink;
  for (HeadState& h : L.hs) {
    if (h.window < 0 || h.len < n_sink + h.window) {
      h.len += 1;
    } else if (h.window == 0) {
      h.n_drop += 1;
    } else {
      h.n_drop += 1;
      h.ring_head = (h.ring_head + 1 == h.window) ? 0 : h.ring_head + 1;
    }
  }
  L.appended += 1;
  L.growth_tokens += 1;
  return RAZOR_OK;
}

int razor_append_many(razor_cache_t* c, int32_t layer, const void* k_new, const void* v_new, int32_t n_tokens,
                      void* stream) {
  if (!c || !k_new || !v_new) return RAZOR_E_NULL_PTR;
  int rc = layer_ready(c, layer);
  if (rc) return rc;
  if (n_tokens < 1) return RAZOR_E_INVALID_ARG;
  if (((uintptr_t)k_new | (uintptr_t)v_new) & 15) return RAZOR_E_MISALIGNED;
  LayerHost& L = c->layers[layer];
  if ((long long)L.appended + n_tokens > c->cfg.max_new_tokens) return RAZOR_E_CAPACITY;
  // Long runs go to the kernel that is parallel over the tokens: about eight CTAs per SM in all, slices of
  // at least 32 tokens, no more slice sums than the scratch holds.
  int slices = 0;
  if (n_tokens >= kAppendChunkMin) {
    const long long nh = c->dv.n_heads;
    const long long room = ((long long)kCompressSliceBudget + nh) / (2 * nh);   // two sets of sums per slice
    const long long cap = std::max(1LL, std::min(room, (long long)(n_tokens / 32)));
    const long long s0 = std::max(1LL, std::min((long long)ceil_div((long long)c->n_sms * 8, nh), cap));
    // two CTAs of the kernel are resident per SM: among s0 .. 1.5 s0 slices take the count whose CTAs fill their
    // last wave best
    const long long resident = 2LL * c->n_sms;
    long long best = s0;
    double best_fill = 0.0;
    for (long long sl = s0; sl <= std::min(cap, s0 + s0 / 2); ++sl) {
      const long long n = sl * nh, waves = (n + resident - 1) / resident;
      const double fill = (double)n / (double)(waves * resident);
      if (fill > best_fill + 1e-9) { best_fill = fill; best = sl; }
    }
    slices = (int)best;
  }
  RZ_CUDA(launch_append_many(c->dv, c->cfg.dtype, layer, k_new, v_new, n_tokens, slices, (cudaStream_t)stream));
  c->note_write(layer, razor_cache::kWriteBulk);
  const int n_sink = c->cfg.n_sink;
  for (HeadState& h : L.hs) h = state_after_run(h, n_sink, n_tokens);   // host mirror of the kernels' state update
  L.appended += n_tokens;
  L.growth_tokens += n_tokens;
  return RAZOR_OK;
}

int razor_append_plan(int32_t len, int32_t n_drop, int32_t ring_head, int32_t window, int32_t n_sink, int32_t n_tokens,
                      int32_t* slot, uint8_t* evicts_old, int32_t* len_after, int32_t* n_drop_after,
                      int32_t* ring_head_after) {
  if (len < 0 || n_drop < 0 || n_sink < 0 || n_tokens < 0) return RAZOR_E_INVALID_ARG;
  if (window >= 0 && (len > n_sink + window || ring_head < 0 || (window > 0 && ring_head >= window)))
    return RAZOR_E_INVALID_ARG;
  if (window >= 0 && len < n_sink + window && ring_head != 0) return RAZOR_E_INVALID_ARG;   // a ring that fills starts at 0
  const HeadState st{len, n_drop, ring_head, window};
  for (int a = 0; a < n_tokens; ++a) {
    const AppendFate f = append_fate(st, n_sink, n_tokens, a);
    if (slot) slot[a] = f.slot;
    if (evicts_old) evicts_old[a] = f.evicts_old ? 1 : 0;
  }
  const HeadState nx = state_after_run(st, n_sink, n_tokens);
  if (len_after) *len_after = nx.len;
  if (n_drop_after) *n_drop_after = nx.n_drop;
  if (ring_head_after) *ring_head_after = nx.ring_head;
  return RAZOR_OK;
}

static int decode_impl(razor_cache_t* c, int32_t layer, const void* q, float* out, int32_t n_tokens,
                       int32_t tok_stride, int32_t q_after, void* stream, const void* k_new = nullptr,
                       const void* v_new = nullptr);

// A long round on the query-tiled kernel.  Work items are (KV head, tile of 128 query rows, run of 128-token
// blocks): every (head, tile) unit is cut into parts of about equal size so that there are a few items per SM,
// the items are handed out longest first, and units in several parts get partial records (128 rows per part)
// that a merge kernel folds.  For a head whose slots are in position order (nothing dropped) the blocks that
// lie wholly after the tile's last query are left out.
static int round_impl(razor_cache_t* c, int32_t layer, const void* q, float* out, int32_t n_tokens, void* stream) {
  if (((uintptr_t)q | (uintptr_t)out) & 15) return RAZOR_E_MISALIGNED;
  const LayerHost& L = c->layers[layer];
  const int G = c->cfg.n_q_heads / c->cfg.n_kv_heads, nh = c->dv.n_heads;
  const int tok_per_tile = kRoundTileRows / G;
  const int n_tiles = ceil_div(n_tokens, tok_per_tile);
  struct Unit { int head, tile, blocks; };
  std::vector<Unit> units;
  units.reserve((size_t)nh * n_tiles);
  long long total_blocks = 0;
  for (int h = 0; h < nh; ++h) {
    const HeadState& st = L.hs[h];
    const int all_blocks = ceil_div(st.len, kRoundBlockTokens);
    for (int t = 0; t < n_tiles; ++t) {
      int blocks = all_blocks;
      if (st.window < 0 || st.n_drop == 0) {   // slot = position: nothing beyond the tile's last query is visible
        const int last_q = std::min(n_tokens, (t + 1) * tok_per_tile) - 1;
        const long long q_pos = (long long)st.len + st.n_drop - n_tokens + last_q;
        blocks = (int)std::min<long long>(all_blocks, q_pos / kRoundBlockTokens + 1);
      }
      units.push_back({h, t, std::max(blocks, 0)});
      total_blocks += std::max(blocks, 0);
    }
  }
  // Parts.  Two CTAs run per SM, and an item costs some ten steps' worth of set-up and read-out, a unit in several
  // parts a merge pass besides.  So a unit is cut only where balance asks for it: into parts of a CTA's average
  // load when the longest unit is at most one and a half times that load (a round of many tiles: usually no cut at
  // all), into parts of half of it otherwise; never more parts than fit the item list or the record rows.
  const long long rec_rows = (long long)c->lay.max_items * kMaxGroup;
  long long longest = 0;
  for (const Unit& u : units) longest = std::max<long long>(longest, u.blocks);
  const long long per_cta = std::max<long long>(1, ceil_div(total_blocks, (long long)c->n_sms * 2));
  long long chunk = 2 * longest <= 3 * per_cta ? per_cta : std::max<long long>(1, ceil_div(per_cta, 2));
  std::vector<RoundItem> items;
  std::vector<RoundUnit> multi;
  for (;;) {
    items.clear();
    multi.clear();
    long long rec = 0;
    for (const Unit& u : units) {
      const int parts = std::max(1, ceil_div(u.blocks, chunk));
      const int per = u.blocks > 0 ? ceil_div(u.blocks, parts) : 0;
      if (parts > 1) {
        multi.push_back(RoundUnit{u.head, u.tile, (int32_t)rec, parts});
      }
      for (int p = 0; p < parts; ++p) {
        RoundItem it;
        it.head = u.head; it.q_tile = u.tile;
        it.blk_begin = std::min(u.blocks, p * per); it.blk_end = std::min(u.blocks, (p + 1) * per);
        it.part_idx = p; it.n_parts = parts; it.rec_base = (int32_t)rec; it.pad = 0;
        items.push_back(it);
      }
      if (parts > 1) rec += (long long)parts * kRoundTileRows;
    }
    if ((long long)items.size() <= kRoundMaxItems && (long long)multi.size() <= kRoundMaxUnits && rec <= rec_rows) break;
    if (chunk > total_blocks) return RAZOR_E_CAPACITY;   // even unsplit units do not fit the work list
    chunk *= 2;
  }
  std::stable_sort(items.begin(), items.end(), [](const RoundItem& a, const RoundItem& b) {
    return a.blk_end - a.blk_begin > b.blk_end - b.blk_begin;
  });
  cudaStream_t s = (cudaStream_t)stream;
  const int slot = c->round_slot;
  c->round_slot = (slot + 1) % kRoundSlots;
  if (c->round_done[slot]) RZ_CUDA(cudaEventSynchronize(c->round_done[slot]));   // the upload that used this area last has left it
  else RZ_CUDA(cudaEventCreateWithFlags(&c->round_done[slot], cudaEventDisableTiming));
  uint8_t* area = c->pinned_round + (size_t)slot * kRoundSlotBytes;
  RoundItem* st_items = (RoundItem*)area;
  RoundUnit* st_units = (RoundUnit*)(area + (size_t)kRoundMaxItems * sizeof(RoundItem));
  std::memcpy(st_items, items.data(), items.size() * sizeof(RoundItem));
  if (!multi.empty()) std::memcpy(st_units, multi.data(), multi.size() * sizeof(RoundUnit));
  RZ_CUDA(cudaMemcpyAsync(c->dv.round_items, st_items, items.size() * sizeof(RoundItem), cudaMemcpyHostToDevice, s));
  if (!multi.empty())
    RZ_CUDA(cudaMemcpyAsync(c->dv.round_units, st_units, multi.size() * sizeof(RoundUnit), cudaMemcpyHostToDevice, s));
  RZ_CUDA(cudaEventRecord(c->round_done[slot], s));
  const RoundJobs jb{(int32_t)items.size(), (int32_t)multi.size(), n_tokens, 0};
  RZ_CUDA(launch_round(c->dv, c->pool_pages, layer, jb, q, out, c->n_sms, s));
  c->last_writer_layer = -1;
  c->writes_since_decode.clear();   // an ordinary launch: everything before it has completed when it starts
  c->writes_overflow = false;
  return RAZOR_OK;
}

// Which pages a span CTA may copy before the decode kernel waits for the launch it depends on.  While that part
// of the kernel runs, the library kernels launched since the previous decode (and that decode itself, when it
// appended a token) may still be writing.  If none of them wrote this layer, every page of it is stable.  If the
// only writes were single-token appends, at most two of them, the only pages they write are the ones holding the
// rows appended last, and the host mirror says which: the slots before `len` for a head that grew, the ring slots
// before ring_head for a head that evicted.  Anything else (a bulk append, a compression, more appends): no early
// copies.  For CTA i the count covers the leading pages of its span's first work item, cut at the first such
// page and at the item's length as it is now.
static void plan_early_prefetch(const razor_cache* c, int layer, DecodeJobs& jb) {
  std::memset(jb.early, 0, sizeof(jb.early));
  jb.state_stable = 0;
  if (c->tune.early_prefetch <= 0 || c->writes_overflow) return;
  int n_writes = 0;
  bool only_appends = true;
  for (const auto& wr : c->writes_since_decode) {
    if (wr.first != layer) continue;
    only_appends &= wr.second == razor_cache::kWriteOneToken;
    n_writes += 1;
  }
  jb.state_stable = n_writes == 0 ? 1 : 0;   // nothing in flight writes this layer's head states
  if (!only_appends) return;
  if (n_writes > 2) return;
  // rows written by appends that may be in flight: the newest n_writes ones; one more is left out for good
  // measure (in a launch that appends itself the mirror is already one token ahead)
  const int n_recent = n_writes > 0 || jb.k_new ? n_writes + 1 : 0;
  const LayerHost& L = c->layers[layer];
  const int n_sink = c->cfg.n_sink;
  const int n = std::min({L.n_spans, c->n_sms, (int)kEarlyCtas});
  for (int i = 0; i < n; ++i) {
    const WorkItem& w = L.items[L.jobs[i]];
    const HeadState& st = L.hs[w.head];
    const int head_pages = ceil_div(st.len, kPageTokens);
    const int page_end = w.page_end < 0 ? head_pages : std::min(w.page_end, head_pages);
    int e = std::min(c->tune.early_prefetch, std::max(0, page_end - w.page_begin));
    for (int j = 0; j < n_recent && e > 0; ++j) {
      int slot = -1;   // slot of the (j + 1)-th newest row
      if (st.window < 0 || st.n_drop == 0) {
        slot = st.len - 1 - j;                                                   // the head grew
      } else if (st.window > 0) {
        if (st.n_drop <= j) { e = 0; break; }                                    // it only just began to evict: leave it
        const long long r = ((long long)st.ring_head - 1 - j) % st.window;
        slot = n_sink + (int)(r < 0 ? r + st.window : r);
      }
      if (slot >= 0) {
        const int tp = slot / kPageTokens - w.page_begin;
        if (tp >= 0 && tp < e) e = tp;
      }
    }
    jb.early[i] = (uint8_t)e;
  }
}

int razor_decode_attention_multi(razor_cache_t* c, int32_t layer, const void* q, float* out, int32_t n_tokens,
                                 void* stream) {
  if (!c || !q || !out) return RAZOR_E_NULL_PTR;
  int rc = layer_ready(c, layer);
  if (rc) return rc;
  if (n_tokens < 1) return RAZOR_E_INVALID_ARG;
  if (n_tokens == 1) return decode_impl(c, layer, q, out, 1, 1, 0, stream);
  if (c->cfg.dtype != RAZOR_BF16) return RAZOR_E_UNSUPPORTED_DIM;
  for (const HeadState& h : c->layers[layer].hs) {
    if (h.len + h.n_drop < n_tokens) return RAZOR_E_INVALID_ARG;          // fewer tokens cached than queries
    if (h.n_drop > 0 && h.window < n_tokens) return RAZOR_E_INVALID_ARG;  // the mean would hold tokens after a query
  }
  const int group0 = c->cfg.n_q_heads / c->cfg.n_kv_heads;
  // A round of more query rows per KV head than one launch of the streaming kernel takes goes to the query-tiled
  // kernel, which streams the cache once per 128 rows (tensor cores).  (An ALiBi cache with sink tokens stays on the
  // path below.)
  // (From 9 rows, a second launch of the streaming kernel: 32K MHA, 256 heads, 12 rows: 0.31 against 0.44 ms; 128K
  // GQA, 16 heads, 16 rows: 113 against 128 us.)
  if ((long long)group0 * n_tokens >= c->round_tiled_min_rows && (!c->dv.alibi || c->cfg.n_sink == 0))
    return round_impl(c, layer, q, out, n_tokens, stream);
  // One launch takes a tile of 2, 4 or 8 rows per KV head (query heads of the group x query tokens).  A
  // longer round runs block by block, the largest block that fits; when the round is not a multiple of
  // the block, the last block is moved back to end with the round and recomputes a few tokens.
  const int group = c->cfg.n_q_heads / c->cfg.n_kv_heads;
  int block = 0;
  for (int rows = 8; rows >= 2 && !block; rows >>= 1)
    if (rows % group == 0 && rows / group <= n_tokens) block = rows / group;
  if (!block) return RAZOR_E_UNSUPPORTED_DIM;
  const size_t row_elems = (size_t)c->cfg.n_q_heads * c->cfg.head_dim;
  for (int start = 0;; start += block) {
    if (start + block > n_tokens) start = n_tokens - block;
    rc = decode_impl(c, layer, (const char*)q + (size_t)start * row_elems * esz(c->cfg), out + (size_t)start * row_elems,
                     block, n_tokens, n_tokens - start - block, stream);
    if (rc || start + block >= n_tokens) return rc;
  }
}

int razor_decode_attention(razor_cache_t* c, int32_t layer, const void* q, float* out, void* stream) {
  if (!c || !q || !out) return RAZOR_E_NULL_PTR;
  int rc = layer_ready(c, layer);
  if (rc) return rc;
  return decode_impl(c, layer, q, out, 1, 1, 0, stream);
}

static int decode_impl(razor_cache_t* c, int32_t layer, const void* q, float* out, int32_t n_tokens,
                       int32_t tok_stride, int32_t q_after, void* stream, const void* k_new, const void* v_new) {
  int rc;
  if (((uintptr_t)q | (uintptr_t)out) & 15) return RAZOR_E_MISALIGNED;
  rc = ensure_schedule(c, layer, (cudaStream_t)stream, true, (c->cfg.n_q_heads / c->cfg.n_kv_heads) * n_tokens);
  if (rc) return rc;
  const LayerHost& L = c->layers[layer];
  DecodeJobs jb{L.n_items, L.n_jobs, L.n_spans, L.jobs[L.n_spans], L.n_multi, n_tokens, tok_stride, q_after, 0, {},
                k_new, v_new};
  plan_early_prefetch(c, layer, jb);
  RZ_CUDA(launch_decode(c->dv, c->cfg.dtype, layer, jb, q, out, c->n_sms, c->tune,
                        (cudaStream_t)stream));
  c->last_writer_layer = -1;
  c->writes_since_decode.clear();
  c->writes_overflow = false;
  return RAZOR_OK;
}

int razor_decode_step(razor_cache_t* c, int32_t layer, const void* k_new, const void* v_new, const void* q, float* out,
                      void* stream) {
  if (!c || !k_new || !v_new || !q || !out) return RAZOR_E_NULL_PTR;
  int rc = layer_ready(c, layer);
  if (rc) return rc;
  if (((uintptr_t)k_new | (uintptr_t)v_new) & 15) return RAZOR_E_MISALIGNED;
  LayerHost& L = c->layers[layer];
  if (L.appended >= c->cfg.max_new_tokens) return RAZOR_E_CAPACITY;
  // A head with no recent window at all drops the new token at once (nothing is stored, only the sums change):
  // that corner stays with the two separate kernels.
  bool plain = false;
  for (const HeadState& h : L.hs) plain |= (h.window == 0);
  if (plain) {
    rc = razor_append(c, layer, k_new, v_new, stream);
    return rc ? rc : razor_decode_attention(c, layer, q, out, stream);
  }
  // The host mirror moves first (the schedule and the early copies are planned for the lengths the launch
  // will see) and moves back if the launch fails.
  const std::vector<HeadState> before = L.hs;
  const int n_sink = c->cfg.n_sink;
  for (HeadState& h : L.hs) {
    if (h.window < 0 || h.len < n_sink + h.window) {
      h.len += 1;
    } else {
      h.n_drop += 1;
      h.ring_head = (h.ring_head + 1 == h.window) ? 0 : h.ring_head + 1;
    }
  }
  L.appended += 1;
  L.growth_tokens += 1;
  rc = decode_impl(c, layer, q, out, 1, 1, 0, stream, k_new, v_new);
  if (rc) {
    L.hs = before;
    L.appended -= 1;
    L.growth_tokens -= 1;
    L.sched_valid = false;
    return rc;
  }
  c->note_write(layer, razor_cache::kWriteOneToken);   // the launch stores the new rows late: the next one must leave them alone
  return RAZOR_OK;
}

int razor_cache_export(razor_cache_t* c, int32_t layer, int32_t b, int32_t kv_head, int32_t* kept_pos, void* K,
                       void* V, float* comp_mean_k, float* comp_mean_v, float* comp_sum_k, float* comp_sum_v,
                       int32_t* n_kept, int32_t* n_drop, void* stream) {
  if (!c) return RAZOR_E_NULL_PTR;
  if (layer < 0 || layer >= c->cfg.n_layers || b < 0 || b >= c->cfg.batch || kv_head < 0 ||
      kv_head >= c->cfg.n_kv_heads)
    return RAZOR_E_INVALID_ARG;
  const LayerHost& L = c->layers[layer];
  if (!L.any || !L.seq_done[b]) return RAZOR_E_NOT_COMPRESSED;
  const int head = b * c->cfg.n_kv_heads + kv_head;
  if (n_kept) *n_kept = L.hs[head].len;
  if (n_drop) *n_drop = L.hs[head].n_drop;
  if (kept_pos || K || V || comp_mean_k || comp_mean_v || comp_sum_k || comp_sum_v) {
    if (((uintptr_t)K | (uintptr_t)V) & 15) return RAZOR_E_MISALIGNED;
    RZ_CUDA(launch_export(c->dv, c->cfg.dtype, layer, head, kept_pos, K, V, comp_mean_k, comp_mean_v, comp_sum_k,
                          comp_sum_v, (cudaStream_t)stream));
  }
  return RAZOR_OK;
}

int razor_cache_stats(const razor_cache_t* c, int32_t layer, size_t* kept_bytes, size_t* dense_bytes) {
  if (!c) return RAZOR_E_NULL_PTR;
  if (layer < 0 || layer >= c->cfg.n_layers) return RAZOR_E_INVALID_ARG;
  const LayerHost& L = c->layers[layer];
  if (!L.any) return RAZOR_E_NOT_COMPRESSED;
  size_t kept = 0, dense = 0;
  for (const HeadState& h : L.hs) {
    kept += (size_t)h.len;
    dense += (size_t)h.len + (size_t)h.n_drop;
  }
  const size_t per_token = 2 * row_bytes(c->cfg);
  if (kept_bytes) *kept_bytes = kept * per_token;
  if (dense_bytes) *dense_bytes = dense * per_token;
  return RAZOR_OK;
}

int razor_schedule_plan(const int32_t* tokens, int32_t n_heads, int32_t n_ctas, int32_t static_percent,
                        int32_t tail_items_per_cta, int32_t min_chunk_pages, int32_t* items, int32_t max_items,
                        int32_t* n_items, int32_t* n_spans) {
  if (!tokens || !n_items) return RAZOR_E_NULL_PTR;
  if (n_heads < 1 || n_ctas < 1 || static_percent < 0 || static_percent > 100 || tail_items_per_cta < 1 ||
      min_chunk_pages < 1)
    return RAZOR_E_INVALID_ARG;
  std::vector<int32_t> pages(n_heads);
  for (int h = 0; h < n_heads; ++h) {
    if (tokens[h] < 0) return RAZOR_E_INVALID_ARG;
    pages[h] = ceil_div(tokens[h], kPageTokens);
  }
  const int cap = n_heads + kItemBudget;
  std::vector<WorkItem> w(cap);
  std::vector<int32_t> jobs(cap + 1);
  std::vector<MultiHead> multi(n_heads);
  const SchedParams sp{n_ctas, static_percent, tail_items_per_cta, min_chunk_pages, kMergeInKernelMaxParts};
  SchedInfo info{};
  const int n = build_schedule(pages.data(), n_heads, sp, cap, w.data(), jobs.data(), multi.data(), &info);
  if (n < 0) return RAZOR_E_INVALID_ARG;
  if (n_spans) *n_spans = info.n_spans;
  return emit_items(w.data(), n, jobs.data(), info.n_jobs, items, max_items, n_items);
}

int razor_cache_set_option(razor_cache_t* c, int32_t option, int32_t value) {
  if (!c) return RAZOR_E_NULL_PTR;
  switch (option) {
    case RAZOR_OPT_DECODE_TAIL_ITEMS_PER_SM:
      if (value < 1 || value > 1024) return RAZOR_E_INVALID_ARG;
      c->tune.tail_items_per_sm = value;
      break;
    case RAZOR_OPT_DECODE_STATIC_PERCENT:
      if (value < 0 || value > 100) return RAZOR_E_INVALID_ARG;
      c->tune.static_pct = value;
      break;
    case RAZOR_OPT_DECODE_MIN_CHUNK_PAGES:
      if (value < 1 || value > (1 << 20)) return RAZOR_E_INVALID_ARG;
      c->tune.min_chunk_pages = value;
      break;
    case RAZOR_OPT_DECODE_RING_KB:
      if (value < 0 || value > 227) return RAZOR_E_INVALID_ARG;
      c->tune.ring_kb = value;
      break;
    case RAZOR_OPT_DECODE_CONSUMER_WARPS:
      if (value != 0 && value != 4 && value != 8 && value != 12 && value != 16) return RAZOR_E_INVALID_ARG;
      c->tune.consumer_warps = value;
      break;
    case RAZOR_OPT_DECODE_TENSOR_CORES:
      if (value < 0 || value > 2) return RAZOR_E_INVALID_ARG;
      c->tune.tensor_cores = value;
      break;
    case RAZOR_OPT_DECODE_EARLY_PREFETCH:
      if (value < 0 || value > 64) return RAZOR_E_INVALID_ARG;
      c->tune.early_prefetch = value;
      break;
    case RAZOR_OPT_ROUND_TILED_MIN_ROWS:
      if (value < 1) return RAZOR_E_INVALID_ARG;
      c->round_tiled_min_rows = value;
      break;
    default:
      return RAZOR_E_INVALID_ARG;
  }
  for (LayerHost& L : c->layers) L.sched_valid = false;   // the next decode re-plans
  return RAZOR_OK;
}

int razor_cache_device_status(razor_cache_t* c, int32_t* status, void* stream) {
  if (!c || !status) return RAZOR_E_NULL_PTR;
  int32_t host = 0;
  RZ_CUDA(cudaMemcpyAsync(&host, c->dv.status, sizeof(host), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  RZ_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  *status = host;
  if (host != 0) {
    // A kernel gave up part-way: its job queue may be left non-zero.  Put it back.
    RZ_CUDA(cudaMemsetAsync(c->dv.queue, 0, 8 * sizeof(int32_t), (cudaStream_t)stream));
    RZ_CUDA(cudaMemsetAsync(c->dv.tickets, 0, (size_t)c->dv.n_heads * sizeof(int32_t), (cudaStream_t)stream));
    RZ_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  }
  return RAZOR_OK;
}

int razor_cache_set_alibi(razor_cache_t* c, const float* slopes, void* stream) {
  if (!c) return RAZOR_E_NULL_PTR;
  if (!slopes) {
    c->dv.alibi = 0;
    return RAZOR_OK;
  }
  if (c->cfg.use_compensation) return RAZOR_E_INVALID_ARG;   // the compensation token has no position to penalise
  const size_t n = (size_t)c->cfg.n_layers * c->cfg.n_q_heads;
  std::vector<float> scaled(n);
  for (size_t i = 0; i < n; ++i) {
    if (!(slopes[i] >= 0.f) || std::isinf(slopes[i])) return RAZOR_E_INVALID_ARG;
    scaled[i] = slopes[i] * 1.4426950408889634f;   // the kernels work in the log2 domain
  }
  RZ_CUDA(cudaMemcpyAsync(c->dv.alibi_slopes, scaled.data(), n * sizeof(float), cudaMemcpyHostToDevice,
                          (cudaStream_t)stream));   // pageable source: staged before the call returns
  c->dv.alibi = 1;
  return RAZOR_OK;
}

int razor_cache_set_head_windows(razor_cache_t* c, int32_t layer, const int32_t* window_h) {
  if (!c) return RAZOR_E_NULL_PTR;
  if (layer < 0 || layer >= c->cfg.n_layers) return RAZOR_E_INVALID_ARG;
  LayerHost& L = c->layers[layer];
  if (!window_h) {
    L.head_window.clear();
    return RAZOR_OK;
  }
  for (int g = 0; g < c->cfg.n_kv_heads; ++g)
    if (window_h[g] < 0) return RAZOR_E_INVALID_ARG;
  L.head_window.assign(window_h, window_h + c->cfg.n_kv_heads);
  return RAZOR_OK;
}

int razor_cache_wait_selftest(razor_cache_t* c, int64_t limit_ns, void* stream) {
  if (!c) return RAZOR_E_NULL_PTR;
  if (limit_ns < 1000 || limit_ns > 1000000000ll) return RAZOR_E_INVALID_ARG;
  RZ_CUDA(launch_wait_selftest(c->dv, (unsigned long long)limit_ns, (cudaStream_t)stream));
  return RAZOR_OK;
}

int razor_schedule_query(razor_cache_t* c, int32_t layer, int32_t* items, int32_t max_items, int32_t* n_items) {
  if (!c || !n_items) return RAZOR_E_NULL_PTR;
  int rc = layer_ready(c, layer);
  if (rc) return rc;
  rc = ensure_schedule(c, layer, nullptr, false, c->cfg.n_q_heads / c->cfg.n_kv_heads);
  if (rc) return rc;
  const LayerHost& L = c->layers[layer];
  return emit_items(L.items, L.n_items, L.jobs, L.n_jobs, items, max_items, n_items);
}

int razor_schedule_combine_heads(razor_cache_t* c, int32_t layer, int32_t* heads, int32_t max_heads, int32_t* n_heads) {
  if (!c || !n_heads) return RAZOR_E_NULL_PTR;
  int rc = layer_ready(c, layer);
  if (rc) return rc;
  rc = ensure_schedule(c, layer, nullptr, false, c->cfg.n_q_heads / c->cfg.n_kv_heads);
  if (rc) return rc;
  const LayerHost& L = c->layers[layer];
  *n_heads = L.n_multi;
  if (!heads) return RAZOR_OK;
  if (max_heads < L.n_multi) return RAZOR_E_INVALID_ARG;
  for (int i = 0; i < L.n_multi; ++i) heads[i] = L.multi[i].head;
  return RAZOR_OK;
}

}  // extern "C"
