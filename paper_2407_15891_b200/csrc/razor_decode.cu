// Decode attention over the compressed cache (Eq. 5; Algorithm 1): split-K flash decoding as a
// persistent producer / consumer kernel, one CTA per SM.
//
// One launch covers every (sequence, KV head) of a layer, full-length retrieval heads and short heads
// alike.  The host lays the heads' page streams end to end and cuts them into one equal span per CTA
// plus a tail of small items; a CTA pulls its span, then tail items, from a queue.  Inside a CTA
//   * the PRODUCER warp pops items, publishes each item's descriptor, query rows and compensation
//     token in a small shared-memory slot, and streams the item's pages (one contiguous K|V block
//     each) into a shared-memory ring with bulk asynchronous copies that complete on mbarriers.  It
//     runs ahead across item boundaries, so the ring never drains;
//   * NC CONSUMER warps take the ring's pages round-robin; each keeps an online-softmax state
//     (m, l, o) per query head of the group in registers and hands it over at the end of the item;
//   * the REDUCER warp merges the NC states of an item into one state and writes it out: as the head's
//     output when the head is in one part, else as a partial record.
// Heads cut into several parts are finished by combine_kernel, a small dependent launch that merges
// their records (one CTA per head) as soon as the streaming kernel has drained.
//
// The compensation token of a non-retrieval head is folded into the online softmax as the initial
// state of the head's first part: m = s_c + log2(N_d), l = 1, o = v_hat, which is the term
// N_d * exp(s_c) * v_hat of Eq. 5 with the count moved onto the logit.
//
// Logits live in the log2 domain: q is pre-multiplied by sm_scale * log2(e) and exp is ex2.
//
// Every wait on an mbarrier is bounded in time.  A wait that runs out sets a CTA-wide abort flag and a
// bit of the device status word; the other warps see the flag in their own waits and leave, and the
// producer waits (again bounded) for its copies in flight before the CTA exits.
#include <math_constants.h>

#include <algorithm>

#include "razor_common.cuh"
#include "razor_sync.cuh"

namespace razor {

namespace {

constexpr int kItemSlots = 2;            // item descriptors in flight between producer and consumers
constexpr int kMaxMergeBufs = 2;         // consumer -> reducer hand-over buffers (one where they are large)
template <int G>
constexpr int merge_bufs() { return G >= 4 ? 1 : 2; }
constexpr int kMaxStages = 64;           // ring stages (pages in flight per CTA)
// Ring position -> (stage, use).  Position p is always consumed by warp p % NC, and a stage must always
// be consumed by the same warp: a warp then never waits on a barrier that is more than one phase behind
// it, which a parity wait could not tell from "done".  So the ring is NC interleaved sub-rings: warp w
// owns stages w, w + NC, w + 2 NC, ... below n_stages (the sub-rings differ in length by at most one
// when n_stages is not a multiple of NC) and walks them round-robin.
template <int NC>
__device__ __forceinline__ void ring_slot(unsigned pos, unsigned n_stages, unsigned& stage, unsigned& use) {
  const unsigned w = pos % NC, k = pos / NC;
  const unsigned cnt = (n_stages - w + NC - 1) / NC;   // stages of warp w's sub-ring (n_stages >= NC)
  stage = w + NC * (k % cnt);
  use = k / cnt;
}

// ------------------------------------------------------------------------------------------ shared layout
struct ItemDesc {
  int32_t head;        // < 0: no more items
  int32_t page_begin;
  int32_t n_pages;
  int32_t len;         // tokens the head holds (masks the tail of its last page)
  int32_t part_idx;
  int32_t n_parts;
  int32_t rec_base;
  int32_t ring_head;   // ring index of the oldest recent token (slot -> position, multi-token rounds)
  int32_t seed;        // 1: this part starts from the compensation token
  int32_t n_drop;
  int32_t window;      // recent-window length, < 0: the head keeps everything
  // a launch that also appends a token: the part that holds the page the new row goes to stores it
  int32_t tp_index;    // that page, counted from page_begin; -1: not in this part (or nothing is appended)
  int32_t tp_slot;     // slot of the new row
  int32_t tp_pid;      // pool page of that slot
  int32_t fold;        // 1: the slot holds the oldest recent token, which joins the dropped set first (Eq. 4)
  int32_t merge_here;  // 1: the part that is written last folds the head's records itself
};

template <typename T, int D, int G>
struct alignas(16) ItemSlot {
  ItemDesc desc;
  alignas(16) T q[G][D];
  alignas(16) float mean[2][D];   // k_hat, v_hat (a part that folds a row receives the sums here and turns them into means)
  alignas(16) T new_kv[2][D];     // the appended K and V row, for the part that stores it
  alignas(16) T old_kv[2][D];     // the row it evicts, as it lies in its page (16-byte chunks swizzled)
};

struct Barriers {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t item_full[kItemSlots];
  uint64_t item_empty[kItemSlots];
  uint64_t merge_full[kMaxMergeBufs];
  uint64_t merge_free[kMaxMergeBufs];
};

// Hand-over buffer: the descriptor of the item, then per consumer warp and query head (m, l) and o[D].
template <int D, int G, int NC>
struct alignas(16) MergeBuf {
  ItemDesc desc;
  float2 ml[NC][G];
  alignas(16) float o[NC][G][D];
};

// Dynamic shared memory: the hand-over buffers, then the page ring (1 KiB aligned).
template <typename T, int D, int G, int NC>
constexpr size_t decode_ring_offset() {
  return (sizeof(MergeBuf<D, G, NC>) * merge_bufs<G>() + 1023) & ~(size_t)1023;
}

template <int G, int EPL>
struct SoftmaxState {
  float m[G], l[G], o[G][EPL];
  __device__ __forceinline__ void clear() {
#pragma unroll
    for (int j = 0; j < G; ++j) {
      m[j] = -CUDART_INF_F;
      l[j] = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) o[j][e] = 0.f;
    }
  }
};

// Merge (m2, l2, o2) into (m, l, o); either side may be empty (m = -inf, l = 0).
template <int EPL>
__device__ __forceinline__ void merge_state(float& m, float& l, float (&o)[EPL], float m2, float l2,
                                            const float (&o2)[EPL]) {
  const float mm = fmaxf(m, m2);
  const float mu = (mm == -CUDART_INF_F) ? 0.f : mm;
  const float c1 = fast_exp2(m - mu), c2 = fast_exp2(m2 - mu);
  l = l * c1 + l2 * c2;
#pragma unroll
  for (int e = 0; e < EPL; ++e) o[e] = o[e] * c1 + o2[e] * c2;
  m = mm;
}

// What a consumer needs to apply causality inside a round of several query tokens, or the distance
// penalty of ALiBi heads (Eq. 1): the position of a slot's token and the position of each query row.
struct RoundMask {
  int n_tok, g_real;            // query tokens of the round; query heads per KV head
  int alibi;                    // 1: add the ALiBi distance penalty
  int total;                    // tokens the head has seen (len + n_drop)
  int q_after;                  // tokens of the round after this launch's block: query t sits at total - q_after - n_tok + t
  int n_sink, ring_head, window, n_drop;
  int slot0;                    // slot of the page's first token
  // position of the token in slot s (Algorithm 1 keeps sinks + a ring of the recent tokens)
  __device__ __forceinline__ int pos(int s) const {
    if (window < 0 || n_drop == 0 || s < n_sink) return s;
    int j = s - n_sink - ring_head;
    if (j < 0) j += window;
    return total - window + j;
  }
};

// One page (16 tokens) from shared memory into the running state of a consumer warp (CUDA cores).
// `page` is the page's first 16-byte chunk; this lane reads logical chunk lir of the rows i*RG + rg.
template <typename T, int D, int G>
__device__ __forceinline__ void consume_page(const uint4* page, int valid, int rg, int lir,
                                             const float (&qf)[G][Elem<T>::kEpl], SoftmaxState<G, Elem<T>::kEpl>& S,
                                             bool alibi, const RoundMask& mk, const float (&slope)[G]) {
  using Geo = RowGeom<T, D>;
  constexpr int LPR = Geo::kLpr, EPL = Geo::kEpl, RG = Geo::kRg, RPG = Geo::kRowsPerGroup;
  uint4 kf[RPG], vf[RPG];
#pragma unroll
  for (int i = 0; i < RPG; ++i) kf[i] = page[(i * RG + rg) * LPR + swz(i * RG + rg, lir)];
#pragma unroll
  for (int i = 0; i < RPG; ++i) vf[i] = page[(kPageTokens + i * RG + rg) * LPR + swz(i * RG + rg, lir)];

  float s[G][RPG];
#pragma unroll
  for (int i = 0; i < RPG; ++i) {
    float a[EPL];
    Elem<T>::unpack(kf[i], a);
#pragma unroll
    for (int j = 0; j < G; ++j) {
      float acc = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc += a[e] * qf[j][e];
      s[j][i] = acc;
    }
  }
#pragma unroll
  for (int j = 0; j < G; ++j)
#pragma unroll
    for (int i = 0; i < RPG; ++i) s[j][i] = row_sum<LPR>(s[j][i]);

  if (alibi) {   // Eq. 1: - l_h (m - n), slopes already in the log2 domain; one query token on this path
    const int q_pos = mk.total - 1;
#pragma unroll
    for (int i = 0; i < RPG; ++i) {
      const float dist = (float)(mk.pos(mk.slot0 + i * RG + rg) - q_pos);
#pragma unroll
      for (int j = 0; j < G; ++j) s[j][i] += slope[j] * dist;
    }
  }
  if (valid < kPageTokens) {   // rows of this page beyond the head's length
#pragma unroll
    for (int i = 0; i < RPG; ++i) {
      if (i * RG + rg >= valid) {
#pragma unroll
        for (int j = 0; j < G; ++j) s[j][i] = -CUDART_INF_F;
        vf[i] = make_uint4(0u, 0u, 0u, 0u);   // unused slots may hold anything, NaN patterns included
      }
    }
  }

#pragma unroll
  for (int j = 0; j < G; ++j) {
    float mx = s[j][0];
#pragma unroll
    for (int i = 1; i < RPG; ++i) mx = fmaxf(mx, s[j][i]);
    const float m_new = fmaxf(S.m[j], mx);
    const float m_use = (m_new == -CUDART_INF_F) ? 0.f : m_new;
    const float corr = fast_exp2(S.m[j] - m_use);
    float psum = 0.f;
#pragma unroll
    for (int i = 0; i < RPG; ++i) {
      s[j][i] = fast_exp2(s[j][i] - m_use);
      psum += s[j][i];
    }
    S.l[j] = S.l[j] * corr + psum;
    S.m[j] = m_new;
#pragma unroll
    for (int e = 0; e < EPL; ++e) S.o[j][e] *= corr;
  }
#pragma unroll
  for (int i = 0; i < RPG; ++i) {
    float v[EPL];
    Elem<T>::unpack(vf[i], v);
#pragma unroll
    for (int j = 0; j < G; ++j)
#pragma unroll
      for (int e = 0; e < EPL; ++e) S.o[j][e] += s[j][i] * v[e];
  }
}

// ------------------------------------------------------------------------------------------ tensor-core path
// Grouped-query heads (bf16, G >= 2): the query heads that share a KV head make a dense tile with the
// page's 16 tokens, so a page is consumed with warp-level matrix instructions (m16n8k16, bf16 in,
// fp32 accumulate):
//   S[token][head]  = K[token][:] . Q[head][:]       A = K rows as they lie, B = Q (heads >= G are zero)
//   O^T[d][head]   += V^T[d][token] * P[token][head]  A = V through a transposing load, B = P
// P goes from the accumulator layout of S to the B layout through an 8x8 register transpose, and is
// split into a bf16 head and a bf16 remainder (two products), so the weights keep fp32-like accuracy.
// Lane (g = lane / 4, t = lane % 4) owns query heads 2t, 2t+1: tokens g, g+8 of S and rows g, g+8 of
// every 16-row tile of O^T.
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
// Transpose of an 8x8 matrix of 16-bit elements held one row-pair per lane.
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
  return y;
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);   // .x = lo (low half), .y = hi
  return *(const uint32_t*)&v;
}

template <int D>
struct MmaState {
  static constexpr int kMT = D / 16;   // 16-row tiles of O^T along the head dimension
  float m[2], l[2];                     // heads 2t, 2t+1: running max (log2 domain), this lane's share of the denominator
  float o[kMT][4];                      // o[mt] = O^T[mt*16 + {g, g, g+8, g+8}][head {2t, 2t+1, 2t, 2t+1}]
  __device__ __forceinline__ void clear() {
    m[0] = m[1] = -CUDART_INF_F;
    l[0] = l[1] = 0.f;
#pragma unroll
    for (int i = 0; i < kMT; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  }
};

// qb[kk][0] = Q[head g][kk*16 + 2t, +1], qb[kk][1] = Q[head g][kk*16 + 8 + 2t, +1] (bf16 pairs; zero for g >= G).
template <int D>
__device__ __forceinline__ void consume_page_mma(uint32_t page_addr, int valid, int lane, float scale_log2,
                                                 const uint32_t (&qb)[D / 16][2], MmaState<D>& S, const RoundMask& mk,
                                                 float slope0, float slope1) {
  constexpr int ROW = D * 2;          // bytes per row
  constexpr int KS = D / 16;          // k-steps of the K.Q product
  constexpr int MT = D / 16;
  const int r = lane & 7, mi = lane >> 3, g = lane >> 2;

  // ---- S = K Q^T, two accumulation chains
  float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
  {
    // matrices of one load: (tokens 0-7, chunk 2kk), (tokens 8-15, 2kk), (tokens 0-7, 2kk+1), (tokens 8-15, 2kk+1)
    const uint32_t row_addr = page_addr + (((mi & 1) << 3) + r) * ROW;
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
      uint32_t a[4];
      ldmatrix_x4(a, row_addr + (((2 * kk + (mi >> 1)) ^ r) << 4));
      if (kk & 1) mma_bf16(s1, a, qb[kk][0], qb[kk][1]);
      else mma_bf16(s0, a, qb[kk][0], qb[kk][1]);
    }
  }
  // s[0], s[1]: token g, heads 2t, 2t+1;  s[2], s[3]: token g+8
  float s[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) s[i] = (s0[i] + s1[i]) * scale_log2;
  if (valid < kPageTokens) {   // tokens of this page beyond the head's length
    if (g >= valid) s[0] = s[1] = -CUDART_INF_F;
    if (g + 8 >= valid) s[2] = s[3] = -CUDART_INF_F;
  }
  if (mk.n_tok > 1 || mk.alibi || mk.q_after > 0) {
    const int t2 = (lane & 3) * 2, q_first = mk.total - mk.q_after - mk.n_tok;
    const int qp0 = q_first + t2 / mk.g_real, qp1 = q_first + (t2 + 1) / mk.g_real;
    const int p0 = mk.pos(mk.slot0 + g), p1 = mk.pos(mk.slot0 + g + 8);
    if (mk.alibi) {            // Eq. 1: - l_h (m - n); slope0/1 belong to this lane's two rows, log2 domain
      s[0] += slope0 * (float)(p0 - qp0);
      s[1] += slope1 * (float)(p0 - qp1);
      s[2] += slope0 * (float)(p1 - qp0);
      s[3] += slope1 * (float)(p1 - qp1);
    }
    // causality inside the round: a query does not see the tokens after it
    if (p0 > qp0) s[0] = -CUDART_INF_F;
    if (p0 > qp1) s[1] = -CUDART_INF_F;
    if (p1 > qp0) s[2] = -CUDART_INF_F;
    if (p1 > qp1) s[3] = -CUDART_INF_F;
  }
  // ---- online softmax of heads 2t, 2t+1 (the eight lanes with the same t share them)
  float mx0 = fmaxf(s[0], s[2]), mx1 = fmaxf(s[1], s[3]);
#pragma unroll
  for (int off = 4; off < 32; off <<= 1) {
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
  }
  const float mn0 = fmaxf(S.m[0], mx0), mn1 = fmaxf(S.m[1], mx1);
  const float mu0 = (mn0 == -CUDART_INF_F) ? 0.f : mn0, mu1 = (mn1 == -CUDART_INF_F) ? 0.f : mn1;
  const float corr0 = fast_exp2(S.m[0] - mu0), corr1 = fast_exp2(S.m[1] - mu1);
  const float p0 = fast_exp2(s[0] - mu0), p1 = fast_exp2(s[1] - mu1);
  const float p2 = fast_exp2(s[2] - mu0), p3 = fast_exp2(s[3] - mu1);
  S.l[0] = S.l[0] * corr0 + (p0 + p2);
  S.l[1] = S.l[1] * corr1 + (p1 + p3);
  S.m[0] = mn0;
  S.m[1] = mn1;
#pragma unroll
  for (int i = 0; i < MT; ++i) {
    S.o[i][0] *= corr0;
    S.o[i][1] *= corr1;
    S.o[i][2] *= corr0;
    S.o[i][3] *= corr1;
  }
  // P as a bf16 head plus a bf16 remainder, transposed into the B layout:
  // b0 = P[tokens 2t, 2t+1][head g], b1 = P[tokens 8+2t, 9+2t][head g]
  const float h0 = __bfloat162float(__float2bfloat16_rn(p0)), h1 = __bfloat162float(__float2bfloat16_rn(p1));
  const float h2 = __bfloat162float(__float2bfloat16_rn(p2)), h3 = __bfloat162float(__float2bfloat16_rn(p3));
  const uint32_t bh0 = movmatrix_trans(pack_bf16(h0, h1)), bh1 = movmatrix_trans(pack_bf16(h2, h3));
  const uint32_t bl0 = movmatrix_trans(pack_bf16(p0 - h0, p1 - h1)), bl1 = movmatrix_trans(pack_bf16(p2 - h2, p3 - h3));
  // ---- O^T += V^T P
  {
    // matrices of one load: (tokens 0-7, chunk 2mt), (tokens 0-7, 2mt+1), (tokens 8-15, 2mt), (tokens 8-15, 2mt+1)
    const uint32_t row_addr = page_addr + (kPageTokens + ((mi >> 1) << 3) + r) * ROW;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      uint32_t a[4];
      ldmatrix_x4_trans(a, row_addr + (((2 * mt + (mi & 1)) ^ r) << 4));
      mma_bf16(S.o[mt], a, bh0, bh1);
      mma_bf16(S.o[mt], a, bl0, bl1);
    }
  }
}

// The part of a launch-that-appends which evicts a row: sums so far (in mean[]) + the evicted row -> new sums
// and means (Eq. 4 over every token dropped so far), stored for later launches and left in mean[] for the
// seed below.  Same arithmetic, in the same order, as the append kernel's.  One warp, D / 32 elements per lane.
template <typename T, int D>
__device__ __forceinline__ void fold_evicted_row(float (&mean)[2][D], const T (&old_kv)[2][D], int slot, int n_drop,
                                                 float* __restrict__ g_sum, float* __restrict__ g_mean, int lane) {
  constexpr int PER = D / 32, EPC = 16 / (int)sizeof(T);   // elements per lane; elements per 16-byte chunk
  const float cnt = (float)n_drop;
#pragma unroll
  for (int kv = 0; kv < 2; ++kv) {
#pragma unroll
    for (int i = 0; i < PER; ++i) {
      const int e = lane * PER + i;
      const int pos = (((e / EPC) ^ (slot & 7)) * EPC) + e % EPC;   // where the page's swizzle put element e
      const float s = mean[kv][e] + (float)old_kv[kv][pos];
      const float m = __fdiv_rn(s, cnt);
      g_sum[kv * D + e] = s;
      g_mean[kv * D + e] = m;
      mean[kv][e] = m;
    }
  }
  __syncwarp();
}

// The appended row into the page that holds its slot: into the copy in shared memory (this launch attends to
// it) and into the pool (for the launches to come).  Lane c < LPR holds 16-byte chunk c of the K and V row.
template <int LPR>
__device__ __forceinline__ void store_new_row(uint8_t* page, uint8_t* pool_page, int slot, const uint4& k, const uint4& v,
                                              int lane) {
  if (lane < LPR) {
    const int t = slot & 15, at = t * LPR + swz(slot, lane);
    ((uint4*)page)[at] = k;
    ((uint4*)page)[kPageTokens * LPR + at] = v;
    ((uint4*)pool_page)[at] = k;
    ((uint4*)pool_page)[kPageTokens * LPR + at] = v;
  }
  __syncwarp();
}

// ------------------------------------------------------------------------------------------ the kernel
template <typename T, int D, int G, int NC, bool MMA>
__global__ void __launch_bounds__((NC + 2) * 32, 1)
decode_kernel(DeviceView dv, int layer, DecodeJobs jb, const T* __restrict__ q, float* __restrict__ out, int n_stages) {
  static_assert(!MMA || sizeof(T) == 2, "the tensor-core path is for bf16 heads");
  using Geo = RowGeom<T, D>;
  constexpr int LPR = Geo::kLpr, EPL = Geo::kEpl;
  constexpr uint32_t PB = Geo::kPageBytes;
  using Slot = ItemSlot<T, D, G>;
  using MBuf = MergeBuf<D, G, NC>;
  constexpr int kMergeBufs = merge_bufs<G>();

  extern __shared__ __align__(1024) uint8_t dyn_smem[];
  __shared__ Barriers bars;
  __shared__ Slot slots[kItemSlots];
  __shared__ int abort_flag_s;
  volatile int* abort_flag = &abort_flag_s;

  MBuf* mbufs = (MBuf*)dyn_smem;
  uint8_t* ring = dyn_smem + decode_ring_offset<T, D, G, NC>();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < n_stages; ++s) {
      mbar_init(&bars.full[s], 1);
      mbar_init(&bars.empty[s], 1);
    }
    for (int s = 0; s < kItemSlots; ++s) {
      mbar_init(&bars.item_full[s], 1);
      mbar_init(&bars.item_empty[s], NC);
    }
    for (int s = 0; s < kMergeBufs; ++s) {
      mbar_init(&bars.merge_full[s], NC);
      mbar_init(&bars.merge_free[s], 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  const bool fused = jb.k_new != nullptr;   // this launch also appends a token
  const WorkItem* items = dv.items + (size_t)layer * dv.max_items;
  const int32_t* jobs = dv.jobs + (size_t)layer * (dv.max_items + 1);
  const int n_items = jb.n_items;
  const WorkItem no_item = {0, 0, 0, 0, 1, 0, 0, 0};   // (merge_here = 0)
  auto row_of = [&](const WorkItem& w) { return (size_t)layer * dv.n_heads + w.head; };
  auto first_pids = [&](const WorkItem& w) {
    return dv.page_table[row_of(w) * dv.max_pages + min(w.page_begin + lane, dv.max_pages - 1)];
  };
  // A job is a run of consecutive items: a span (looked up in jobs[]) or a single tail item (tail
  // jobs follow the spans and map to consecutive items, so they need no lookup).
  auto job_range = [&](int j, int& first, int& end) {
    if (j >= jb.n_jobs) {
      first = end = n_items;
    } else if (j >= jb.n_spans) {
      first = jb.tail_first + (j - jb.n_spans);
      end = first + 1;
    } else {
      first = jobs[j];
      end = jobs[j + 1];
    }
  };
  // The spans are handed out by CTA index and the queue counts tail jobs only, so the producer can look
  // up its span, the span's first item and that item's first page ids right here: the schedule is written
  // by host copies only and the page table by host copies or the compression's plan kernel, which lies
  // whole kernels back in the stream, so both may be read before the dependency below is resolved.  The head
  // state of the first item too, when the host says that nothing in flight writes this layer's states.
  int it0 = n_items, job_end0 = n_items;
  WorkItem w0 = no_item;
  int32_t pid0 = 0;
  HeadState st0 = {0, 0, 0, 0};
  const bool has_span = (int)blockIdx.x < jb.n_spans;
  const bool state_early = has_span && jb.state_stable != 0;   // the head states of this layer are at rest
  if (warp == NC && has_span) {
    job_range((int)blockIdx.x, it0, job_end0);
    w0 = it0 < n_items ? items[it0] : no_item;
    pid0 = first_pids(w0);
    if (state_early) st0 = dv.state[row_of(w0)];
  }
  __syncthreads();
  // The first pages of the span go into the (still empty) ring right away: the host has named a run of
  // leading pages of the span's first item that exist and that no kernel still in flight writes (an append
  // before this launch touches one known page per head).  Positions below the ring length use every stage at
  // most once, so nothing has to be waited for.  The pages' descriptor, which needs the head's state as the
  // append leaves it, follows after the dependency wait; the consumers then find these pages already landed.
  unsigned early_done = 0;
  if (warp == NC && has_span && blockIdx.x < kEarlyCtas) {
    const int n_early = min((int)jb.early[blockIdx.x], n_stages);   // the host has applied its own cap already
    const int32_t* pt0 = dv.page_table + row_of(w0) * dv.max_pages + w0.page_begin;
    for (int p = lane; p < n_early; p += 32) {
      unsigned stage, use;
      ring_slot<NC>((unsigned)p, (unsigned)n_stages, stage, use);
      mbar_arrive_expect_tx(&bars.full[stage], PB);
      bulk_load(ring + (size_t)stage * PB, dv.pool + (size_t)pt0[p] * dv.page_bytes, PB, &bars.full[stage]);
    }
    early_done = (unsigned)n_early;
    if (n_early > 0) pid0 = pt0[min(n_early + lane, dv.max_pages - 1 - w0.page_begin)];   // ids of the round that follows
  }
  // This kernel is launched as a programmatic dependent of whatever precedes it on the stream (the
  // append or an earlier combine), so everything above overlaps that kernel's tail; nothing a kernel
  // still in flight writes is touched before this point.
  cudaGridDependencySynchronize();
  // The combine kernel that follows may be made resident as soon as SMs free up; it waits for this whole
  // grid to finish before it reads anything this grid writes.
  cudaTriggerProgrammaticLaunchCompletion();

  // Row r of a KV head's tile is query token r / g_real, query head r % g_real of the group (one token
  // per sequence: g_real = G).  Offset, in elements, of that row in q and in out ([B, n_tok, Hq, D]).
  const int g_real = G / jb.n_tok;
  auto row_offset = [&](int head, int r) {
    const int b = head / dv.n_kv_heads, g = head % dv.n_kv_heads;
    return (((size_t)b * jb.tok_stride + r / g_real) * ((size_t)dv.n_kv_heads * g_real) + (size_t)g * g_real + r % g_real) * D;
  };
  // Warp-uniform bounded wait: false for every lane if any lane's wait failed.
  auto warp_wait = [&](uint64_t* bar, uint32_t parity) -> bool {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
  };

  if (warp == NC) {
    // ======================================================================== producer
    const unsigned ns = (unsigned)n_stages;
    // positions issued per round: never more than one lap of the shortest sub-ring, so that no lane of
    // a round waits for a stage that another lane of the same round is about to fill
    const int batch = min(32, NC * (n_stages / NC));
    unsigned c = early_done;                             // ring positions issued so far by this CTA (exact)
    unsigned seq_issued = 0;                             // item slots whose copies were issued
    int marker_slot = -1;                                // slot that received the end marker
    bool ok = true;
    // Look-ahead of one item: the next item's queue pop, its descriptor, its head state and its first
    // page ids are requested while the current item's pages are being issued, so that the ring is not
    // left to drain over a chain of dependent global loads at every item boundary.
    int it = it0, job_end = job_end0;
    WorkItem w = w0;
    int32_t pid_first = pid0;
    if (!has_span) {   // more CTAs than spans: start on the tail
      int j = 0;
      if (lane == 0) j = atomicAdd(dv.queue, 1);
      job_range(jb.n_spans + __shfl_sync(0xffffffffu, j, 0), it, job_end);
      w = it < n_items ? items[it] : no_item;
      pid_first = first_pids(w);
    }
    // The query rows of the first item do not depend on the head's state: their copy is issued now, next to the
    // load of that state, instead of behind it.
    constexpr uint32_t kQBytes = G * D * sizeof(T);
    bool q_issued = false;
    if (lane == 0 && it < n_items) {
      mbar_expect_tx(&bars.item_full[0], kQBytes);
      for (int t = 0; t < jb.n_tok; ++t)
        bulk_load(&slots[0].q[t * g_real][0], q + row_offset(w.head, t * g_real), kQBytes / jb.n_tok, &bars.item_full[0]);
      q_issued = true;
    }
    HeadState st = state_early ? st0 : dv.state[row_of(w)];
    for (unsigned seq = 0; ok; ++seq) {
      const int slot = seq % kItemSlots;
      const bool need_pop = it < n_items && it + 1 >= job_end;   // the job ends with this item
      int next_raw = jb.n_jobs;
      if (lane == 0 && need_pop) next_raw = atomicAdd(dv.queue, 1);   // result is picked up below
      if (seq >= kItemSlots) ok = warp_wait(&bars.item_empty[slot], ((seq / kItemSlots) - 1) & 1);
      if (!ok) break;
      Slot& sl = slots[slot];
      if (it >= n_items) {
        if (lane == 0) {
          sl.desc.head = -1;
          mbar_arrive(&bars.item_full[slot]);
        }
        marker_slot = slot;
        break;
      }
      const size_t hs = row_of(w);
      // A launch that appends: `st` becomes the state the append leaves (the stored state stays as it was until
      // the last CTA of the launch advances every head), tp_slot the slot the new row goes to.
      int tp_slot = -1;
      bool evicts = false;
      if (fused) {
        if (st.window < 0 || st.len < dv.n_sink + st.window) {
          tp_slot = st.len;
          st.len += 1;
        } else if (st.window > 0) {
          tp_slot = dv.n_sink + st.ring_head;
          evicts = true;
          st.n_drop += 1;
          st.ring_head = (st.ring_head + 1 == st.window) ? 0 : st.ring_head + 1;
        }   // (a head with sinks only and no window is not run through this path: the host sees to that)
      }
      const int head_pages = (st.len + kPageTokens - 1) / kPageTokens;
      const int page_end = w.page_end < 0 ? head_pages : min(w.page_end, head_pages);
      const int n = max(0, page_end - w.page_begin);
      const int tp_rel = tp_slot >= 0 ? (tp_slot >> 4) - w.page_begin : -1;
      const bool owns = tp_rel >= 0 && tp_rel < n;   // this part holds the page the new row goes to
      const int p_first = seq == 0 ? (int)early_done : 0;   // pages of this item already on their way
      if (p_first > n) {   // the host's count and the device's lengths disagree: stop rather than mix items up
        if (lane == 0) {
          atomicOr(dv.status, kStatusEarlyMismatch);
          if (q_issued) mbar_arrive(&bars.item_full[slot]);   // lets the exit path wait for the query copy in flight
        }
        if (__shfl_sync(0xffffffffu, (int)q_issued, 0)) seq_issued = seq + 1;
        *abort_flag = 1;
        ok = false;
        break;
      }
      // The compensation token enters the head's first part; in a launch that evicts a row into the sums it
      // enters the part that holds that row instead, which computes the new mean itself.
      const bool fold = evicts && owns;
      const bool seed = dv.use_comp && st.n_drop > 0 && st.window >= 0 && (evicts ? owns : w.part_idx == 0);
      if (lane == 0) {
        ItemDesc d;
        d.head = w.head; d.page_begin = w.page_begin; d.n_pages = n; d.len = st.len;
        d.part_idx = w.part_idx; d.n_parts = w.n_parts; d.rec_base = w.rec_base; d.ring_head = st.ring_head;
        d.seed = seed ? 1 : 0; d.n_drop = st.n_drop; d.window = st.window; d.merge_here = w.merge_here;
        d.tp_index = owns ? tp_rel : -1; d.tp_slot = tp_slot; d.fold = fold ? 1 : 0;
        d.tp_pid = owns ? dv.page_table[hs * dv.max_pages + (tp_slot >> 4)] : 0;
        sl.desc = d;
        constexpr uint32_t q_bytes = kQBytes, mean_bytes = 2 * D * sizeof(float), row_bytes = D * sizeof(T);
        const bool q_now = !(seq == 0 && q_issued);   // the first item's query rows are on their way already
        mbar_arrive_expect_tx(&bars.item_full[slot], (q_now ? q_bytes : 0u) + ((seed || fold) ? mean_bytes : 0u) +
                                                         (owns ? 2 * row_bytes : 0u) + (fold ? 2 * row_bytes : 0u));
        if (q_now)
          for (int t = 0; t < jb.n_tok; ++t)   // the g_real rows of one query token are contiguous
            bulk_load(&sl.q[t * g_real][0], q + row_offset(w.head, t * g_real), q_bytes / jb.n_tok, &bars.item_full[slot]);
        if (fold) {   // the sums so far and the row that leaves the window
          const uint8_t* old_row = dv.pool + (size_t)d.tp_pid * dv.page_bytes + (size_t)(tp_slot & 15) * row_bytes;
          bulk_load(&sl.mean[0][0], dv.comp_sum + hs * 2 * D, mean_bytes, &bars.item_full[slot]);
          bulk_load(&sl.old_kv[0][0], old_row, row_bytes, &bars.item_full[slot]);
          bulk_load(&sl.old_kv[1][0], old_row + kPageTokens * row_bytes, row_bytes, &bars.item_full[slot]);
        } else if (seed) {
          bulk_load(&sl.mean[0][0], dv.comp_mean + hs * 2 * D, mean_bytes, &bars.item_full[slot]);
        }
        if (owns) {
          bulk_load(&sl.new_kv[0][0], (const T*)jb.k_new + (size_t)w.head * D, row_bytes, &bars.item_full[slot]);
          bulk_load(&sl.new_kv[1][0], (const T*)jb.v_new + (size_t)w.head * D, row_bytes, &bars.item_full[slot]);
        }
      }
      seq_issued = seq + 1;
      const int32_t* pt = dv.page_table + hs * dv.max_pages + w.page_begin;
      // Page i of an item always goes to consumer warp i % NC (so a part's result does not depend on
      // which CTA streamed it or on what that CTA streamed before): the item starts on a ring position
      // that is a multiple of NC, and the positions left over in its last round are passed on empty.
      const int n_pad = (n + NC - 1) / NC * NC;
      int it_next = it + 1, end_next = job_end;   // the next item of this job, unless the job ends here
      WorkItem w_next = no_item;
      bool have_next = false;
      int32_t pid_cur = pid_first;
      for (int p0 = p_first; p0 < n_pad; p0 += batch) {
        const int in_batch = min(batch, n_pad - p0);
        const bool mine = lane < in_batch;
        const bool real = mine && p0 + lane < n;
        const int32_t pid_after = (p0 + batch + lane < n) ? pt[p0 + batch + lane] : 0;   // ids of the next round
        unsigned stage = 0, use_cur = 0;
        bool ready = true;
        if (mine) {
          // Each lane waits for its own stage and issues at once, inside the same divergent region: a freed
          // stage is refilled whatever the other stages of the round are doing.
          ring_slot<NC>(c + lane, ns, stage, use_cur);
          if (use_cur > 0) ready = mbar_wait(&bars.empty[stage], (use_cur - 1) & 1, abort_flag);
          if (ready) {
            if (real) {
              mbar_arrive_expect_tx(&bars.full[stage], PB);
              bulk_load(ring + (size_t)stage * PB, dv.pool + (size_t)pid_cur * dv.page_bytes, PB, &bars.full[stage]);
            } else {
              mbar_arrive(&bars.full[stage]);
            }
          }
        }
        ok = __all_sync(0xffffffffu, ready);
        if (!ok) {
          // Some lane gave up, so `c` no longer says exactly which positions were issued: the lanes that
          // did issue a copy in this round wait (bounded) for it here, before the common exit path.
          if (ready && real && !mbar_wait_drain(&bars.full[stage], use_cur & 1)) atomicOr(dv.status, kStatusDrainTimeout);
          break;
        }
        c += in_batch;
        pid_cur = pid_after;
        if (!have_next) {   // the pop issued above has had a round of copies to come back
          if (need_pop) job_range(jb.n_spans + __shfl_sync(0xffffffffu, next_raw, 0), it_next, end_next);
          w_next = it_next < n_items ? items[it_next] : no_item;
          have_next = true;
        }
      }
      if (!ok) break;
      if (!have_next) {
        if (need_pop) job_range(jb.n_spans + __shfl_sync(0xffffffffu, next_raw, 0), it_next, end_next);
        w_next = it_next < n_items ? items[it_next] : no_item;
      }
      it = it_next;
      job_end = end_next;
      w = w_next;
      st = dv.state[row_of(w)];
      pid_first = first_pids(w);
    }
    if (!ok && lane == 0) atomicOr(dv.status, kStatusProducerTimeout);
    // Wait (bounded) until every copy this warp issued has landed: the CTA's shared memory must not be
    // released under a copy in flight.  In a healthy run the consumers have waited for all of them already.
    bool drained = true;
    for (unsigned s = lane; s < ns; s += 32) {
      const unsigned w = s % NC, j = s / NC, cnt = (ns - w + NC - 1) / NC;
      const unsigned kw = c > w ? (c - w + NC - 1) / NC : 0;   // positions issued so far on warp w's sub-ring
      if (kw > j) {
        const unsigned k_last = j + cnt * ((kw - 1 - j) / cnt);   // latest of them that used stage s
        if (!mbar_wait_drain(&bars.full[s], (k_last / cnt) & 1)) drained = false;
      }
    }
    // (The slot that took the end marker was first waited free, so its earlier copies have landed; its
    // barrier has since moved on a phase and must not be asked about the earlier one.)
    if (lane < kItemSlots && (unsigned)lane < seq_issued && lane != marker_slot) {
      const unsigned last = lane + kItemSlots * ((seq_issued - 1 - lane) / kItemSlots);
      if (!mbar_wait_drain(&bars.item_full[lane], (last / kItemSlots) & 1)) drained = false;
    }
    if (!__all_sync(0xffffffffu, drained) && lane == 0) atomicOr(dv.status, kStatusDrainTimeout);
    // Queue reset for the next launch: every CTA has made its last pop before it counts itself done.
    // In a launch that appends, the stored head states must stay as they were while any CTA still builds
    // descriptors from them; the CTA that counts itself done last knows that nobody does any more and advances
    // every head by the append.
    int done = 0;
    if (lane == 0) {
      __threadfence();
      done = atomicAdd(dv.queue + 1, 1);
    }
    done = __shfl_sync(0xffffffffu, done, 0);
    if (done == (int)gridDim.x - 1) {
      if (lane == 0) {
        dv.queue[0] = 0;
        dv.queue[1] = 0;
      }
      if (fused) {
        HeadState* states = dv.state + (size_t)layer * dv.n_heads;
        for (int h = lane; h < dv.n_heads; h += 32) {
          HeadState s = states[h];
          if (s.window < 0 || s.len < dv.n_sink + s.window) {
            s.len += 1;
          } else if (s.window > 0) {
            s.n_drop += 1;
            s.ring_head = (s.ring_head + 1 == s.window) ? 0 : s.ring_head + 1;
          }
          states[h] = s;
          dv.ring_valid[(size_t)layer * dv.n_heads + h] = 0;   // the window's content changed and its sum was not kept up
        }
      }
    }
  } else if (warp < NC) {
    // ======================================================================== consumers
    const unsigned ns = (unsigned)n_stages;
    const int lir = lane % LPR, rg = lane / LPR;
    unsigned c = 0;   // ring positions of all items so far (the same count in every consumer warp)
    bool ok = true;
    for (unsigned seq = 0;; ++seq) {
      const int slot = seq % kItemSlots;
      const int mb = seq % kMergeBufs;
      MBuf& M = mbufs[mb];
      if (!warp_wait(&bars.item_full[slot], (seq / kItemSlots) & 1)) { ok = false; break; }
      Slot& sl = slots[slot];
      const ItemDesc d = sl.desc;
      if (d.head < 0) {
        // pass the end marker on to the reducer
        if (seq >= kMergeBufs && !warp_wait(&bars.merge_free[mb], ((seq / kMergeBufs) - 1) & 1)) { ok = false; break; }
        if (warp == 0 && lane == 0) M.desc.head = -1;
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars.merge_full[mb]);
        break;
      }
      if constexpr (MMA) {
        // ---------------------------------------------------------------- tensor-core consumer
        const int g = lane >> 2, t = lane & 3;
        uint32_t qa[D / 16][2];   // B fragments of Q: head g
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          qa[kk][0] = qa[kk][1] = 0u;
          if (g < G) {
            const uint32_t* qrow = (const uint32_t*)&sl.q[g][0];
            qa[kk][0] = qrow[kk * 8 + t];
            qa[kk][1] = qrow[kk * 8 + 4 + t];
          }
        }
        float slope0 = 0.f, slope1 = 0.f;   // ALiBi slopes of this lane's rows 2t, 2t+1 (query head = row % g_real)
        if (dv.alibi) {
          const float* sl_h = dv.alibi_slopes + (size_t)layer * dv.n_kv_heads * g_real + (size_t)(d.head % dv.n_kv_heads) * g_real;
          slope0 = sl_h[(2 * t) % g_real];
          slope1 = sl_h[(2 * t + 1) % g_real];
        }
        MmaState<D> S;
        S.clear();
        const bool first = warp == 0;
        // a launch that appends: the warp that will meet the new row's page takes the row out of the slot now
        // (the slot is handed back below), and the first warp folds the evicted row into the sums
        uint4 new_k = make_uint4(0u, 0u, 0u, 0u), new_v = new_k;
        if (d.tp_index >= 0 && warp == d.tp_index % NC && lane < LPR) {
          new_k = ((const uint4*)&sl.new_kv[0][0])[lane];
          new_v = ((const uint4*)&sl.new_kv[1][0])[lane];
        }
        if (d.fold && first) {
          const size_t hs2 = ((size_t)layer * dv.n_heads + d.head) * 2 * D;
          fold_evicted_row<T, D>(sl.mean, sl.old_kv, d.tp_slot, d.n_drop, dv.comp_sum + hs2, dv.comp_mean + hs2, lane);
        }
        // Compensation token (Eq. 4, Eq. 5) seeds the first part of a head that dropped tokens.
        if (d.seed && first) {
          constexpr int PER = D / 32;
          const float log_cnt = log2f((float)d.n_drop);
#pragma unroll
          for (int j = 0; j < G; ++j) {
            float sc = 0.f;
#pragma unroll
            for (int e = 0; e < PER; ++e)
              sc += __bfloat162float(sl.q[j][lane * PER + e]) * sl.mean[0][lane * PER + e];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) sc += __shfl_xor_sync(0xffffffffu, sc, off);
            if (t == (j >> 1)) {   // head j lives in slot j & 1 of the lanes with t = j / 2
              S.m[j & 1] = sc * dv.scale_log2 + log_cnt;
              S.l[j & 1] = (g == 0) ? 1.f : 0.f;
#pragma unroll
              for (int mt = 0; mt < D / 16; ++mt) {
                S.o[mt][j & 1] = sl.mean[1][mt * 16 + g];
                S.o[mt][2 + (j & 1)] = sl.mean[1][mt * 16 + 8 + g];
              }
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars.item_empty[slot]);   // this warp holds all it needs from the slot

        const int n_pad = (d.n_pages + NC - 1) / NC * NC;
        for (int i = warp; i < n_pad; i += NC) {
          unsigned stage, use;
          ring_slot<NC>(c + i, ns, stage, use);
          if (!warp_wait(&bars.full[stage], use & 1)) { ok = false; break; }
          if (i < d.n_pages) {
            uint8_t* page = ring + (size_t)stage * PB;
            if (i == d.tp_index)
              store_new_row<LPR>(page, dv.pool + (size_t)d.tp_pid * dv.page_bytes, d.tp_slot, new_k, new_v, lane);
            const int valid = d.len - (d.page_begin + i) * kPageTokens;
            if (valid < kPageTokens) {
              // V rows beyond the head's length may hold anything; a zero weight times a NaN is a NaN
              uint4* vrows = (uint4*)page + (kPageTokens + max(valid, 0)) * LPR;
              for (int idx = lane; idx < (kPageTokens - max(valid, 0)) * LPR; idx += 32)
                vrows[idx] = make_uint4(0u, 0u, 0u, 0u);
              __syncwarp();
            }
            const RoundMask mk{jb.n_tok, g_real, dv.alibi, d.len + d.n_drop, jb.q_after, dv.n_sink, d.ring_head, d.window,
                               d.n_drop, (d.page_begin + i) * kPageTokens};
            consume_page_mma<D>(smem_u32(page), valid, lane, dv.scale_log2, qa, S, mk, slope0, slope1);
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars.empty[stage]);
        }
        if (!ok) break;
        c += n_pad;

#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
          S.l[0] += __shfl_xor_sync(0xffffffffu, S.l[0], off);
          S.l[1] += __shfl_xor_sync(0xffffffffu, S.l[1], off);
        }
        // Hand the state over to the reducer.
        if (seq >= kMergeBufs && !warp_wait(&bars.merge_free[mb], ((seq / kMergeBufs) - 1) & 1)) { ok = false; break; }
        if (first && lane == 0) M.desc = d;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int h = 2 * t + e;
          if (h < G) {
            if (g == 0) M.ml[warp][h] = make_float2(S.m[e], S.l[e]);
#pragma unroll
            for (int mt = 0; mt < D / 16; ++mt) {
              M.o[warp][h][mt * 16 + g] = S.o[mt][e];
              M.o[warp][h][mt * 16 + 8 + g] = S.o[mt][2 + e];
            }
          }
        }
      } else {
        // ---------------------------------------------------------------- CUDA-core consumer
        float qf[G][EPL];
#pragma unroll
        for (int j = 0; j < G; ++j) {
          const uint4 u = ((const uint4*)&sl.q[j][0])[lir];
          Elem<T>::unpack(u, qf[j]);
#pragma unroll
          for (int e = 0; e < EPL; ++e) qf[j][e] *= dv.scale_log2;
        }
        float slope[G];   // ALiBi slopes of the group's query heads (log2 domain); zero when ALiBi is off
#pragma unroll
        for (int j = 0; j < G; ++j)
          slope[j] = dv.alibi ? dv.alibi_slopes[(size_t)layer * dv.n_kv_heads * G + (size_t)(d.head % dv.n_kv_heads) * G + j] : 0.f;
        SoftmaxState<G, EPL> S;
        S.clear();
        const bool first = warp == 0;   // the warp that takes the item's first page also takes its seed
        // a launch that appends: the warp that will meet the new row's page takes the row out of the slot now
        // (the slot is handed back below), and the first warp folds the evicted row into the sums
        uint4 new_k = make_uint4(0u, 0u, 0u, 0u), new_v = new_k;
        if (d.tp_index >= 0 && warp == d.tp_index % NC && lane < LPR) {
          new_k = ((const uint4*)&sl.new_kv[0][0])[lane];
          new_v = ((const uint4*)&sl.new_kv[1][0])[lane];
        }
        if (d.fold && first) {
          const size_t hs2 = ((size_t)layer * dv.n_heads + d.head) * 2 * D;
          fold_evicted_row<T, D>(sl.mean, sl.old_kv, d.tp_slot, d.n_drop, dv.comp_sum + hs2, dv.comp_mean + hs2, lane);
        }
        // Compensation token (Eq. 4, Eq. 5) seeds the first part of a head that dropped tokens.
        if (d.seed && first) {
          float kh[EPL], vh[EPL];
#pragma unroll
          for (int e = 0; e < EPL; ++e) { kh[e] = sl.mean[0][lir * EPL + e]; vh[e] = sl.mean[1][lir * EPL + e]; }
          const float log_cnt = log2f((float)d.n_drop);
#pragma unroll
          for (int j = 0; j < G; ++j) {
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) s += qf[j][e] * kh[e];
            s = row_sum<LPR>(s);
            if (rg == 0) {
              S.m[j] = s + log_cnt;
              S.l[j] = 1.f;
#pragma unroll
              for (int e = 0; e < EPL; ++e) S.o[j][e] = vh[e];
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars.item_empty[slot]);   // this warp holds all it needs from the slot

        const int n_pad = (d.n_pages + NC - 1) / NC * NC;
        for (int i = warp; i < n_pad; i += NC) {
          unsigned stage, use;
          ring_slot<NC>(c + i, ns, stage, use);
          if (!warp_wait(&bars.full[stage], use & 1)) { ok = false; break; }
          if (i < d.n_pages) {
            if (i == d.tp_index)
              store_new_row<LPR>(ring + (size_t)stage * PB, dv.pool + (size_t)d.tp_pid * dv.page_bytes, d.tp_slot, new_k,
                                 new_v, lane);
            const RoundMask mk{1, G, dv.alibi, d.len + d.n_drop, 0, dv.n_sink, d.ring_head, d.window, d.n_drop,
                               (d.page_begin + i) * kPageTokens};
            consume_page<T, D, G>((const uint4*)(ring + (size_t)stage * PB), d.len - (d.page_begin + i) * kPageTokens,
                                  rg, lir, qf, S, dv.alibi != 0, mk, slope);
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars.empty[stage]);
        }
        if (!ok) break;
        c += n_pad;

        // Row groups of the warp hold disjoint token subsets: merge them.
#pragma unroll
        for (int off = LPR; off < 32; off <<= 1) {
#pragma unroll
          for (int j = 0; j < G; ++j) {
            const float m2 = __shfl_xor_sync(0xffffffffu, S.m[j], off);
            const float l2 = __shfl_xor_sync(0xffffffffu, S.l[j], off);
            float o2[EPL];
#pragma unroll
            for (int e = 0; e < EPL; ++e) o2[e] = __shfl_xor_sync(0xffffffffu, S.o[j][e], off);
            merge_state<EPL>(S.m[j], S.l[j], S.o[j], m2, l2, o2);
          }
        }
        // Hand the state over to the reducer.
        if (seq >= kMergeBufs && !warp_wait(&bars.merge_free[mb], ((seq / kMergeBufs) - 1) & 1)) { ok = false; break; }
        if (first && lane == 0) M.desc = d;
        if (rg == 0) {
#pragma unroll
          for (int j = 0; j < G; ++j) {
            if (lir == 0) M.ml[warp][j] = make_float2(S.m[j], S.l[j]);
#pragma unroll
            for (int e = 0; e < EPL; e += 4)
              *(float4*)&M.o[warp][j][lir * EPL + e] = make_float4(S.o[j][e], S.o[j][e + 1], S.o[j][e + 2], S.o[j][e + 3]);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars.merge_full[mb]);
    }
    if (!ok && lane == 0) atomicOr(dv.status, kStatusConsumerTimeout);
  } else {
    // ======================================================================== reducer
    bool ok = true;
    for (unsigned seq = 0;; ++seq) {
      const int mb = seq % kMergeBufs;
      if (!warp_wait(&bars.merge_full[mb], (seq / kMergeBufs) & 1)) { ok = false; break; }
      const MBuf& M = mbufs[mb];
      const ItemDesc d = M.desc;
      if (d.head < 0) break;
      // NC warp states -> one state per query head of the group
      float m_tot[G], l_tot[G];
      LaneVec<D> acc[G];
#pragma unroll
      for (int j = 0; j < G; ++j) {
        float mx = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < NC; ++w) mx = fmaxf(mx, M.ml[w][j].x);
        const float mu = (mx == -CUDART_INF_F) ? 0.f : mx;
        float l = 0.f;
        acc[j].zero();
#pragma unroll
        for (int w = 0; w < NC; ++w) {
          const float2 ml = M.ml[w][j];
          const float cw = fast_exp2(ml.x - mu);
          l += ml.y * cw;
          LaneVec<D> o;
          o.load_shared(&M.o[w][j][0], lane);
          acc[j].fma(cw, o);
        }
        m_tot[j] = mx;
        l_tot[j] = l;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars.merge_free[mb]);

      if (d.n_parts == 1) {   // the head's only part: this is its output
#pragma unroll
        for (int j = 0; j < G; ++j) {
          acc[j].scale(l_tot[j] > 0.f ? 1.f / l_tot[j] : 0.f);
          acc[j].store(out + row_offset(d.head, j), lane);
        }
      } else {                // one of several parts: its record
#pragma unroll
        for (int j = 0; j < G; ++j) {
          const size_t r = (size_t)(d.rec_base + d.part_idx) * G + j;
          if (lane == 0) dv.rec_ml[r] = make_float2(m_tot[j], l_tot[j]);
          acc[j].store(dv.rec_o + r * D, lane);
        }
        if (d.merge_here) {
          // A head in few parts is finished here, by whichever part is written last: every part publishes its
          // record (fence), then takes a ticket; the holder of the last ticket sees all records and folds them
          // in part order, so the result does not depend on who that is.  Nobody waits for anybody.
          __threadfence();
          __syncwarp();
          int ticket = 0;
          if (lane == 0) ticket = atomicAdd(dv.tickets + d.head, 1);
          ticket = __shfl_sync(0xffffffffu, ticket, 0);
          if (ticket == d.n_parts - 1) {
            if (lane == 0) dv.tickets[d.head] = 0;   // at rest again for the next launch
            __threadfence();
#pragma unroll
            for (int j = 0; j < G; ++j) {
              float2 ml[kMergeInKernelMaxParts];
              LaneVec<D> rows[kMergeInKernelMaxParts];
#pragma unroll
              for (int p = 0; p < kMergeInKernelMaxParts; ++p) {
                const size_t r = (size_t)(d.rec_base + min(p, d.n_parts - 1)) * G + j;   // beyond the end: re-read, unused
                ml[p] = __ldcg(&dv.rec_ml[r]);
                rows[p].load_l2(dv.rec_o + r * D, lane);
              }
              float mx = -CUDART_INF_F;
#pragma unroll
              for (int p = 0; p < kMergeInKernelMaxParts; ++p)
                if (p < d.n_parts) mx = fmaxf(mx, ml[p].x);
              const float mu = (mx == -CUDART_INF_F) ? 0.f : mx;
              float lt = 0.f;
              LaneVec<D> sum;
              sum.zero();
#pragma unroll
              for (int p = 0; p < kMergeInKernelMaxParts; ++p) {
                if (p < d.n_parts) {
                  const float cw = fast_exp2(ml[p].x - mu);
                  lt += ml[p].y * cw;
                  sum.fma(cw, rows[p]);
                }
              }
              sum.scale(lt > 0.f ? 1.f / lt : 0.f);
              sum.store(out + row_offset(d.head, j), lane);
            }
          }
        }
      }
    }
    if (!ok && lane == 0) atomicOr(dv.status, kStatusReducerTimeout);
  }
}

// ------------------------------------------------------------------------------------------ combine
// Merges the partial records of the heads that were cut into several parts (Eq. 5 regrouped: sums of
// exponentials under a common maximum).  One CTA per (such head, query row of its tile); warp w folds
// records w, w + 16, ... in that order and the warp states are folded in warp order, so the result
// does not depend on timing.  Launched as a programmatic dependent of the streaming kernel: its CTAs become
// resident as that kernel's CTAs leave and wait for all of its writes at cudaGridDependencySynchronize().
// (CTAs small enough to sit beside a streaming CTA were tried - four warps, 2 KB of shared memory, the same
// shared-memory split requested: they still only started as streaming CTAs left, and took three times as long.)
constexpr int kCombineWarps = 16;

template <int D>
__global__ void __launch_bounds__(kCombineWarps * 32) combine_kernel(DeviceView dv, int layer, int n_tok,
                                                                     int tok_stride, float* __restrict__ out) {
  __shared__ float2 s_ml[kCombineWarps];
  __shared__ __align__(16) float s_o[kCombineWarps][D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = dv.group * n_tok, j = blockIdx.y;   // rows per KV head: query tokens x query heads of the group
  const MultiHead mh = dv.multi[(size_t)layer * dv.n_heads + blockIdx.x];   // uploaded before either kernel
  cudaTriggerProgrammaticLaunchCompletion();   // whatever is queued behind this kernel may set itself up
  cudaGridDependencySynchronize();   // the streaming kernel's records are complete and visible from here on
  float m = -CUDART_INF_F, l = 0.f;
  LaneVec<D> acc;
  acc.zero();
  constexpr int U = 8;   // records in flight per warp
  for (int r0 = warp; r0 < mh.n_parts; r0 += kCombineWarps * U) {
    float2 ml[U];
    LaneVec<D> rows[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int r = min(r0 + u * kCombineWarps, mh.n_parts - 1);   // beyond the end: re-read the last one, unused
      const size_t idx = (size_t)(mh.rec_base + r) * G + j;
      ml[u] = __ldcg(&dv.rec_ml[idx]);
      rows[u].load_l2(dv.rec_o + idx * D, lane);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (r0 + u * kCombineWarps < mh.n_parts) {
        const float mn = fmaxf(m, ml[u].x);
        const float mu = (mn == -CUDART_INF_F) ? 0.f : mn;
        const float c_old = fast_exp2(m - mu), c_new = fast_exp2(ml[u].x - mu);
        l = l * c_old + ml[u].y * c_new;
        acc.scale(c_old);
        acc.fma(c_new, rows[u]);
        m = mn;
      }
    }
  }
  if (lane == 0) s_ml[warp] = make_float2(m, l);
  acc.store(&s_o[warp][0], lane);
  __syncthreads();
  if (warp == 0) {
    float mx = -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < kCombineWarps; ++w) mx = fmaxf(mx, s_ml[w].x);
    const float mu = (mx == -CUDART_INF_F) ? 0.f : mx;
    float lt = 0.f;
    LaneVec<D> sum;
    sum.zero();
#pragma unroll
    for (int w = 0; w < kCombineWarps; ++w) {
      const float cw = fast_exp2(s_ml[w].x - mu);
      lt += s_ml[w].y * cw;
      LaneVec<D> o;
      o.load_shared(&s_o[w][0], lane);
      sum.fma(cw, o);
    }
    sum.scale(lt > 0.f ? 1.f / lt : 0.f);
    const int b = mh.head / dv.n_kv_heads, g = mh.head % dv.n_kv_heads, gr = dv.group;
    sum.store(out + (((size_t)b * tok_stride + j / gr) * ((size_t)dv.n_kv_heads * gr) + (size_t)g * gr + j % gr) * D, lane);
  }
}

template <int D>
cudaError_t combine_launch(const DeviceView& dv, int layer, int n_multi, int n_tok, int tok_stride, float* out,
                           cudaStream_t s) {
  if (n_multi <= 0) return cudaSuccess;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_multi, dv.group * n_tok);
  cfg.blockDim = dim3(kCombineWarps * 32);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, combine_kernel<D>, dv, layer, n_tok, tok_stride, out);
}

// ------------------------------------------------------------------------------------------ launch
constexpr int kSmemOptIn = 232448;   // 227 KiB: the most one CTA may hold on sm_100

template <typename T, int D, int G, int NC, bool MMA>
cudaError_t decode_launch(const DeviceView& dv, int layer, const DecodeJobs& jb, const void* q, float* out, int n_sms,
                          const DecodeTuning& tune, cudaStream_t s) {
  auto kern = decode_kernel<T, D, G, NC, MMA>;
  constexpr size_t PB = RowGeom<T, D>::kPageBytes;
  constexpr size_t ring_off = decode_ring_offset<T, D, G, NC>();
  static int static_smem = -1;        // per instantiation
  static bool opted_in[64] = {};
  cudaError_t e;
  if (static_smem < 0) {
    cudaFuncAttributes fa;
    if ((e = cudaFuncGetAttributes(&fa, kern)) != cudaSuccess) return e;
    static_smem = (int)fa.sharedSizeBytes;
  }
  const long long avail = (long long)kSmemOptIn - static_smem - (long long)ring_off;
  long long stages = avail / (long long)PB;
  if (tune.ring_kb > 0) stages = std::min<long long>(stages, (long long)tune.ring_kb * 1024 / (long long)PB);
  stages = std::min<long long>(stages, kMaxStages);
  if (stages < NC) return cudaErrorInvalidConfiguration;   // every consumer warp owns at least one stage
  const size_t dyn = ring_off + (size_t)stages * PB;
  int dev = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !opted_in[dev]) {
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)(kSmemOptIn - static_smem))) != cudaSuccess)
      return e;
    if (dev >= 0 && dev < 64) opted_in[dev] = true;
  }
  int grid = std::min(n_sms, (int)jb.n_jobs);
  if (grid < 1) grid = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3((NC + 2) * 32);
  cfg.dynamicSmemBytes = dyn;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if ((e = cudaLaunchKernelEx(&cfg, kern, dv, layer, jb, (const T*)q, out, (int)stages)) != cudaSuccess) return e;
  return combine_launch<D>(dv, layer, jb.n_multi, jb.n_tok, jb.tok_stride, out, s);
}

template <typename T, int D, int G>
cudaError_t decode_nc(const DeviceView& dv, int layer, const DecodeJobs& jb, const void* q, float* out, int n_sms,
                      const DecodeTuning& tune, cudaStream_t s) {
  // Consumer warps.  The ring holds a multiple of NC pages and (NC + 2) warps share the register file,
  // so the choice trades pages in flight against registers per thread.
  const int nc = tune.consumer_warps;
  if constexpr (sizeof(T) == 2 && G >= 2) {
    // Grouped heads: the tensor-core consumer unless switched off (default on from group 4 up).
    // (rounds of several query tokens always take it: only that consumer applies their causal mask)
    const bool mma = jb.n_tok > 1 || jb.q_after > 0 || tune.tensor_cores == 1 || (tune.tensor_cores == 0 && G >= 4);
    if (mma) {
      if (nc == 4) return decode_launch<T, D, G, 4, true>(dv, layer, jb, q, out, n_sms, tune, s);
      return decode_launch<T, D, G, 8, true>(dv, layer, jb, q, out, n_sms, tune, s);
    }
  }
  if constexpr (sizeof(T) == 2 && G == 1) {
    if (tune.tensor_cores == 1) return decode_launch<T, D, G, 8, true>(dv, layer, jb, q, out, n_sms, tune, s);
    if (nc == 8) return decode_launch<T, D, G, 8, false>(dv, layer, jb, q, out, n_sms, tune, s);
    if (nc == 16) return decode_launch<T, D, G, 16, false>(dv, layer, jb, q, out, n_sms, tune, s);
    return decode_launch<T, D, G, 12, false>(dv, layer, jb, q, out, n_sms, tune, s);
  } else if constexpr (sizeof(T) == 2) {
    return decode_launch<T, D, G, 8, false>(dv, layer, jb, q, out, n_sms, tune, s);
  } else {
    return decode_launch<T, D, G, 4, false>(dv, layer, jb, q, out, n_sms, tune, s);
  }
}

template <typename T, int D>
cudaError_t decode_g(const DeviceView& dv, int layer, const DecodeJobs& jb, const void* q, float* out, int n_sms,
                     const DecodeTuning& tune, cudaStream_t s) {
  switch (dv.group * jb.n_tok) {   // rows of a KV head's tile
    case 1: return decode_nc<T, D, 1>(dv, layer, jb, q, out, n_sms, tune, s);
    case 2: return decode_nc<T, D, 2>(dv, layer, jb, q, out, n_sms, tune, s);
    case 4: return decode_nc<T, D, 4>(dv, layer, jb, q, out, n_sms, tune, s);
    case 8: return decode_nc<T, D, 8>(dv, layer, jb, q, out, n_sms, tune, s);
  }
  return cudaErrorInvalidValue;
}

// One warp waits, with the decode kernel's own bounded wait, on a barrier that nothing will ever arrive
// on.  The wait must give up after limit_ns, raise the abort flag and report through the status word:
// a check that the safety net under every wait of the decode kernel works, without hanging anything.
__global__ void wait_selftest_kernel(DeviceView dv, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag_s;
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool ok = mbar_wait(&bar, 0, &abort_flag_s, limit_ns);
  if (!ok && threadIdx.x == 0) atomicOr(dv.status, kStatusSelfTest);
}

}  // namespace

cudaError_t launch_wait_selftest(const DeviceView& dv, unsigned long long limit_ns, cudaStream_t s) {
  wait_selftest_kernel<<<1, 32, 0, s>>>(dv, limit_ns);
  return cudaGetLastError();
}

cudaError_t launch_decode(const DeviceView& dv, int dtype, int layer, const DecodeJobs& jb, const void* q, float* out,
                          int n_sms, const DecodeTuning& tune, cudaStream_t s) {
  if (dtype == RAZOR_BF16) {
    return dv.head_dim == 128 ? decode_g<__nv_bfloat16, 128>(dv, layer, jb, q, out, n_sms, tune, s)
                              : decode_g<__nv_bfloat16, 64>(dv, layer, jb, q, out, n_sms, tune, s);
  }
  return dv.head_dim == 128 ? decode_g<float, 128>(dv, layer, jb, q, out, n_sms, tune, s)
                            : decode_g<float, 64>(dv, layer, jb, q, out, n_sms, tune, s);
}

}  // namespace razor
