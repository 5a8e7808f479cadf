// Attention of a long round of new tokens (a follow-up prompt, a prefill chunk) over the compressed cache:
// the rows of a KV head's queries (query tokens x query heads of the group) are tiled 128 at a time, so
// the cache is streamed once per 128 query rows and the work is a real dense contraction.  It runs on the
// 5th-generation tensor cores: S = Q K^T with both operands in shared memory, O = P V with P read out of
// tensor memory and V out of shared memory, accumulators in tensor memory.  Same arithmetic as the decode kernel
// otherwise: causal mask inside the round (Section 3.1), compensation token with its count as the initial
// softmax state of a head's first part (Eq. 5), split over the tokens with partial records merged afterwards;
// for ALiBi caches (Section 3.1) a second instantiation adds Eq. 1's distance penalty to every score.
//
// A work item is (KV head, tile of 128 query rows, a run of 128-token blocks of the head's slot stream); a CTA
// takes it in steps of 64 tokens.  Persistent CTAs pull items from a queue (longest first), TWO CTAs to an SM:
// each has half of the tensor memory (256 columns) and less than half of the shared memory, and because the
// two run independently, one's softmax (transcendental unit, ALU) overlaps the other's waits and matrix
// products - inside one CTA the phases of a step follow each other.  Roles in a CTA of six warps:
//   * warp 0: TMA copies of K and V, one 16-token page at a time.  A page of the pool is [16 K rows][16 V rows]
//     with the 16-byte chunks of a row XOR-swizzled by the token index; a tensor map over the pool with a box of
//     (64 elements, 16 tokens) lands each half row at a 128-byte pitch, which is exactly the 128-byte-swizzled
//     operand layout of the matrix unit: K as a K-major operand of S = Q K^T, V as an MN-major operand of
//     O = P V.  Two stages of 64 tokens each for K and for V;
//   * warp 1, one thread: issues the matrix instructions and commits them onto the barriers;
//   * warps 2-5: softmax, a thread per query row (tensor-memory lane).  It reads its 64 scores of S, masks, keeps
//     a reference max and the sum, and writes P - a bf16 head plus a bf16 remainder per weight - into tensor
//     memory in the layout the matrix unit reads operand A in.  Scale, subtraction, sums and remainders work on
//     two scores per instruction (f32x2).  O accumulates in tensor memory over the item's steps; the reference
//     max may lag the true one by a factor of 2^8, and only when a row outruns it is the accumulator rescaled.
// Tensor memory of a CTA (256 columns): S in [0, 64), P in [64, 128) (heads, then remainders), O in [128, 256).
// (Tried and dropped: P through shared memory - the matrix unit's own operand reads, the TMA writes and the
// softmax stores then share the shared-memory port; one CTA per SM with 128-token steps, first with a thread per
// row, then with eight softmax warps and four threads per row - its warps move through the phases of a step
// together; exponentials partly as a polynomial on the FMA pipe.)
// Every wait is bounded in time; a wait that runs out sets the CTA's abort flag and a bit of the device status
// word, copies and instructions in flight are waited for, tensor memory is released.
#include <math_constants.h>

#include <algorithm>

#include "razor_common.cuh"
#include "razor_sync.cuh"
#include "razor_tc.cuh"

namespace razor {
namespace {

constexpr int kRows = kRoundTileRows;      // query rows per tile = accumulator rows = tensor-memory lanes
constexpr int kBlk = kRoundBlockTokens;    // tokens per block of a work item
constexpr int kStep = 64;                  // tokens per step = columns of S
constexpr int kStepsPerBlock = kBlk / kStep;
constexpr int kKvStages = 2;
constexpr int kRoundThreads = 6 * 32;
constexpr int kSoftmaxThreads = 128;
constexpr int kCtasPerSm = 2;
constexpr int kQHalfBytes = kRows * 128;   // one 64-element half of the 128-row query tile
constexpr int kKvHalfBytes = kStep * 128;  // one 64-element half of a 64-token K or V stage

struct RoundCtl {
  uint64_t q_ready;               // softmax threads -> MMA: the query tile is in shared memory
  uint64_t k_full[kKvStages];     // TMA -> MMA: the stage holds 64 tokens of K
  uint64_t k_empty[kKvStages];    // MMA (commit of S = Q K^T) -> TMA
  uint64_t v_full[kKvStages];     // the same for V; a V stage is free once O += P V has run
  uint64_t v_empty[kKvStages];
  uint64_t s_full;                // MMA (commit) -> softmax: S holds a step's scores
  uint64_t s_empty;               // softmax -> MMA: S read out into registers
  uint64_t p_full;                // softmax -> MMA: P of the step is in tensor memory
  uint64_t p_empty;               // MMA (commit) -> softmax: the product that read P has run
  uint64_t o_read;                // softmax -> MMA: the item's output accumulator has been read out of tensor memory
  uint64_t item_ready;            // producer -> everyone: the next item index is in `item`
  uint64_t item_taken;            // MMA warp + softmax threads -> producer: `item` has been read
  uint64_t blk_sync;              // the softmax threads among themselves, once per masked step (a bounded wait, unlike bar.sync)
  uint64_t drain;
  uint32_t tmem_base;
  int abort_flag;
  int item;                       // index of the current work item, -1: no more
  int32_t col_pos[2][kStep];      // token position of each column of a masked step (two may be in progress)
};

template <int D>
constexpr size_t round_smem_bytes() {
  // 1 KB alignment slack, Q tile, K and V stages, control block
  return 1024 + (size_t)kRows * D * 2 + (size_t)kKvStages * 2 * kStep * D * 2 + sizeof(RoundCtl);
}

// One page half: 16 tokens x 64 elements of K or V of pool page `pid` into shared memory (2 KB).
template <int D>
__device__ __forceinline__ void tma_load_page_half(void* dst, const CUtensorMap* map, int half, int kv, int pid,
                                                   uint64_t* bar) {
  if constexpr (D == 128) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];" ::
            "r"(smem_u32(dst)),
        "l"(map), "r"(0), "r"(0), "r"(half), "r"(kv), "r"(pid), "r"(smem_u32(bar))
        : "memory");
  } else {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::
            "r"(smem_u32(dst)),
        "l"(map), "r"(0), "r"(0), "r"(kv), "r"(pid), "r"(smem_u32(bar))
        : "memory");
  }
}

__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *(const uint32_t*)&v;
}

// 32 consecutive columns of this thread's lane into tensor memory; complete after tmem_st_wait_all().
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      :
      : "r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
        "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
        "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait_all() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Position of the token in slot s of a head (Algorithm 1 keeps the sinks and a ring of the recent tokens).
__device__ __forceinline__ int slot_pos(int s, int n_sink, int ring_head, int window, int n_drop, int total) {
  if (window < 0 || n_drop == 0 || s < n_sink) return s;
  int j = s - n_sink - ring_head;
  if (j < 0) j += window;
  return total - window + j;
}

template <int D, bool kAlibi>
__global__ void __launch_bounds__(kRoundThreads, kCtasPerSm)
    round_kernel(DeviceView dv, const __grid_constant__ CUtensorMap map_pool, int layer, RoundJobs jb,
                 const __nv_bfloat16* __restrict__ q, float* __restrict__ out) {
  constexpr int HALVES = D / 64;
  constexpr int Q_BYTES = kRows * D * 2, KV_TILE = kStep * D * 2;
  constexpr uint32_t kIdescQK = instr_desc_bf16(kRows, kStep, false);
  constexpr uint32_t kIdescPV = instr_desc_bf16(kRows, D, true);
  // tensor memory: S in columns [0, 64), P in [64, 128) - a row's 64 weights as 32 columns of bf16 pairs (the
  // heads) and 32 more (the remainders) -, the output accumulator in [128, 128 + D)
  constexpr uint32_t kTmemCols = 256;
  constexpr uint32_t kPCol = kStep, kPLo = kStep / 2, kOCol = 2 * kStep;

  extern __shared__ uint8_t round_smem_raw[];
  uint8_t* base = round_smem_raw + ((1024u - (smem_u32(round_smem_raw) & 1023u)) & 1023u);
  uint8_t* q_tile = base;
  uint8_t* k_tile = q_tile + Q_BYTES;                    // [stage][half][64 tokens][128 B]
  uint8_t* v_tile = k_tile + kKvStages * KV_TILE;
  RoundCtl* ctl = (RoundCtl*)(v_tile + kKvStages * KV_TILE);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &ctl->abort_flag;
  const RoundItem* items = dv.round_items;

  if (threadIdx.x == 0) {
    mbar_init(&ctl->q_ready, kSoftmaxThreads);
    for (int s = 0; s < kKvStages; ++s) {
      mbar_init(&ctl->k_full[s], 1);
      mbar_init(&ctl->k_empty[s], 1);
      mbar_init(&ctl->v_full[s], 1);
      mbar_init(&ctl->v_empty[s], 1);
    }
    mbar_init(&ctl->s_full, 1);
    mbar_init(&ctl->s_empty, kSoftmaxThreads);
    mbar_init(&ctl->p_full, kSoftmaxThreads);
    mbar_init(&ctl->p_empty, 1);
    mbar_init(&ctl->o_read, kSoftmaxThreads);
    mbar_init(&ctl->item_ready, 1);
    mbar_init(&ctl->item_taken, kSoftmaxThreads + 1);
    mbar_init(&ctl->blk_sync, kSoftmaxThreads);
    mbar_init(&ctl->drain, 1);
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // the MMA warp owns the tensor-memory allocation (half of the SM's: the other CTA has the rest)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  const int G = dv.group;               // query heads per KV head
  const int tok_per_tile = kRows / G;   // query tokens of a tile
  // Steps of a work item: its blocks in halves, without the steps that lie wholly beyond the head's length.
  auto first_step = [](const RoundItem& w) { return w.blk_begin * kStepsPerBlock; };
  auto end_step = [](const RoundItem& w, int len) {
    return max(w.blk_begin * kStepsPerBlock, min(w.blk_end * kStepsPerBlock, (len + kStep - 1) / kStep));
  };

  if (warp == 0) {
    // ================================================================ producer: work items and TMA copies
    unsigned gb = 0;       // steps issued so far by this CTA
    unsigned issued_k = 0, issued_v = 0;
    for (unsigned gi = 0;; ++gi) {
      int it = 0;
      if (lane == 0) it = atomicAdd(dv.queue + 2, 1);
      it = __shfl_sync(0xffffffffu, it, 0);
      if (it >= jb.n_items) it = -1;
      // publish the item
      if (gi > 0 && !__all_sync(0xffffffffu, mbar_wait(&ctl->item_taken, (gi - 1) & 1, abort_flag))) break;
      if (lane == 0) {
        ctl->item = it;
        mbar_arrive(&ctl->item_ready);
      }
      if (it < 0) break;
      const RoundItem w = items[it];
      const size_t hs = (size_t)layer * dv.n_heads + w.head;
      const HeadState st = dv.state[hs];
      const int head_pages = (st.len + kPageTokens - 1) / kPageTokens;
      const int32_t* pt = dv.page_table + hs * dv.max_pages;
      bool ok = true;
      // lane p < 4 handles page p of a step (past the head's end: a page of it again - finite data, masked);
      // the ids of the next step are fetched while this one is being issued
      constexpr int kStepPages = kStep / kPageTokens;
      auto page_of = [&](int step) { return lane < kStepPages ? pt[min(step * kStepPages + lane, max(head_pages - 1, 0))] : 0; };
      const int s_begin = first_step(w), s_end = end_step(w, st.len);
      int pid = s_begin < s_end ? page_of(s_begin) : 0;
      for (int step = s_begin; step < s_end && ok; ++step, ++gb) {
        const int s = gb % kKvStages;
        const unsigned use = gb / kKvStages;   // how often the stage has been filled before
        const int pid_next = step + 1 < s_end ? page_of(step + 1) : 0;
        // K of the step: its stage is free as soon as the scores of two steps ago have been computed
        if (gb >= kKvStages) ok = __all_sync(0xffffffffu, mbar_wait(&ctl->k_empty[s], (use - 1) & 1, abort_flag));
        if (!ok) break;
        if (lane == 0) mbar_arrive_expect_tx(&ctl->k_full[s], (uint32_t)KV_TILE);
        __syncwarp();
        if (lane < kStepPages) {
#pragma unroll
          for (int h = 0; h < HALVES; ++h)
            tma_load_page_half<D>(k_tile + s * KV_TILE + h * kKvHalfBytes + lane * 2048, &map_pool, h, 0, pid, &ctl->k_full[s]);
        }
        issued_k = gb + 1;
        // V of the step: its stage is free once the product of two steps ago has run
        if (gb >= kKvStages) ok = __all_sync(0xffffffffu, mbar_wait(&ctl->v_empty[s], (use - 1) & 1, abort_flag));
        if (!ok) break;
        if (lane == 0) mbar_arrive_expect_tx(&ctl->v_full[s], (uint32_t)KV_TILE);
        __syncwarp();
        if (lane < kStepPages) {
#pragma unroll
          for (int h = 0; h < HALVES; ++h)
            tma_load_page_half<D>(v_tile + s * KV_TILE + h * kKvHalfBytes + lane * 2048, &map_pool, h, 1, pid, &ctl->v_full[s]);
        }
        issued_v = gb + 1;
        pid = pid_next;
      }
      if (!ok) break;
    }
    if (*abort_flag) {   // copies in flight must land before the CTA may exit
      if (lane == 0) {
        atomicOr(dv.status, kStatusProducerTimeout);
        for (unsigned g = issued_k > kKvStages ? issued_k - kKvStages : 0; g < issued_k; ++g)
          if (!mbar_wait_drain(&ctl->k_full[g % kKvStages], (g / kKvStages) & 1)) atomicOr(dv.status, kStatusDrainTimeout);
        for (unsigned g = issued_v > kKvStages ? issued_v - kKvStages : 0; g < issued_v; ++g)
          if (!mbar_wait_drain(&ctl->v_full[g % kKvStages], (g / kKvStages) & 1)) atomicOr(dv.status, kStatusDrainTimeout);
      }
    }
    // queue at rest again for the next launch
    if (lane == 0) {
      __threadfence();
      const int done = atomicAdd(dv.queue + 3, 1);
      if (done == (int)gridDim.x - 1) {
        dv.queue[2] = 0;
        dv.queue[3] = 0;
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ================================================================ MMA issue: one thread
    if (lane == 0) {
      unsigned gb = 0;
      bool ok = true;
      const uint32_t q0 = smem_u32(q_tile);
      // O = sum over the item's steps of P V, accumulated in tensor memory (the softmax threads rescale it there on
      // the rare occasions a row's reference maximum moves).  P is read out of tensor memory (operand A), V out of
      // shared memory.
      auto issue_pv = [&](unsigned g, bool first_of_item, unsigned gi) -> bool {
        const int s = g % kKvStages;
        if (!mbar_wait(&ctl->p_full, g & 1, abort_flag)) return false;
        if (!mbar_wait(&ctl->v_full[s], (g / kKvStages) & 1, abort_flag)) return false;
        // the first product of an item overwrites the accumulator: the item before must have been read out
        if (first_of_item && gi >= 1 && !mbar_wait(&ctl->o_read, (gi - 1) & 1, abort_flag)) return false;
        tc_fence_after();
        const uint32_t v0 = smem_u32(v_tile + s * KV_TILE);
        const uint32_t p0 = tmem + kPCol;
#pragma unroll
        for (int kk = 0; kk < kStep / 16; ++kk) {   // 16 tokens per instruction: 8 columns of bf16 pairs
          const uint64_t db = operand_desc_mn(v0 + (uint32_t)(kk * 16 * 128), kKvHalfBytes, 1024);
          umma_bf16_tmem_a(tmem + kOCol, p0 + (uint32_t)(kk * 8), db, kIdescPV, (kk > 0 || !first_of_item) ? 1u : 0u);
          umma_bf16_tmem_a(tmem + kOCol, p0 + kPLo + (uint32_t)(kk * 8), db, kIdescPV, 1);
        }
        umma_commit(&ctl->v_empty[s]);
        umma_commit(&ctl->p_empty);
        return true;
      };
      for (unsigned gi = 0; ok; ++gi) {
        ok = mbar_wait(&ctl->item_ready, gi & 1, abort_flag);
        if (!ok) break;
        const int it = ctl->item;
        mbar_arrive(&ctl->item_taken);
        if (it < 0) break;
        const RoundItem w = items[it];
        const HeadState st = dv.state[(size_t)layer * dv.n_heads + w.head];
        const int nb = end_step(w, st.len) - first_step(w);
        ok = mbar_wait(&ctl->q_ready, gi & 1, abort_flag);
        for (int i = 0; i < nb && ok; ++i) {
          const unsigned g = gb + i;
          const int s = g % kKvStages;
          ok = mbar_wait(&ctl->k_full[s], (g / kKvStages) & 1, abort_flag);
          // S is overwritten: the softmax threads must have the scores of the step before in registers
          if (ok && g >= 1) ok = mbar_wait(&ctl->s_empty, (g - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t k0 = smem_u32(k_tile + s * KV_TILE);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {   // 16 elements = 32 bytes along the swizzled half row
            const uint32_t q_off = (uint32_t)((kk >> 2) * kQHalfBytes + (kk & 3) * 32);
            const uint32_t k_off = (uint32_t)((kk >> 2) * kKvHalfBytes + (kk & 3) * 32);
            umma_bf16_desc(tmem, operand_desc(q0 + q_off), operand_desc(k0 + k_off), kIdescQK, kk > 0);
          }
          umma_commit(&ctl->k_empty[s]);
          umma_commit(&ctl->s_full);
          if (i >= 1) ok = issue_pv(g - 1, i == 1, gi);   // behind the next step's scores, so that its softmax overlaps this product
        }
        if (ok && nb > 0) ok = issue_pv(gb + nb - 1, nb == 1, gi);
        gb += nb;
      }
      if (!ok) {   // leaving early: let the instructions in flight finish before tensor memory is released
        atomicOr(dv.status, kStatusConsumerTimeout);
        umma_commit(&ctl->drain);
        (void)mbar_wait_drain(&ctl->drain, 0);
      }
    }
    __syncwarp();
  } else {
    // ================================================================ softmax and epilogue: a thread per query row
    const int sw = warp & 3;                     // tensor-memory lane quarter this warp may access
    const int row = sw * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(sw * 32) << 16);
    const float scale_log2 = dv.scale_log2;
    unsigned gb = 0, n_sync = 0;   // steps so far; exchanges of column positions so far
    bool ok = true;
    for (unsigned gi = 0; ok; ++gi) {
      ok = mbar_wait(&ctl->item_ready, gi & 1, abort_flag);
      if (!ok) break;
      const int it = ctl->item;
      mbar_arrive(&ctl->item_taken);
      if (it < 0) break;
      const RoundItem w = items[it];
      const size_t hs = (size_t)layer * dv.n_heads + w.head;
      const HeadState st = dv.state[hs];
      const int b = w.head / dv.n_kv_heads, g_kv = w.head % dv.n_kv_heads;
      const int total = st.len + st.n_drop;
      // this row: query token t (within the round), query head j of the group
      const int t = w.q_tile * tok_per_tile + row / G, j = row % G;
      const bool row_live = t < jb.n_tok;
      // A warp none of whose rows is a query of the round (the last tile of a round is seldom full) keeps the pace of
      // the barriers and computes nothing: its rows of P and O hold whatever they held, and nobody reads them.
      const bool warp_live = __any_sync(0xffffffffu, row_live);
      const int q_pos = total - jb.n_tok + t;
      const size_t row_off = (((size_t)b * jb.n_tok + min(t, jb.n_tok - 1)) * ((size_t)dv.n_kv_heads * G) + (size_t)g_kv * G + j) * D;

      // ---- the query row into shared memory (operand layout: 128-byte half rows, chunks swizzled by the row)
      const bool seed = w.part_idx == 0 && dv.use_comp && st.n_drop > 0 && st.window >= 0;
      float s_c = 0.f;
      {
        const uint4* src = (const uint4*)(q + row_off);
        const float* k_hat = dv.comp_mean + hs * 2 * D;
#pragma unroll
        for (int c = 0; c < D / 8; ++c) {
          uint4 u = row_live ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
          *(uint4*)(q_tile + (c >> 3) * kQHalfBytes + row * 128 + (((c & 7) ^ (row & 7)) << 4)) = u;
          if (seed) {
            float f[8];
            Elem<__nv_bfloat16>::unpack(u, f);
#pragma unroll
            for (int e = 0; e < 8; ++e) s_c = fmaf(f[e], k_hat[c * 8 + e], s_c);
          }
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(&ctl->q_ready);

      // Online softmax against a reference maximum m_ref that is allowed to lag: weights are 2^(s - m_ref), at
      // most 2^kLag, and the accumulator in tensor memory is rescaled only when a row's maximum has outrun the
      // reference by more than kLag (rare after the first steps).  The compensation token (Eq. 4, Eq. 5: weight
      // N_d exp(s_c), value v_hat) is carried as a scalar weight w_seed and added at the end.
      constexpr float kLag = 8.f;
      float m_ref = -CUDART_INF_F, l_run = 0.f, w_seed = 0.f;
      if (seed) {
        m_ref = s_c * scale_log2 + log2f((float)st.n_drop);
        l_run = 1.f;
        w_seed = 1.f;
      }
      const bool in_order = st.window < 0 || st.n_drop == 0;               // slot = position
      float slope_l2 = 0.f;   // ALiBi slope of this row's query head (Section 3.1), log2 domain
      if constexpr (kAlibi) slope_l2 = dv.alibi_slopes[((size_t)layer * dv.n_kv_heads + g_kv) * G + j];
      const int q_pos_min = total - jb.n_tok + w.q_tile * tok_per_tile;    // the tile's earliest query
      int new_lo = 0, new_hi = 0, new_lo2 = 0, new_hi2 = 0;                // slot ranges [lo, hi) holding the round's tokens
      if (!in_order) {
        const int lo = ((st.ring_head - jb.n_tok) % st.window + st.window) % st.window;
        if (jb.n_tok >= st.window) { new_lo = dv.n_sink; new_hi = dv.n_sink + st.window; }
        else if (lo < st.ring_head) { new_lo = dv.n_sink + lo; new_hi = dv.n_sink + st.ring_head; }
        else { new_lo = dv.n_sink + lo; new_hi = dv.n_sink + st.window; new_lo2 = dv.n_sink; new_hi2 = dv.n_sink + st.ring_head; }
      }
      const int s_begin = first_step(w);
      const int nb = end_step(w, st.len) - s_begin;
      // V rows of slots beyond the head's length may hold anything (a zero weight times a NaN is a NaN): the softmax
      // threads zero them in shared memory before the step's product is released.
      auto zero_rows_beyond_the_end = [&](unsigned g, int slot0) -> bool {
        if (slot0 + kStep <= st.len) return true;
        if (!mbar_wait(&ctl->v_full[g % kKvStages], (g / kKvStages) & 1, abort_flag)) return false;   // the rows must have landed before they are overwritten
        const int first_bad = max(st.len - slot0, 0);
        uint8_t* vt = v_tile + (g % kKvStages) * KV_TILE;
        for (int idx = first_bad * 8 + row; idx < kStep * 8; idx += kSoftmaxThreads) {   // 16-byte chunks of the bad rows
#pragma unroll
          for (int h = 0; h < HALVES; ++h) *(uint4*)(vt + h * kKvHalfBytes + idx * 16) = make_uint4(0u, 0u, 0u, 0u);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        return true;
      };
      for (int i = 0; i < nb && ok; ++i) {
        const unsigned g = gb + i;
        const int slot0 = (s_begin + i) * kStep;
        // Does the step need masking?  Slots beyond the head's length, or tokens of the round (the newest n_tok: the
        // last slots of a head whose slots are in position order, a cyclic run of the ring otherwise) that come
        // after some query of the tile.  Every thread finds the same answer from the head's state, so the common
        // case costs no exchange; in a step that does need it each of the first 64 threads works out the position
        // of one column and the four warps trade them through shared memory.
        const int slot1 = slot0 + kStep;
        bool masked = slot1 > st.len;
        if (in_order) masked |= slot1 - 1 > q_pos_min;
        else masked |= (slot0 < new_hi && new_lo < slot1) || (slot0 < new_hi2 && new_lo2 < slot1);
        const int32_t* col_pos = ctl->col_pos[n_sync & 1];
        if (masked) {
          // (double-buffered: a thread may still be reading the positions of the masked step before)
          if (row < kStep) {
            const int s = slot0 + row;   // column `row` of the step
            ctl->col_pos[n_sync & 1][row] = s < st.len ? slot_pos(s, dv.n_sink, st.ring_head, st.window, st.n_drop, total) : 0x7fffffff;
          }
          mbar_arrive(&ctl->blk_sync);
          ok = mbar_wait(&ctl->blk_sync, n_sync & 1, abort_flag);
          if (!ok) break;
          n_sync += 1;
        }
        ok = mbar_wait(&ctl->s_full, g & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        if (!warp_live) {
          tc_fence_before();
          mbar_arrive(&ctl->s_empty);
          if (g >= 1) ok = mbar_wait(&ctl->p_empty, (g - 1) & 1, abort_flag);   // (an arrival must not run into the phase before)
          if (ok) ok = zero_rows_beyond_the_end(g, slot0);   // (every softmax thread has a share of that)
          if (!ok) break;
          mbar_arrive(&ctl->p_full);
          continue;
        }

        // ---- this row's 64 scores, in registers
        uint32_t v[kStep];
#pragma unroll
        for (int c = 0; c < kStep / 32; ++c) tmem_ld32_issue(lane_addr + (uint32_t)(c * 32), v + c * 32);
        tmem_ld_wait_all();
#pragma unroll
        for (int e = 0; e < kStep; ++e) asm volatile("" : "+r"(v[e]));
        tc_fence_before();
        mbar_arrive(&ctl->s_empty);
        if (masked) {
#pragma unroll
          for (int e = 0; e < kStep; ++e)
            if (col_pos[e] > q_pos) v[e] = 0xff800000u;   // -inf
        }
        if constexpr (kAlibi) {
          // Eq. 1: the logit of column e gets - l_h (m - n), with the slope already in the log2 domain.  The position
          // n of column e runs up with e: slot0 + e in position order; in a ring total - window + (x0 + e), plus window
          // for the columns before the wrap (x0 + e < 0).  (No sink tokens in an ALiBi cache on this path.)  The scores
          // are put into the log2 domain here, so the scale below is one.
          float pen_base, pen_wrap = 0.f;
          int wrap_end = 0;
          if (in_order) {
            pen_base = slope_l2 * (float)(slot0 - q_pos);
          } else {
            const int x0 = slot0 - st.ring_head;
            pen_base = slope_l2 * (float)(total - st.window + x0 - q_pos);
            pen_wrap = slope_l2 * (float)st.window;
            wrap_end = -x0;
          }
#pragma unroll
          for (int e = 0; e < kStep; ++e) {
            float pen = fmaf(slope_l2, (float)e, pen_base);
            if (e < wrap_end) pen += pen_wrap;
            v[e] = __float_as_uint(fmaf(__uint_as_float(v[e]), scale_log2, pen));
          }
        }
        const float sc = kAlibi ? 1.f : scale_log2;
        float mx0 = -CUDART_INF_F, mx1 = -CUDART_INF_F;
#pragma unroll
        for (int e = 0; e < kStep; e += 4) {
          mx0 = max3(mx0, __uint_as_float(v[e]), __uint_as_float(v[e + 1]));
          mx1 = max3(mx1, __uint_as_float(v[e + 2]), __uint_as_float(v[e + 3]));
        }
        // (the scale is positive: the max of the scaled scores is the scaled max)
        const float m_blk = fmaxf(mx0, mx1) * sc;

        // The product of the step before must have run before P is overwritten and before O is touched.  The
        // weights themselves need neither, so in the common case (no rescaling) they are computed into registers
        // first and the wait comes just before the stores: the product's latency hides behind the arithmetic.
        bool p_free = g == 0;
        // ---- move the reference maximum?  Tensor-memory loads and stores are warp-wide, so the warp decides as one.
        const bool want = m_blk > m_ref + kLag || (m_ref == -CUDART_INF_F && m_blk > -CUDART_INF_F);
        if (__any_sync(0xffffffffu, want)) {
          if (!p_free) {
            ok = mbar_wait(&ctl->p_empty, (g - 1) & 1, abort_flag);
            if (!ok) break;
            p_free = true;
          }
          const float m_to = fmaxf(m_ref, m_blk);
          const float f = (m_to == -CUDART_INF_F || m_ref == -CUDART_INF_F) ? 0.f : fast_exp2(m_ref - m_to);   // 1 for a row that stays
          if (i >= 1) {   // the accumulator holds products of this item: rescale this warp's rows
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
              uint32_t o[32];
              tmem_ld32_issue(lane_addr + kOCol + (uint32_t)(c * 32), o);
              tmem_ld_wait_all();
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                asm volatile("" : "+r"(o[e]));
                o[e] = __float_as_uint(__uint_as_float(o[e]) * f);
              }
              tmem_st32(lane_addr + kOCol + (uint32_t)(c * 32), o);
            }
            tmem_st_wait_all();
            tc_fence_before();
          }
          l_run *= f;
          w_seed *= f;
          m_ref = m_to;
        }
        const float m_use = (m_ref == -CUDART_INF_F) ? 0.f : m_ref;

        // ---- weights, their sum, and P into tensor memory: column c of the head half holds the bf16 pair of tokens
        // 2c and 2c + 1 (the operand-A layout of the matrix unit), the remainder half the same.  A weight goes into
        // the product as a bf16 head (its upper 16 bits) plus a bf16 remainder - two products - so that it keeps
        // fp32-like accuracy: a single bf16 would put 2^-9 of a large weight times its V row into the result.
        const uint64_t scale2 = f2_pack(sc, sc), neg_m2 = f2_pack(-m_use, -m_use);
        uint64_t psum2[2] = {f2_pack(0.f, 0.f), f2_pack(0.f, 0.f)};
        const uint32_t p_addr = lane_addr + kPCol;
        uint32_t hi[kStep / 2], lo[kStep / 2];
#pragma unroll
        for (int e2 = 0; e2 < kStep / 2; ++e2) {
          const int e = e2 * 2;
          float t0, t1, l0, l1;
          f2_unpack(f2_fma(f2_pack(__uint_as_float(v[e]), __uint_as_float(v[e + 1])), scale2, neg_m2), t0, t1);
          const float w0 = fast_exp2(t0), w1 = fast_exp2(t1);
          const uint64_t w2 = f2_pack(w0, w1);
          psum2[e2 & 1] = f2_add(psum2[e2 & 1], w2);
          const uint32_t b0 = __float_as_uint(w0), b1 = __float_as_uint(w1);
          hi[e2] = __byte_perm(b0, b1, 0x7632);
          f2_unpack(f2_sub(w2, f2_pack(__uint_as_float(b0 & 0xffff0000u), __uint_as_float(b1 & 0xffff0000u))), l0, l1);
          lo[e2] = pack2_bf16(l0, l1);
        }
        if (!p_free) {
          ok = mbar_wait(&ctl->p_empty, (g - 1) & 1, abort_flag);
          if (!ok) break;
        }
        tmem_st32(p_addr, hi);
        tmem_st32(p_addr + kPLo, lo);
        {
          float a0, a1;
          f2_unpack(f2_add(psum2[0], psum2[1]), a0, a1);
          l_run += a0 + a1;
        }
        ok = zero_rows_beyond_the_end(g, slot0);
        if (!ok) break;
        tmem_st_wait_all();
        tc_fence_before();
        mbar_arrive(&ctl->p_full);
      }
      if (!ok) break;
      // ---- the row's result: accumulator out of tensor memory once the last product is done, plus the
      // compensation token's share; the output when the unit is in one part, else a partial record
      if (nb > 0) {
        ok = mbar_wait(&ctl->p_empty, (gb + nb - 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
      }
      gb += nb;
      const bool direct = w.n_parts == 1;
      const float inv = direct ? (l_run > 0.f ? 1.f / l_run : 0.f) : 1.f;
      const size_t r = (size_t)w.rec_base + (size_t)w.part_idx * kRows + row;
      float* dst = direct ? out + row_off : dv.rec_o + r * D;
      const float* v_hat = dv.comp_mean + hs * 2 * D + D;
#pragma unroll
      for (int c = 0; c < (warp_live ? D / 32 : 0); ++c) {
        uint32_t o[32];
        if (nb > 0) {
          tmem_ld32_issue(lane_addr + kOCol + (uint32_t)(c * 32), o);
          tmem_ld_wait_all();
        }
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          asm volatile("" : "+r"(o[e]));
          float x = nb > 0 ? __uint_as_float(o[e]) : 0.f;
          if (seed) x = fmaf(w_seed, v_hat[c * 32 + e], x);
          o[e] = __float_as_uint(x * inv);
        }
        if (direct ? row_live : true) {
#pragma unroll
          for (int e = 0; e < 32; e += 4)
            *(float4*)(dst + c * 32 + e) = make_float4(__uint_as_float(o[e]), __uint_as_float(o[e + 1]), __uint_as_float(o[e + 2]), __uint_as_float(o[e + 3]));
        }
      }
      if (!direct && warp_live) dv.rec_ml[r] = make_float2(m_ref, l_run);
      tc_fence_before();
      mbar_arrive(&ctl->o_read);
    }
    if (!ok && lane == 0) atomicOr(dv.status, kStatusReducerTimeout);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// Merges the partial records of the (head, query tile) units that were cut into several parts: a warp per
// query row, parts folded in order.  grid = (units, 32), block = 128.
template <int D>
__global__ void __launch_bounds__(128) round_combine_kernel(DeviceView dv, RoundJobs jb, float* __restrict__ out) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const RoundUnit u = dv.round_units[blockIdx.x];
  const int row = blockIdx.y * 4 + warp;
  const int G = dv.group, tok_per_tile = kRows / G;
  const int t = u.q_tile * tok_per_tile + row / G, j = row % G;
  if (t >= jb.n_tok) return;
  float m = -CUDART_INF_F, l = 0.f;
  LaneVec<D> acc;
  acc.zero();
  constexpr int U = 8;   // records in flight (a unit of a long head may be in a hundred parts)
  for (int p0 = 0; p0 < u.n_parts; p0 += U) {
    float2 mls[U];
    LaneVec<D> os[U];
#pragma unroll
    for (int i = 0; i < U; ++i) {
      const size_t r = (size_t)u.rec_base + (size_t)min(p0 + i, u.n_parts - 1) * kRows + row;   // beyond the end: re-read, unused
      mls[i] = __ldcg(&dv.rec_ml[r]);
      os[i].load_l2(dv.rec_o + r * D, lane);
    }
#pragma unroll
    for (int i = 0; i < U; ++i) {
      if (p0 + i < u.n_parts) {
        const float2 ml = mls[i];
        const float mn = fmaxf(m, ml.x);
        const float mu = (mn == -CUDART_INF_F) ? 0.f : mn;
        const float c_old = fast_exp2(m - mu), c_new = fast_exp2(ml.x - mu);
        l = l * c_old + ml.y * c_new;
        acc.scale(c_old);
        acc.fma(c_new, os[i]);
        m = mn;
      }
    }
  }
  acc.scale(l > 0.f ? 1.f / l : 0.f);
  const int b = u.head / dv.n_kv_heads, g_kv = u.head % dv.n_kv_heads;
  acc.store(out + (((size_t)b * jb.n_tok + t) * ((size_t)dv.n_kv_heads * G) + (size_t)g_kv * G + j) * D, lane);
}

// Tensor map over the page pool as (64 elements, 16 tokens, [2 halves,] K|V, pages): a box of 64 x 16 is one
// half of the K or V rows of a page; no swizzle on top (the pool's pages are stored swizzled already).
template <int D>
bool make_pool_map(CUtensorMap* map, const void* pool, long long n_pages) {
  const EncodeTiledFn encode = encode_tiled_fn();
  if (!encode) return false;
  constexpr cuuint64_t RB = D * 2;   // bytes per row
  if constexpr (D == 128) {
    const cuuint64_t dims[5] = {64, 16, 2, 2, (cuuint64_t)n_pages};
    const cuuint64_t strides[4] = {RB, 128, 16 * RB, 32 * RB};
    const cuuint32_t box[5] = {64, 16, 1, 1, 1};
    const cuuint32_t es[5] = {1, 1, 1, 1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(pool), dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  } else {
    const cuuint64_t dims[4] = {64, 16, 2, (cuuint64_t)n_pages};
    const cuuint64_t strides[3] = {RB, 16 * RB, 32 * RB};
    const cuuint32_t box[4] = {64, 16, 1, 1};
    const cuuint32_t es[4] = {1, 1, 1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(pool), dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  }
}

template <int D, bool kAlibi>
cudaError_t round_launch(const DeviceView& dv, long long pool_pages, int layer, const RoundJobs& jb, const void* q,
                         float* out, int n_sms, cudaStream_t s) {
  CUtensorMap map;
  if (!make_pool_map<D>(&map, dv.pool, pool_pages)) return cudaErrorInvalidValue;
  static bool opted_in[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !opted_in[dev]) {
    e = cudaFuncSetAttribute(round_kernel<D, kAlibi>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)round_smem_bytes<D>());
    if (e != cudaSuccess) return e;
    // two CTAs to an SM need the largest shared-memory split
    e = cudaFuncSetAttribute(round_kernel<D, kAlibi>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) opted_in[dev] = true;
  }
  const int grid = std::max(1, std::min(n_sms * kCtasPerSm, jb.n_items));
  round_kernel<D, kAlibi><<<grid, kRoundThreads, round_smem_bytes<D>(), s>>>(dv, map, layer, jb, (const __nv_bfloat16*)q, out);
  e = cudaGetLastError();
  if (e != cudaSuccess || jb.n_units == 0) return e;
  round_combine_kernel<D><<<dim3(jb.n_units, kRows / 4), 128, 0, s>>>(dv, jb, out);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_round(const DeviceView& dv, long long pool_pages, int layer, const RoundJobs& jb, const void* q,
                         float* out, int n_sms, cudaStream_t s) {
  if (dv.alibi)
    return dv.head_dim == 128 ? round_launch<128, true>(dv, pool_pages, layer, jb, q, out, n_sms, s)
                              : round_launch<64, true>(dv, pool_pages, layer, jb, q, out, n_sms, s);
  return dv.head_dim == 128 ? round_launch<128, false>(dv, pool_pages, layer, jb, q, out, n_sms, s)
                            : round_launch<64, false>(dv, pool_pages, layer, jb, q, out, n_sms, s);
}

}  // namespace razor
