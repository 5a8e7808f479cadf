// Cache-building kernels: prefill-end compression (Algorithm 1, Eq. 4), decode-token
// append with fold-on-evict, and the logical-order export used for snapshots and parity checks.
#include "razor_common.cuh"
#include "razor_sync.cuh"

namespace razor {

// ---------------------------------------------------------------------------------------------
// Compression.  grid = (slices, Hkv, sequences); a CTA streams one slice of the rows of one
// (sequence, KV head).  Every dense row is read exactly once: a kept row is copied bit for bit to its
// page slot, a dropped row is added into per-thread fp32 accumulators.  The per-slice sums go to
// scratch and are reduced in a fixed order by compress_finalize_kernel, so the compensation token
// (Eq. 4) is reproducible from run to run.
// Slot of a kept position p (ascending position order): retrieval head or N <= N0 + W: slot = p;
// otherwise sinks p < N0 keep slot p and recent tokens p >= N - W go to N0 + (p - (N - W)).
//
// The rows come in through the bulk-copy engine: a producer warp copies blocks of 16 rows (their K
// rows, then their V rows: one copy each when the rows are contiguous in the source, one per row
// otherwise) into a ring of shared-memory stages that complete on mbarriers, and kCompressWarps
// consumer warps take the blocks round-robin, 16 bytes of a row per lane.  Block i always goes to warp
// i % kCompressWarps and the ring length is a multiple of that, so the sums are added in the same
// order every run.  All waits are bounded (status bits as in the decode kernel).
constexpr int kCompressWarps = 4;
constexpr int kCompressThreads = (kCompressWarps + 1) * 32;
constexpr int kCompressRingBytes = 64 * 1024;

template <typename T, int D>
struct CompressSmem {
  static constexpr int kBlockBytes = 2 * kPageTokens * RowGeom<T, D>::kRowBytes;   // 16 K rows + 16 V rows
  static constexpr int kStages = kCompressRingBytes / kBlockBytes;
  static_assert(kStages >= kCompressWarps && kStages % kCompressWarps == 0, "a stage belongs to one warp");
  alignas(128) uint8_t ring[kStages][kBlockBytes];
  float red[kCompressWarps][RowGeom<T, D>::kRg][2][D];   // [warp][row within a pass][K | V][D]
  uint64_t full[kStages], empty[kStages];
  int abort_flag;
};

template <typename T, int D>
__global__ void __launch_bounds__(kCompressThreads) compress_kernel(DeviceView dv, int layer, int n_slices) {
  using Geo = RowGeom<T, D>;
  using Smem = CompressSmem<T, D>;
  constexpr int LPR = Geo::kLpr, RG = Geo::kRg, EPL = Geo::kEpl, RB = Geo::kRowBytes, S = Smem::kStages;
  extern __shared__ __align__(128) uint8_t compress_smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>(compress_smem_raw);

  const SeqDesc sd = dv.seq_desc[blockIdx.z];
  const int g = blockIdx.y;
  const int head = sd.b * dv.n_kv_heads + g;
  const HeadState st = dv.state[(size_t)layer * dv.n_heads + head];
  const int N = sd.n_ctx, n_sink = dv.n_sink;
  const bool keep_all = st.window < 0 || N <= n_sink + st.window;
  const int recent0 = keep_all ? 0 : N - st.window;

  const int rows_per_slice = (((N + n_slices - 1) / n_slices) + 15) & ~15;
  const int r0 = blockIdx.x * rows_per_slice;
  const int r1 = min(N, r0 + rows_per_slice);
  const int n_blocks = r1 > r0 ? (r1 - r0 + kPageTokens - 1) / kPageTokens : 0;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  const char* Kb = (const char*)sd.K + (size_t)g * sd.stride_h * sizeof(T);
  const char* Vb = (const char*)sd.V + (size_t)g * sd.stride_h * sizeof(T);
  const size_t row_stride = (size_t)sd.stride_n * sizeof(T);
  volatile int* abort_flag = &sm.abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(&sm.full[s], 1);
      mbar_init(&sm.empty[s], 1);
    }
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == kCompressWarps) {
    // ---- producer
    if (lane == 0) {
      const bool contiguous = row_stride == (size_t)RB;
      int issued = 0;
      for (int i = 0; i < n_blocks; ++i) {
        const int s = i % S, use = i / S;
        if (use > 0 && !mbar_wait(&sm.empty[s], (use - 1) & 1, abort_flag)) {
          atomicOr(dv.status, kStatusProducerTimeout);
          break;
        }
        const int p = r0 + i * kPageTokens, rows = min(kPageTokens, r1 - p);
        mbar_arrive_expect_tx(&sm.full[s], (uint32_t)(2 * rows * RB));
        uint8_t* dstK = sm.ring[s];
        uint8_t* dstV = dstK + kPageTokens * RB;
        if (contiguous) {
          bulk_load(dstK, Kb + (size_t)p * row_stride, (uint32_t)(rows * RB), &sm.full[s]);
          bulk_load(dstV, Vb + (size_t)p * row_stride, (uint32_t)(rows * RB), &sm.full[s]);
        } else {
          for (int t = 0; t < rows; ++t) {
            bulk_load(dstK + t * RB, Kb + (size_t)(p + t) * row_stride, RB, &sm.full[s]);
            bulk_load(dstV + t * RB, Vb + (size_t)(p + t) * row_stride, RB, &sm.full[s]);
          }
        }
        issued = i + 1;
      }
      if (*abort_flag) {   // the copies in flight must land before the CTA may exit
        for (int i = max(0, issued - S); i < issued; ++i)
          if (!mbar_wait_drain(&sm.full[i % S], (i / S) & 1)) atomicOr(dv.status, kStatusDrainTimeout);
      }
    }
  } else {
    // ---- consumers: LPR lanes per row, so a warp takes RG rows of a block per pass
    const int lir = lane % LPR, par = lane / LPR;
    const int32_t* pt = dv.page_table + ((size_t)layer * dv.n_heads + head) * dv.max_pages;
    float accK[EPL], accV[EPL];
#pragma unroll
    for (int i = 0; i < EPL; ++i) accK[i] = accV[i] = 0.f;
    for (int i = warp; i < n_blocks; i += kCompressWarps) {
      const int s = i % S, use = i / S;
      if (!__all_sync(0xffffffffu, mbar_wait(&sm.full[s], use & 1, abort_flag))) {
        if (lane == 0) atomicOr(dv.status, kStatusConsumerTimeout);
        break;
      }
      const int p0 = r0 + i * kPageTokens;
      const uint4* rowsK = (const uint4*)sm.ring[s];
      const uint4* rowsV = rowsK + kPageTokens * LPR;
      // The block goes to registers (eight passes at a time) and the stage back to the producer before
      // the rows are looked at, so that a stage is held only for the time of a few shared-memory loads.
      constexpr int PASSES = kPageTokens / RG, CH = PASSES < 8 ? PASSES : 8;
#pragma unroll
      for (int c = 0; c < PASSES / CH; ++c) {
        uint4 kf[CH], vf[CH];
#pragma unroll
        for (int it = 0; it < CH; ++it) {
          const int t = RG * (c * CH + it) + par;
          kf[it] = rowsK[t * LPR + lir];
          vf[it] = rowsV[t * LPR + lir];
        }
        if (c == PASSES / CH - 1) {
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.empty[s]);
        }
#pragma unroll
        for (int it = 0; it < CH; ++it) {
          const int t = RG * (c * CH + it) + par, p = p0 + t;
          if (p >= r1) continue;
          int slot;
          if (keep_all || p < n_sink) slot = p;
          else if (p >= recent0) slot = n_sink + (p - recent0);
          else slot = -1;
          if (slot >= 0) {
            const size_t page = (size_t)pt[slot >> 4];
            uint4* dst = (uint4*)(dv.pool + page * dv.page_bytes + (size_t)(slot & 15) * RB) + swz(slot, lir);
            dst[0] = kf[it];
            dst[kPageTokens * LPR] = vf[it];   // V rows follow the 16 K rows of the page
          } else {
            float a[EPL], b[EPL];
            Elem<T>::unpack(kf[it], a);
            Elem<T>::unpack(vf[it], b);
#pragma unroll
            for (int e = 0; e < EPL; ++e) { accK[e] += a[e]; accV[e] += b[e]; }
          }
        }
      }
    }
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      sm.red[warp][par][0][lir * EPL + e] = accK[e];
      sm.red[warp][par][1][lir * EPL + e] = accV[e];
    }
  }
  __syncthreads();
  float* scratch =
      dv.compress_scratch + (((size_t)blockIdx.z * dv.n_kv_heads + g) * n_slices + blockIdx.x) * 2 * D;
  for (int e = threadIdx.x; e < 2 * D; e += kCompressThreads) {
    float sum = 0.f;
#pragma unroll
    for (int w = 0; w < kCompressWarps; ++w)
#pragma unroll
      for (int r = 0; r < RG; ++r) sum += sm.red[w][r][e / D][e % D];
    scratch[e] = sum;
  }
}

// grid = planned heads, block = 256: the head's state and its page-table row (consecutive pool pages), so
// that a compression call sends a few bytes per head to the device instead of whole page-table rows.
__global__ void __launch_bounds__(256) compress_plan_kernel(DeviceView dv, int layer) {
  const HeadPlan pl = dv.plan[blockIdx.x];
  const size_t hs = (size_t)layer * dv.n_heads + pl.head;
  int32_t* row = dv.page_table + hs * dv.max_pages;
  for (int k = threadIdx.x; k < pl.n_pages; k += 256) row[k] = pl.first_page + k;
  if (threadIdx.x == 0) {
    dv.state[hs] = HeadState{pl.len, pl.n_drop, 0, pl.window};
    dv.ring_valid[hs] = 0;   // nobody has summed the rows of the new window
  }
}

// grid = (Hkv, sequences), block = 2*D threads: fixed-order sum of the slice partials, then the
// means of Eq. 4 (zero when nothing was dropped, so no 0/0 is ever formed).
template <int D>
__global__ void compress_finalize_kernel(DeviceView dv, int layer, int n_slices) {
  const SeqDesc sd = dv.seq_desc[blockIdx.y];
  const int head = sd.b * dv.n_kv_heads + blockIdx.x;
  const size_t hs = (size_t)layer * dv.n_heads + head;
  const int n_drop = dv.state[hs].n_drop;
  const float* scratch = dv.compress_scratch + ((size_t)blockIdx.y * dv.n_kv_heads + blockIdx.x) * n_slices * 2 * D;
  const int e = threadIdx.x;
  float s = 0.f;
  for (int i = 0; i < n_slices; ++i) s += scratch[(size_t)i * 2 * D + e];
  if (n_drop == 0) s = 0.f;
  dv.comp_sum[hs * 2 * D + e] = s;
  dv.comp_mean[hs * 2 * D + e] = n_drop > 0 ? __fdiv_rn(s, (float)n_drop) : 0.f;
}

// ---------------------------------------------------------------------------------------------
// Append: one warp per (sequence, KV head).  A head that keeps everything, or whose window is not
// full yet, stores the new row in slot `len`.  Otherwise the oldest recent token (ring slot
// ring_head) is folded into the fp32 compensation sums, the count grows by one, the means are
// recomputed (Eq. 4 over every token dropped so far) and the new row takes that slot.
template <typename T, int D>
__global__ void __launch_bounds__(64) append_kernel(DeviceView dv, int layer, const T* __restrict__ k_new,
                                                     const T* __restrict__ v_new, int early_reads) {
  using Geo = RowGeom<T, D>;
  constexpr int LPR = Geo::kLpr, EPL = Geo::kEpl;
  const int lane = threadIdx.x & 31;
  const int head = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  // Launched as a programmatic dependent of the kernel before it on the stream, which may still be running
  // when this kernel starts.  Two kinds of memory are read here:
  //   * the library's own state of this layer (head state, page id, the row about to be evicted, the
  //     compensation sums), last written by this layer's compression or previous append.  Unless that writer
  //     is the kernel directly before this one (early_reads = 0) it finished long ago, so these reads and the
  //     arithmetic on them may run ahead of the dependency wait;
  //   * the caller's k_new / v_new.  Whatever produced them (in a model: the K/V projection, the kernel
  //     directly before this one) is not known to the library, so they are read only after the wait.
  // Every write comes after the wait as well, which keeps completion in stream order.
  // The kernel queued behind this one (the layer's decode kernel) may start right away: ahead of its own wait
  // it touches nothing this kernel writes (it is told which page of each head the append stores into).
  cudaTriggerProgrammaticLaunchCompletion();
  if (!early_reads) cudaGridDependencySynchronize();
  const bool active = head < dv.n_heads;
  const size_t hs = (size_t)layer * dv.n_heads + (active ? head : 0);
  HeadState st = dv.state[hs];
  const int n_sink = dv.n_sink;
  const bool keeps_all = st.window < 0;

  int slot = -1;
  bool evict = false, fold_new = false;
  if (keeps_all || st.len < n_sink + st.window) {
    slot = st.len;
    st.len += 1;
  } else if (st.window == 0) {
    fold_new = true;                 // no recent window at all: the token is dropped at once
    st.n_drop += 1;
  } else {
    slot = n_sink + st.ring_head;
    evict = true;
    st.n_drop += 1;
    st.ring_head = (st.ring_head + 1 == st.window) ? 0 : st.ring_head + 1;
  }

  const bool row_lane = active && lane < LPR;
  uint4* krow = nullptr;
  float fold[2][EPL], old_sum[2][EPL];   // the row that joins the dropped set (K, V) and the sums so far
  if (row_lane) {
    if (slot >= 0) {
      const size_t page = (size_t)dv.page_table[hs * dv.max_pages + (slot >> 4)];
      krow = (uint4*)(dv.pool + page * dv.page_bytes + (size_t)(slot & 15) * Geo::kRowBytes) + swz(slot, lane);
    }
    if (evict || fold_new) {
      const float* sum = dv.comp_sum + hs * 2 * D + lane * EPL;
#pragma unroll
      for (int i = 0; i < EPL; ++i) { old_sum[0][i] = sum[i]; old_sum[1][i] = sum[D + i]; }
    }
    if (evict) {
      Elem<T>::unpack(krow[0], fold[0]);
      Elem<T>::unpack(krow[kPageTokens * LPR], fold[1]);
    }
  }
  if (early_reads) cudaGridDependencySynchronize();
  if (row_lane) {
    const uint4 kf = ((const uint4*)(k_new + (size_t)head * D))[lane];
    const uint4 vf = ((const uint4*)(v_new + (size_t)head * D))[lane];
    if (fold_new) {
      Elem<T>::unpack(kf, fold[0]);
      Elem<T>::unpack(vf, fold[1]);
    }
    if (evict || fold_new) {
      float* sum = dv.comp_sum + hs * 2 * D + lane * EPL;
      float* mean = dv.comp_mean + hs * 2 * D + lane * EPL;
      const float cnt = (float)st.n_drop;
#pragma unroll
      for (int i = 0; i < EPL; ++i) {
        const float sk = old_sum[0][i] + fold[0][i], sv = old_sum[1][i] + fold[1][i];
        sum[i] = sk;
        sum[D + i] = sv;
        mean[i] = __fdiv_rn(sk, cnt);
        mean[D + i] = __fdiv_rn(sv, cnt);
      }
    }
    if (slot >= 0) {
      krow[0] = kf;
      krow[kPageTokens * LPR] = vf;
    }
  }
  if (active && lane == 0) {
    dv.state[hs] = st;
    dv.ring_valid[hs] = 0;   // the window's content changed and its sum was not kept up
  }
}

// ---------------------------------------------------------------------------------------------
// Append of a round of n_tok tokens per sequence (a second prompt, a verify step): one warp per
// (sequence, KV head) applies the single-token rule n_tok times in order, so the state afterwards is
// what n_tok razor_append calls would leave.  k_new, v_new: [B, n_tok, Hkv, D].
template <typename T, int D>
__global__ void __launch_bounds__(128) append_many_kernel(DeviceView dv, int layer, const T* __restrict__ k_new,
                                                          const T* __restrict__ v_new, int n_tok) {
  using Geo = RowGeom<T, D>;
  constexpr int LPR = Geo::kLpr, EPL = Geo::kEpl;
  const int lane = threadIdx.x & 31;
  const int head = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  cudaGridDependencySynchronize();
  cudaTriggerProgrammaticLaunchCompletion();
  if (head >= dv.n_heads) return;
  const size_t hs = (size_t)layer * dv.n_heads + head;
  HeadState st = dv.state[hs];
  __syncwarp();
  const int n_sink = dv.n_sink;
  const bool keeps_all = st.window < 0;
  const int b = head / dv.n_kv_heads, g = head % dv.n_kv_heads;
  float* sum = dv.comp_sum + hs * 2 * D + lane * EPL;
  float* mean = dv.comp_mean + hs * 2 * D + lane * EPL;
  for (int t = 0; t < n_tok; ++t) {
    int slot = -1;
    bool evict = false, fold_new = false;
    if (keeps_all || st.len < n_sink + st.window) {
      slot = st.len;
      st.len += 1;
    } else if (st.window == 0) {
      fold_new = true;
      st.n_drop += 1;
    } else {
      slot = n_sink + st.ring_head;
      evict = true;
      st.n_drop += 1;
      st.ring_head = (st.ring_head + 1 == st.window) ? 0 : st.ring_head + 1;
    }
    if (lane < LPR) {
      const size_t row = (((size_t)b * n_tok + t) * dv.n_kv_heads + g) * D;
      const uint4 kf = ((const uint4*)(k_new + row))[lane];
      const uint4 vf = ((const uint4*)(v_new + row))[lane];
      uint4* krow = nullptr;
      if (slot >= 0) {
        const size_t page = (size_t)dv.page_table[hs * dv.max_pages + (slot >> 4)];
        krow = (uint4*)(dv.pool + page * dv.page_bytes + (size_t)(slot & 15) * Geo::kRowBytes) + swz(slot, lane);
      }
      if (evict || fold_new) {
        const uint4 ok = evict ? krow[0] : kf;
        const uint4 ov = evict ? krow[kPageTokens * LPR] : vf;
        float a[EPL], c[EPL];
        Elem<T>::unpack(ok, a);
        Elem<T>::unpack(ov, c);
        const float cnt = (float)st.n_drop;
#pragma unroll
        for (int i = 0; i < EPL; ++i) {
          const float sk = sum[i] + a[i], sv = sum[D + i] + c[i];
          sum[i] = sk;
          sum[D + i] = sv;
          mean[i] = __fdiv_rn(sk, cnt);
          mean[D + i] = __fdiv_rn(sv, cnt);
        }
      }
      if (slot >= 0) {
        krow[0] = kf;
        krow[kPageTokens * LPR] = vf;
      }
    }
    __syncwarp();   // a later token of the round may evict a row this one just stored
  }
  if (lane == 0) {
    dv.state[hs] = st;
    dv.ring_valid[hs] = 0;
  }
}

// ---------------------------------------------------------------------------------------------
// Append of a long run of tokens (a prompt chunk of a chunked prefill, a long second prompt), in
// parallel over the tokens.  The state afterwards is what n_tok single appends would leave; append_fate()
// decides per token, in closed form, where it ends up.  A token that does not stay is added to the
// compensation sums straight from the input; a token that stays in a ring slot that held a token from
// before the call adds that old row to the sums first.  Every slot is written by exactly one thread group,
// after it has read the old row, so there is no order between CTAs to keep.  grid = (slices, heads);
// per-slice sums go to the compression scratch and append_chunk_finalize_kernel adds them to the running
// sums (Eq. 4 over everything dropped so far).
// Old rows are not read back when the run evicts the whole window and the sum of the window's rows is on
// record (ring_sum, kept by this kernel: every slice also sums the rows it stores into the window): that sum
// is then the old rows' share of the dropped set.  A prefill handed over in chunks of at least the window
// length therefore reads every row once and writes it once.
template <typename T, int D>
__global__ void __launch_bounds__(256) append_chunk_kernel(DeviceView dv, int layer, const T* __restrict__ k_new,
                                                           const T* __restrict__ v_new, int n_tok, int n_slices) {
  using Geo = RowGeom<T, D>;
  constexpr int LPR = Geo::kLpr, EPL = Geo::kEpl, NGRP = 256 / LPR;
  __shared__ float red[NGRP][2][D];
  const int head = blockIdx.y;
  const size_t hs = (size_t)layer * dv.n_heads + head;
  const HeadState st = dv.state[hs];
  const int n_sink = dv.n_sink;
  const int b = head / dv.n_kv_heads, g = head % dv.n_kv_heads;
  const int32_t* pt = dv.page_table + hs * dv.max_pages;
  const int per = (n_tok + n_slices - 1) / n_slices;
  const int a0 = min(n_tok, (int)blockIdx.x * per), a1 = min(n_tok, a0 + per);
  const int lir = threadIdx.x % LPR, grp = threadIdx.x / LPR;
  // the whole old window leaves and its sum is known: no need to read its rows
  const int ring_fill = st.window >= 0 && st.len > n_sink ? st.len - n_sink : 0;
  const int n_evict = n_tok - append_run_fits(st, n_sink, n_tok);
  const bool skip_old = st.window >= 0 && n_evict >= ring_fill && dv.ring_valid[hs] != 0;

  float accK[EPL], accV[EPL], ringK[EPL], ringV[EPL];
#pragma unroll
  for (int i = 0; i < EPL; ++i) accK[i] = accV[i] = ringK[i] = ringV[i] = 0.f;
  constexpr int U = 4;   // rows of a thread group in flight
  for (int a_first = a0 + grp; a_first < a1; a_first += NGRP * U) {
    uint4 kfs[U], vfs[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int a = a_first + u * NGRP;
      if (a < a1) {
        const size_t row = (((size_t)b * n_tok + a) * dv.n_kv_heads + g) * D;
        kfs[u] = ld_stream((const uint4*)(k_new + row) + lir);
        vfs[u] = ld_stream((const uint4*)(v_new + row) + lir);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int a = a_first + u * NGRP;
      if (a >= a1) break;
      const uint4 kf = kfs[u], vf = vfs[u];
      const AppendFate fate = append_fate(st, n_sink, n_tok, a);
      const int slot = fate.slot;
      const bool stays = slot >= 0, had_old = fate.evicts_old;
      float a_k[EPL], a_v[EPL];
      if (stays) {
        const size_t page = (size_t)pt[slot >> 4];
        uint4* dst = (uint4*)(dv.pool + page * dv.page_bytes + (size_t)(slot & 15) * Geo::kRowBytes) + swz(slot, lir);
        if (had_old && !skip_old) {
          Elem<T>::unpack(dst[0], a_k);
          Elem<T>::unpack(dst[kPageTokens * LPR], a_v);
#pragma unroll
          for (int i = 0; i < EPL; ++i) { accK[i] += a_k[i]; accV[i] += a_v[i]; }
        }
        dst[0] = kf;
        dst[kPageTokens * LPR] = vf;
        if (st.window >= 0 && slot >= n_sink) {   // a row of the new window
          Elem<T>::unpack(kf, a_k);
          Elem<T>::unpack(vf, a_v);
#pragma unroll
          for (int i = 0; i < EPL; ++i) { ringK[i] += a_k[i]; ringV[i] += a_v[i]; }
        }
      } else {
        Elem<T>::unpack(kf, a_k);
        Elem<T>::unpack(vf, a_v);
#pragma unroll
        for (int i = 0; i < EPL; ++i) { accK[i] += a_k[i]; accV[i] += a_v[i]; }
      }
    }
  }
  // two sets of sums per slice: rows that join the dropped set, rows stored into the window
  float* scratch = dv.compress_scratch + ((size_t)head * n_slices + blockIdx.x) * 4 * D;
#pragma unroll
  for (int set = 0; set < 2; ++set) {
    if (set) __syncthreads();
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
      red[grp][0][lir * EPL + i] = set ? ringK[i] : accK[i];
      red[grp][1][lir * EPL + i] = set ? ringV[i] : accV[i];
    }
    __syncthreads();
    for (int e = threadIdx.x; e < 2 * D; e += 256) {
      float sum = 0.f;
#pragma unroll
      for (int r = 0; r < NGRP; ++r) sum += (&red[r][0][0])[e];
      scratch[set * 2 * D + e] = sum;
    }
  }
}

// grid = heads, block = 2*D: slice sums added in a fixed order onto the running sums, means recomputed,
// state advanced by n_tok appends.
template <int D>
__global__ void append_chunk_finalize_kernel(DeviceView dv, int layer, int n_tok, int n_slices) {
  const int head = blockIdx.x, e = threadIdx.x;
  const size_t hs = (size_t)layer * dv.n_heads + head;
  const HeadState st = dv.state[hs];
  const int E = n_tok - append_run_fits(st, dv.n_sink, n_tok);
  const int ring_fill = st.window >= 0 && st.len > dv.n_sink ? st.len - dv.n_sink : 0;
  const bool all_old_gone = st.window >= 0 && E >= ring_fill;        // the window holds rows of this run only
  const bool skip_old = all_old_gone && dv.ring_valid[hs] != 0;      // (the streaming kernel decided the same)
  const float* scratch = dv.compress_scratch + (size_t)head * n_slices * 4 * D;
  if (E > 0) {
    float s = dv.comp_sum[hs * 2 * D + e];
    if (skip_old) s += dv.ring_sum[hs * 2 * D + e];   // the old window's rows, summed when they were stored
    for (int i = 0; i < n_slices; ++i) s += scratch[(size_t)i * 4 * D + e];
    dv.comp_sum[hs * 2 * D + e] = s;
    dv.comp_mean[hs * 2 * D + e] = __fdiv_rn(s, (float)(st.n_drop + E));
  }
  if (all_old_gone) {
    float r = 0.f;
    for (int i = 0; i < n_slices; ++i) r += scratch[(size_t)i * 4 * D + 2 * D + e];
    dv.ring_sum[hs * 2 * D + e] = r;
  }
  __syncthreads();   // every thread has read the old state and flag
  if (e == 0) {
    dv.state[hs] = state_after_run(st, dv.n_sink, n_tok);
    dv.ring_valid[hs] = all_old_gone ? 1 : 0;
  }
}

// ---------------------------------------------------------------------------------------------
// Export in logical order (ascending original position).  With T = len + n_drop tokens seen so far:
// logical index i < N0 (or any i while nothing has been dropped) is position i in slot i; otherwise
// j = i - N0 is the j-th oldest recent token: slot N0 + (ring_head + j) mod W, position T - W + j.
template <typename T, int D>
__global__ void __launch_bounds__(256) export_kernel(DeviceView dv, int layer, int head, int32_t* kept_pos, T* K,
                                                     T* V, float* mean_k, float* mean_v, float* sum_k, float* sum_v) {
  using Geo = RowGeom<T, D>;
  constexpr int LPR = Geo::kLpr, NGRP = 256 / LPR;
  const size_t hs = (size_t)layer * dv.n_heads + head;
  const HeadState st = dv.state[hs];
  const int n_sink = dv.n_sink;
  const int lir = threadIdx.x % LPR, grp = threadIdx.x / LPR;
  const int total = st.len + st.n_drop;
  for (int i = blockIdx.x * NGRP + grp; i < st.len; i += gridDim.x * NGRP) {
    int slot = i, pos = i;
    if (st.n_drop > 0 && i >= n_sink) {
      const int j = i - n_sink;
      slot = n_sink + (st.ring_head + j) % st.window;
      pos = total - st.window + j;
    }
    const size_t page = (size_t)dv.page_table[hs * dv.max_pages + (slot >> 4)];
    const uint4* src =
        (const uint4*)(dv.pool + page * dv.page_bytes + (size_t)(slot & 15) * Geo::kRowBytes) + swz(slot, lir);
    if (K) ((uint4*)(K + (size_t)i * D))[lir] = src[0];
    if (V) ((uint4*)(V + (size_t)i * D))[lir] = src[kPageTokens * LPR];
    if (kept_pos && lir == 0) kept_pos[i] = pos;
  }
  if (blockIdx.x == 0) {
    for (int e = threadIdx.x; e < D; e += 256) {
      if (mean_k) mean_k[e] = dv.comp_mean[hs * 2 * D + e];
      if (mean_v) mean_v[e] = dv.comp_mean[hs * 2 * D + D + e];
      if (sum_k) sum_k[e] = dv.comp_sum[hs * 2 * D + e];
      if (sum_v) sum_v[e] = dv.comp_sum[hs * 2 * D + D + e];
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Launch as a programmatic dependent of the preceding kernel on the stream: the launch latency and the
// kernel's first instructions overlap that kernel's tail.  Before its cudaGridDependencySynchronize() such a
// kernel touches at most memory that the library itself wrote whole kernels earlier; the caller's buffers
// are read, and everything is written, only after that wait.
template <typename... KArgs, typename... Args>
static cudaError_t launch_dependent(void (*kernel)(KArgs...), int grid, int block, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <typename T, int D>
static cudaError_t compress_t(const DeviceView& dv, int layer, int n_seqs, int n_slices, int n_plan, cudaStream_t s) {
  dim3 grid(n_slices, dv.n_kv_heads, n_seqs);
  const size_t smem = sizeof(CompressSmem<T, D>);
  cudaError_t e = cudaFuncSetAttribute(compress_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  if (n_plan > 0) {
    compress_plan_kernel<<<n_plan, 256, 0, s>>>(dv, layer);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  compress_kernel<T, D><<<grid, kCompressThreads, smem, s>>>(dv, layer, n_slices);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  compress_finalize_kernel<D><<<dim3(dv.n_kv_heads, n_seqs), 2 * D, 0, s>>>(dv, layer, n_slices);
  return cudaGetLastError();
}

cudaError_t launch_compress(const DeviceView& dv, int dtype, int layer, int n_seqs, int n_slices, int n_plan,
                            cudaStream_t s) {
  if (dtype == RAZOR_BF16) {
    return dv.head_dim == 128 ? compress_t<__nv_bfloat16, 128>(dv, layer, n_seqs, n_slices, n_plan, s)
                              : compress_t<__nv_bfloat16, 64>(dv, layer, n_seqs, n_slices, n_plan, s);
  }
  return dv.head_dim == 128 ? compress_t<float, 128>(dv, layer, n_seqs, n_slices, n_plan, s)
                            : compress_t<float, 64>(dv, layer, n_seqs, n_slices, n_plan, s);
}

template <typename T, int D>
static cudaError_t append_t(const DeviceView& dv, int layer, const void* k, const void* v, int early_reads,
                            cudaStream_t s) {
  const int warps = 2;
  return launch_dependent(append_kernel<T, D>, (dv.n_heads + warps - 1) / warps, warps * 32, s, dv, layer, (const T*)k,
                          (const T*)v, early_reads);
}

cudaError_t launch_append(const DeviceView& dv, int dtype, int layer, const void* k, const void* v, int early_reads,
                          cudaStream_t s) {
  if (dtype == RAZOR_BF16) {
    return dv.head_dim == 128 ? append_t<__nv_bfloat16, 128>(dv, layer, k, v, early_reads, s)
                              : append_t<__nv_bfloat16, 64>(dv, layer, k, v, early_reads, s);
  }
  return dv.head_dim == 128 ? append_t<float, 128>(dv, layer, k, v, early_reads, s)
                            : append_t<float, 64>(dv, layer, k, v, early_reads, s);
}

template <typename T, int D>
static cudaError_t append_many_t(const DeviceView& dv, int layer, const void* k, const void* v, int n_tok, int n_slices,
                                 cudaStream_t s) {
  if (n_slices > 0) {   // a long run: parallel over the tokens
    append_chunk_kernel<T, D><<<dim3(n_slices, dv.n_heads), 256, 0, s>>>(dv, layer, (const T*)k, (const T*)v, n_tok,
                                                                         n_slices);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    append_chunk_finalize_kernel<D><<<dv.n_heads, 2 * D, 0, s>>>(dv, layer, n_tok, n_slices);
    return cudaGetLastError();
  }
  const int warps = 4;
  return launch_dependent(append_many_kernel<T, D>, (dv.n_heads + warps - 1) / warps, warps * 32, s, dv, layer,
                          (const T*)k, (const T*)v, n_tok);
}

cudaError_t launch_append_many(const DeviceView& dv, int dtype, int layer, const void* k, const void* v, int n_tok,
                               int n_slices, cudaStream_t s) {
  if (dtype == RAZOR_BF16) {
    return dv.head_dim == 128 ? append_many_t<__nv_bfloat16, 128>(dv, layer, k, v, n_tok, n_slices, s)
                              : append_many_t<__nv_bfloat16, 64>(dv, layer, k, v, n_tok, n_slices, s);
  }
  return dv.head_dim == 128 ? append_many_t<float, 128>(dv, layer, k, v, n_tok, n_slices, s)
                            : append_many_t<float, 64>(dv, layer, k, v, n_tok, n_slices, s);
}

template <typename T, int D>
static cudaError_t export_t(const DeviceView& dv, int layer, int head, int32_t* kp, void* K, void* V, float* mk,
                            float* mv, float* sk, float* sv, cudaStream_t s) {
  export_kernel<T, D><<<64, 256, 0, s>>>(dv, layer, head, kp, (T*)K, (T*)V, mk, mv, sk, sv);
  return cudaGetLastError();
}

cudaError_t launch_export(const DeviceView& dv, int dtype, int layer, int head, int32_t* kp, void* K, void* V,
                          float* mk, float* mv, float* sk, float* sv, cudaStream_t s) {
  if (dtype == RAZOR_BF16) {
    return dv.head_dim == 128 ? export_t<__nv_bfloat16, 128>(dv, layer, head, kp, K, V, mk, mv, sk, sv, s)
                              : export_t<__nv_bfloat16, 64>(dv, layer, head, kp, K, V, mk, mv, sk, sv, s);
  }
  return dv.head_dim == 128 ? export_t<float, 128>(dv, layer, head, kp, K, V, mk, mv, sk, sv, s)
                            : export_t<float, 64>(dv, layer, head, kp, K, V, mk, mv, sk, sv, s);
}

}  // namespace razor
