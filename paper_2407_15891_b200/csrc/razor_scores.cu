// Retrieval-head identification (Section 3.3), the part that is pure arithmetic: given a head's queries
// and keys on a sequence of `period` random tokens repeated several times, the echo score (attention
// weight on the earlier copies of the current token, positions m - j*period) and the induction score
// (weight on the tokens right after them, m - j*period + 1), averaged over the queries m >= period.
//
// The weights need the causal softmax denominator of every query over all earlier keys: an N x N score
// matrix per head.  That is a dense contraction, so it runs on the tensor cores: tcgen05.mma with both
// operands in shared memory and the 128 x 128 fp32 score tile in tensor memory.
//
// A CTA owns 128 queries of one head (the rows of the accumulator, one per tensor-memory lane) and walks
// the key tiles up to its own diagonal.  Three roles, connected by mbarriers:
//   * one thread issues the TMA copies: the query tile once, then 128 keys at a time into one of two
//     shared-memory stages.  The tensor map's 128-byte swizzle puts them in the layout the matrix unit
//     reads (rows of 128 bytes, eight rows to a 1 KB group, 16-byte chunks XOR-swizzled by the row
//     number within the group; a row of D = 128 elements is two such half rows, one box each), and
//     rows beyond the sequence arrive as zeros;
//   * one thread issues the D / 16 matrix instructions of a tile (K = 16 each) into one of two
//     accumulator buffers and commits them onto the barriers that free the stage and publish the tile;
//   * eight SOFTMAX warps read the tile out of tensor memory: warps w and w + 4 share lanes
//     32 (w % 4) .. + 31, i.e. 32 queries, and take one half of the 128 columns each, so a thread sees
//     half a row of its query and keeps a running max and sum without shuffles; the two halves are
//     merged once at the end.  Only the diagonal tile needs the causal mask.
// The denominators go to scratch; a second, small kernel computes the handful of target logits per query
// as plain dot products and sums the weights per block; the blocks are added in a fixed order (reproducible).
//
// Every barrier wait is bounded in time; a wait that runs out makes the CTA leave through the common
// exit (copies in flight are waited for, tensor memory is always released) and sets a flag in scratch,
// which turns the scores into NaN.
#include <cuda.h>
#include <math_constants.h>

#include "razor_common.cuh"
#include "razor_sync.cuh"
#include "razor_tc.cuh"

namespace razor {
namespace {

constexpr int kQTile = 128;         // queries per CTA = accumulator rows = tensor-memory lanes
constexpr int kKTile = 128;         // keys per tile = accumulator columns
constexpr int kStages = 2;          // key stages in shared memory and accumulator buffers in tensor memory
constexpr int kSoftmaxWarps = 8;    // warp w: lanes 32 (w % 4) .. + 31, columns 64 (w / 4) .. + 63
constexpr int kCopyWarp = kSoftmaxWarps, kMmaWarp = kSoftmaxWarps + 1;
constexpr int kScoreWarps = kSoftmaxWarps + 2;
constexpr int kScoreThreads = kScoreWarps * 32;
constexpr uint32_t kTmemCols = kStages * kKTile;   // a power of two >= 32
constexpr int kHalfRowBytes = 128;                 // one swizzle row: 64 bf16
constexpr int kHalfTileBytes = 128 * kHalfRowBytes;

// Barriers and small exchange areas behind the tiles.
struct ScoreCtl {
  uint64_t q_full;             // copy -> MMA: the query tile has landed
  uint64_t k_full[kStages];    // copy -> MMA: the stage holds its keys
  uint64_t k_empty[kStages];   // MMA (commit) -> copy: the stage has been read
  uint64_t t_full[kStages];    // MMA (commit) -> softmax: the accumulator buffer holds a tile
  uint64_t t_empty[kStages];   // softmax -> MMA: the buffer has been read out
  uint64_t drain;              // abort path: MMAs in flight have finished
  uint32_t tmem_base;
  int abort_flag;
  float2 half_ml[kQTile];      // (max, sum) of the upper column half, for the merge
};

template <int D>
__host__ __device__ constexpr int score_tile_bytes() { return (D / 64) * kHalfTileBytes; }
template <int D>
constexpr size_t score_smem_bytes() {
  // 1 KB of slack to align the tiles; at least 80 KB so that no more than two CTAs share an SM and
  // their accumulators (kTmemCols columns each) always fit the 512 columns of tensor memory
  const size_t need = 1024 + (size_t)(1 + kStages) * score_tile_bytes<D>() + sizeof(ScoreCtl);
  return need < 80 * 1024 ? 80 * 1024 : need;
}

// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, N / 8 at bit 17, M / 16 at bit 24.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kKTile >> 3) << 17) |
                                ((uint32_t)(kQTile >> 4) << 24);

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t accumulate) {
  umma_bf16_desc(tmem_d, desc_a, desc_b, kInstrDesc, accumulate);
}
// The transcendental unit is the busiest pipe of this kernel (one ex2 per score), so of every kPolyEvery pairs of
// exponentials one pair is computed as a polynomial on the FMA and integer pipes instead (f2_exp2_poly).
constexpr int kPolyEvery = 3;

// Completes the loads issued so far.  The registers pass through the statement so that no use of them
// can be scheduled ahead of it.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&v)[64]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int j = 0; j < 64; ++j) asm volatile("" : "+r"(v[j]));
}

// One box of the [heads][tokens][D] tensor (64 elements x 128 rows of one head) into shared memory;
// completion is counted in bytes on `bar`.  x is a multiple of 64 elements, i.e. of 128 bytes.
__device__ __forceinline__ void tma_load_box(void* dst, const CUtensorMap* map, int x, int row, int head, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::
          "r"(smem_u32(dst)),
      "l"(map), "r"(x), "r"(row), "r"(head), "r"(smem_u32(bar))
      : "memory");
}
template <int D>
__device__ __forceinline__ void tma_load_tile(uint8_t* tile, const CUtensorMap* map, int row0, int head, uint64_t* bar) {
  mbar_arrive_expect_tx(bar, (uint32_t)score_tile_bytes<D>());
#pragma unroll
  for (int h = 0; h < D / 64; ++h) tma_load_box(tile + h * kHalfTileBytes, map, h * 64, row0, head, bar);
}

// grid = (heads, query tiles), block = kScoreThreads.  Writes lse[head][m], the log2 of the causal softmax
// denominator of query m (scaled logits in the log2 domain); *fault is set when a wait gave up.
template <int D>
__global__ void __launch_bounds__(kScoreThreads, 2)
    head_lse_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, int n_tokens,
                    int period, float scale_log2, float* __restrict__ lse, int* fault) {
  constexpr int TB = score_tile_bytes<D>();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  uint8_t* qtile = base;
  uint8_t* ktile = base + TB;
  ScoreCtl* ctl = (ScoreCtl*)(base + (1 + kStages) * TB);

  // Heads vary fastest in the launch order: the longest row of the triangle of every head first, then the next
  // one of every head, so that the grid ends on the short rows.
  const int head = blockIdx.x, n_tiles = gridDim.y;
  const int tile = n_tiles - 1 - (int)blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = tile * kQTile;
  if (q0 + kQTile <= period) return;   // none of these queries has an earlier copy of its token
  volatile int* abort_flag = &ctl->abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&ctl->q_full, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&ctl->k_full[s], 1);
      mbar_init(&ctl->k_empty[s], 1);
      mbar_init(&ctl->t_full[s], 1);
      mbar_init(&ctl->t_empty[s], kSoftmaxWarps * 32);
    }
    mbar_init(&ctl->drain, 1);
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {   // the MMA warp owns the tensor-memory allocation
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  const int n_kt = tile + 1;   // key tiles up to and including the diagonal

  if (warp < kSoftmaxWarps) {
    // ---- softmax: query q0 + row, columns [col0, col0 + 64) of every tile
    const int row = (warp & 3) * 32 + lane, col0 = (warp >> 2) * 64;
    float m_run = -CUDART_INF_F, l_run = 0.f;
    const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)col0;
    for (int kt = 0; kt < n_kt; ++kt) {
      const int b = kt & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(&ctl->t_full[b], (kt >> 1) & 1, abort_flag))) break;
      tc_fence_after();
      uint32_t v[64];
      tmem_ld32_issue(lane_addr + (uint32_t)(b * kKTile), v);
      tmem_ld32_issue(lane_addr + (uint32_t)(b * kKTile + 32), v + 32);
      tmem_ld_wait(v);
      tc_fence_before();
      mbar_arrive(&ctl->t_empty[b]);   // the buffer is in registers: hand it back
      if (kt == tile) {   // causality: key q0 + column against query q0 + row
#pragma unroll
        for (int j = 0; j < 64; ++j)
          if (col0 + j > row) v[j] = 0xff800000u;   // -inf
      }
      float mx[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
      for (int j = 0; j < 64; j += 2) mx[(j >> 1) & 3] = max3(mx[(j >> 1) & 3], __uint_as_float(v[j]), __uint_as_float(v[j + 1]));
      // the scale is positive, so the max of the scaled logits is the scaled max
      const float tile_max = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale_log2;
      const float mn = fmaxf(m_run, tile_max);
      const float mu = (mn == -CUDART_INF_F) ? 0.f : mn;   // a fully masked half row so far
      // two scores per instruction: scale and subtract, exponentials, sums
      const uint64_t scale2 = f2_pack(scale_log2, scale_log2), neg_mu2 = f2_pack(-mu, -mu);
      uint64_t sum2[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) sum2[k] = f2_pack(0.f, 0.f);
#pragma unroll
      for (int j = 0; j < 64; j += 2) {
        const uint64_t t2 = f2_fma(f2_pack(__uint_as_float(v[j]), __uint_as_float(v[j + 1])), scale2, neg_mu2);
        uint64_t w2;
        if ((j >> 1) % kPolyEvery == kPolyEvery - 1) {
          w2 = f2_exp2_poly(t2);
        } else {
          float t0, t1;
          f2_unpack(t2, t0, t1);
          w2 = f2_pack(fast_exp2(t0), fast_exp2(t1));
        }
        sum2[(j >> 1) & 3] = f2_add(sum2[(j >> 1) & 3], w2);
      }
      float sum[4];
      {
        float a0, a1, b0, b1;
        f2_unpack(f2_add(sum2[0], sum2[1]), a0, a1);
        f2_unpack(f2_add(sum2[2], sum2[3]), b0, b1);
        sum[0] = a0; sum[1] = a1; sum[2] = b0; sum[3] = b1;
      }
      l_run = l_run * fast_exp2(m_run - mu) + ((sum[0] + sum[1]) + (sum[2] + sum[3]));
      m_run = mn;
    }
    if (col0) ctl->half_ml[row] = make_float2(m_run, l_run);
    asm volatile("bar.sync 1, %0;" ::"n"(kSoftmaxWarps * 32) : "memory");   // the softmax warps only
    if (!col0 && q0 + row < n_tokens) {
      const float2 o = ctl->half_ml[row];
      const float mn = fmaxf(m_run, o.x);   // finite: column 0 of tile 0 is never masked
      const float l = l_run * fast_exp2(m_run - mn) + o.y * fast_exp2(o.x - mn);
      lse[(size_t)head * n_tokens + q0 + row] = mn + log2f(l);
    }
  } else if (warp == kCopyWarp) {
    // ---- TMA issue: one thread
    if (lane == 0) {
      tma_load_tile<D>(qtile, &map_q, q0, head, &ctl->q_full);
      int issued = 0;
      for (int kt = 0; kt < n_kt; ++kt) {
        const int s = kt & 1;
        if (kt >= kStages && !mbar_wait(&ctl->k_empty[s], ((kt >> 1) - 1) & 1, abort_flag)) break;
        tma_load_tile<D>(ktile + s * TB, &map_k, kt * kKTile, head, &ctl->k_full[s]);
        issued = kt + 1;
      }
      if (*abort_flag) {   // leaving early: the copies in flight must land before the CTA may exit
        (void)mbar_wait_drain(&ctl->q_full, 0);
        for (int kt = max(0, issued - kStages); kt < issued; ++kt) (void)mbar_wait_drain(&ctl->k_full[kt & 1], (kt >> 1) & 1);
      }
    }
    __syncwarp();
  } else {
    // ---- MMA issue: one thread
    if (lane == 0) {
      bool ok = mbar_wait(&ctl->q_full, 0, abort_flag);
      for (int kt = 0; kt < n_kt && ok; ++kt) {
        const int s = kt & 1;
        ok = mbar_wait(&ctl->k_full[s], (kt >> 1) & 1, abort_flag);
        if (ok && kt >= kStages) ok = mbar_wait(&ctl->t_empty[s], ((kt >> 1) - 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a0 = smem_u32(qtile), b0 = smem_u32(ktile + s * TB);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {   // 16 elements = 32 bytes along the swizzled half row
          const uint32_t off = (uint32_t)((kk >> 2) * kHalfTileBytes + (kk & 3) * 32);
          umma_bf16(tmem + (uint32_t)(s * kKTile), operand_desc(a0 + off), operand_desc(b0 + off), kk > 0);
        }
        umma_commit(&ctl->k_empty[s]);
        umma_commit(&ctl->t_full[s]);
      }
      if (!ok) {   // leaving early: let the instructions in flight finish before tensor memory is released
        umma_commit(&ctl->drain);
        (void)mbar_wait_drain(&ctl->drain, 0);
      }
    }
    __syncwarp();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
  if (*abort_flag && threadIdx.x == 0) atomicOr(fault, 1);
}

// E = 4 or 8 consecutive bf16 (8 or 16 bytes, aligned) as floats.
template <int E>
__device__ __forceinline__ void load_bf16(const __nv_bfloat16* p, float (&f)[E]) {
  static_assert(E == 4 || E == 8, "one 8- or 16-byte load");
  uint32_t w[E / 2];
  if constexpr (E == 8) {
    const uint4 u = __ldg((const uint4*)p);
    w[0] = u.x; w[1] = u.y; w[2] = u.z; w[3] = u.w;
  } else {
    const uint2 u = __ldg((const uint2*)p);
    w[0] = u.x; w[1] = u.y;
  }
#pragma unroll
  for (int i = 0; i < E / 2; ++i) {   // bf16 -> fp32 is a 16-bit shift
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

constexpr int kTargetQueries = 64;   // queries per CTA of the target kernel (8 warps x 8 queries)

// The handful of target logits per query, as plain dot products, turned into attention weights with the
// denominators from head_lse_kernel.  A warp takes a query and one earlier copy of its token at a time:
// its lower 16 lanes hold the copy's key (echo), its upper 16 lanes the key after it (induction), each
// lane D / 16 elements.  grid = (ceil(n_tokens / 64), heads), block = 256;
// partial[(head * n_blocks + block) * 2 + {0: echo, 1: induction}] = the block's sums of weights.
template <int D>
__global__ void __launch_bounds__(256) head_targets_kernel(const __nv_bfloat16* __restrict__ Q,
                                                           const __nv_bfloat16* __restrict__ K,
                                                           const float* __restrict__ lse, int n_tokens, int period,
                                                           float scale_log2, float* __restrict__ partial) {
  constexpr int E = D / 16;   // elements per lane
  __shared__ float red[8][2];
  const int head = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kind = lane >> 4, l16 = lane & 15;
  const __nv_bfloat16* Qh = Q + (size_t)head * n_tokens * D;
  const __nv_bfloat16* Kh = K + (size_t)head * n_tokens * D;
  // The warp's 8 queries are consecutive, so are their targets in every earlier period: one batch of 8
  // independent row loads per period.
  const int m0 = (int)blockIdx.x * kTargetQueries + warp * 8;
  float qf[8][E], lse_m[8];
#pragma unroll
  for (int qi = 0; qi < 8; ++qi) {
    const int m = min(m0 + qi, n_tokens - 1);
    load_bf16<E>(Qh + (size_t)m * D + l16 * E, qf[qi]);
    lse_m[qi] = lse[(size_t)head * n_tokens + m];
  }
  float acc = 0.f;
  for (int c0 = m0 - period; c0 + 7 >= 0; c0 -= period) {   // c0 + qi: the copy of query m0 + qi's token
    float dot[8];
#pragma unroll
    for (int qi = 0; qi < 8; ++qi) {
      const int c = max(c0 + qi, 0);   // clamped rows are discarded below; c + kind <= m - period + 1
      float kf[E];
      load_bf16<E>(Kh + (size_t)(c + kind) * D + l16 * E, kf);
      dot[qi] = 0.f;
#pragma unroll
      for (int e = 0; e < E; ++e) dot[qi] = fmaf(qf[qi][e], kf[e], dot[qi]);
    }
#pragma unroll
    for (int off = 8; off > 0; off >>= 1)
#pragma unroll
      for (int qi = 0; qi < 8; ++qi) dot[qi] += __shfl_xor_sync(0xffffffffu, dot[qi], off);
#pragma unroll
    for (int qi = 0; qi < 8; ++qi)
      if (c0 + qi >= 0 && m0 + qi < n_tokens) acc += fast_exp2(dot[qi] * scale_log2 - lse_m[qi]);
  }
  if (l16 == 0) red[warp][kind] = acc;
  __syncthreads();
  if (threadIdx.x < 2) {
    float sum = 0.f;
    for (int w = 0; w < 8; ++w) sum += red[w][threadIdx.x];
    partial[((size_t)head * gridDim.x + blockIdx.x) * 2 + threadIdx.x] = sum;
  }
}

// grid = heads, block = 32: the blocks' sums added, then the mean over the queries m >= period.
// A launch in which some wait gave up has no valid partial sums: its scores are NaN.
__global__ void head_scores_finalize_kernel(const float* __restrict__ scratch, const int* __restrict__ fault,
                                            int n_blocks, int n_queries, float* __restrict__ echo,
                                            float* __restrict__ induction) {
  const int lane = threadIdx.x;
  const float* src = scratch + (size_t)blockIdx.x * n_blocks * 2;
  float e = 0.f, i = 0.f;
  for (int b = lane; b < n_blocks; b += 32) {   // lane-strided, then a fixed tree: the same order every run
    e += src[2 * b];
    i += src[2 * b + 1];
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    e += __shfl_xor_sync(0xffffffffu, e, off);
    i += __shfl_xor_sync(0xffffffffu, i, off);
  }
  if (lane == 0) {
    const bool bad = *fault != 0;
    echo[blockIdx.x] = bad ? CUDART_NAN_F : (n_queries > 0 ? e / (float)n_queries : 0.f);
    induction[blockIdx.x] = bad ? CUDART_NAN_F : (n_queries > 0 ? i / (float)n_queries : 0.f);
  }
}

// Tensor map of X[n_heads][n_tokens][D] bf16 with boxes of 64 elements x 128 rows of one head, written
// to shared memory with the 128-byte swizzle; rows beyond n_tokens read as zeros.
template <int D>
bool make_tile_map(CUtensorMap* map, const void* X, int n_heads, int n_tokens) {
  const EncodeTiledFn encode = encode_tiled_fn();
  if (!encode) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)n_tokens, (cuuint64_t)n_heads};
  const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)n_tokens * D * 2};   // bytes, dimensions 1 and 2
  const cuuint32_t box[3] = {64, 128, 1};
  const cuuint32_t elem_strides[3] = {1, 1, 1};
  return encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(X), dims, strides, box, elem_strides,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
cudaError_t run_head_scores(const void* Q, const void* K, int n_heads, int n_tokens, int period, float scale_log2,
                            float* echo, float* induction, float* partial, float* lse, int* fault, cudaStream_t s) {
  const int tiles = (n_tokens + kQTile - 1) / kQTile, blocks = (n_tokens + kTargetQueries - 1) / kTargetQueries;
  CUtensorMap map_q, map_k;
  if (!make_tile_map<D>(&map_q, Q, n_heads, n_tokens) || !make_tile_map<D>(&map_k, K, n_heads, n_tokens))
    return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(head_lse_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)score_smem_bytes<D>());
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(fault, 0, sizeof(int), s);
  if (e != cudaSuccess) return e;
  head_lse_kernel<D><<<dim3(n_heads, tiles), kScoreThreads, score_smem_bytes<D>(), s>>>(map_q, map_k, n_tokens, period,
                                                                                        scale_log2, lse, fault);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  head_targets_kernel<D><<<dim3(blocks, n_heads), 256, 0, s>>>((const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, lse,
                                                              n_tokens, period, scale_log2, partial);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  head_scores_finalize_kernel<<<n_heads, 32, 0, s>>>(partial, fault, blocks, n_tokens - period, echo, induction);
  return cudaGetLastError();
}

}  // namespace
}  // namespace razor

namespace {
// Scratch layout: per-block partial sums | lse[n_heads][n_tokens] | fault word.
size_t partial_bytes(int n_heads, int n_tokens) {
  const size_t blocks = ((size_t)n_tokens + razor::kTargetQueries - 1) / razor::kTargetQueries;
  return ((size_t)n_heads * blocks * 2 * sizeof(float) + 255) / 256 * 256;
}
size_t lse_bytes(int n_heads, int n_tokens) {
  return ((size_t)n_heads * (size_t)n_tokens * sizeof(float) + 255) / 256 * 256;
}
}  // namespace

extern "C" int razor_head_scores_scratch_bytes(int32_t n_heads, int32_t n_tokens, size_t* bytes) {
  if (!bytes) return RAZOR_E_NULL_PTR;
  if (n_heads < 1 || n_tokens < 1) return RAZOR_E_INVALID_ARG;
  *bytes = partial_bytes(n_heads, n_tokens) + lse_bytes(n_heads, n_tokens) + 256;
  return RAZOR_OK;
}

extern "C" int razor_head_scores(const void* Q, const void* K, int32_t n_heads, int32_t n_tokens, int32_t head_dim,
                                 int32_t dtype, int32_t period, float sm_scale, float* echo, float* induction,
                                 void* scratch, size_t scratch_bytes, void* stream) {
  using namespace razor;
  if (!Q || !K || !echo || !induction || !scratch) return RAZOR_E_NULL_PTR;
  if (n_heads < 1 || n_heads > 65535 || n_tokens < 2 || period < 2 || period >= n_tokens) return RAZOR_E_INVALID_ARG;
  if (n_tokens > 65535 * razor::kQTile) return RAZOR_E_CAPACITY;   // query tiles are a grid y dimension
  if (!(sm_scale >= 0.f)) return RAZOR_E_INVALID_ARG;
  if (dtype != RAZOR_BF16 || (head_dim != 64 && head_dim != 128)) return RAZOR_E_UNSUPPORTED_DIM;
  if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)scratch) & 15) return RAZOR_E_MISALIGNED;
  size_t need = 0;
  razor_head_scores_scratch_bytes(n_heads, n_tokens, &need);
  if (scratch_bytes < need) return RAZOR_E_POOL_TOO_SMALL;
  const float scale = sm_scale == 0.f ? 1.0f / sqrtf((float)head_dim) : sm_scale;
  const float scale_log2 = scale * 1.4426950408889634f;
  float* partial = (float*)scratch;
  float* lse = (float*)((uint8_t*)scratch + partial_bytes(n_heads, n_tokens));
  int* fault = (int*)((uint8_t*)lse + lse_bytes(n_heads, n_tokens));
  cudaStream_t s = (cudaStream_t)stream;
  const cudaError_t e =
      head_dim == 128 ? run_head_scores<128>(Q, K, n_heads, n_tokens, period, scale_log2, echo, induction, partial, lse, fault, s)
                      : run_head_scores<64>(Q, K, n_heads, n_tokens, period, scale_log2, echo, induction, partial, lse, fault, s);
  if (e != cudaSuccess) {
    razor::note_cuda_error(e);   // razor_last_cuda_error() reports it
    return RAZOR_E_CUDA;
  }
  return RAZOR_OK;
}

extern "C" int razor_select_retrieval_heads(const float* echo, const float* induction, int32_t n_heads,
                                            float frac_induction, float frac_echo, uint8_t* mask) {
  if (!echo || !induction || !mask) return RAZOR_E_NULL_PTR;
  if (n_heads < 1 || !(frac_induction >= 0.f && frac_induction <= 1.f) || !(frac_echo >= 0.f && frac_echo <= 1.f))
    return RAZOR_E_INVALID_ARG;
  auto top = [&](const float* score, float frac) {
    int k = (int)lrintf(frac * (float)n_heads);
    if (k < 1) k = 1;
    if (k > n_heads) k = n_heads;
    for (int pick = 0; pick < k; ++pick) {   // selection by repeated maximum: ties go to the lower index
      int best = -1;
      for (int h = 0; h < n_heads; ++h)
        if (!(mask[h] & 2) && (best < 0 || score[h] > score[best])) best = h;
      mask[best] |= 3;
    }
    for (int h = 0; h < n_heads; ++h) mask[h] &= 1;   // bit 1 marked "taken in this pass"
  };
  for (int h = 0; h < n_heads; ++h) mask[h] = 0;
  top(induction, frac_induction);
  top(echo, frac_echo);
  return RAZOR_OK;
}
