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
//   * four LOADER warps copy the next 128 keys into one of two shared-memory stages, in the layout the
//     matrix unit reads (rows of 128 bytes, eight rows to a 1 KB group, 16-byte chunks XOR-swizzled
//     by the row number within the group; a row of D = 128 elements is two such half rows);
//   * one thread of the MMA warp issues the D / 16 instructions of a tile (K = 16 each) into one of two
//     accumulator buffers and commits them onto the barriers that free the stage and publish the tile;
//   * four SOFTMAX warps read the tile out of tensor memory, a thread per query: it sees its whole row,
//     so the running max and sum need no shuffles.  Only the diagonal tile needs the causal mask.
// The handful of target logits per query are then plain dot products.  Per-CTA partial sums go to
// caller-provided scratch and are added in a fixed order (reproducible).
//
// Every barrier wait is bounded in time; a wait that runs out makes the CTA leave through the common
// exit (tensor memory is always released) and sets a flag in scratch, which turns the scores into NaN.
#include <math_constants.h>

#include "razor_common.cuh"
#include "razor_sync.cuh"

namespace razor {
namespace {

constexpr int kQTile = 128;         // queries per CTA = accumulator rows = tensor-memory lanes
constexpr int kKTile = 128;         // keys per tile = accumulator columns
constexpr int kStages = 2;          // key stages in shared memory and accumulator buffers in tensor memory
constexpr int kSoftmaxWarps = 4;    // warp w reads tensor-memory lanes 32 w .. 32 w + 31
constexpr int kLoaderWarps = 4;
constexpr int kScoreWarps = kSoftmaxWarps + kLoaderWarps + 1;
constexpr int kScoreThreads = kScoreWarps * 32;
constexpr uint32_t kTmemCols = kStages * kKTile;   // a power of two >= 32
constexpr int kHalfRowBytes = 128;                 // one swizzle row: 64 bf16
constexpr int kHalfTileBytes = 128 * kHalfRowBytes;

// Barriers and small exchange areas behind the tiles.
struct ScoreCtl {
  uint64_t k_full[kStages];    // loaders -> MMA: the stage holds its keys
  uint64_t k_empty[kStages];   // MMA (commit) -> loaders: the stage has been read
  uint64_t t_full[kStages];    // MMA (commit) -> softmax: the accumulator buffer holds a tile
  uint64_t t_empty[kStages];   // softmax -> MMA: the buffer has been read out
  uint64_t drain;              // abort path: MMAs in flight have finished
  uint32_t tmem_base;
  int abort_flag;
  float lse[kQTile];           // log2 of each query's softmax denominator
  float red[kScoreWarps][2];
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

// Shared-memory matrix descriptor of a K-major operand in the 128-byte swizzled layout: start address
// and strides in 16-byte units; consecutive 8-row groups are 1 KB apart; descriptor version 1.
__device__ __forceinline__ uint64_t operand_desc(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, N / 8 at bit 17, M / 16 at bit 24.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kKTile >> 3) << 17) |
                                ((uint32_t)(kQTile >> 4) << 24);

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      :
      : "r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(kInstrDesc), "r"(accumulate)
      : "memory");
}
// Arrives on `bar` once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// 32 consecutive columns of this thread's lane, complete on return.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}

// Rows [row0, row0 + 128) of X[n_tokens][D] into a tile in the matrix unit's layout; rows beyond the
// sequence are zero.  Called by `n_thr` threads with ranks `t`.
template <int D>
__device__ __forceinline__ void stage_tile(uint8_t* tile, const __nv_bfloat16* __restrict__ X, int row0, int n_tokens,
                                           int t, int n_thr) {
  constexpr int CH = D / 8;   // 16-byte chunks per row
  for (int idx = t; idx < 128 * CH; idx += n_thr) {
    const int r = idx / CH, c = idx % CH;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row0 + r < n_tokens) v = ((const uint4*)(X + (size_t)(row0 + r) * D))[c];
    *(uint4*)(tile + (c >> 3) * kHalfTileBytes + r * kHalfRowBytes + (((c & 7) ^ (r & 7)) << 4)) = v;
  }
}

// grid = (query tiles, heads), block = kScoreThreads.
// scratch[(head * n_tiles + tile) * 2 + {0: echo, 1: induction}]; *fault is set when a wait gave up.
template <int D>
__global__ void __launch_bounds__(kScoreThreads, 2) head_scores_kernel(const __nv_bfloat16* __restrict__ Q,
                                                                       const __nv_bfloat16* __restrict__ K,
                                                                       int n_tokens, int period, float scale_log2,
                                                                       float* __restrict__ scratch, int* fault) {
  constexpr int TB = score_tile_bytes<D>();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  uint8_t* qtile = base;
  uint8_t* ktile = base + TB;
  ScoreCtl* ctl = (ScoreCtl*)(base + (1 + kStages) * TB);

  const int head = blockIdx.y, n_tiles = gridDim.x;
  const int tile = n_tiles - 1 - (int)blockIdx.x;   // the long rows of the triangle first
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = tile * kQTile;
  const __nv_bfloat16* Qh = Q + (size_t)head * n_tokens * D;
  const __nv_bfloat16* Kh = K + (size_t)head * n_tokens * D;
  float* dst = scratch + ((size_t)head * n_tiles + tile) * 2;
  if (q0 + kQTile <= period) {   // none of these queries has an earlier copy of its token
    if (threadIdx.x == 0) dst[0] = dst[1] = 0.f;
    return;
  }
  volatile int* abort_flag = &ctl->abort_flag;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&ctl->k_full[s], kLoaderWarps * 32);
      mbar_init(&ctl->k_empty[s], 1);
      mbar_init(&ctl->t_full[s], 1);
      mbar_init(&ctl->t_empty[s], kSoftmaxWarps * 32);
    }
    mbar_init(&ctl->drain, 1);
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kScoreWarps - 1) {   // the MMA warp owns the tensor-memory allocation
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  stage_tile<D>(qtile, Qh, q0, n_tokens, threadIdx.x, kScoreThreads);
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  const int n_kt = tile + 1;   // key tiles up to and including the diagonal

  if (warp < kSoftmaxWarps) {
    // ---- softmax: thread = query q0 + threadIdx.x, lane threadIdx.x of the accumulator
    const int row = threadIdx.x;
    float m_run = -CUDART_INF_F, l_run = 0.f;
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    for (int kt = 0; kt < n_kt; ++kt) {
      const int b = kt & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(&ctl->t_full[b], (kt >> 1) & 1, abort_flag))) break;
      tc_fence_after();
      const bool diag = kt == tile;
#pragma unroll 1
      for (int c4 = 0; c4 < kKTile / 32; ++c4) {
        uint32_t v[32];
        tmem_ld32(lane_addr + (uint32_t)(b * kKTile + c4 * 32), v);
        if (c4 == kKTile / 32 - 1) {   // the buffer is in registers: hand it back
          tc_fence_before();
          mbar_arrive(&ctl->t_empty[b]);
        }
        float x[32];
        float mx = -CUDART_INF_F;
#pragma unroll
        for (int j = 0; j < 32; ++j) x[j] = __uint_as_float(v[j]) * scale_log2;
        if (diag) {   // causality: key q0 + column against query q0 + row
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (c4 * 32 + j > row) x[j] = -CUDART_INF_F;
        }
#pragma unroll
        for (int j = 0; j < 32; ++j) mx = fmaxf(mx, x[j]);
        const float mn = fmaxf(m_run, mx);   // finite: column 0 of tile 0 is never masked
        float sum = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) sum += fast_exp2(x[j] - mn);
        l_run = l_run * fast_exp2(m_run - mn) + sum;
        m_run = mn;
      }
    }
    ctl->lse[row] = m_run + log2f(l_run);
  } else if (warp < kSoftmaxWarps + kLoaderWarps) {
    // ---- loaders
    const int t = threadIdx.x - kSoftmaxWarps * 32;
    for (int kt = 0; kt < n_kt; ++kt) {
      const int s = kt & 1;
      if (kt >= kStages && !__all_sync(0xffffffffu, mbar_wait(&ctl->k_empty[s], ((kt >> 1) - 1) & 1, abort_flag)))
        break;
      stage_tile<D>(ktile + s * TB, Kh, kt * kKTile, n_tokens, t, kLoaderWarps * 32);
      fence_async_smem();
      mbar_arrive(&ctl->k_full[s]);
    }
  } else {
    // ---- MMA issue: one thread
    if (lane == 0) {
      bool ok = true;
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
  if (warp == kScoreWarps - 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
  if (*abort_flag) {
    if (threadIdx.x == 0) {
      atomicOr(fault, 1);
      dst[0] = dst[1] = 0.f;
    }
    return;
  }
  // ---- the target logits: a few plain dot products per query, lanes splitting the head dimension
  constexpr int PER = D / 32;
  float echo = 0.f, induction = 0.f;
  for (int qi = warp; qi < kQTile; qi += kScoreWarps) {
    const int m = q0 + qi;
    if (m < period || m >= n_tokens) continue;   // warp-uniform
    const float lse = ctl->lse[qi];
    float qv[PER];
#pragma unroll
    for (int e = 0; e < PER; ++e) qv[e] = __bfloat162float(Qh[(size_t)m * D + lane * PER + e]);
    for (int n = m - period; n >= 0; n -= period) {
      float de = 0.f, di = 0.f;
#pragma unroll
      for (int e = 0; e < PER; ++e) {
        de += qv[e] * __bfloat162float(Kh[(size_t)n * D + lane * PER + e]);
        di += qv[e] * __bfloat162float(Kh[(size_t)(n + 1) * D + lane * PER + e]);
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        de += __shfl_xor_sync(0xffffffffu, de, off);
        di += __shfl_xor_sync(0xffffffffu, di, off);
      }
      echo += fast_exp2(de * scale_log2 - lse);
      induction += fast_exp2(di * scale_log2 - lse);
    }
  }
  if (lane == 0) {
    ctl->red[warp][0] = echo;
    ctl->red[warp][1] = induction;
  }
  __syncthreads();
  if (threadIdx.x < 2) {
    float sum = 0.f;
    for (int w = 0; w < kScoreWarps; ++w) sum += ctl->red[w][threadIdx.x];
    dst[threadIdx.x] = sum;
  }
}

// grid = heads, block = 32: tiles added in order, then the mean over the queries m >= period.
// A launch in which some wait gave up has no valid partial sums: its scores are NaN.
__global__ void head_scores_finalize_kernel(const float* __restrict__ scratch, const int* __restrict__ fault,
                                            int n_tiles, int n_queries, float* __restrict__ echo,
                                            float* __restrict__ induction) {
  if (threadIdx.x >= 2) return;
  const float* src = scratch + (size_t)blockIdx.x * n_tiles * 2 + threadIdx.x;
  float s = 0.f;
  for (int i = 0; i < n_tiles; ++i) s += src[(size_t)i * 2];
  float mean = n_queries > 0 ? s / (float)n_queries : 0.f;
  if (*fault) mean = CUDART_NAN_F;
  (threadIdx.x == 0 ? echo : induction)[blockIdx.x] = mean;
}

template <int D>
cudaError_t run_head_scores(const void* Q, const void* K, int n_heads, int n_tokens, int period, float scale_log2,
                            float* echo, float* induction, float* partial, int* fault, cudaStream_t s) {
  const int tiles = (n_tokens + kQTile - 1) / kQTile;
  cudaError_t e = cudaFuncSetAttribute(head_scores_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)score_smem_bytes<D>());
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(fault, 0, sizeof(int), s);
  if (e != cudaSuccess) return e;
  head_scores_kernel<D><<<dim3(tiles, n_heads), kScoreThreads, score_smem_bytes<D>(), s>>>(
      (const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, n_tokens, period, scale_log2, partial, fault);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  head_scores_finalize_kernel<<<n_heads, 32, 0, s>>>(partial, fault, tiles, n_tokens - period, echo, induction);
  return cudaGetLastError();
}

}  // namespace
}  // namespace razor

namespace {
size_t partial_bytes(int n_heads, int n_tokens) {
  const size_t tiles = ((size_t)n_tokens + razor::kQTile - 1) / razor::kQTile;
  return ((size_t)n_heads * tiles * 2 * sizeof(float) + 255) / 256 * 256;
}
}  // namespace

extern "C" int razor_head_scores_scratch_bytes(int32_t n_heads, int32_t n_tokens, size_t* bytes) {
  if (!bytes) return RAZOR_E_NULL_PTR;
  if (n_heads < 1 || n_tokens < 1) return RAZOR_E_INVALID_ARG;
  *bytes = partial_bytes(n_heads, n_tokens) + 256;   // per-tile partial sums, then the fault word
  return RAZOR_OK;
}

extern "C" int razor_head_scores(const void* Q, const void* K, int32_t n_heads, int32_t n_tokens, int32_t head_dim,
                                 int32_t dtype, int32_t period, float sm_scale, float* echo, float* induction,
                                 void* scratch, size_t scratch_bytes, void* stream) {
  using namespace razor;
  if (!Q || !K || !echo || !induction || !scratch) return RAZOR_E_NULL_PTR;
  if (n_heads < 1 || n_heads > 65535 || n_tokens < 2 || period < 2 || period >= n_tokens) return RAZOR_E_INVALID_ARG;
  if (!(sm_scale >= 0.f)) return RAZOR_E_INVALID_ARG;
  if (dtype != RAZOR_BF16 || (head_dim != 64 && head_dim != 128)) return RAZOR_E_UNSUPPORTED_DIM;
  if (((uintptr_t)Q | (uintptr_t)K | (uintptr_t)scratch) & 15) return RAZOR_E_MISALIGNED;
  size_t need = 0;
  razor_head_scores_scratch_bytes(n_heads, n_tokens, &need);
  if (scratch_bytes < need) return RAZOR_E_POOL_TOO_SMALL;
  const float scale = sm_scale == 0.f ? 1.0f / sqrtf((float)head_dim) : sm_scale;
  const float scale_log2 = scale * 1.4426950408889634f;
  float* partial = (float*)scratch;
  int* fault = (int*)((uint8_t*)scratch + partial_bytes(n_heads, n_tokens));
  cudaStream_t s = (cudaStream_t)stream;
  const cudaError_t e =
      head_dim == 128 ? run_head_scores<128>(Q, K, n_heads, n_tokens, period, scale_log2, echo, induction, partial, fault, s)
                      : run_head_scores<64>(Q, K, n_heads, n_tokens, period, scale_log2, echo, induction, partial, fault, s);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
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
