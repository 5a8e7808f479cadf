// Retrieval-head identification (Section 3.3), the part that is pure arithmetic: given a head's queries
// and keys on a sequence of `period` random tokens repeated several times, the echo score (attention
// weight on the earlier copies of the current token, positions m - j*period) and the induction score
// (weight on the tokens right after them, m - j*period + 1), averaged over the queries m >= period.
//
// The weights need the causal softmax denominator of every query over all earlier keys: an N x N score
// matrix per head.  That is a dense contraction, so it runs on warp-level matrix instructions
// (m16n8k16, bf16 in, fp32 out): a CTA takes 64 queries, stages the keys 64 at a time in shared memory
// (rows chunk-swizzled so that the fragment loads are conflict-free), and each warp keeps the running
// max / sum of its 8 queries.  The handful of target logits per query are then plain dot products.
// Per-CTA partial sums go to caller-provided scratch and are added in a fixed order (reproducible).
#include <math_constants.h>

#include "razor_common.cuh"

namespace razor {
namespace {

constexpr int kQTile = 64;   // queries per CTA (8 warps x 8 queries)
constexpr int kKTile = 64;   // keys staged per step

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// grid = (query tiles, heads), block = 256.  scratch[(head * n_tiles + tile) * 2 + {0: echo, 1: induction}].
template <int D>
__global__ void __launch_bounds__(256) head_scores_kernel(const __nv_bfloat16* __restrict__ Q,
                                                          const __nv_bfloat16* __restrict__ K, int n_tokens, int period,
                                                          float scale_log2, float* __restrict__ scratch) {
  constexpr int CH = D * 2 / 16;   // 16-byte chunks per row
  __shared__ __align__(128) uint8_t ktile[kKTile * D * 2];
  __shared__ float red[8][2];
  const int head = blockIdx.y, tile = blockIdx.x, n_tiles = gridDim.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int q0 = tile * kQTile, qw0 = q0 + warp * 8;
  const __nv_bfloat16* Qh = Q + (size_t)head * n_tokens * D;
  const __nv_bfloat16* Kh = K + (size_t)head * n_tokens * D;
  float* dst = scratch + ((size_t)head * n_tiles + tile) * 2;
  if (q0 + kQTile <= period) {   // none of these queries has an earlier copy of its token
    if (threadIdx.x == 0) dst[0] = dst[1] = 0.f;
    return;
  }
  // B fragments: query qw0 + g of this warp
  uint32_t qb[D / 16][2];
#pragma unroll
  for (int kk = 0; kk < D / 16; ++kk) {
    qb[kk][0] = qb[kk][1] = 0u;
    if (qw0 + g < n_tokens) {
      const uint32_t* qrow = (const uint32_t*)(Qh + (size_t)(qw0 + g) * D);
      qb[kk][0] = qrow[kk * 8 + t];
      qb[kk][1] = qrow[kk * 8 + 4 + t];
    }
  }
  // running softmax (log2 domain) of this lane's queries qa = qw0 + 2t and qa + 1
  const int qa = qw0 + 2 * t;
  float m0 = -CUDART_INF_F, m1 = -CUDART_INF_F, l0 = 0.f, l1 = 0.f;
  const int last_key = min(n_tokens, q0 + kQTile) - 1;   // causal limit of the CTA
  const int r8 = lane & 7, mi = lane >> 3;
  for (int k0 = 0; k0 <= last_key; k0 += kKTile) {
    __syncthreads();   // the previous tile has been consumed
    for (int idx = threadIdx.x; idx < kKTile * CH; idx += 256) {
      const int r = idx / CH, c = idx % CH;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (k0 + r < n_tokens) v = ((const uint4*)(Kh + (size_t)(k0 + r) * D))[c];
      ((uint4*)ktile)[r * CH + (c ^ (r & 7))] = v;
    }
    __syncthreads();
    for (int p = 0; p < kKTile / 16; ++p) {
      const int kbase = k0 + p * 16;
      if (kbase > qw0 + 7) break;   // beyond this warp's last query
      float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
      const uint32_t row_addr = smem_addr(ktile) + (p * 16 + ((mi & 1) << 3) + r8) * (D * 2);
#pragma unroll
      for (int kk = 0; kk < D / 16; ++kk) {
        uint32_t a[4];
        ldsm_x4(a, row_addr + (((2 * kk + (mi >> 1)) ^ r8) << 4));
        if (kk & 1) mma_16816(s1, a, qb[kk][0], qb[kk][1]);
        else mma_16816(s0, a, qb[kk][0], qb[kk][1]);
      }
      // s[0], s[1]: key kbase + g against queries qa, qa + 1;  s[2], s[3]: key kbase + g + 8
      float s[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) s[i] = (s0[i] + s1[i]) * scale_log2;
      const int ka = kbase + g, kb = ka + 8;
      if (ka > qa) s[0] = -CUDART_INF_F;   // causality (keys beyond the sequence are beyond every query too)
      if (ka > qa + 1) s[1] = -CUDART_INF_F;
      if (kb > qa) s[2] = -CUDART_INF_F;
      if (kb > qa + 1) s[3] = -CUDART_INF_F;
      float mx0 = fmaxf(s[0], s[2]), mx1 = fmaxf(s[1], s[3]);
#pragma unroll
      for (int off = 4; off < 32; off <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
      }
      const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
      const float mu0 = (mn0 == -CUDART_INF_F) ? 0.f : mn0, mu1 = (mn1 == -CUDART_INF_F) ? 0.f : mn1;
      l0 = l0 * fast_exp2(m0 - mu0) + fast_exp2(s[0] - mu0) + fast_exp2(s[2] - mu0);
      l1 = l1 * fast_exp2(m1 - mu1) + fast_exp2(s[1] - mu1) + fast_exp2(s[3] - mu1);
      m0 = mn0;
      m1 = mn1;
    }
  }
#pragma unroll
  for (int off = 4; off < 32; off <<= 1) {
    l0 += __shfl_xor_sync(0xffffffffu, l0, off);
    l1 += __shfl_xor_sync(0xffffffffu, l1, off);
  }
  const float lse0 = m0 + log2f(l0), lse1 = m1 + log2f(l1);   // log2 of the softmax denominators
  // The target logits: a few plain dot products per query, lanes splitting the head dimension.
  constexpr int PER = D / 32;
  float echo = 0.f, induction = 0.f;
  for (int qi = 0; qi < 8; ++qi) {
    const int m = qw0 + qi;
    const float lse = __shfl_sync(0xffffffffu, (qi & 1) ? lse1 : lse0, qi >> 1);   // lane (g = 0, t = qi / 2)
    if (m < period || m >= n_tokens) continue;   // warp-uniform
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
    red[warp][0] = echo;
    red[warp][1] = induction;
  }
  __syncthreads();
  if (threadIdx.x < 2) {
    float sum = 0.f;
    for (int w = 0; w < 8; ++w) sum += red[w][threadIdx.x];
    dst[threadIdx.x] = sum;
  }
}

// grid = heads, block = 32: tiles added in order, then the mean over the queries m >= period.
__global__ void head_scores_finalize_kernel(const float* __restrict__ scratch, int n_tiles, int n_queries,
                                            float* __restrict__ echo, float* __restrict__ induction) {
  if (threadIdx.x >= 2) return;
  const float* src = scratch + (size_t)blockIdx.x * n_tiles * 2 + threadIdx.x;
  float s = 0.f;
  for (int i = 0; i < n_tiles; ++i) s += src[(size_t)i * 2];
  const float mean = n_queries > 0 ? s / (float)n_queries : 0.f;
  (threadIdx.x == 0 ? echo : induction)[blockIdx.x] = mean;
}

}  // namespace
}  // namespace razor

extern "C" int razor_head_scores_scratch_bytes(int32_t n_heads, int32_t n_tokens, size_t* bytes) {
  if (!bytes) return RAZOR_E_NULL_PTR;
  if (n_heads < 1 || n_tokens < 1) return RAZOR_E_INVALID_ARG;
  const size_t tiles = ((size_t)n_tokens + razor::kQTile - 1) / razor::kQTile;
  *bytes = ((size_t)n_heads * tiles * 2 * sizeof(float) + 255) / 256 * 256;
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
  if (((uintptr_t)Q | (uintptr_t)K) & 15) return RAZOR_E_MISALIGNED;
  size_t need = 0;
  razor_head_scores_scratch_bytes(n_heads, n_tokens, &need);
  if (scratch_bytes < need) return RAZOR_E_POOL_TOO_SMALL;
  const float scale = sm_scale == 0.f ? 1.0f / sqrtf((float)head_dim) : sm_scale;
  const int tiles = (n_tokens + kQTile - 1) / kQTile;
  const dim3 grid(tiles, n_heads);
  cudaStream_t s = (cudaStream_t)stream;
  if (head_dim == 128)
    head_scores_kernel<128><<<grid, 256, 0, s>>>((const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, n_tokens, period,
                                                 scale * 1.4426950408889634f, (float*)scratch);
  else
    head_scores_kernel<64><<<grid, 256, 0, s>>>((const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, n_tokens, period,
                                                scale * 1.4426950408889634f, (float*)scratch);
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) {
    head_scores_finalize_kernel<<<n_heads, 32, 0, s>>>((const float*)scratch, tiles, n_tokens - period, echo, induction);
    e = cudaGetLastError();
  }
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
