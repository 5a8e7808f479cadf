// razor_compensation_mean_static: the compensation token of Eq. 4 for the heads of one sequence,
// computed without any caller-provided or library-allocated scratch memory.
//
// Who needs this: code that runs where device memory cannot be allocated or handed over - a plugin
// inside a host application that owns the allocator and gives out only its input and output
// tensors, a callback running while a stream is being captured, a process whose memory budget was
// fixed at start-up.  Such a caller cannot create the page pool and workspace the cache-building
// calls want, but it can still ask for the one quantity of the method that needs a reduction.
//
// The per-slice partial sums live in a file-scope device array of fixed size, so every GPU that loads
// this library carries that array (kScratchBytes) until the process exits.  All calls on a device
// share it: calls whose kernels overlap on the GPU (different streams) would overwrite each other's
// partial sums, so the caller must order them.  Nothing in the array has to start at zero - every
// slot the second kernel reads is written by the first kernel of the same call.
#include "razor_common.cuh"

namespace razor {
namespace {

constexpr int kStaticMaxHeads = 64;    // KV heads per call
constexpr int kStaticSlices = 32;      // row slices per head
constexpr int kStaticMaxDim = 128;
constexpr size_t kScratchFloats = (size_t)kStaticMaxHeads * kStaticSlices * 2 * kStaticMaxDim;   // 2 MiB

static __device__ __align__(256) float g_static_scratch[kScratchFloats];

// grid = (kStaticSlices, n_heads): sums of the K and V rows [r0, r1) of one slice of the dropped range.
template <typename T, int D>
__global__ void __launch_bounds__(256) static_slice_sum_kernel(const T* __restrict__ K, const T* __restrict__ V,
                                                               int64_t stride_h, int64_t stride_n, int first, int last,
                                                               float* __restrict__ scratch) {
  using Geo = RowGeom<T, D>;
  constexpr int LPR = Geo::kLpr, EPL = Geo::kEpl, NGRP = 256 / LPR;
  __shared__ float red[NGRP][2][D];
  const int n = last - first;
  const int per = (n + kStaticSlices - 1) / kStaticSlices;
  const int r0 = first + min(n, (int)blockIdx.x * per), r1 = first + min(n, ((int)blockIdx.x + 1) * per);
  const int lir = threadIdx.x % LPR, grp = threadIdx.x / LPR;
  const char* Kb = (const char*)(K + (size_t)blockIdx.y * stride_h);
  const char* Vb = (const char*)(V + (size_t)blockIdx.y * stride_h);
  const size_t row_stride = (size_t)stride_n * sizeof(T);
  float accK[EPL], accV[EPL];
#pragma unroll
  for (int i = 0; i < EPL; ++i) accK[i] = accV[i] = 0.f;
  for (int p = r0 + grp; p < r1; p += NGRP) {
    float a[EPL], b[EPL];
    Elem<T>::unpack(ld_stream((const uint4*)(Kb + (size_t)p * row_stride) + lir), a);
    Elem<T>::unpack(ld_stream((const uint4*)(Vb + (size_t)p * row_stride) + lir), b);
#pragma unroll
    for (int i = 0; i < EPL; ++i) { accK[i] += a[i]; accV[i] += b[i]; }
  }
#pragma unroll
  for (int i = 0; i < EPL; ++i) {
    red[grp][0][lir * EPL + i] = accK[i];
    red[grp][1][lir * EPL + i] = accV[i];
  }
  __syncthreads();
  float* dst = scratch + ((size_t)blockIdx.y * kStaticSlices + blockIdx.x) * 2 * D;
  for (int e = threadIdx.x; e < 2 * D; e += 256) {
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < NGRP; ++r) s += (&red[r][0][0])[e];
    dst[e] = s;
  }
}

// grid = n_heads, block = 2*D: slices added in a fixed order, then the division of Eq. 4.
template <int D>
__global__ void static_finalize_kernel(const float* __restrict__ scratch, int n_drop, float* __restrict__ mean_k,
                                       float* __restrict__ mean_v) {
  const int e = threadIdx.x;
  const float* src = scratch + (size_t)blockIdx.x * kStaticSlices * 2 * D;
  float s = 0.f;
  for (int i = 0; i < kStaticSlices; ++i) s += src[(size_t)i * 2 * D + e];
  const float m = n_drop > 0 ? __fdiv_rn(s, (float)n_drop) : 0.f;
  if (e < D) mean_k[(size_t)blockIdx.x * D + e] = m;
  else mean_v[(size_t)blockIdx.x * D + (e - D)] = m;
}

template <typename T, int D>
cudaError_t run_static(const void* K, const void* V, int64_t stride_h, int64_t stride_n, int n_heads, int first,
                       int last, float* scratch, float* mean_k, float* mean_v, cudaStream_t s) {
  static_slice_sum_kernel<T, D><<<dim3(kStaticSlices, n_heads), 256, 0, s>>>((const T*)K, (const T*)V, stride_h,
                                                                             stride_n, first, last, scratch);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  static_finalize_kernel<D><<<n_heads, 2 * D, 0, s>>>(scratch, last - first, mean_k, mean_v);
  return cudaGetLastError();
}

// Device address of the scratch array, looked up once per device (the array's name is only a
// host-side handle in host code; kernels must be given the address the runtime reports).  The address
// is remembered per device ordinal for the life of the process: it assumes the device's primary context
// is not destroyed (cudaDeviceReset) while the library stays loaded.
cudaError_t scratch_address(float** out) {
  static float* cached[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64 && cached[dev]) {
    *out = cached[dev];
    return cudaSuccess;
  }
  void* p = nullptr;
  e = cudaGetSymbolAddress(&p, g_static_scratch);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < 64) cached[dev] = (float*)p;
  *out = (float*)p;
  return cudaSuccess;
}

}  // namespace
}  // namespace razor

extern "C" int razor_compensation_mean_static(const void* K, const void* V, int64_t stride_h, int64_t stride_n,
                                              int32_t n_kv_heads, int32_t head_dim, int32_t dtype, int32_t ctx_len,
                                              int32_t n_sink, int32_t window, float* mean_k, float* mean_v,
                                              int32_t* n_drop, void* stream) {
  using namespace razor;
  if (!mean_k || !mean_v) return RAZOR_E_NULL_PTR;
  if (n_kv_heads < 1 || ctx_len < 0 || n_sink < 0 || window < 0) return RAZOR_E_INVALID_ARG;
  if (n_kv_heads > kStaticMaxHeads) return RAZOR_E_CAPACITY;   // beyond the built-in scratch
  if (head_dim != 64 && head_dim != 128) return RAZOR_E_UNSUPPORTED_DIM;
  if (dtype != RAZOR_F32 && dtype != RAZOR_BF16) return RAZOR_E_UNSUPPORTED_DIM;
  const size_t es = dtype == RAZOR_BF16 ? 2 : 4;
  const bool keep_all = (long long)ctx_len <= (long long)n_sink + window;
  const int first = keep_all ? 0 : n_sink, last = keep_all ? 0 : ctx_len - window;   // dropped rows [first, last)
  if (last > first) {
    if (!K || !V) return RAZOR_E_NULL_PTR;
    if (((uintptr_t)K | (uintptr_t)V) & 15) return RAZOR_E_MISALIGNED;
    if (((stride_h * (int64_t)es) | (stride_n * (int64_t)es)) & 15) return RAZOR_E_MISALIGNED;
    if (stride_n < head_dim || stride_h < 0) return RAZOR_E_INVALID_ARG;
  }
  if (((uintptr_t)mean_k | (uintptr_t)mean_v) & 3) return RAZOR_E_MISALIGNED;
  float* scratch = nullptr;
  cudaError_t e = scratch_address(&scratch);
  if (e == cudaSuccess) {
    cudaStream_t s = (cudaStream_t)stream;
    if (dtype == RAZOR_BF16)
      e = head_dim == 128 ? run_static<__nv_bfloat16, 128>(K, V, stride_h, stride_n, n_kv_heads, first, last, scratch, mean_k, mean_v, s)
                          : run_static<__nv_bfloat16, 64>(K, V, stride_h, stride_n, n_kv_heads, first, last, scratch, mean_k, mean_v, s);
    else
      e = head_dim == 128 ? run_static<float, 128>(K, V, stride_h, stride_n, n_kv_heads, first, last, scratch, mean_k, mean_v, s)
                          : run_static<float, 64>(K, V, stride_h, stride_n, n_kv_heads, first, last, scratch, mean_k, mean_v, s);
  }
  if (e != cudaSuccess) {
    note_cuda_error(e);   // razor_last_cuda_error() reports it
    return RAZOR_E_CUDA;
  }
  if (n_drop) *n_drop = last - first;
  return RAZOR_OK;
}
