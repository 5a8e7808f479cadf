// Device helpers shared by the kernels: 16-byte row fragments, unpacking, warp reductions.
#ifndef RAZOR_COMMON_CUH_
#define RAZOR_COMMON_CUH_

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "razor_internal.h"

namespace razor {

// A K or V row is read as 16-byte fragments, one per lane: LPR lanes cover a row, each lane owns
// EPL consecutive dimensions.
template <typename T>
struct Elem;
template <>
struct Elem<float> {
  static constexpr int kEpl = 4;  // elements per 16-byte fragment
  static __device__ __forceinline__ void unpack(const uint4& u, float (&f)[4]) {
    f[0] = __uint_as_float(u.x);
    f[1] = __uint_as_float(u.y);
    f[2] = __uint_as_float(u.z);
    f[3] = __uint_as_float(u.w);
  }
};
template <>
struct Elem<__nv_bfloat16> {
  static constexpr int kEpl = 8;
  // bf16 -> fp32 is a 16-bit shift: the low half of a word is element 2i, the high half 2i+1.
  static __device__ __forceinline__ void unpack(const uint4& u, float (&f)[8]) {
    f[0] = __uint_as_float(u.x << 16);
    f[1] = __uint_as_float(u.x & 0xffff0000u);
    f[2] = __uint_as_float(u.y << 16);
    f[3] = __uint_as_float(u.y & 0xffff0000u);
    f[4] = __uint_as_float(u.z << 16);
    f[5] = __uint_as_float(u.z & 0xffff0000u);
    f[6] = __uint_as_float(u.w << 16);
    f[7] = __uint_as_float(u.w & 0xffff0000u);
  }
};

template <typename T, int D>
struct RowGeom {
  static constexpr int kEpl = Elem<T>::kEpl;
  static constexpr int kRowBytes = D * (int)sizeof(T);
  static constexpr int kLpr = kRowBytes / 16;      // lanes per row
  static constexpr int kRg = 32 / kLpr;            // rows a warp reads per load instruction
  static constexpr int kRowsPerGroup = kPageTokens / kRg;
  static constexpr int kPageBytes = 2 * kPageTokens * kRowBytes;
  static_assert(kLpr == 8 || kLpr == 16 || kLpr == 32, "row must be 128, 256 or 512 bytes");
};

// In-page placement of 16-byte chunks.  A page is stored as [16 K rows][16 V rows]; chunk c of the row
// of token t (t = slot & 15) sits at chunk position c ^ (t & 7).  The page travels to shared memory
// as one flat block, and with this placement eight rows read at the same logical chunk fall into
// eight different bank groups, which is what the matrix-fragment loads of the grouped-query path
// need; row-wise readers just permute their lanes.
__device__ __forceinline__ int swz(int token, int chunk) { return chunk ^ (token & 7); }

// Streaming 16-byte load: the KV cache is read once per step, keep it out of L1.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// Load that must see other SMs' writes from this launch (partial records): L2 only.
__device__ __forceinline__ float ld_cg(const float* p) { return __ldcg(p); }
__device__ __forceinline__ float4 ld_cg4(const float4* p) { return __ldcg(p); }

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Sum over the kLpr lanes that share a row (butterfly; every lane ends with the total).
template <int LPR>
__device__ __forceinline__ float row_sum(float x) {
#pragma unroll
  for (int off = LPR / 2; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
  return x;
}

// A row of D floats spread over a warp: D/32 consecutive floats per lane.
template <int D>
struct LaneVec;
template <>
struct LaneVec<128> {
  float4 v;
  __device__ __forceinline__ void zero() { v = make_float4(0.f, 0.f, 0.f, 0.f); }
  __device__ __forceinline__ void fma(float c, const LaneVec& o) {
    v.x += c * o.v.x; v.y += c * o.v.y; v.z += c * o.v.z; v.w += c * o.v.w;
  }
  __device__ __forceinline__ void scale(float c) { v.x *= c; v.y *= c; v.z *= c; v.w *= c; }
  __device__ __forceinline__ void load_shared(const float* row, int lane) { v = *(const float4*)(row + lane * 4); }
  __device__ __forceinline__ void load_l2(const float* row, int lane) { v = __ldcg((const float4*)(row + lane * 4)); }
  __device__ __forceinline__ void store(float* row, int lane) const { *(float4*)(row + lane * 4) = v; }
};
template <>
struct LaneVec<64> {
  float2 v;
  __device__ __forceinline__ void zero() { v = make_float2(0.f, 0.f); }
  __device__ __forceinline__ void fma(float c, const LaneVec& o) { v.x += c * o.v.x; v.y += c * o.v.y; }
  __device__ __forceinline__ void scale(float c) { v.x *= c; v.y *= c; }
  __device__ __forceinline__ void load_shared(const float* row, int lane) { v = *(const float2*)(row + lane * 2); }
  __device__ __forceinline__ void load_l2(const float* row, int lane) { v = __ldcg((const float2*)(row + lane * 2)); }
  __device__ __forceinline__ void store(float* row, int lane) const { *(float2*)(row + lane * 2) = v; }
};

}  // namespace razor
#endif
