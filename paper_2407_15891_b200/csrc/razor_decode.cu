// Decode attention over the compressed cache (Eq. 5; Algorithm 1 line 5): split-K flash decoding.
//
// One launch covers every (sequence, KV head) of a layer, full-length retrieval heads and short
// heads alike.  The host cuts the token streams into page ranges of near-equal size (work items);
// warps pull items from a queue.  A warp streams its pages once, keeps an online softmax state
// (m, l, o) per query head of the group in registers, and either writes the output directly (head
// not split) or writes a partial record and takes a ticket; the warp that draws the head's last
// ticket merges the partials, so there is no second launch and no spin-wait anywhere.
//
// The compensation token of a non-retrieval head is folded into the online softmax as the initial
// state of the head's first part: m = s_c + log2(N_d), l = 1, o = v_hat, which is the term
// N_d * exp(s_c) * v_hat of Eq. 5 with the count moved onto the logit.
//
// Logits live in the log2 domain: q is pre-multiplied by sm_scale * log2(e) and exp is ex2.
#include <math_constants.h>

#include "razor_common.cuh"

namespace razor {

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

template <typename T, int D, int G>
__global__ void __launch_bounds__(128, (G == 1 ? 4 : 2))
decode_kernel(DeviceView dv, int layer, int n_items, const T* __restrict__ q, float* __restrict__ out) {
  using Geo = RowGeom<T, D>;
  constexpr int LPR = Geo::kLpr, EPL = Geo::kEpl, RG = Geo::kRg, RPG = Geo::kRowsPerGroup;
  constexpr int REC = kPartialPad + D;   // floats per partial record
  const int lane = threadIdx.x & 31;
  const int lir = lane % LPR, rg = lane / LPR;
  const int n_q_heads = dv.n_kv_heads * G;
  const WorkItem* items = dv.items + (size_t)layer * dv.max_items;
  const int total_warps = gridDim.x * (blockDim.x >> 5);

  for (;;) {
    int it = 0;
    if (lane == 0) it = atomicAdd(dv.queue, 1);
    it = __shfl_sync(0xffffffffu, it, 0);
    if (it >= n_items) break;

    const WorkItem w = items[it];
    const size_t hs = (size_t)layer * dv.n_heads + w.head;
    const HeadState st = dv.state[hs];
    const int n_pages = (st.len + kPageTokens - 1) / kPageTokens;
    const int page_end = w.page_end < 0 ? n_pages : min(w.page_end, n_pages);
    const int b = w.head / dv.n_kv_heads, g = w.head % dv.n_kv_heads;
    const size_t q_row = (size_t)b * n_q_heads + (size_t)g * G;

    float qf[G][EPL];
#pragma unroll
    for (int j = 0; j < G; ++j) {
      const uint4 u = ((const uint4*)(q + (q_row + j) * D))[lir];
      Elem<T>::unpack(u, qf[j]);
#pragma unroll
      for (int e = 0; e < EPL; ++e) qf[j][e] *= dv.scale_log2;
    }

    SoftmaxState<G, EPL> S;
    S.clear();

    // Compensation token (Eq. 4, Eq. 5) seeds the first part of a head that dropped tokens.
    if (w.part_idx == 0 && dv.use_comp && st.n_drop > 0 && st.window >= 0) {
      const float* mean = dv.comp_mean + hs * 2 * D + lir * EPL;
      float kh[EPL], vh[EPL];
#pragma unroll
      for (int e = 0; e < EPL; ++e) { kh[e] = mean[e]; vh[e] = mean[D + e]; }
      const float log_cnt = log2f((float)st.n_drop);
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

    const int32_t* pt = dv.page_table + hs * dv.max_pages;
    for (int p = w.page_begin; p < page_end; ++p) {
      const uint4* kp = (const uint4*)(dv.pool + (size_t)pt[p] * dv.page_bytes) + rg * LPR + lir;
      uint4 kf[RPG], vf[RPG];
#pragma unroll
      for (int i = 0; i < RPG; ++i) kf[i] = ld_stream(kp + i * 32);
#pragma unroll
      for (int i = 0; i < RPG; ++i) vf[i] = ld_stream(kp + kPageTokens * LPR + i * 32);

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

      const int valid = st.len - p * kPageTokens;   // rows of this page that hold tokens
      if (valid < kPageTokens) {
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

    if (w.n_parts == 1) {
      if (rg == 0) {
#pragma unroll
        for (int j = 0; j < G; ++j) {
          const float inv = S.l[j] > 0.f ? 1.f / S.l[j] : 0.f;
          float* dst = out + (q_row + j) * D + lir * EPL;
#pragma unroll
          for (int e = 0; e < EPL; e += 4)
            *(float4*)(dst + e) = make_float4(S.o[j][e] * inv, S.o[j][e + 1] * inv, S.o[j][e + 2] * inv,
                                              S.o[j][e + 3] * inv);
        }
      }
      continue;
    }

    float* rec0 = dv.partials + (size_t)w.part_base * G * REC;
    if (rg == 0) {
#pragma unroll
      for (int j = 0; j < G; ++j) {
        float* rec = rec0 + ((size_t)w.part_idx * G + j) * REC;
        if (lir == 0) { rec[0] = S.m[j]; rec[1] = S.l[j]; }
#pragma unroll
        for (int e = 0; e < EPL; e += 4)
          *(float4*)(rec + kPartialPad + lir * EPL + e) =
              make_float4(S.o[j][e], S.o[j][e + 1], S.o[j][e + 2], S.o[j][e + 3]);
      }
    }
    __threadfence();
    __syncwarp();
    int ticket = 0;
    if (lane == 0) ticket = atomicAdd(&dv.tickets[w.head], 1);
    ticket = __shfl_sync(0xffffffffu, ticket, 0);
    if (ticket != w.n_parts - 1) continue;

    // Last part of this head to finish: merge all partial records (read through L2).
    __threadfence();
    if (lane == 0) dv.tickets[w.head] = 0;
    if (rg == 0) {
#pragma unroll 1
      for (int j = 0; j < G; ++j) {
        float M = -CUDART_INF_F, L = 0.f, acc[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
        for (int i = 0; i < w.n_parts; ++i) {
          const float* rec = rec0 + ((size_t)i * G + j) * REC;
          const float mi = ld_cg(rec), li = ld_cg(rec + 1);
          float oi[EPL];
#pragma unroll
          for (int e = 0; e < EPL; e += 4) {
            const float4 t = ld_cg4((const float4*)(rec + kPartialPad + lir * EPL + e));
            oi[e] = t.x; oi[e + 1] = t.y; oi[e + 2] = t.z; oi[e + 3] = t.w;
          }
          merge_state<EPL>(M, L, acc, mi, li, oi);
        }
        const float inv = L > 0.f ? 1.f / L : 0.f;
        float* dst = out + (q_row + j) * D + lir * EPL;
#pragma unroll
        for (int e = 0; e < EPL; e += 4)
          *(float4*)(dst + e) = make_float4(acc[e] * inv, acc[e + 1] * inv, acc[e + 2] * inv, acc[e + 3] * inv);
      }
    }
  }

  // Queue reset for the next launch: every warp has made its last pop before it counts itself done.
  if (lane == 0) {
    const int done = atomicAdd(dv.queue + 1, 1);
    if (done == total_warps - 1) {
      dv.queue[0] = 0;
      dv.queue[1] = 0;
    }
  }
}

template <typename T, int D, int G>
static cudaError_t decode_t(const DeviceView& dv, int layer, int n_items, const void* q, float* out, int n_sms,
                            cudaStream_t s) {
  const int ctas_per_sm = (G == 1) ? 4 : 2;
  int grid = n_sms * ctas_per_sm;
  const int need = (n_items + 3) / 4;
  if (grid > need) grid = need;
  if (grid < 1) grid = 1;
  decode_kernel<T, D, G><<<grid, 128, 0, s>>>(dv, layer, n_items, (const T*)q, out);
  return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t decode_g(const DeviceView& dv, int layer, int n_items, const void* q, float* out, int n_sms,
                            cudaStream_t s) {
  switch (dv.group) {
    case 1: return decode_t<T, D, 1>(dv, layer, n_items, q, out, n_sms, s);
    case 2: return decode_t<T, D, 2>(dv, layer, n_items, q, out, n_sms, s);
    case 4: return decode_t<T, D, 4>(dv, layer, n_items, q, out, n_sms, s);
    case 8: return decode_t<T, D, 8>(dv, layer, n_items, q, out, n_sms, s);
  }
  return cudaErrorInvalidValue;
}

cudaError_t launch_decode(const DeviceView& dv, int dtype, int layer, int n_items, const void* q, float* out,
                          int n_sms, cudaStream_t s) {
  if (dtype == RAZOR_BF16) {
    return dv.head_dim == 128 ? decode_g<__nv_bfloat16, 128>(dv, layer, n_items, q, out, n_sms, s)
                              : decode_g<__nv_bfloat16, 64>(dv, layer, n_items, q, out, n_sms, s);
  }
  return dv.head_dim == 128 ? decode_g<float, 128>(dv, layer, n_items, q, out, n_sms, s)
                            : decode_g<float, 64>(dv, layer, n_items, q, out, n_sms, s);
}

}  // namespace razor
