// Masked attention of Section 3.2 on CUDA cores (fp32 FMA), for fp32 tensors.
//
// One CTA per (b, h, query tile) walks the tile list of its (h, qt) row.  Two
// threads share a query row, each owning alternate 4-element groups of the head
// dimension (q and the output accumulator stay in registers).  K and V tiles
// are staged in shared memory as fp32; for every key of a tile whose bitmap bit
// is set the pair computes the logit, updates the running maximum / sum
// (online softmax) and adds p*V.  Pruned keys are skipped, which is exactly a
// weight of zero; rows that never see a kept key output zeros.
#include <math_constants.h>

#include "ap_common.cuh"

namespace ap {

namespace {

constexpr int kThreads = 256;

template <typename T>
__device__ __forceinline__ float4 load4(const T *p);
template <>
__device__ __forceinline__ float4 load4<float>(const float *p) {
  return *reinterpret_cast<const float4 *>(p);
}

template <typename T>
__device__ __forceinline__ void store4(T *p, float4 v);
template <>
__device__ __forceinline__ void store4<float>(float *p, float4 v) {
  *reinterpret_cast<float4 *>(p) = v;
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads) fwd_simt_kernel(const T *__restrict__ Q, const T *__restrict__ K,
                                                            const T *__restrict__ V,
                                                            const int32_t *__restrict__ row_ptr,
                                                            const int32_t *__restrict__ col_idx,
                                                            const uint8_t *__restrict__ flags,
                                                            const uint32_t *__restrict__ bitmap, T *__restrict__ O,
                                                            int H, int Lq, int Lk, int n_qt, float scale) {
  constexpr int G = D / 8;  // 4-element groups per thread
  extern __shared__ __align__(16) float smem[];
  float *k_s = smem;               // [128][D]
  float *v_s = smem + kTile * D;   // [128][D]
  const int qt = blockIdx.x % n_qt;
  const int h = (blockIdx.x / n_qt) % H;
  const int b = blockIdx.x / (n_qt * H);
  const int r = threadIdx.x >> 1, half = threadIdx.x & 1;
  const int i = qt * kTile + r;
  const size_t bh = (size_t)b * H + h;

  float4 q[G], o[G];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    o[g] = make_float4(0.f, 0.f, 0.f, 0.f);
    q[g] = i < Lq ? load4<T>(Q + (bh * Lq + i) * D + 4 * (2 * g + half)) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float m = -CUDART_INF_F, l = 0.f;

  const int t_begin = row_ptr[h * n_qt + qt], t_end = row_ptr[h * n_qt + qt + 1];
  for (int t = t_begin; t < t_end; ++t) {
    const int kt = col_idx[t];
    __syncthreads();  // previous tile fully consumed
    for (int e = threadIdx.x; e < kTile * D / 4; e += kThreads) {
      const int jj = e / (D / 4), c = e % (D / 4);
      const int j = kt * kTile + jj;
      float4 kv = make_float4(0.f, 0.f, 0.f, 0.f), vv = kv;
      if (j < Lk) {
        kv = load4<T>(K + (bh * Lk + j) * D + 4 * c);
        vv = load4<T>(V + (bh * Lk + j) * D + 4 * c);
      }
      reinterpret_cast<float4 *>(k_s)[e] = kv;
      reinterpret_cast<float4 *>(v_s)[e] = vv;
    }
    const bool full = flags[t] & 1;
    const uint4 bw = reinterpret_cast<const uint4 *>(bitmap + (size_t)t * kBitmapWords)[r];
    const uint32_t words[4] = {bw.x, bw.y, bw.z, bw.w};
    __syncthreads();
#pragma unroll 1
    for (int w = 0; w < 4; ++w) {
      const uint32_t bits = full ? 0xffffffffu : words[w];
      if (!__any_sync(0xffffffffu, bits != 0u)) continue;
#pragma unroll 1
      for (int c = 0; c < 32; ++c) {
        const bool keep = (bits >> c) & 1u;
        if (!__any_sync(0xffffffffu, keep)) continue;
        const int jj = 32 * w + c;
        const float4 *krow = reinterpret_cast<const float4 *>(k_s + jj * D);
        float dot = 0.f;
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const float4 kv = krow[2 * g + half];
          dot = fmaf(q[g].x, kv.x, dot); dot = fmaf(q[g].y, kv.y, dot);
          dot = fmaf(q[g].z, kv.z, dot); dot = fmaf(q[g].w, kv.w, dot);
        }
        dot += __shfl_xor_sync(0xffffffffu, dot, 1);
        if (keep) {
          const float s = dot * scale;
          if (s > m) {
            const float alpha = expf(m - s);  // exp(-inf) = 0 on the first kept key
            l *= alpha;
#pragma unroll
            for (int g = 0; g < G; ++g) {
              o[g].x *= alpha; o[g].y *= alpha; o[g].z *= alpha; o[g].w *= alpha;
            }
            m = s;
          }
          const float p = expf(s - m);
          l += p;
          const float4 *vrow = reinterpret_cast<const float4 *>(v_s + jj * D);
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const float4 vv = vrow[2 * g + half];
            o[g].x = fmaf(p, vv.x, o[g].x); o[g].y = fmaf(p, vv.y, o[g].y);
            o[g].z = fmaf(p, vv.z, o[g].z); o[g].w = fmaf(p, vv.w, o[g].w);
          }
        }
      }
    }
  }
  if (i < Lq) {
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float4 out = make_float4(0.f, 0.f, 0.f, 0.f);
      if (l > 0.f) out = make_float4(o[g].x / l, o[g].y / l, o[g].z / l, o[g].w / l);
      store4<T>(O + (bh * Lq + i) * D + 4 * (2 * g + half), out);
    }
  }
}

// The same attention with 1.5-entmax as the normaliser (the section on sparse normalisation):
// p_j = max(s_j / 2 - tau, 0)^2 over the kept keys, tau such that the row sums to 1.  tau depends
// on all kept scores of a row, so the CTA walks its tiles once per sweep: row maxima first
// (tau = max/2 - 0.625; the root lies in [max/2 - 1, max/2)), then sweeps that collect the size n of the support of the
// trial threshold and its sums S1, S2 of (s_j/2 - tau) and of its square and move tau to the smaller
// root of the support's parabola, tau + (S2 - 1) / (S1 + sqrt(S1^2 - n (S2 - 1))) (Newton's step
// (S2 - 1) / (2 S1) where it has none), until no row of the CTA moves by more than
// 5e-7 max(1, |tau|) (at most 30 sweeps), then the sweep that forms the weights and adds p V.
// Both threads of a row see the same scores and keep the same statistics.
template <typename T, int D>
__global__ void __launch_bounds__(kThreads) fwd_entmax_simt_kernel(const T *__restrict__ Q, const T *__restrict__ K,
                                                                   const T *__restrict__ V,
                                                                   const int32_t *__restrict__ row_ptr,
                                                                   const int32_t *__restrict__ col_idx,
                                                                   const uint8_t *__restrict__ flags,
                                                                   const uint32_t *__restrict__ bitmap,
                                                                   T *__restrict__ O, int H, int Lq, int Lk, int n_qt,
                                                                   float half_scale) {
  constexpr int G = D / 8;
  extern __shared__ __align__(16) float smem[];
  float *k_s = smem;               // [128][D]
  float *v_s = smem + kTile * D;   // [128][D]
  const int qt = blockIdx.x % n_qt;
  const int h = (blockIdx.x / n_qt) % H;
  const int b = blockIdx.x / (n_qt * H);
  const int r = threadIdx.x >> 1, half = threadIdx.x & 1;
  const int i = qt * kTile + r;
  const size_t bh = (size_t)b * H + h;

  float4 q[G], o[G];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    o[g] = make_float4(0.f, 0.f, 0.f, 0.f);
    q[g] = i < Lq ? load4<T>(Q + (bh * Lq + i) * D + 4 * (2 * g + half)) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float m = -CUDART_INF_F, tau = 0.f, l = 0.f;
  const int t_begin = row_ptr[h * n_qt + qt], t_end = row_ptr[h * n_qt + qt + 1];
  int kind = 0;  // 0 maxima, 1 sums over the support, 2 weights
  for (int sw = 0;; ++sw) {
    float n = 0.f, S1 = 0.f, S2 = 0.f;
    for (int t = t_begin; t < t_end; ++t) {
      const int kt = col_idx[t];
      __syncthreads();  // previous tile fully consumed
      for (int e = threadIdx.x; e < kTile * D / 4; e += kThreads) {
        const int jj = e / (D / 4), c = e % (D / 4);
        const int j = kt * kTile + jj;
        float4 kv = make_float4(0.f, 0.f, 0.f, 0.f), vv = kv;
        if (j < Lk) {
          kv = load4<T>(K + (bh * Lk + j) * D + 4 * c);
          if (kind == 2) vv = load4<T>(V + (bh * Lk + j) * D + 4 * c);
        }
        reinterpret_cast<float4 *>(k_s)[e] = kv;
        if (kind == 2) reinterpret_cast<float4 *>(v_s)[e] = vv;
      }
      const bool full = flags[t] & 1;
      const uint4 bw = reinterpret_cast<const uint4 *>(bitmap + (size_t)t * kBitmapWords)[r];
      const uint32_t words[4] = {bw.x, bw.y, bw.z, bw.w};
      __syncthreads();
#pragma unroll 1
      for (int w = 0; w < 4; ++w) {
        const uint32_t bits = full ? 0xffffffffu : words[w];
        if (!__any_sync(0xffffffffu, bits != 0u)) continue;
#pragma unroll 1
        for (int c = 0; c < 32; ++c) {
          const bool keep = (bits >> c) & 1u;
          if (!__any_sync(0xffffffffu, keep)) continue;
          const int jj = 32 * w + c;
          const float4 *krow = reinterpret_cast<const float4 *>(k_s + jj * D);
          float dot = 0.f;
#pragma unroll
          for (int g = 0; g < G; ++g) {
            const float4 kv = krow[2 * g + half];
            dot = fmaf(q[g].x, kv.x, dot); dot = fmaf(q[g].y, kv.y, dot);
            dot = fmaf(q[g].z, kv.z, dot); dot = fmaf(q[g].w, kv.w, dot);
          }
          dot += __shfl_xor_sync(0xffffffffu, dot, 1);
          if (!keep) continue;
          const float x = dot * half_scale;
          if (kind == 0) {
            m = fmaxf(m, x);
          } else {
            const float u = x - tau;
            if (u > 0.f) {
              if (kind == 1) {
                n += 1.f;
                S1 += u;
                S2 = fmaf(u, u, S2);
              } else {
                const float p = u * u;
                l += p;
                const float4 *vrow = reinterpret_cast<const float4 *>(v_s + jj * D);
#pragma unroll
                for (int g = 0; g < G; ++g) {
                  const float4 vv = vrow[2 * g + half];
                  o[g].x = fmaf(p, vv.x, o[g].x); o[g].y = fmaf(p, vv.y, o[g].y);
                  o[g].z = fmaf(p, vv.z, o[g].z); o[g].w = fmaf(p, vv.w, o[g].w);
                }
              }
            }
          }
        }
      }
    }
    if (kind == 2) break;
    bool moved = false;
    if (kind == 0) {
      // no kept key: every weight is 0 whatever the threshold
      tau = m == -CUDART_INF_F ? CUDART_INF_F : m - 0.625f;
    } else {
      const float disc = S1 * S1 - n * (S2 - 1.f);
      const float step = S1 > 0.f ? (S2 - 1.f) / (S1 + (disc >= 0.f ? sqrtf(disc) : S1)) : 0.f;
      tau += step;
      moved = i < Lq && fabsf(step) > 5e-7f * fmaxf(1.f, fabsf(tau));
    }
    const int more = __syncthreads_or(moved ? 1 : 0);
    kind = kind == 0 ? 1 : ((more && sw < 30) ? 1 : 2);
  }
  if (i < Lq) {
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float4 out = make_float4(0.f, 0.f, 0.f, 0.f);
      if (l > 0.f) out = make_float4(o[g].x / l, o[g].y / l, o[g].z / l, o[g].w / l);
      store4<T>(O + (bh * Lq + i) * D + 4 * (2 * g + half), out);
    }
  }
}

template <typename T, int D>
cudaError_t launch_entmax(const void *Q, const void *K, const void *V, const ap_tiles &t, void *O, int B, int H, int Lq,
                          int Lk, float scale, cudaStream_t s) {
  const size_t smem = 2 * (size_t)kTile * D * sizeof(float);
  auto kern = fwd_entmax_simt_kernel<T, D>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<B * H * t.n_qt, kThreads, smem, s>>>(static_cast<const T *>(Q), static_cast<const T *>(K),
                                              static_cast<const T *>(V), t.row_ptr, t.col_idx, t.flags, t.bitmap,
                                              static_cast<T *>(O), H, Lq, Lk, t.n_qt, 0.5f * scale);
  count_launches(1);
  return cudaGetLastError();
}

template <typename T, int D>
cudaError_t launch(const void *Q, const void *K, const void *V, const ap_tiles &t, void *O, int B, int H, int Lq,
                   int Lk, float scale, cudaStream_t s) {
  const size_t smem = 2 * (size_t)kTile * D * sizeof(float);
  auto kern = fwd_simt_kernel<T, D>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<B * H * t.n_qt, kThreads, smem, s>>>(static_cast<const T *>(Q), static_cast<const T *>(K),
                                              static_cast<const T *>(V), t.row_ptr, t.col_idx, t.flags, t.bitmap,
                                              static_cast<T *>(O), H, Lq, Lk, t.n_qt, scale);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fwd_simt(const void *Q, const void *K, const void *V, const ap_tiles &t, void *O, int B, int H,
                            int Lq, int Lk, int d, float scale, cudaStream_t s) {
  return d == 64 ? launch<float, 64>(Q, K, V, t, O, B, H, Lq, Lk, scale, s)
                 : launch<float, 128>(Q, K, V, t, O, B, H, Lq, Lk, scale, s);
}

cudaError_t launch_fwd_entmax_simt(const void *Q, const void *K, const void *V, const ap_tiles &t, void *O, int B,
                                   int H, int Lq, int Lk, int d, float scale, cudaStream_t s) {
  return d == 64 ? launch_entmax<float, 64>(Q, K, V, t, O, B, H, Lq, Lk, scale, s)
                 : launch_entmax<float, 128>(Q, K, V, t, O, B, H, Lq, Lk, scale, s);
}

}  // namespace ap
