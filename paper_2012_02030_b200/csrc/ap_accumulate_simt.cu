// Eq. 1 as a running sum, CUDA-core (fp32 FMA) version.
//
// One CTA owns up to 8 query rows of one head and loops over the B samples in
// ascending order, so every accumulator entry is updated by exactly one thread
// in a fixed order (no floating-point atomics; results are reproducible).  Per
// sample: scores of the rows against all keys of the row domain go to shared
// memory, then one warp per row takes the row maximum, the sum of exponentials
// and adds the normalised row to the accumulator with coalesced read-modify-
// writes.  Used for fp32 inputs, where tensor-core precision would not do.
//
// kEntmax: the same sum with 1.5-entmax as the normaliser (the section on sparse normalisation),
// p_j = max(s_j / 2 - tau, 0)^2 with tau such that the row sums to 1.  The row's scores are in
// shared memory, so the warp iterates on tau there: from max/2 - 0.625 (the root lies in [max/2 - 1, max/2)) to the
// smaller root of the parabola of the current support, tau + (S2 - 1) / (S1 + sqrt(S1^2 - n (S2 - 1)))
// with n, S1, S2 the support's size and its sums of (s_j/2 - tau) and of its square (Newton's
// step (S2 - 1) / (2 S1) where the parabola has no root), until the step falls under
// 5e-7 max(1, |tau|) (at most 30 steps).
#include <math_constants.h>

#include "ap_common.cuh"

namespace ap {

namespace {

constexpr int kRows = 8;
constexpr int kThreads = 256;

template <typename T>
__device__ __forceinline__ void load8(const T *p, float v[8]);

template <>
__device__ __forceinline__ void load8<float>(const float *p, float v[8]) {
  float4 a = *reinterpret_cast<const float4 *>(p), b = *reinterpret_cast<const float4 *>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

template <>
__device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16 *p, float v[8]) {
  uint4 u = *reinterpret_cast<const uint4 *>(p);
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    v[2 * c] = __uint_as_float(w[c] << 16);
    v[2 * c + 1] = __uint_as_float(w[c] & 0xffff0000u);
  }
}

template <typename T, int D, bool kEntmax>
__global__ void __launch_bounds__(kThreads) accumulate_simt_kernel(float *__restrict__ acc, const T *__restrict__ Q,
                                                                   const T *__restrict__ K,
                                                                   const float *__restrict__ bias, int B, int H,
                                                                   int Lq, int Lk, int rows, int causal,
                                                                   float scale) {
  extern __shared__ __align__(16) float smem[];
  float *q_s = smem;                 // [rows][D]
  float *s_s = smem + kRows * D;     // [rows][Lk]
  const int h = blockIdx.y;
  const int i0 = blockIdx.x * rows;
  const int n_rows = min(rows, Lq - i0);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // keys any row of this block may look at
  const int off = causal ? Lk - Lq : 0;  // causal: row i looks at keys j <= i + (Lk - Lq)
  const int jmax = causal ? min(Lk, i0 + n_rows + off) : Lk;

  for (int b = 0; b < B; ++b) {
    const T *Qb = Q + (((size_t)b * H + h) * Lq + i0) * D;
    const T *Kb = K + ((size_t)b * H + h) * (size_t)Lk * D;
    for (int e = threadIdx.x; e < kRows * D; e += kThreads) {
      const int r = e / D;
      q_s[e] = r < n_rows ? (float)Qb[e] : 0.f;
    }
    __syncthreads();
    for (int j = threadIdx.x; j < jmax; j += kThreads) {
      float dot[kRows];
#pragma unroll
      for (int r = 0; r < kRows; ++r) dot[r] = 0.f;
      const T *krow = Kb + (size_t)j * D;
#pragma unroll 2
      for (int t = 0; t < D; t += 8) {
        float kv[8];
        load8<T>(krow + t, kv);
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
          const float4 qa = *reinterpret_cast<const float4 *>(q_s + r * D + t);
          const float4 qb = *reinterpret_cast<const float4 *>(q_s + r * D + t + 4);
          dot[r] = fmaf(qa.x, kv[0], dot[r]); dot[r] = fmaf(qa.y, kv[1], dot[r]);
          dot[r] = fmaf(qa.z, kv[2], dot[r]); dot[r] = fmaf(qa.w, kv[3], dot[r]);
          dot[r] = fmaf(qb.x, kv[4], dot[r]); dot[r] = fmaf(qb.y, kv[5], dot[r]);
          dot[r] = fmaf(qb.z, kv[6], dot[r]); dot[r] = fmaf(qb.w, kv[7], dot[r]);
        }
      }
#pragma unroll
      for (int r = 0; r < kRows; ++r) {
        if (r < n_rows) {
          float s = dot[r] * scale;
          if (bias) s += bias[((size_t)h * Lq + i0 + r) * Lk + j];
          s_s[(size_t)r * Lk + j] = s;
        }
      }
    }
    __syncthreads();
    // warp r normalises row r and adds it to the accumulator
    for (int r = warp; r < n_rows; r += kThreads / 32) {
      const int i = i0 + r;
      const int jend = causal ? min(Lk, i + 1 + off) : Lk;
      const float *srow = s_s + (size_t)r * Lk;
      float m = -CUDART_INF_F;
      for (int j = lane; j < jend; j += 32) m = fmaxf(m, srow[j]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      float *arow = acc + ((size_t)h * Lq + i) * Lk;
      if (kEntmax) {
        float tau = 0.5f * m - 0.625f;  // the root lies in [max/2 - 1, max/2)
        for (int it = 0; it < 30; ++it) {
          float n = 0.f, S1 = 0.f, S2 = 0.f;
          for (int j = lane; j < jend; j += 32) {
            const float u = fmaf(0.5f, srow[j], -tau);
            if (u > 0.f) {
              n += 1.f;
              S1 += u;
              S2 = fmaf(u, u, S2);
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {  // every lane ends with the same bits
            n += __shfl_xor_sync(0xffffffffu, n, o);
            S1 += __shfl_xor_sync(0xffffffffu, S1, o);
            S2 += __shfl_xor_sync(0xffffffffu, S2, o);
          }
          const float disc = S1 * S1 - n * (S2 - 1.f);
          const float step = S1 > 0.f ? (S2 - 1.f) / (S1 + (disc >= 0.f ? sqrtf(disc) : S1)) : 0.f;
          tau += step;
          if (fabsf(step) <= 5e-7f * fmaxf(1.f, fabsf(tau))) break;
        }
        for (int j = lane; j < jend; j += 32) {
          const float u = fmaf(0.5f, srow[j], -tau);
          if (u > 0.f) arow[j] += u * u;
        }
        continue;
      }
      float z = 0.f;
      for (int j = lane; j < jend; j += 32) z += expf(srow[j] - m);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
      for (int j = lane; j < jend; j += 32) arow[j] += expf(srow[j] - m) / z;
    }
    __syncthreads();
  }
}

template <typename T, int D, bool kEntmax>
cudaError_t launch(float *acc, const void *Q, const void *K, const float *bias, int B, int H, int Lq, int Lk,
                   int causal, float scale, cudaStream_t s) {
  // as many rows per CTA (up to 8) as the score rows allow in shared memory
  int rows = kRows;
  const size_t budget = 200 * 1024;
  while (rows > 1 && (size_t)(kRows * D + (size_t)rows * Lk) * sizeof(float) > budget) rows >>= 1;
  const size_t smem = (size_t)(kRows * D + (size_t)rows * Lk) * sizeof(float);
  if (smem > budget) return cudaErrorInvalidValue;
  auto kern = accumulate_simt_kernel<T, D, kEntmax>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(ceil_div(Lq, rows), H);
  kern<<<grid, kThreads, smem, s>>>(acc, static_cast<const T *>(Q), static_cast<const T *>(K), bias, B, H, Lq, Lk,
                                    rows, causal, scale);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_accumulate_simt(float *acc, const void *Q, const void *K, const float *bias, int B, int H,
                                   int Lq, int Lk, int d, ap_dtype dt, int causal, float scale,
                                   cudaStream_t s, int entmax) {
  if (entmax) {  // fp32 tensors only
    return d == 64 ? launch<float, 64, true>(acc, Q, K, bias, B, H, Lq, Lk, causal, scale, s)
                   : launch<float, 128, true>(acc, Q, K, bias, B, H, Lq, Lk, causal, scale, s);
  }
  if (dt == AP_F32) {
    return d == 64 ? launch<float, 64, false>(acc, Q, K, bias, B, H, Lq, Lk, causal, scale, s)
                   : launch<float, 128, false>(acc, Q, K, bias, B, H, Lq, Lk, causal, scale, s);
  }
  return d == 64 ? launch<__nv_bfloat16, 64, false>(acc, Q, K, bias, B, H, Lq, Lk, causal, scale, s)
                 : launch<__nv_bfloat16, 128, false>(acc, Q, K, bias, B, H, Lq, Lk, causal, scale, s);
}

}  // namespace ap
