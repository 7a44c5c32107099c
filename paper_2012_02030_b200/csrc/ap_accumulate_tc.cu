// Eq. 1 as a running sum for bf16 and fp16 tensors, on the tcgen05 tensor cores.
//
// One CTA owns one (head, 128-row query tile) and adds, for up to 16 samples b per launch,
// the normalised softmax rows to the accumulator.  A softmax row needs its
// maximum and its sum of exponentials over ALL keys before any entry can be
// normalised, and the sum over b needs each sample normalised separately, so
// the CTA sweeps its key tiles twice:
//   sweep 1  for every key tile kt, for every b:  S = Q_b K_b(kt)^T  (tcgen05.mma,
//            operands staged by TMA, accumulator in TMEM) -> per-row running
//            maximum and sum of exp2 of the scaled, biased logits
//   sweep 2  the same visits again: p = exp2(logit - max - log2 sum) is the
//            normalised weight; the sum over b is kept in TMEM and added to the
//            accumulator once per key tile (one global update per entry and
//            call instead of one per sample).
// The bias tile of a key tile is staged once per sweep and key tile by TMA (fp32,
// 128-byte swizzle, so that a thread reads its own row without bank conflicts),
// copied to registers and reused for all b.  Samples are added in ascending b by
// a fixed thread and every accumulator entry receives exactly one addition per
// launch (a fire-and-forget red.global.add), so results are reproducible bit for bit.
//
// Warp roles (320 threads, one CTA per SM): warps 0-7 softmax; thread (wg, r)
// with wg = warp / 4 owns row r of the tile and columns [64 wg, 64 wg + 64) of
// every key tile; warp 8 TMA producer; warp 9 MMA issuer and TMEM owner.  S is
// double-buffered in TMEM (2 x 128 columns) so the MMA of the next visit runs
// under the softmax of the current one.  Every mbarrier wait is bounded.
#include <math_constants.h>

#include "ap_common.cuh"
#include "ap_sm100.cuh"

namespace ap {

namespace {

using namespace sm100;

constexpr int kThreads = 320;
constexpr int kSoftmaxThreads = 256;
constexpr int kSubBytes = 128 * 128;
constexpr uint32_t kTmemCols = 512;  // S x 2 (columns 0..255), running sum over b (columns 256..383)
constexpr uint32_t kMaxPolls = 1u << 22;
constexpr int kMaxB = 16;  // samples per launch (statistics live in shared memory)
constexpr int kBiasBytes = 128 * 128 * 4;  // one fp32 bias tile: 4 boxes of 128 rows x 32 columns
constexpr float kLog2e = 1.4426950408889634f;

template <int D>
struct Cfg {
  static constexpr int kSub = D / 64;
  static constexpr int kTileBytes = kSub * kSubBytes;    // one operand tile (Q or K)
  static constexpr int kStages = D == 64 ? 3 : 2;        // (Q, K) pairs in flight
  static constexpr int kBiasOffset = 2 * kStages * kTileBytes;
  static constexpr int kStatsOffset = kBiasOffset + kBiasBytes;
  static constexpr int kStatsBytes = 2 * kMaxB * 128 * 8;  // [wg][b][row] (max, sum)
  static constexpr int kBarOffset = kStatsOffset + kStatsBytes;
  static constexpr int kSmemBytes = kBarOffset + 256 + 1024;
  static_assert(kSmemBytes <= 227 * 1024, "within the shared memory of one CTA");
};

struct Barriers {
  uint64_t s_full[2], s_empty[2];
  uint64_t in_full[3], in_empty[3];
  uint64_t sweep1_done;  // all 256 softmax threads have stored their sweep-1 statistics
  uint64_t bias_full, bias_empty;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ bool wait_or_abort(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                              unsigned *err) {
  for (uint32_t i = 0; i < kMaxPolls; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (i > 64) __nanosleep(64);
  }
  *abort_flag = 1;
  atomicOr(err, kDevErrTimeout);
  return false;
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
accumulate_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_bias, int bias_by_tma, float *__restrict__ acc,
                     const float *__restrict__ bias, int b0, int Bc, int H, int Lq, int Lk,
                     int n_qt, int n_kt, int causal, int f16, float scale_log2, unsigned *err) {
  using C = Cfg<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem =
      reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char *bias_s = smem + C::kBiasOffset;
  float2 *stats = reinterpret_cast<float2 *>(smem + C::kStatsOffset);  // [wg][b][row]
  Barriers *bars = reinterpret_cast<Barriers *>(smem + C::kBarOffset);

  // late query tiles (most key tiles under a causal mask) first
  const int qt = n_qt - 1 - (int)(blockIdx.x / H);
  const int h = blockIdx.x % H;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // causal: row i looks at keys j <= i + (Lk - Lq), i.e. Lk - Lq memory keys, then its own segment
  const int off = causal ? Lk - Lq : 0;
  const int n_k = causal ? min(n_kt, (qt * kTile + kTile - 1 + off) / kTile + 1) : n_kt;  // key tiles of this query tile
  const int visits_per_sweep = n_k * Bc;
  const int n_visits = 2 * visits_per_sweep;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->s_full[s], 1);
      mbar_init(&bars->s_empty[s], kSoftmaxThreads);
    }
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&bars->in_full[s], 1);
      mbar_init(&bars->in_empty[s], 1);
    }
    mbar_init(&bars->sweep1_done, kSoftmaxThreads);
    mbar_init(&bars->bias_full, 1);
    mbar_init(&bars->bias_empty, kSoftmaxThreads);
    bars->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 9) {
    tmem_alloc(&bars->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = bars->tmem_base;
  volatile int *abort_flag = &bars->abort_flag;

  if (warp == 8) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tensormap(&map_q);
      prefetch_tensormap(&map_k);
      if (bias_by_tma) prefetch_tensormap(&map_bias);
      int v = 0, bias_loads = 0;
      for (; v < n_visits; ++v) {
        const int st = v % C::kStages;
        const uint32_t ph = (uint32_t)(v / C::kStages) & 1u;
        const int vv = v % visits_per_sweep;
        const int kt = vv / Bc, b = b0 + vv % Bc;
        if (bias_by_tma && v % Bc == 0) {
          // bias tile of the key tile whose visits start here; the buffer is free once all
          // softmax threads have copied the previous tile to registers
          const int tl = v / Bc;
          if (!wait_or_abort(&bars->bias_empty, ((uint32_t)tl & 1u) ^ 1u, abort_flag, err)) break;
          mbar_arrive_expect_tx(&bars->bias_full, kBiasBytes);
#pragma unroll
          for (int q = 0; q < 4; ++q)
            tma_load_3d(bias_s + q * (kBiasBytes / 4), &map_bias, &bars->bias_full, kt * kTile + 32 * q, qt * kTile, h);
          bias_loads = tl + 1;
        }
        if (!wait_or_abort(&bars->in_empty[st], ph ^ 1u, abort_flag, err)) break;
        unsigned char *q_s = smem + (2 * st) * C::kTileBytes, *k_s = q_s + C::kTileBytes;
        mbar_arrive_expect_tx(&bars->in_full[st], 2 * C::kTileBytes);
#pragma unroll
        for (int s = 0; s < C::kSub; ++s) {
          tma_load_3d(q_s + s * kSubBytes, &map_q, &bars->in_full[st], 64 * s, qt * kTile, b * H + h);
          tma_load_3d(k_s + s * kSubBytes, &map_k, &bars->in_full[st], 64 * s, kt * kTile, b * H + h);
        }
      }
      if (*abort_flag) {  // winding down: let the copies in flight land (bounded)
        for (int j = max(0, v - C::kStages); j < v; ++j)
          mbar_wait(&bars->in_full[j % C::kStages], (uint32_t)(j / C::kStages) & 1u, kMaxPolls);
        if (bias_loads > 0) mbar_wait(&bars->bias_full, (uint32_t)(bias_loads - 1) & 1u, kMaxPolls);
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(128, 128, false, false, f16 != 0);
      for (int v = 0; v < n_visits; ++v) {
        const int st = v % C::kStages;
        const uint32_t ph = (uint32_t)(v / C::kStages) & 1u;
        const int buf = v & 1;
        if (!wait_or_abort(&bars->in_full[st], ph, abort_flag, err)) break;
        if (!wait_or_abort(&bars->s_empty[buf], ((uint32_t)(v >> 1) & 1u) ^ 1u, abort_flag, err)) break;
        tc_fence_after_sync();
        const unsigned char *q_s = smem + (2 * st) * C::kTileBytes, *k_s = q_s + C::kTileBytes;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const int sub = ks / 4, off = (ks % 4) * 32;
          const uint64_t da = smem_desc_sw128(smem_u32(q_s + sub * kSubBytes + off), 16, 1024);
          const uint64_t db = smem_desc_sw128(smem_u32(k_s + sub * kSubBytes + off), 16, 1024);
          mma_ss(tmem + 128 * buf, da, db, idesc, ks > 0);
        }
        mma_commit(&bars->in_empty[st]);
        mma_commit(&bars->s_full[buf]);
      }
    }
  } else {
    // ------------------------------------------------------------ softmax (256 threads)
    const int wg = warp >> 2;
    const int r = (warp & 3) * 32 + lane;  // row of the tile == TMEM lane
    const int i = qt * kTile + r;
    const bool row_ok = i < Lq;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const int jend = causal ? min(Lk, i + 1 + off) : Lk;  // first key outside this row's domain
    const bool vec = (Lk & 3) == 0;
    float2 *my_stats = stats + (size_t)wg * kMaxB * 128 + r;  // + b * 128
    for (int b = 0; b < Bc; ++b) my_stats[b * 128] = make_float2(-CUDART_INF_F, 0.f);

    float bias2[64];  // bias * log2(e) of this thread's 64 columns of the current key tile
    float ref = 0.f;  // sweep 2: max + log2(sum) of the current sample's row
    bool ok = true;
    // (sweep, key tile, sample) of the visit, stepped rather than divided out of v: an integer
    // division per visit is a hundred cycles on this thread's critical path
    int sweep = 0, kt = 0, b = -1;
    for (int v = 0; v < n_visits && ok; ++v) {
      if (++b == Bc) {
        b = 0;
        if (++kt == n_k) {
          kt = 0;
          sweep = 1;
        }
      }
      const int buf = v & 1;
      const int j0 = kt * kTile + 64 * wg;  // first column of this thread's slice
      if (v == visits_per_sweep) {
        // every statistic of sweep 1 is final once both column halves of every row are done
        mbar_arrive(&bars->sweep1_done);
        ok = wait_or_abort(&bars->sweep1_done, 0, abort_flag, err);
        if (!ok) break;
      }
      if (b == 0) {  // new key tile: fetch this thread's bias slice once for all samples
        if (bias_by_tma) {
          const int tl = sweep * n_k + kt;
          ok = wait_or_abort(&bars->bias_full, (uint32_t)tl & 1u, abort_flag, err);
          if (!ok) break;
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const unsigned char *box = bias_s + (2 * wg + q) * (kBiasBytes / 4) + r * 128;
#pragma unroll
            for (int k = 0; k < 8; ++k) {  // 16-byte chunk k of the row sits at position k ^ (r % 8)
              const float4 t = *reinterpret_cast<const float4 *>(box + ((k ^ (r & 7)) << 4));
              bias2[32 * q + 4 * k] = t.x * kLog2e; bias2[32 * q + 4 * k + 1] = t.y * kLog2e;
              bias2[32 * q + 4 * k + 2] = t.z * kLog2e; bias2[32 * q + 4 * k + 3] = t.w * kLog2e;
            }
          }
          mbar_arrive(&bars->bias_empty);
        } else {
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            const int j = j0 + 4 * c;
            if (bias && row_ok) {
              const float *brow = bias + ((size_t)h * Lq + i) * Lk;
              if (j < Lk) t.x = brow[j];
              if (j + 1 < Lk) t.y = brow[j + 1];
              if (j + 2 < Lk) t.z = brow[j + 2];
              if (j + 3 < Lk) t.w = brow[j + 3];
            }
            bias2[4 * c] = t.x * kLog2e; bias2[4 * c + 1] = t.y * kLog2e;
            bias2[4 * c + 2] = t.z * kLog2e; bias2[4 * c + 3] = t.w * kLog2e;
          }
        }
      }
      if (sweep == 1) {
        // combine the two column halves' statistics of sample b: max + log2(sum)
        const float2 s0 = stats[(size_t)b * 128 + r], s1 = stats[(size_t)(kMaxB + b) * 128 + r];
        const float mm = fmaxf(s0.x, s1.x);
        const float z = s0.y * ex2_approx(s0.x - mm) + s1.y * ex2_approx(s1.x - mm);
        ref = mm + lg2_approx(z);
      }
      ok = wait_or_abort(&bars->s_full[buf], (uint32_t)(v >> 1) & 1u, abort_flag, err);
      if (!ok) break;
      tc_fence_after_sync();
      // columns of this slice inside the row's domain; whole warp inside => no masking
      const int n_valid = max(0, min(64, jend - j0));
      const bool interior = __all_sync(0xffffffffu, n_valid == 64);
      float2 st = sweep == 0 ? my_stats[b * 128] : make_float2(0.f, 0.f);
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t x[32];
        tmem_ld32(tmem + 128 * buf + 64 * wg + 32 * c + lane_addr, x);
        tmem_wait_ld();
        float t[32];
        if (interior) {  // the usual case: nothing to mask, no per-entry comparison
#pragma unroll
          for (int e = 0; e < 32; e += 2)
            ffma2(t[e], t[e + 1], __uint_as_float(x[e]), __uint_as_float(x[e + 1]), scale_log2, bias2[32 * c + e],
                  bias2[32 * c + e + 1]);
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e)
            t[e] = 32 * c + e < n_valid ? fmaf(__uint_as_float(x[e]), scale_log2, bias2[32 * c + e]) : -CUDART_INF_F;
        }
        if (sweep == 0) {
          // four independent chains each for the maximum and for the sum
          float m0 = st.x, m1 = -CUDART_INF_F, m2 = -CUDART_INF_F, m3 = -CUDART_INF_F;
#pragma unroll
          for (int e = 0; e < 32; e += 8) {  // three-input maxima: half the instructions
            m0 = fmax3(m0, t[e], t[e + 4]);
            m1 = fmax3(m1, t[e + 1], t[e + 5]);
            m2 = fmax3(m2, t[e + 2], t[e + 6]);
            m3 = fmax3(m3, t[e + 3], t[e + 7]);
          }
          const float cm = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
          const float cm_safe = cm == -CUDART_INF_F ? 0.f : cm;
          float z0 = st.y * ex2_approx(st.x - cm_safe), z1 = 0.f, z2 = 0.f, z3 = 0.f;
          const float neg_cm = -cm_safe;
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            float a0, a1, a2, a3;
            fadd2(a0, a1, t[e], t[e + 1], neg_cm, neg_cm);
            fadd2(a2, a3, t[e + 2], t[e + 3], neg_cm, neg_cm);
            fadd2(z0, z1, z0, z1, ex2_approx(a0), ex2_approx(a1));
            fadd2(z2, z3, z2, z3, ex2_approx(a2), ex2_approx(a3));
          }
          st = make_float2(cm, (z0 + z1) + (z2 + z3));
        } else {
          // running sum over b of the normalised weights, kept in TMEM next to S
          const uint32_t ps_addr = tmem + 256 + 64 * wg + 32 * c + lane_addr;
          uint32_t ps[32];
          if (b > 0) {
            tmem_ld32(ps_addr, ps);
            tmem_wait_ld();
          }
          const float neg_ref = -ref;
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            float a0, a1;
            fadd2(a0, a1, t[e], t[e + 1], neg_ref, neg_ref);
            float p0 = ex2_approx(a0), p1 = ex2_approx(a1);
            if (b > 0) fadd2(p0, p1, __uint_as_float(ps[e]), __uint_as_float(ps[e + 1]), p0, p1);
            ps[e] = __float_as_uint(p0);
            ps[e + 1] = __float_as_uint(p1);
          }
          if (b < Bc - 1) {
            tmem_st32(ps_addr, ps);
          } else if (row_ok) {
            // last sample of this key tile: one addition per accumulator entry and launch,
            // performed in L2 (entries outside the domain are not touched)
            float *arow = acc + ((size_t)h * Lq + i) * Lk + j0 + 32 * c;
            const int nv = n_valid - 32 * c;
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              const int jj = 4 * g;
              if (jj >= nv) break;
              if (vec && jj + 4 <= nv) {
                asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(arow + jj),
                             "f"(__uint_as_float(ps[jj])), "f"(__uint_as_float(ps[jj + 1])),
                             "f"(__uint_as_float(ps[jj + 2])), "f"(__uint_as_float(ps[jj + 3]))
                             : "memory");
              } else {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                  if (jj + e < nv)
                    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(arow + jj + e), "f"(__uint_as_float(ps[jj + e]))
                                 : "memory");
              }
            }
          }
        }
      }
      // S[buf] is consumed: the MMA of visit v + 2 may overwrite it
      if (sweep == 1 && b < Bc - 1) tmem_wait_st();
      tc_fence_before_sync();
      mbar_arrive(&bars->s_empty[buf]);
      if (sweep == 0) my_stats[b * 128] = st;
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 9) tmem_dealloc(tmem, kTmemCols);
}

template <int D>
cudaError_t launch(const CUtensorMap &mq, const CUtensorMap &mk, const CUtensorMap &mb, int bias_by_tma, float *acc,
                   const float *bias, int B, int H, int Lq, int Lk, int causal, int f16, float scale, unsigned *err,
                   cudaStream_t s) {
  auto kern = accumulate_tc_kernel<D>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D>::kSmemBytes);
  if (e != cudaSuccess) return e;
  const int n_qt = ceil_div(Lq, kTile), n_kt = ceil_div(Lk, kTile);
  // samples in ascending order, at most kMaxB per launch; launches on one stream run in order
  for (int b0 = 0; b0 < B; b0 += kMaxB) {
    const int Bc = B - b0 < kMaxB ? B - b0 : kMaxB;
    kern<<<H * n_qt, kThreads, Cfg<D>::kSmemBytes, s>>>(mq, mk, mb, bias_by_tma, acc, bias, b0, Bc, H, Lq, Lk, n_qt,
                                                       n_kt, causal, f16, scale * kLog2e, err);
    count_launches(1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace

cudaError_t launch_accumulate_tc(float *acc, const void *Q, const void *K, const float *bias, int B, int H, int Lq,
                                 int Lk, int d, int causal, int f16, float scale, cudaStream_t s) {
  unsigned *err = device_error_word();
  if (!err) return cudaErrorUnknown;
  CUtensorMap mq, mk;
  if (!make_tile_map_bf16(&mq, Q, B * H, Lq, d) || !make_tile_map_bf16(&mk, K, B * H, Lk, d)) return cudaErrorUnknown;
  // the bias goes through TMA when its rows are 16-byte multiples; otherwise threads load it directly
  CUtensorMap mb = mq;
  const int bias_by_tma = (bias && (Lk & 3) == 0) ? 1 : 0;
  if (bias_by_tma && !make_tile_map_f32(&mb, bias, H, Lq, Lk)) return cudaErrorUnknown;
  return d == 64 ? launch<64>(mq, mk, mb, bias_by_tma, acc, bias, B, H, Lq, Lk, causal, f16, scale, err, s)
                 : launch<128>(mq, mk, mb, bias_by_tma, acc, bias, B, H, Lq, Lk, causal, f16, scale, err, s);
}

}  // namespace ap
