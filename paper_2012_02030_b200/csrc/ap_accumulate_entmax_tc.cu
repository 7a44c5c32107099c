// Eq. 1 with 1.5-entmax in place of the softmax (the section on sparse normalisation), for bf16
// and fp16 tensors, on the tcgen05 tensor cores.
//
// 1.5-entmax of a row of scores z is p_j = max(z_j / 2 - tau, 0)^2 with tau the one number for
// which the row sums to 1.  f(tau) = sum_j max(x_j - tau, 0)^2 - 1 (x = z / 2) is convex and
// decreasing and its root lies in [max x - 1, max x).  On the support of a trial threshold c (the
// n entries with x_j > c) f is the parabola sum (x_j - tau)^2 - 1, whose smaller root is
//     c + (S2 - 1) / (S1 + sqrt(S1^2 - n (S2 - 1))),   S1 = sum (x_j - c), S2 = sum (x_j - c)^2 over the support.
// That root is the answer when the support is the right one; otherwise it lies on the other side
// of the answer than c (too many entries in the support push it right, too few left), the trial
// thresholds left of the answer rise and those right of it fall, so the iteration ends after a
// few supports wherever in [max x - 1, max x) it starts (it starts at max x - 0.625).  Where the parabola has no root (a support far too wide)
// the step is Newton's, (S2 - 1) / (2 S1), which stays left of the answer.
// The scores of a row (up to Lk of them, for every sample) do not fit on the chip, but QK^T is
// cheap on the tensor cores, so the CTA recomputes them: one (head, 128-row query tile) per CTA,
// up to 8 samples per launch,
//   sweep 0          S = Q_b K_b(kt)^T for every key tile and sample -> row maxima, tau = max - 0.625
//   sweeps 1 .. n    the same visits -> n, S1, S2 of every (sample, row) -> one step; repeated
//                    until no row of the CTA moves any more (or kMaxNewton sweeps)
//   last sweep       p = max(x - tau, 0)^2; the sum over samples is kept in TMEM and added to the
//                    accumulator once per key tile (one red.global.add per entry and launch).
// Warp roles, operand staging, bias handling and TMEM layout are those of the softmax kernel:
// warps 0-7 normalise (thread (wg, r) owns row r and columns [64 wg, 64 wg + 64) of every key
// tile), warp 8 copies with TMA, warp 9 issues the products.  The two column halves of a row meet
// in shared memory at the end of every sweep; the copy and product warps learn there whether
// another sweep of the iteration follows.  Every mbarrier wait is bounded.
#include <math_constants.h>

#include "ap_common.cuh"
#include "ap_sm100.cuh"

namespace ap {

namespace {

using namespace sm100;

constexpr int kThreads = 320;
constexpr int kNormThreads = 256;
constexpr int kSubBytes = 128 * 128;
constexpr uint32_t kTmemCols = 512;  // S x 2 (columns 0..255), running sum over b (columns 256..383)
constexpr uint32_t kMaxPolls = 1u << 22;
constexpr int kMaxB = 8;         // samples per launch (row statistics and thresholds live in shared memory)
constexpr int kMaxNewton = 30;   // sweeps of the iteration at most (fp32 steps stop moving long before)
constexpr int kBiasBytes = 128 * 128 * 4;
// The first trial threshold: this far below the row maximum.  The root lies between max - 1 (all the
// weight on one entry) and max; from either side of it the iteration below lands on the other side
// or on the root, and starting in the middle of that range saves a sweep on most rows.
constexpr float kFirstGap = 0.625f;

template <int D>
struct Cfg {
  static constexpr int kSub = D / 64;
  static constexpr int kTileBytes = kSub * kSubBytes;
  static constexpr int kStages = D == 64 ? 3 : 2;
  static constexpr int kBiasOffset = 2 * kStages * kTileBytes;
  static constexpr int kStatsOffset = kBiasOffset + kBiasBytes;
  static constexpr int kStatsBytes = 2 * kMaxB * 128 * 8;  // [wg][b][row] (max, -) or (S1, S2)
  static constexpr int kCntOffset = kStatsOffset + kStatsBytes;
  static constexpr int kCntBytes = 2 * kMaxB * 128 * 4;    // [wg][b][row] support size n
  static constexpr int kTauOffset = kCntOffset + kCntBytes;
  static constexpr int kTauBytes = 2 * kMaxB * 128 * 4;    // [wg][b][row]: each half keeps its own copy
  static constexpr int kBarOffset = kTauOffset + kTauBytes;
  static constexpr int kSmemBytes = kBarOffset + 512 + 1024;
  static_assert(kSmemBytes <= 227 * 1024, "within the shared memory of one CTA");
};

struct Barriers {
  uint64_t s_full[2], s_empty[2];
  uint64_t in_full[3], in_empty[3];
  uint64_t sweep_done;  // all statistics of the sweep are in shared memory
  uint64_t decided;     // all rows have taken their step and said whether they need another
  uint64_t bias_full, bias_empty;
  uint32_t tmem_base;
  int abort_flag;
  int more[kMaxNewton + 2];  // more[s] != 0: some row still moved after sweep s
};

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

// Sweep s + 1 is the last one when sweep s was a sweep of the iteration after which nothing moved.
__device__ __forceinline__ bool last_follows(const Barriers *bars, int s) {
  return s >= 1 && (s >= kMaxNewton || *reinterpret_cast<const volatile int *>(&bars->more[s]) == 0);
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
accumulate_entmax_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                         const __grid_constant__ CUtensorMap map_bias, int bias_by_tma, float *__restrict__ acc,
                         const float *__restrict__ bias, int b0, int Bc, int H, int Lq, int Lk, int n_qt, int n_kt,
                         int causal, int f16, float half_scale, unsigned *err) {
  using C = Cfg<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem =
      reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char *bias_s = smem + C::kBiasOffset;
  float2 *stats = reinterpret_cast<float2 *>(smem + C::kStatsOffset);  // [wg][b][row]
  float *cnts = reinterpret_cast<float *>(smem + C::kCntOffset);       // [wg][b][row]
  float *taus = reinterpret_cast<float *>(smem + C::kTauOffset);       // [wg][b][row]
  Barriers *bars = reinterpret_cast<Barriers *>(smem + C::kBarOffset);

  const int qt = n_qt - 1 - (int)(blockIdx.x / H);  // late query tiles (most key tiles when causal) first
  const int h = blockIdx.x % H;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int off = causal ? Lk - Lq : 0;
  const int n_k = causal ? min(n_kt, (qt * kTile + kTile - 1 + off) / kTile + 1) : n_kt;
  const int visits_per_sweep = n_k * Bc;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->s_full[s], 1);
      mbar_init(&bars->s_empty[s], kNormThreads);
    }
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&bars->in_full[s], 1);
      mbar_init(&bars->in_empty[s], 1);
    }
    mbar_init(&bars->sweep_done, kNormThreads);
    mbar_init(&bars->decided, kNormThreads);
    mbar_init(&bars->bias_full, 1);
    mbar_init(&bars->bias_empty, kNormThreads);
    bars->abort_flag = 0;
    for (int s = 0; s < kMaxNewton + 2; ++s) bars->more[s] = 0;
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
      int v = 0, tl = 0;  // visits issued, bias tiles issued
      bool last = false, ok = true;
      for (int sw = 0; ok; ++sw) {
        for (int vv = 0; vv < visits_per_sweep && ok; ++vv, ++v) {
          const int st = v % C::kStages;
          const uint32_t ph = (uint32_t)(v / C::kStages) & 1u;
          const int kt = vv / Bc, b = b0 + vv % Bc;
          if (bias_by_tma && vv % Bc == 0) {
            if (!wait_or_abort(&bars->bias_empty, ((uint32_t)tl & 1u) ^ 1u, abort_flag, err)) { ok = false; break; }
            mbar_arrive_expect_tx(&bars->bias_full, kBiasBytes);
#pragma unroll
            for (int q = 0; q < 4; ++q)
              tma_load_3d(bias_s + q * (kBiasBytes / 4), &map_bias, &bars->bias_full, kt * kTile + 32 * q, qt * kTile, h);
            ++tl;
          }
          if (!wait_or_abort(&bars->in_empty[st], ph ^ 1u, abort_flag, err)) { ok = false; break; }
          unsigned char *q_s = smem + (2 * st) * C::kTileBytes, *k_s = q_s + C::kTileBytes;
          mbar_arrive_expect_tx(&bars->in_full[st], 2 * C::kTileBytes);
#pragma unroll
          for (int s = 0; s < C::kSub; ++s) {
            tma_load_3d(q_s + s * kSubBytes, &map_q, &bars->in_full[st], 64 * s, qt * kTile, b * H + h);
            tma_load_3d(k_s + s * kSubBytes, &map_k, &bars->in_full[st], 64 * s, kt * kTile, b * H + h);
          }
        }
        if (!ok || last) break;
        if (!wait_or_abort(&bars->decided, (uint32_t)sw & 1u, abort_flag, err)) break;
        last = last_follows(bars, sw);
      }
      if (*abort_flag) {  // winding down: let the copies in flight land (bounded)
        for (int j = max(0, v - C::kStages); j < v; ++j)
          mbar_wait(&bars->in_full[j % C::kStages], (uint32_t)(j / C::kStages) & 1u, kMaxPolls);
        if (tl > 0) mbar_wait(&bars->bias_full, (uint32_t)(tl - 1) & 1u, kMaxPolls);
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(128, 128, false, false, f16 != 0);
      int v = 0;
      bool last = false, ok = true;
      for (int sw = 0; ok; ++sw) {
        for (int vv = 0; vv < visits_per_sweep; ++vv, ++v) {
          const int st = v % C::kStages;
          const uint32_t ph = (uint32_t)(v / C::kStages) & 1u;
          const int buf = v & 1;
          if (!wait_or_abort(&bars->in_full[st], ph, abort_flag, err)) { ok = false; break; }
          if (!wait_or_abort(&bars->s_empty[buf], ((uint32_t)(v >> 1) & 1u) ^ 1u, abort_flag, err)) { ok = false; break; }
          tc_fence_after_sync();
          const unsigned char *q_s = smem + (2 * st) * C::kTileBytes, *k_s = q_s + C::kTileBytes;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const int sub = ks / 4, o = (ks % 4) * 32;
            const uint64_t da = smem_desc_sw128(smem_u32(q_s + sub * kSubBytes + o), 16, 1024);
            const uint64_t db = smem_desc_sw128(smem_u32(k_s + sub * kSubBytes + o), 16, 1024);
            mma_ss(tmem + 128 * buf, da, db, idesc, ks > 0);
          }
          mma_commit(&bars->in_empty[st]);
          mma_commit(&bars->s_full[buf]);
        }
        if (!ok || last) break;
        if (!wait_or_abort(&bars->decided, (uint32_t)sw & 1u, abort_flag, err)) break;
        last = last_follows(bars, sw);
      }
    }
  } else {
    // ------------------------------------------------------------ normalisation (256 threads)
    const int wg = warp >> 2;
    const int r = (warp & 3) * 32 + lane;  // row of the tile == TMEM lane
    const int i = qt * kTile + r;
    const bool row_ok = i < Lq;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const int jend = causal ? min(Lk, i + 1 + off) : Lk;  // first key outside this row's domain
    const bool vec = (Lk & 3) == 0;
    float2 *my_stats = stats + (size_t)wg * kMaxB * 128 + r;  // + b * 128
    float *my_cnt = cnts + (size_t)wg * kMaxB * 128 + r;      // + b * 128
    float *my_tau = taus + (size_t)wg * kMaxB * 128 + r;      // + b * 128

    float hbias[64];  // half the bias of this thread's 64 columns of the current key tile
    int v = 0, tl = 0;
    bool last = false, ok = true;
    for (int sw = 0; ok; ++sw) {
      const int kind = sw == 0 ? 0 : (last ? 2 : 1);  // 0 maxima, 1 sums over the support, 2 weights
      // (key tile, sample) of the visit, stepped rather than divided out of vv: an integer division per
      // visit is a hundred cycles on this thread's critical path
      int kt = 0, b = -1;
      for (int vv = 0; vv < visits_per_sweep && ok; ++vv, ++v) {
        if (++b == Bc) {
          b = 0;
          ++kt;
        }
        const int buf = v & 1;
        const int j0 = kt * kTile + 64 * wg;  // first column of this thread's slice
        if (b == 0) {  // new key tile: fetch this thread's bias slice once for all samples
          if (bias_by_tma) {
            ok = wait_or_abort(&bars->bias_full, (uint32_t)tl & 1u, abort_flag, err);
            if (!ok) break;
            ++tl;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const unsigned char *box = bias_s + (2 * wg + q) * (kBiasBytes / 4) + r * 128;
#pragma unroll
              for (int k = 0; k < 8; ++k) {  // 16-byte chunk k of the row sits at position k ^ (r % 8)
                const float4 t = *reinterpret_cast<const float4 *>(box + ((k ^ (r & 7)) << 4));
                hbias[32 * q + 4 * k] = t.x * 0.5f; hbias[32 * q + 4 * k + 1] = t.y * 0.5f;
                hbias[32 * q + 4 * k + 2] = t.z * 0.5f; hbias[32 * q + 4 * k + 3] = t.w * 0.5f;
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
              hbias[4 * c] = t.x * 0.5f; hbias[4 * c + 1] = t.y * 0.5f;
              hbias[4 * c + 2] = t.z * 0.5f; hbias[4 * c + 3] = t.w * 0.5f;
            }
          }
        }
        const float neg_tau = kind == 0 ? 0.f : -my_tau[b * 128];
        // statistics of (sample b, this half of the row): fresh at the first key tile of a sweep
        float2 st = kt == 0 ? make_float2(kind == 0 ? -CUDART_INF_F : 0.f, 0.f) : my_stats[b * 128];
        float cnt = (kind != 1 || kt == 0) ? 0.f : my_cnt[b * 128];
        ok = wait_or_abort(&bars->s_full[buf], (uint32_t)(v >> 1) & 1u, abort_flag, err);
        if (!ok) break;
        tc_fence_after_sync();
        const int n_valid = max(0, min(64, jend - j0));  // columns of this slice inside the row's domain
        const bool interior = __all_sync(0xffffffffu, n_valid == 64);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t x[32];
          tmem_ld32(tmem + 128 * buf + 64 * wg + 32 * c + lane_addr, x);
          tmem_wait_ld();
          float t[32];  // x_j = (scale * q.k_j + bias_j) / 2, -inf outside the domain
          if (interior) {
#pragma unroll
            for (int e = 0; e < 32; e += 2)
              ffma2(t[e], t[e + 1], __uint_as_float(x[e]), __uint_as_float(x[e + 1]), half_scale, hbias[32 * c + e],
                    hbias[32 * c + e + 1]);
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e)
              t[e] = 32 * c + e < n_valid ? fmaf(__uint_as_float(x[e]), half_scale, hbias[32 * c + e]) : -CUDART_INF_F;
          }
          if (kind == 0) {
            float m0 = st.x, m1 = -CUDART_INF_F, m2 = -CUDART_INF_F, m3 = -CUDART_INF_F;
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
              m0 = fmax3(m0, t[e], t[e + 4]);
              m1 = fmax3(m1, t[e + 1], t[e + 5]);
              m2 = fmax3(m2, t[e + 2], t[e + 6]);
              m3 = fmax3(m3, t[e + 3], t[e + 7]);
            }
            st.x = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
          } else if (kind == 1) {
            // four independent chains each for S1 and S2
            float a0 = st.x, a1 = 0.f, a2 = 0.f, a3 = 0.f, q0 = st.y, q1 = 0.f, q2 = 0.f, q3 = 0.f;
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
              // max(x - tau, 0) as a saturating add: every trial threshold is at least max - 1 (the
              // root's lower bound), so x - tau <= 1 and clamping to [0, 1] clamps at 0 only; the add
              // runs on the FMA pipe, a separate maximum would load the half-rate ALU pipe
              const float u0 = __saturatef(t[e] + neg_tau), u1 = __saturatef(t[e + 1] + neg_tau);
              const float u2 = __saturatef(t[e + 2] + neg_tau), u3 = __saturatef(t[e + 3] + neg_tau);
              fadd2(a0, a1, a0, a1, u0, u1);
              fadd2(a2, a3, a2, a3, u2, u3);
              ffma2v(q0, q1, u0, u1, u0, u1, q0, q1);
              ffma2v(q2, q3, u2, u3, u2, u3, q2, q3);
              cnt += ((u0 > 0.f ? 1.f : 0.f) + (u1 > 0.f ? 1.f : 0.f)) + ((u2 > 0.f ? 1.f : 0.f) + (u3 > 0.f ? 1.f : 0.f));
            }
            st = make_float2((a0 + a1) + (a2 + a3), (q0 + q1) + (q2 + q3));
          } else {
            // running sum over b of the weights, kept in TMEM next to S
            const uint32_t ps_addr = tmem + 256 + 64 * wg + 32 * c + lane_addr;
            uint32_t ps[32];
            if (b > 0) {
              tmem_ld32(ps_addr, ps);
              tmem_wait_ld();
            }
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              float p0, p1;
              const float u0 = __saturatef(t[e] + neg_tau), u1 = __saturatef(t[e + 1] + neg_tau);
              if (b > 0) {
                ffma2v(p0, p1, u0, u1, u0, u1, __uint_as_float(ps[e]), __uint_as_float(ps[e + 1]));
              } else {
                p0 = u0 * u0; p1 = u1 * u1;
              }
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
        // S[buf] is consumed: the product of visit v + 2 may overwrite it
        if (kind == 2 && b < Bc - 1) tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(&bars->s_empty[buf]);
        if (kind != 2) my_stats[b * 128] = st;
        if (kind == 1) my_cnt[b * 128] = cnt;
      }
      if (!ok || last) break;
      // ---- end of a sweep: the two halves of every row meet, every (sample, row) takes its step
      mbar_arrive(&bars->sweep_done);
      ok = wait_or_abort(&bars->sweep_done, (uint32_t)sw & 1u, abort_flag, err);
      if (!ok) break;
      bool moved = false;
      for (int b = 0; b < Bc; ++b) {
        const float2 s0 = stats[(size_t)b * 128 + r], s1 = stats[(size_t)(kMaxB + b) * 128 + r];
        float tau;
        if (sw == 0) {
          tau = fmaxf(s0.x, s1.x) - kFirstGap;
        } else {
          tau = my_tau[b * 128];
          const float S1 = s0.x + s1.x, S2 = s0.y + s1.y;
          const float n = cnts[(size_t)b * 128 + r] + cnts[(size_t)(kMaxB + b) * 128 + r];
          // root of the support's parabola; Newton's step where it has none
          const float disc = S1 * S1 - n * (S2 - 1.f);
          const float step = S1 > 0.f ? (S2 - 1.f) / (S1 + (disc >= 0.f ? sqrtf(disc) : S1)) : 0.f;
          tau += step;
          // below the resolution of tau itself a step is rounding noise of the sums
          moved = moved || fabsf(step) > 2e-6f * fmaxf(1.f, fabsf(tau));
        }
        my_tau[b * 128] = tau;
      }
      if (moved && row_ok) *reinterpret_cast<volatile int *>(&bars->more[sw]) = 1;
      mbar_arrive(&bars->decided);  // release: the flag and the old statistics' last reads precede it
      ok = wait_or_abort(&bars->decided, (uint32_t)sw & 1u, abort_flag, err);
      if (!ok) break;
      last = last_follows(bars, sw);
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
  auto kern = accumulate_entmax_kernel<D>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D>::kSmemBytes);
  if (e != cudaSuccess) return e;
  const int n_qt = ceil_div(Lq, kTile), n_kt = ceil_div(Lk, kTile);
  // samples in ascending order, at most kMaxB per launch; launches on one stream run in order
  for (int b0 = 0; b0 < B; b0 += kMaxB) {
    const int Bc = B - b0 < kMaxB ? B - b0 : kMaxB;
    kern<<<H * n_qt, kThreads, Cfg<D>::kSmemBytes, s>>>(mq, mk, mb, bias_by_tma, acc, bias, b0, Bc, H, Lq, Lk, n_qt,
                                                       n_kt, causal, f16, 0.5f * scale, err);
    count_launches(1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace

cudaError_t launch_accumulate_entmax_tc(float *acc, const void *Q, const void *K, const float *bias, int B, int H,
                                        int Lq, int Lk, int d, int causal, int f16, float scale, cudaStream_t s) {
  unsigned *err = device_error_word();
  if (!err) return cudaErrorUnknown;
  CUtensorMap mq, mk;
  if (!make_tile_map_bf16(&mq, Q, B * H, Lq, d) || !make_tile_map_bf16(&mk, K, B * H, Lk, d)) return cudaErrorUnknown;
  CUtensorMap mb = mq;
  const int bias_by_tma = (bias && (Lk & 3) == 0) ? 1 : 0;
  if (bias_by_tma && !make_tile_map_f32(&mb, bias, H, Lq, Lk)) return cudaErrorUnknown;
  return d == 64 ? launch<64>(mq, mk, mb, bias_by_tma, acc, bias, B, H, Lq, Lk, causal, f16, scale, err, s)
                 : launch<128>(mq, mk, mb, bias_by_tma, acc, bias, B, H, Lq, Lk, causal, f16, scale, err, s);
}

}  // namespace ap
