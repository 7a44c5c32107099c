// Eq. 1 as a running sum for bf16 and fp16 tensors, on the tcgen05 tensor cores.
//
// One CTA owns one (head, 128-row query tile) and adds, for up to 32 samples b per launch,
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
// a fixed thread and every accumulator entry receives exactly one addition per CTA that
// owns it, so results are reproducible bit for bit.  Shapes with few (head, query tile)
// pairs would leave most SMs idle; for them a launch's samples are cut into chunks, one
// CTA per (chunk, head, query tile), and the chunks' sums are added to the accumulator
// in ascending chunk order: per key tile a counter in global memory says how many warps
// of lower chunks have finished their addition, and a CTA waits (bounded) for its turn
// before it issues its own.  Where the accumulator's rows are
// 16-byte multiples that addition is a TMA reduction: each softmax warp stages its
// 32 rows x 32 columns in shared memory (128-byte swizzle again) and one lane issues
// cp.reduce.async.bulk.tensor ... add, which updates whole 128-byte lines in L2;
// a lane per row adding 16 bytes at a time would touch 32 lines per instruction.  Inside
// a tile that straddles the edge of a causal domain the reduction adds exact zeros to the
// entries outside the domain (boxes wholly outside are skipped).  Other shapes keep the
// per-row red.global.add.
//
// Warp roles (320 threads, one CTA per SM): warps 0-7 softmax; thread (wg, r)
// with wg = warp / 4 owns row r of the tile and columns [64 wg, 64 wg + 64) of
// every key tile; warp 8 TMA producer; warp 9 MMA issuer and TMEM owner.  S is
// double-buffered in TMEM (2 x 128 columns) so the MMA of the next visit runs
// under the softmax of the current one; a visit's 64 columns are copied to registers in one
// go and S is handed back before the arithmetic starts.  TMEM columns 256-383 hold the running
// sum over b, columns 384-511 the per-sample (maximum, sum) pairs of both column halves, which
// a thread reads back for its own row (lane) at the start of sweep 2.  Every mbarrier wait is
// bounded.
#include <math_constants.h>

#include <atomic>

#include "ap_common.cuh"
#include "ap_sm100.cuh"

namespace ap {

namespace {

using namespace sm100;

constexpr int kThreads = 320;
constexpr int kSoftmaxThreads = 256;
constexpr int kSoftmaxWarps = kSoftmaxThreads / 32;
constexpr int kSubBytes = 128 * 128;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kSumCol = 256;    // running sum over b: 128 columns
constexpr uint32_t kStatsCol = 384;  // (max, sum) pairs: 64 columns per column half, 2 per sample
constexpr int kMaxB = 32;            // samples per launch (what the spare tensor-memory columns hold)
constexpr int kBiasBytes = 128 * 128 * 4;  // one fp32 bias tile: 4 boxes of 128 rows x 32 columns
constexpr int kRedBytes = 32 * 128;        // per softmax warp: 32 rows x 32 fp32 columns on their way to the accumulator
constexpr float kLog2e = 1.4426950408889634f;

template <int D>
struct Cfg {
  static constexpr int kSub = D / 64;
  static constexpr int kTileBytes = kSub * kSubBytes;    // one operand tile (Q or K)
  static constexpr int kStages = D == 64 ? 4 : 2;        // (Q, K) pairs in flight
  static constexpr int kBiasOffset = 2 * kStages * kTileBytes;
  static constexpr int kRedOffset = kBiasOffset + kBiasBytes;
  static constexpr int kBarOffset = kRedOffset + kSoftmaxWarps * kRedBytes;
  static constexpr int kSmemBytes = kBarOffset + 256 + 1024;
  static_assert(kSmemBytes <= 227 * 1024, "within the shared memory of one CTA");
};

struct Barriers {
  uint64_t s_full[2], s_empty[2];
  uint64_t in_full[4], in_empty[4];
  uint64_t sweep1_done;  // all softmax warps have stored their sweep-1 statistics
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

__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned *p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Turn counters of the chunked launches: one word per (head, query tile, key tile), zeroed before every
// such launch.  Launches that overlap on the GPU (different streams) take different sets.
constexpr size_t kTurnWords = 8192;
constexpr int kTurnSets = 8;
constexpr int kMinChunk = 2;  // samples per CTA at least
__device__ unsigned g_turn[kTurnSets][kTurnWords];

unsigned *turn_words() {
  static std::atomic<unsigned> next{0};
  static unsigned *base[16] = {nullptr};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 16) return nullptr;
  if (!base[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_turn) != cudaSuccess) return nullptr;
    base[dev] = static_cast<unsigned *>(p);
  }
  return base[dev] + (size_t)(next.fetch_add(1) % kTurnSets) * kTurnWords;
}

// Bounded wait that also gives up as soon as another thread of the CTA has.
__device__ __noinline__ bool wait_or_abort(uint64_t *bar, uint32_t parity, volatile int *abort_flag, unsigned *err,
                                           uint32_t max_polls) {
  for (uint32_t i = 0; i < max_polls; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (i > 1024) __nanosleep(64);
  }
  *abort_flag = 1;
  atomicOr(err, kDevErrTimeout);
  return false;
}

// The same wait for a whole (converged) warp: one lane polls - 32 lanes polling one barrier would
// serialise - and the outcome is shared.
__device__ __forceinline__ bool warp_wait(uint64_t *bar, uint32_t parity, int lane, volatile int *abort_flag,
                                          unsigned *err, uint32_t max_polls) {
  bool ok = true;
  if (lane == 0 && !mbar_try_wait(bar, parity)) ok = wait_or_abort(bar, parity, abort_flag, err, max_polls);
  return __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
}

// dbg_skip != 0 (test hook): the copies of the first visit are never issued, so the MMA issuer's
// first wait runs out and the CTA leaves through its error path.
// kChunked: the instantiation for launches whose samples are cut into chunks (see below); a
// separate one so that its extra code costs the plain launches nothing.
template <int D, bool kChunked>
__global__ void __launch_bounds__(kThreads, 1)
accumulate_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_bias, const __grid_constant__ CUtensorMap map_acc,
                     int bias_by_tma, int acc_by_tma, float *__restrict__ acc, const float *__restrict__ bias, int b0,
                     int Bc_all, int chunk_samples, unsigned *__restrict__ turn, int H, int Lq, int Lk, int n_qt,
                     int n_kt, int causal, int f16, float scale_log2, unsigned *err, uint32_t max_polls, int dbg_skip) {
  using C = Cfg<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem =
      reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char *bias_s = smem + C::kBiasOffset;
  Barriers *bars = reinterpret_cast<Barriers *>(smem + C::kBarOffset);

  // Small shapes have fewer (head, query tile) pairs than the GPU has SMs; the launch's samples are
  // then cut into chunks, CTA (chunk, head, query tile) takes chunk_samples of them, and the chunks'
  // sums are added to the accumulator in ascending order of the chunks (turn[], see below), so that
  // the result does not depend on which CTA finishes first.  Lower chunks have lower block indices.
  const int unit = kChunked ? (int)blockIdx.x % (H * n_qt) : (int)blockIdx.x;
  const int chunk = kChunked ? (int)blockIdx.x / (H * n_qt) : 0;
  if (kChunked) b0 += chunk * chunk_samples;
  const int Bc = kChunked ? min(chunk_samples, Bc_all - chunk * chunk_samples) : Bc_all;
  // late query tiles (most key tiles under a causal mask) first
  const int qt = n_qt - 1 - unit / H;
  const int h = unit % H;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // causal: row i looks at keys j <= i + (Lk - Lq), i.e. Lk - Lq memory keys, then its own segment
  const int off = causal ? Lk - Lq : 0;
  const int n_k = causal ? min(n_kt, (qt * kTile + kTile - 1 + off) / kTile + 1) : n_kt;  // key tiles of this query tile
  const int visits_per_sweep = n_k * Bc;
  const int n_visits = 2 * visits_per_sweep;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&bars->s_full[s], 1);
      mbar_init(&bars->s_empty[s], kSoftmaxWarps);  // one arrival per softmax warp
    }
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&bars->in_full[s], 1);
      mbar_init(&bars->in_empty[s], 1);
    }
    mbar_init(&bars->sweep1_done, kSoftmaxWarps);
    mbar_init(&bars->bias_full, 1);
    mbar_init(&bars->bias_empty, kSoftmaxWarps);
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
          if (!wait_or_abort(&bars->bias_empty, ((uint32_t)tl & 1u) ^ 1u, abort_flag, err, max_polls)) break;
          mbar_arrive_expect_tx(&bars->bias_full, kBiasBytes);
#pragma unroll
          for (int q = 0; q < 4; ++q)
            tma_load_3d(bias_s + q * (kBiasBytes / 4), &map_bias, &bars->bias_full, kt * kTile + 32 * q, qt * kTile, h);
          bias_loads = tl + 1;
        }
        if (!wait_or_abort(&bars->in_empty[st], ph ^ 1u, abort_flag, err, max_polls)) break;
        if (dbg_skip != 0 && v == 0) continue;
        unsigned char *q_s = smem + (2 * st) * C::kTileBytes, *k_s = q_s + C::kTileBytes;
        mbar_arrive_expect_tx(&bars->in_full[st], 2 * C::kTileBytes);
#pragma unroll
        for (int s = 0; s < C::kSub; ++s) {
          tma_load_3d(q_s + s * kSubBytes, &map_q, &bars->in_full[st], 64 * s, qt * kTile, b * H + h);
          tma_load_3d(k_s + s * kSubBytes, &map_k, &bars->in_full[st], 64 * s, kt * kTile, b * H + h);
        }
      }
      if (*abort_flag) {  // winding down: let the copies in flight land (bounded)
        for (int j = max(0, v - C::kStages); j < v; ++j) {
          if (dbg_skip != 0 && j == 0) continue;
          mbar_wait(&bars->in_full[j % C::kStages], (uint32_t)(j / C::kStages) & 1u, max_polls);
        }
        if (bias_loads > 0) mbar_wait(&bars->bias_full, (uint32_t)(bias_loads - 1) & 1u, max_polls);
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
        if (!wait_or_abort(&bars->in_full[st], ph, abort_flag, err, max_polls)) break;
        if (!wait_or_abort(&bars->s_empty[buf], ((uint32_t)(v >> 1) & 1u) ^ 1u, abort_flag, err, max_polls)) break;
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
    const uint32_t s_addr = tmem + lane_addr + 64 * wg;                   // + 128 * buf
    const uint32_t sum_addr = tmem + lane_addr + kSumCol + 64 * wg;       // + 32 * c
    const uint32_t my_stats = tmem + lane_addr + kStatsCol + 64 * wg;     // + 2 * b
    const uint32_t other_stats = tmem + lane_addr + kStatsCol + 64 * (1 - wg);
    // this warp's 32 rows x 32 columns on their way to the accumulator, and the rows' place in it
    unsigned char *red_s = smem + C::kRedOffset + warp * kRedBytes;
    const int red_y = qt * kTile + (warp & 3) * 32;
    const int red_jend = causal ? min(Lk, red_y + 32 + off) : Lk;  // first key outside the domain of all 32 rows

    for (int b = 0; b < Bc; ++b) tmem_st2(my_stats + 2 * b, __float_as_uint(-CUDART_INF_F), 0u);

    float bias2[64];  // bias * log2(e) of this thread's 64 columns of the current key tile
    bool ok = true;
    // the bias slice of key tile kt (tl: how many tiles were staged before it), once for all samples
    auto fetch_bias = [&](int kt, int tl) {
      const int j0 = kt * kTile + 64 * wg;
      if (bias_by_tma) {
        ok = warp_wait(&bars->bias_full, (uint32_t)tl & 1u, lane, abort_flag, err, max_polls);
        if (!ok) return;
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
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->bias_empty);
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
    };
    // S of visit v is ready: copy this thread's 64 columns to registers and hand S back.  The MMA of
    // visit v + 2 may then overwrite the buffer while the arithmetic on the copy is still going on
    // (one arrival per warp: 256 threads arriving one by one would take longer than a visit's MMAs).
    auto take_s = [&](int v, uint32_t (&xs)[64]) {
      const int buf = v & 1;
      ok = warp_wait(&bars->s_full[buf], (uint32_t)(v >> 1) & 1u, lane, abort_flag, err, max_polls);
      if (!ok) return;
      tc_fence_after_sync();
      tmem_ld32(s_addr + 128 * buf, xs);
      tmem_ld32(s_addr + 128 * buf + 32, xs + 32);
    };
    auto release_s = [&](int v) {
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->s_empty[v & 1]);
    };

    // ---- sweep 1: per sample and row, the maximum and the sum of exp2 over this thread's columns
    int v = 0;
    for (int kt = 0; kt < n_k && ok; ++kt) {
      fetch_bias(kt, kt);
      if (!ok) break;
      // columns of this slice inside the row's domain; whole warp inside => no masking
      const int n_valid = max(0, min(64, jend - (kt * kTile + 64 * wg)));
      const bool interior = __all_sync(0xffffffffu, n_valid == 64);
      for (int b = 0; b < Bc; ++b, ++v) {
        uint32_t xs[64], sv[2];
        take_s(v, xs);
        if (!ok) break;
        tmem_wait_st();  // this sample's pair as the previous key tile left it
        tmem_ld2(my_stats + 2 * b, sv);
        tmem_wait_ld();
        release_s(v);
        float t[64];
#pragma unroll
        for (int e = 0; e < 64; e += 2)
          ffma2(t[e], t[e + 1], __uint_as_float(xs[e]), __uint_as_float(xs[e + 1]), scale_log2, bias2[e], bias2[e + 1]);
        if (!interior) {
#pragma unroll
          for (int e = 0; e < 64; ++e) t[e] = e < n_valid ? t[e] : -CUDART_INF_F;
        }
        const float m_old = __uint_as_float(sv[0]);
        // four independent chains each for the maximum and for the sum
        float m0 = m_old, m1 = -CUDART_INF_F, m2 = -CUDART_INF_F, m3 = -CUDART_INF_F;
#pragma unroll
        for (int e = 0; e < 64; e += 8) {  // three-input maxima: half the instructions
          m0 = fmax3(m0, t[e], t[e + 4]);
          m1 = fmax3(m1, t[e + 1], t[e + 5]);
          m2 = fmax3(m2, t[e + 2], t[e + 6]);
          m3 = fmax3(m3, t[e + 3], t[e + 7]);
        }
        const float cm = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
        const float cm_safe = cm == -CUDART_INF_F ? 0.f : cm;
        float z0 = __uint_as_float(sv[1]) * ex2_approx(m_old - cm_safe), z1 = 0.f, z2 = 0.f, z3 = 0.f;
        const float neg_cm = -cm_safe;
#pragma unroll
        for (int e = 0; e < 64; e += 4) {
          float a0, a1, a2, a3;
          fadd2(a0, a1, t[e], t[e + 1], neg_cm, neg_cm);
          fadd2(a2, a3, t[e + 2], t[e + 3], neg_cm, neg_cm);
          fadd2(z0, z1, z0, z1, ex2_approx(a0), ex2_approx(a1));
          fadd2(z2, z3, z2, z3, ex2_approx(a2), ex2_approx(a3));
        }
        tmem_st2(my_stats + 2 * b, __float_as_uint(cm), __float_as_uint((z0 + z1) + (z2 + z3)));
      }
    }
    if (ok) {
      // every statistic of sweep 1 is final once both column halves of every row are done
      tmem_wait_st();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->sweep1_done);
      ok = warp_wait(&bars->sweep1_done, 0, lane, abort_flag, err, max_polls);
      tc_fence_after_sync();
    }

    // ---- sweep 2: normalised weights, summed over b in TMEM, added to the accumulator per key tile
    for (int kt = 0; kt < n_k && ok; ++kt) {
      fetch_bias(kt, n_k + kt);
      if (!ok) break;
      const int j0 = kt * kTile + 64 * wg;  // first column of this thread's slice
      const int n_valid = max(0, min(64, jend - j0));
      const bool interior = __all_sync(0xffffffffu, n_valid == 64);
      for (int b = 0; b < Bc; ++b, ++v) {
        uint32_t xs[64], s0[2], s1[2];
        take_s(v, xs);
        if (!ok) break;
        tmem_ld2(my_stats + 2 * b, s0);
        tmem_ld2(other_stats + 2 * b, s1);
        tmem_wait_ld();
        release_s(v);
        // both column halves' statistics of sample b combined: max + log2(sum).  A row without any key
        // in its domain (possible when Lk < Lq) gets weight 0 everywhere.
        const float mm = fmaxf(__uint_as_float(s0[0]), __uint_as_float(s1[0]));
        const float z = __uint_as_float(s0[1]) * ex2_approx(__uint_as_float(s0[0]) - mm) +
                        __uint_as_float(s1[1]) * ex2_approx(__uint_as_float(s1[0]) - mm);
        const float neg_ref = jend > 0 ? -(mm + lg2_approx(z)) : -CUDART_INF_F;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          float p[32];
#pragma unroll
          for (int e = 0; e < 32; e += 2)
            ffma2(p[e], p[e + 1], __uint_as_float(xs[32 * c + e]), __uint_as_float(xs[32 * c + e + 1]), scale_log2,
                  bias2[32 * c + e], bias2[32 * c + e + 1]);
          if (!interior) {
#pragma unroll
            for (int e = 0; e < 32; ++e) p[e] = 32 * c + e < n_valid ? p[e] : -CUDART_INF_F;
          }
          uint32_t ps[32];
          if (b > 0) {
            tmem_ld32(sum_addr + 32 * c, ps);
            tmem_wait_ld();
          }
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            float a0, a1;
            fadd2(a0, a1, p[e], p[e + 1], neg_ref, neg_ref);
            float p0 = ex2_approx(a0), p1 = ex2_approx(a1);
            if (b > 0) fadd2(p0, p1, __uint_as_float(ps[e]), __uint_as_float(ps[e + 1]), p0, p1);
            ps[e] = __float_as_uint(p0);
            ps[e + 1] = __float_as_uint(p1);
          }
          if (b < Bc - 1) {
            tmem_st32(sum_addr + 32 * c, ps);
          } else if (acc_by_tma) {
            // last sample of this key tile: one addition per accumulator entry and launch, performed
            // in L2 by a TMA reduction of this warp's 32 x 32 block
            if (lane == 0) bulk_wait_group_read0();  // the block staged before has been read
            __syncwarp();
#pragma unroll
            for (int k = 0; k < 8; ++k)  // 16-byte chunk k of row `lane` goes to position k ^ (lane % 8)
              *reinterpret_cast<uint4 *>(red_s + lane * 128 + ((k ^ (lane & 7)) << 4)) =
                  make_uint4(ps[4 * k], ps[4 * k + 1], ps[4 * k + 2], ps[4 * k + 3]);
            fence_proxy_async_smem();
            __syncwarp();
            const int x = j0 + 32 * c;
            if (kChunked && c == 0) {
              // this key tile's entries have received the sums of all lower chunks once their eight
              // warps each have counted themselves in (bounded wait)
              if (lane == 0) {
                const unsigned *flag = turn + ((size_t)h * n_qt + qt) * n_kt + kt;
                const unsigned want = (unsigned)chunk * kSoftmaxWarps;
                uint32_t polls = 0;
                while (ld_acquire_gpu(flag) < want && ok) {
                  if (*abort_flag || ++polls > max_polls) {
                    if (!*abort_flag) {
                      *abort_flag = 1;
                      atomicOr(err, kDevErrTimeout);
                    }
                    ok = false;
                  } else if (polls > 64) {
                    __nanosleep(128);
                  }
                }
              }
              ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
              if (!ok) break;
            }
            if (lane == 0 && red_y < Lq && x < red_jend) {
              tma_reduce_add_3d(&map_acc, red_s, x, red_y, h);
              bulk_commit_group();
            }
            if (kChunked && c == 1 && lane == 0) {
              // both blocks of this warp are in the accumulator: count this warp in for the next chunk
              bulk_wait_group0();
              __threadfence();
              atomicAdd(turn + ((size_t)h * n_qt + qt) * n_kt + kt, 1u);
            }
          } else if (row_ok) {
            // accumulator rows that are no 16-byte multiples: one red per entry (entries outside the
            // domain are not touched)
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
        // the sums must be in TMEM before the next visit reads them
        if (b < Bc - 1) tmem_wait_st();
      }
    }
    if (lane == 0) bulk_wait_group0();  // shared memory stays valid until the reductions have read it
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 9) tmem_dealloc(tmem, kTmemCols);
}

template <int D>
cudaError_t launch(const CUtensorMap &mq, const CUtensorMap &mk, const CUtensorMap &mb, const CUtensorMap &ma,
                   int bias_by_tma, int acc_by_tma, float *acc, const float *bias, int B, int H, int Lq, int Lk,
                   int causal, int f16, float scale, unsigned *err, cudaStream_t s) {
  auto kern = accumulate_tc_kernel<D, false>;
  auto kern_chunked = accumulate_tc_kernel<D, true>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D>::kSmemBytes);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(kern_chunked, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D>::kSmemBytes);
  if (e != cudaSuccess) return e;
  const int n_qt = ceil_div(Lq, kTile), n_kt = ceil_div(Lk, kTile);
  const DebugKnobs knobs = debug_knobs();
  // Shapes with at most half as many (head, query tile) pairs as SMs: several CTAs per pair, each with
  // a chunk of the samples, taking turns at the accumulator (one wave of CTAs, one per SM).
  const int n_units = H * n_qt, sms = sm_count();
  int max_chunks = 1;
  unsigned *turn = nullptr;
  if (acc_by_tma && !knobs.skip_arrive && sms > 0 && 2 * n_units <= sms && (size_t)n_units * n_kt <= kTurnWords) {
    turn = turn_words();
    if (turn) max_chunks = sms / n_units;
  }
  // samples in ascending order, at most kMaxB per CTA and launch; launches on one stream run in order
  for (int b0 = 0; b0 < B;) {
    const int left = B - b0;
    int chunks = 1, per = left < kMaxB ? left : kMaxB;
    if (max_chunks > 1 && left >= 2 * kMinChunk) {
      chunks = left / kMinChunk < max_chunks ? left / kMinChunk : max_chunks;
      per = ceil_div(left, chunks);
      if (per > kMaxB) per = kMaxB;
      chunks = ceil_div(left < chunks * per ? left : chunks * per, per);
    }
    const int Bc = left < chunks * per ? left : chunks * per;
    unsigned *t = chunks > 1 ? turn : nullptr;
    if (t && (e = cudaMemsetAsync(t, 0, (size_t)n_units * n_kt * sizeof(unsigned), s)) != cudaSuccess) return e;
    (t ? kern_chunked : kern)<<<knobs.skip_arrive ? 1 : n_units * chunks, kThreads, Cfg<D>::kSmemBytes, s>>>(
        mq, mk, mb, ma, bias_by_tma, acc_by_tma, acc, bias, b0, Bc, per, t, H, Lq, Lk, n_qt, n_kt, causal, f16,
        scale * kLog2e, err, knobs.max_polls, knobs.skip_arrive);
    count_launches(1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    b0 += Bc;
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
  // so does the accumulator's update (32-row boxes, one per softmax warp)
  CUtensorMap ma = mq;
  const int acc_by_tma = (Lk & 3) == 0 ? 1 : 0;
  if (acc_by_tma && !make_tile_map_f32(&ma, acc, H, Lq, Lk, 32)) return cudaErrorUnknown;
  return d == 64
             ? launch<64>(mq, mk, mb, ma, bias_by_tma, acc_by_tma, acc, bias, B, H, Lq, Lk, causal, f16, scale, err, s)
             : launch<128>(mq, mk, mb, ma, bias_by_tma, acc_by_tma, acc, bias, B, H, Lq, Lk, causal, f16, scale, err, s);
}

}  // namespace ap
