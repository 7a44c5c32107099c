// Masked attention of Section 3.2 with 1.5-entmax as the normaliser (the section on sparse
// normalisation), for bf16 and fp16 tensors, on the tcgen05 tensor cores:
//   O[b,h,i,:] = sum_j p_j V[b,h,j,:],   p = entmax15( scale * Q[b,h,i,:].K[b,h,j,:] : j kept by the mask ),
//   entmax15(z)_j = max(z_j / 2 - tau, 0)^2 with tau such that the row sums to 1; a row without
//   kept entries outputs 0.
// Unlike a softmax, the weights cannot be formed in one pass with a running correction: tau depends
// on all kept scores of the row.  One CTA owns one (b, h, 128-row query tile) and sweeps the rounds
// of its list row (the schedule of the tile list: up to eight non-empty groups of 16 key columns,
// taken from one or several key tiles, per round) several times, recomputing S = Q K^T on the tensor
// cores each time:
//   sweep 0          row maxima over the kept entries, tau = max - 0.625 (the root lies in [max - 1, max))
//   sweeps 1 .. n    over the support of the trial threshold (the n entries with x > tau):
//                    S1 = sum (x - tau), S2 = sum (x - tau)^2 -> tau moves to the smaller root of the
//                    support's parabola, tau + (S2 - 1) / (S1 + sqrt(S1^2 - n (S2 - 1))), which is the
//                    answer once the support is right and lies on the other side of it otherwise
//                    (Newton's step (S2 - 1) / (2 S1) where the parabola has no root); until no row
//                    of the CTA moves (or kMaxNewton sweeps)
//   last sweep       P = max(x - tau, 0)^2 rounded to the tensors' type, written over S in TMEM;
//                    O += P V (A operand from TMEM); the epilogue divides by the sum of the rounded
//                    weights, so that O is an exact convex combination of V rows.
// Warps 0-7 normalise (thread (wg, r) owns row r and columns [64 wg, 64 wg + 64) of every round),
// warp 8 copies with TMA (Q once; the rounds' K rows every sweep, in boxes of 16 rows per group or
// one box of 128 rows for eight adjacent groups, into a ring of 4 to 6 stages; V rows in the last
// sweep), warp 9 issues the products.
// Every mbarrier wait is bounded.
#include <math_constants.h>

#include "ap_common.cuh"
#include "ap_sm100.cuh"

namespace ap {

namespace {

using namespace sm100;

constexpr int kThreads = 320;
constexpr int kNormThreads = 256;
constexpr int kSubBytes = 128 * 128;
constexpr uint32_t kTmemCols = 512;  // S x 3 (columns 0..383), O (columns 384..384 + d)
constexpr int kSBufs = 3;            // S buffers in flight: a visit's hand-offs take longer than its work
constexpr uint32_t kMaxPolls = 1u << 22;
constexpr int kMaxNewton = 30;
// The first trial threshold: this far below the row maximum (the root lies in [max - 1, max); from
// either side of it the iteration lands on the other side or on the root).
constexpr float kFirstGap = 0.625f;

template <int D>
struct Cfg {
  static constexpr int kSub = D / 64;
  static constexpr int kTileBytes = kSub * kSubBytes;
  // K is copied again in every sweep and a list row is a few rounds long: a ring deep enough to hold
  // a short row whole keeps the copies several visits ahead of the products.  V is needed once.
  static constexpr int kStages = D == 64 ? 6 : 4;         // K ring
  static constexpr int kVStages = D == 64 ? 2 : 1;        // V ring (last sweep)
  static constexpr int kKOffset = kTileBytes;             // after Q
  static constexpr int kVOffset = kKOffset + kStages * kTileBytes;
  static constexpr int kStatsOffset = kVOffset + kVStages * kTileBytes;
  static constexpr int kStatsBytes = 2 * 128 * 8;         // [wg][row] (max, -), (S1, S2) or (sum of weights, -)
  static constexpr int kCntOffset = kStatsOffset + kStatsBytes;
  static constexpr int kCntBytes = 2 * 128 * 4;           // [wg][row] support size n
  static constexpr int kTauOffset = kCntOffset + kCntBytes;
  static constexpr int kTauBytes = 2 * 128 * 4;           // [wg][row]: each half keeps its own copy
  static constexpr int kBarOffset = kTauOffset + kTauBytes;
  static constexpr int kSmemBytes = kBarOffset + 512 + 1024;
  static_assert(kSmemBytes > 114 * 1024 && kSmemBytes <= 227 * 1024, "one CTA per SM, within the limit");
};

struct Barriers {
  uint64_t q_full;
  uint64_t s_full[kSBufs], s_empty[kSBufs];
  uint64_t in_full[6], in_empty[6];  // K ring: rows landed / S = Q K^T of the visit completed
  uint64_t v_full[2], v_empty[2];    // V ring: rows landed / O += P V of the visit completed
  uint64_t sweep_done;  // all statistics of the sweep are in shared memory
  uint64_t decided;     // every row has moved its threshold and said whether it needs another sweep
  uint64_t o_done;
  uint32_t tmem_base;
  int abort_flag;
  int more[kMaxNewton + 2];
};

struct Maps {
  CUtensorMap q;
  CUtensorMap k16, k128, v16, v128;  // K and V in boxes of 16 and of 128 rows
};

// A round's descriptor as loaded (nothing is computed from it here, so that the loads of the next
// round's descriptor stay in flight while the current round is worked on) ...
struct RawRound {
  uint32_t info;
  int4 a, b;
};
__device__ __forceinline__ RawRound load_round(const int32_t *round_rows, const uint8_t *round_info, int t) {
  RawRound r;
  r.info = __ldg(round_info + t);
  r.a = __ldg(reinterpret_cast<const int4 *>(round_rows + (size_t)t * 8));
  r.b = __ldg(reinterpret_cast<const int4 *>(round_rows + (size_t)t * 8) + 1);
  return r;
}
// ... and decoded: its groups and whether they are eight adjacent ones (one box of 128 rows brings them).
struct Round {
  int ng;
  bool run;
  int rows[8];
};
__device__ __forceinline__ Round decode_round(const RawRound &r) {
  Round rd;
  rd.ng = (int)(r.info & 15u);
  rd.rows[0] = r.a.x; rd.rows[1] = r.a.y; rd.rows[2] = r.a.z; rd.rows[3] = r.a.w;
  rd.rows[4] = r.b.x; rd.rows[5] = r.b.y; rd.rows[6] = r.b.z; rd.rows[7] = r.b.w;
  rd.run = rd.ng == 8;
#pragma unroll
  for (int q = 1; q < 8; ++q) rd.run = rd.run && rd.rows[q] == rd.rows[0] + 16 * q;
  return rd;
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

__device__ __forceinline__ bool last_follows(const Barriers *bars, int s) {
  return s >= 1 && (s >= kMaxNewton || *reinterpret_cast<const volatile int *>(&bars->more[s]) == 0);
}

// v when sel < 0, -inf otherwise (one select instruction on the sign of an integer).
__device__ __forceinline__ float keep_if_negative(float v, int sel) {
  float d;
  asm("slct.f32.s32 %0, %1, %2, %3;" : "=f"(d) : "f"(-CUDART_INF_F), "f"(v), "r"(sel));
  return d;
}

template <bool kF16>
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  if constexpr (kF16) {
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
  } else {
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
  }
}
template <bool kF16>
__device__ __forceinline__ float2 unpack2(uint32_t v) {
  if constexpr (kF16) {
    return __half22float2(*reinterpret_cast<const __half2 *>(&v));
  } else {
    return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&v));
  }
}

template <int D, bool kF16>
__global__ void __launch_bounds__(kThreads, 1)
fwd_entmax_kernel(const __grid_constant__ Maps maps, uint16_t *__restrict__ O, const int32_t *__restrict__ round_ptr,
                  const int32_t *__restrict__ round_rows, const uint8_t *__restrict__ round_info,
                  const uint32_t *__restrict__ round_bitmap, int BH, int H, int Lq, int n_qt, float half_scale,
                  unsigned *err) {
  using C = Cfg<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem =
      reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float2 *stats = reinterpret_cast<float2 *>(smem + C::kStatsOffset);  // [wg][row]
  float *cnts = reinterpret_cast<float *>(smem + C::kCntOffset);       // [wg][row]
  float *taus = reinterpret_cast<float *>(smem + C::kTauOffset);       // [wg][row]
  Barriers *bars = reinterpret_cast<Barriers *>(smem + C::kBarOffset);

  const int bh = (int)(blockIdx.x % BH);
  const int qt = n_qt - 1 - (int)(blockIdx.x / BH);  // late query tiles (the longest list rows when causal) first
  const int h = bh % H;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t0 = round_ptr[h * n_qt + qt];
  const int T = round_ptr[h * n_qt + qt + 1] - t0;  // rounds of this query tile: visits per sweep

  if (threadIdx.x == 0) {
    mbar_init(&bars->q_full, 1);
    for (int s = 0; s < kSBufs; ++s) {
      mbar_init(&bars->s_full[s], 1);
      mbar_init(&bars->s_empty[s], kNormThreads);
    }
    for (int s = 0; s < C::kStages; ++s) {
      mbar_init(&bars->in_full[s], 1);
      mbar_init(&bars->in_empty[s], 1);
    }
    for (int s = 0; s < C::kVStages; ++s) {
      mbar_init(&bars->v_full[s], 1);
      mbar_init(&bars->v_empty[s], 1);
    }
    mbar_init(&bars->sweep_done, kNormThreads);
    mbar_init(&bars->decided, kNormThreads + 2);  // + the copy and product threads, which run ahead of it
    mbar_init(&bars->o_done, 1);
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

  if (T == 0) {
    // nothing kept in these 128 rows: the output is exactly 0
    if (warp < 8) {
      const int r = (warp & 3) * 32 + lane, wg = warp >> 2;
      const int i = qt * kTile + r;
      if (i < Lq) {
        uint4 *dst = reinterpret_cast<uint4 *>(O + ((size_t)bh * Lq + i) * D + wg * (D / 2));
#pragma unroll
        for (int c = 0; c < D / 16; ++c) dst[c] = make_uint4(0u, 0u, 0u, 0u);
      }
    }
  } else if (warp == 8) {
    // ------------------------------------------------------------ TMA producer
    // K of visit v goes to stage v % kStages of its ring; V of the j-th visit of the last sweep to stage
    // j % kVStages of its own.  A sweep that is not the last is always followed by another, so the K
    // rows of the first visits of the next sweep are copied before the rows have decided whether that
    // sweep is the last one: the decision costs no copy latency.
    if (lane == 0) {
      prefetch_tensormap(&maps.q);
      prefetch_tensormap(&maps.k16);
      prefetch_tensormap(&maps.k128);
      prefetch_tensormap(&maps.v16);
      prefetch_tensormap(&maps.v128);
      mbar_arrive_expect_tx(&bars->q_full, C::kTileBytes);
#pragma unroll
      for (int s = 0; s < C::kSub; ++s) tma_load_3d(smem + s * kSubBytes, &maps.q, &bars->q_full, 64 * s, qt * kTile, bh);
      // rows of group q of a round land at rows [16 q, 16 q + 16) of the stage: 2048 bytes per group and half
      auto copy_rows = [&](const Round &rd, unsigned char *dst, const CUtensorMap *m16, const CUtensorMap *m128,
                           uint64_t *bar) {
        mbar_arrive_expect_tx(bar, (uint32_t)(rd.ng * 2048 * C::kSub));
        if (rd.run) {
#pragma unroll
          for (int s = 0; s < C::kSub; ++s) tma_load_3d(dst + s * kSubBytes, m128, bar, 64 * s, rd.rows[0], bh);
        } else {
#pragma unroll
          for (int q = 0; q < 8; ++q)
            if (q < rd.ng) {
#pragma unroll
              for (int s = 0; s < C::kSub; ++s) tma_load_3d(dst + s * kSubBytes + q * 2048, m16, bar, 64 * s, rd.rows[q], bh);
            }
        }
      };
      int v = 0;        // visits whose K copy has been issued
      int v_loads = 0;  // V copies issued
      bool ok = true;
      RawRound next = load_round(round_rows, round_info, t0);  // rounds are visited in order, again and again
      int vv_next = 0;
      auto copy_k = [&]() -> bool {
        const Round rd = decode_round(next);
        vv_next = vv_next + 1 == T ? 0 : vv_next + 1;
        next = load_round(round_rows, round_info, t0 + vv_next);
        const int st = v % C::kStages;
        if (!wait_or_abort(&bars->in_empty[st], ((uint32_t)(v / C::kStages) & 1u) ^ 1u, abort_flag, err)) return false;
        copy_rows(rd, smem + C::kKOffset + st * C::kTileBytes, &maps.k16, &maps.k128, &bars->in_full[st]);
        ++v;
        return true;
      };
      auto copy_v = [&](int vv) -> bool {  // V of round vv, the v_loads-th visit of the last sweep
        const int st = v_loads % C::kVStages;
        const Round rd = decode_round(load_round(round_rows, round_info, t0 + vv));
        if (!wait_or_abort(&bars->v_empty[st], ((uint32_t)(v_loads / C::kVStages) & 1u) ^ 1u, abort_flag, err)) return false;
        copy_rows(rd, smem + C::kVOffset + st * C::kTileBytes, &maps.v16, &maps.v128, &bars->v_full[st]);
        ++v_loads;
        return true;
      };
      const int n_ahead = T < C::kStages ? T : C::kStages;
      for (int vv = 0; vv < T && ok; ++vv) ok = copy_k();  // sweep 0
      for (int sw = 0; ok; ++sw) {
        // sweep sw is issued and is not the last: the head of sweep sw + 1, before the decision
        for (int vv = 0; vv < n_ahead && ok; ++vv) ok = copy_k();
        if (!ok) break;
        // (a participant of the barrier: a short sweep could otherwise complete the next phase
        // before this thread has seen this one)
        mbar_arrive(&bars->decided);
        if (!wait_or_abort(&bars->decided, (uint32_t)sw & 1u, abort_flag, err)) break;
        const bool last = last_follows(bars, sw);
        for (int vv = 0; vv < T && ok; ++vv) {
          if (vv >= n_ahead) ok = copy_k();
          if (ok && last) ok = copy_v(vv);
        }
        if (last) break;
      }
      if (*abort_flag) {  // winding down: let the copies in flight land (bounded)
        mbar_wait(&bars->q_full, 0u, kMaxPolls);
        for (int j = max(0, v - C::kStages); j < v; ++j)
          mbar_wait(&bars->in_full[j % C::kStages], (uint32_t)(j / C::kStages) & 1u, kMaxPolls);
        for (int j = max(0, v_loads - C::kVStages); j < v_loads; ++j)
          mbar_wait(&bars->v_full[j % C::kVStages], (uint32_t)(j / C::kVStages) & 1u, kMaxPolls);
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------ MMA issuer
    // S = Q K^T of the first visits of the next sweep is issued before the decision as well
    // (three S buffers).
    if (lane == 0) {
      constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, false, true, kF16);
      const uint32_t q_addr = smem_u32(smem), k_addr = smem_u32(smem + C::kKOffset), v_addr = smem_u32(smem + C::kVOffset);
      bool ok = wait_or_abort(&bars->q_full, 0u, abort_flag, err);
      int v = 0;  // visits whose S has been issued
      auto ng_of = [&](int vv) { return (int)(__ldg(round_info + t0 + vv) & 15u); };
      uint32_t info_next = __ldg(round_info + t0);  // used one visit later: the load stays in flight
      int vv_next = 0;
      auto issue_qk = [&]() -> bool {
        const int st = v % C::kStages, buf = v % kSBufs;
        const uint32_t idesc_qk = idesc_bf16_f32(128, 16 * (int)(info_next & 15u), false, false, kF16);
        vv_next = vv_next + 1 == T ? 0 : vv_next + 1;
        info_next = __ldg(round_info + t0 + vv_next);
        if (!wait_or_abort(&bars->in_full[st], (uint32_t)(v / C::kStages) & 1u, abort_flag, err)) return false;
        // S[buf] was read (and, in the last sweep, its P consumed by a product issued earlier by
        // this thread: products execute in issue order) kSBufs visits ago
        if (!wait_or_abort(&bars->s_empty[buf], ((uint32_t)(v / kSBufs) & 1u) ^ 1u, abort_flag, err)) return false;
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const int sub = ks / 4, o = (ks % 4) * 32;
          mma_ss(tmem + 128 * buf, smem_desc_sw128(q_addr + sub * kSubBytes + o, 16, 1024),
                 smem_desc_sw128(k_addr + st * C::kTileBytes + sub * kSubBytes + o, 16, 1024), idesc_qk, ks > 0);
        }
        mma_commit(&bars->in_empty[st]);
        mma_commit(&bars->s_full[buf]);
        ++v;
        return true;
      };
      // O += P V of visit u = round j of the last sweep: P is in S[u & 1] once the normalising
      // threads have arrived; one contraction step of 16 keys per group; then the V stage is free
      auto issue_pv = [&](int u, int j) -> bool {
        const int sb = u % kSBufs, sv = j % C::kVStages, ng_u = ng_of(j);
        if (!wait_or_abort(&bars->v_full[sv], (uint32_t)(j / C::kVStages) & 1u, abort_flag, err)) return false;
        if (!wait_or_abort(&bars->s_empty[sb], (uint32_t)(u / kSBufs) & 1u, abort_flag, err)) return false;
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          if (ks < ng_u)
            mma_ts(tmem + 128 * kSBufs, tmem + 128 * sb + 32 * (ks >> 1) + 8 * (ks & 1),
                   smem_desc_sw128(v_addr + sv * C::kTileBytes + ks * 2048, kSubBytes, 1024), idesc_pv,
                   (j == 0 && ks == 0) ? 0u : 1u);
        mma_commit(&bars->v_empty[sv]);
        return true;
      };
      const int n_ahead = T < kSBufs ? T : kSBufs;
      for (int vv = 0; vv < T && ok; ++vv) ok = issue_qk();  // sweep 0
      for (int sw = 0; ok; ++sw) {
        const int v_head = v;
        for (int vv = 0; vv < n_ahead && ok; ++vv) ok = issue_qk();
        if (!ok) break;
        mbar_arrive(&bars->decided);
        if (!wait_or_abort(&bars->decided, (uint32_t)sw & 1u, abort_flag, err)) break;
        if (!last_follows(bars, sw)) {
          for (int vv = n_ahead; vv < T && ok; ++vv) ok = issue_qk();
        } else {
          // visit by visit: S of the visit (unless issued above), then O += P V of the one before
          for (int vv = 0; vv < T && ok; ++vv) {
            if (vv >= n_ahead) ok = issue_qk();
            if (ok && vv > 0) ok = issue_pv(v_head + vv - 1, vv - 1);
          }
          if (ok && issue_pv(v_head + T - 1, T - 1)) mma_commit(&bars->o_done);
          break;
        }
      }
    }
  } else {
    // ------------------------------------------------------------ normalisation (256 threads)
    const int wg = warp >> 2;
    const int r = (warp & 3) * 32 + lane;  // row of the tile == TMEM lane
    const int i = qt * kTile + r;
    const bool row_ok = i < Lq;
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    float2 *my_stats = stats + wg * 128 + r;
    float *my_tau = taus + wg * 128 + r;
    float cnt = 0.f;

    // kept-entry bits of this thread's 64 columns of the round (0 for the columns of unused groups),
    // fetched one visit ahead
    // (raw: nothing is computed from the loaded values before the visit that uses them)
    auto fetch = [&](int vv, uint32_t &info, uint2 &bits) {
      const int t = t0 + vv;
      info = __ldg(round_info + t);
      bits = __ldg(reinterpret_cast<const uint2 *>(round_bitmap + ((size_t)t * kTile + r) * 4 + 2 * wg));
    };
    uint32_t info_next;
    uint2 bits_next;
    fetch(0, info_next, bits_next);

    int v = 0;
    bool last = false, ok = true;
    float2 st = make_float2(0.f, 0.f);
    float neg_tau = 0.f;
    for (int sw = 0; ok; ++sw) {
      const int kind = sw == 0 ? 0 : (last ? 2 : 1);  // 0 maxima, 1 sums over the support, 2 weights
      st = make_float2(kind == 0 ? -CUDART_INF_F : 0.f, 0.f);
      cnt = 0.f;
      for (int vv = 0; vv < T && ok; ++vv, ++v) {
        const int buf = v % kSBufs;
        const bool full = (info_next & 0x80u) != 0u;  // every entry of the round is kept
        const uint2 bits = bits_next;
        fetch(vv + 1 == T ? 0 : vv + 1, info_next, bits_next);
        ok = wait_or_abort(&bars->s_full[buf], (uint32_t)(v / kSBufs) & 1u, abort_flag, err);
        if (!ok) break;
        tc_fence_after_sync();
        float psum0 = 0.f, psum1 = 0.f;
#pragma unroll 1
        for (int c = 0; c < 2; ++c) {
          uint32_t x[32];
          tmem_ld32(tmem + 128 * buf + 64 * wg + 32 * c + lane_addr, x);
          tmem_wait_ld();
          const uint32_t w = c == 0 ? bits.x : bits.y;
          float t[32];  // x_j = scale * q.k_j / 2, -inf for pruned entries
#pragma unroll
          for (int e = 0; e < 32; e += 2)
            ffma2(t[e], t[e + 1], __uint_as_float(x[e]), __uint_as_float(x[e + 1]), half_scale, 0.f, 0.f);
          if (!full) {
            // bit e of w moved to the sign position selects between the score and -inf
#pragma unroll
            for (int e = 0; e < 32; ++e) t[e] = keep_if_negative(t[e], (int)(w << (31 - e)));
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
            // P in the tensors' type over the first 16 columns of this chunk of S
            uint32_t pk[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const float u0 = __saturatef(t[2 * e] + neg_tau), u1 = __saturatef(t[2 * e + 1] + neg_tau);
              pk[e] = pack2<kF16>(u0 * u0, u1 * u1);
              const float2 pr = unpack2<kF16>(pk[e]);  // the weights the product will use
              psum0 += pr.x;
              psum1 += pr.y;
            }
            tmem_st16(tmem + 128 * buf + 64 * wg + 32 * c + lane_addr, pk);
          }
        }
        if (kind == 2) {
          st.x += psum0 + psum1;
          tmem_wait_st();
        }
        // S[buf] is read; in the last sweep it now holds P for the product
        tc_fence_before_sync();
        mbar_arrive(&bars->s_empty[buf]);
      }
      if (!ok) break;
      *my_stats = st;
      cnts[wg * 128 + r] = cnt;
      // ---- end of a sweep: the two halves of every row meet
      mbar_arrive(&bars->sweep_done);
      ok = wait_or_abort(&bars->sweep_done, (uint32_t)sw & 1u, abort_flag, err);
      if (!ok) break;
      const float2 s0 = stats[r], s1 = stats[128 + r];
      if (last) {
        // epilogue: O / (sum of the rounded weights); this thread writes half of the row's d columns
        ok = wait_or_abort(&bars->o_done, 0u, abort_flag, err);
        if (!ok) break;
        tc_fence_after_sync();
        const float z = s0.x + s1.x;
        const float inv = z > 0.f ? 1.f / z : 0.f;
#pragma unroll
        for (int c = 0; c < D / 64; ++c) {
          uint32_t o[32];
          tmem_ld32(tmem + 128 * kSBufs + wg * (D / 2) + 32 * c + lane_addr, o);
          tmem_wait_ld();
          if (row_ok) {
            uint4 *dst = reinterpret_cast<uint4 *>(O + ((size_t)bh * Lq + i) * D + wg * (D / 2) + 32 * c);
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint4 pkt;
              pkt.x = pack2<kF16>(__uint_as_float(o[8 * g]) * inv, __uint_as_float(o[8 * g + 1]) * inv);
              pkt.y = pack2<kF16>(__uint_as_float(o[8 * g + 2]) * inv, __uint_as_float(o[8 * g + 3]) * inv);
              pkt.z = pack2<kF16>(__uint_as_float(o[8 * g + 4]) * inv, __uint_as_float(o[8 * g + 5]) * inv);
              pkt.w = pack2<kF16>(__uint_as_float(o[8 * g + 6]) * inv, __uint_as_float(o[8 * g + 7]) * inv);
              dst[g] = pkt;
            }
          }
        }
        break;
      }
      bool moved = false;
      float tau;
      if (sw == 0) {
        const float m = fmaxf(s0.x, s1.x);
        // No kept entry: every weight is 0 whatever the score
        tau = m == -CUDART_INF_F ? CUDART_INF_F : m - kFirstGap;
      } else {
        tau = *my_tau;
        const float S1 = s0.x + s1.x, S2 = s0.y + s1.y, n = cnts[r] + cnts[128 + r];
        // root of the support's parabola; Newton's step where it has none
        const float disc = S1 * S1 - n * (S2 - 1.f);
        const float step = S1 > 0.f ? (S2 - 1.f) / (S1 + (disc >= 0.f ? sqrtf(disc) : S1)) : 0.f;
        tau += step;
        // below the resolution of tau itself a step is rounding noise of the sums
        moved = fabsf(step) > 2e-6f * fmaxf(1.f, fabsf(tau));
      }
      *my_tau = tau;
      neg_tau = -tau;
      if (moved && row_ok) *reinterpret_cast<volatile int *>(&bars->more[sw]) = 1;
      mbar_arrive(&bars->decided);
      ok = wait_or_abort(&bars->decided, (uint32_t)sw & 1u, abort_flag, err);
      if (!ok) break;
      last = last_follows(bars, sw);
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 9) tmem_dealloc(tmem, kTmemCols);
}

template <int D, bool kF16>
cudaError_t launch(const Maps &maps, const ap_tiles &t, void *O, int B, int H, int Lq, float scale, unsigned *err,
                   cudaStream_t s) {
  auto kern = fwd_entmax_kernel<D, kF16>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<D>::kSmemBytes);
  if (e != cudaSuccess) return e;
  kern<<<B * H * t.n_qt, kThreads, Cfg<D>::kSmemBytes, s>>>(maps, static_cast<uint16_t *>(O), t.round_ptr, t.round_rows,
                                                           t.round_info, t.round_bitmap, B * H, H, Lq, t.n_qt,
                                                           0.5f * scale, err);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fwd_entmax_tc(const void *Q, const void *K, const void *V, const ap_tiles &t, void *O, int B, int H,
                                 int Lq, int Lk, int d, int f16, float scale, cudaStream_t s) {
  unsigned *err = device_error_word();
  if (!err) return cudaErrorUnknown;
  Maps maps;
  if (!make_tile_map_bf16(&maps.q, Q, B * H, Lq, d) || !make_tile_map_bf16(&maps.k16, K, B * H, Lk, d, 16) ||
      !make_tile_map_bf16(&maps.k128, K, B * H, Lk, d, 128) || !make_tile_map_bf16(&maps.v16, V, B * H, Lk, d, 16) ||
      !make_tile_map_bf16(&maps.v128, V, B * H, Lk, d, 128))
    return cudaErrorUnknown;
  if (d == 64)
    return f16 ? launch<64, true>(maps, t, O, B, H, Lq, scale, err, s) : launch<64, false>(maps, t, O, B, H, Lq, scale, err, s);
  return f16 ? launch<128, true>(maps, t, O, B, H, Lq, scale, err, s) : launch<128, false>(maps, t, O, B, H, Lq, scale, err, s);
}

}  // namespace ap
