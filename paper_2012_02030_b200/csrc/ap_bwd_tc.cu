// Derivative of the masked attention of Section 3.2 (what retraining under the mask, step 4 of
// the procedure, needs) for bf16 / fp16 tensors, on the tcgen05 tensor cores.
//
// With S = scale Q K^T, P = softmax of S over the kept entries of a row, O = P V and an incoming dO:
//   dV = P^T dO,   dP = dO V^T,   dS = P o (dP - D),  D_i = dO_i . O_i,
//   dQ = scale dS K,   dK = scale dS^T Q.
// Two kernels follow the tile list, both tile by tile and without overlap between their steps (a
// first, plain version: one CTA of 256 threads, two threads per row of the tile, each with two of
// the four 32-column chunks; one thread issues the copies and the MMAs, everybody waits on two
// mbarriers):
//   rows kernel     one CTA per (b, h, query tile), following the query tile's ROUNDS (the forward's
//                   schedule: up to eight non-empty 16-column groups gathered from its key tiles, so
//                   the work follows the slots, not the stored tiles).  Sweep 1 over the rounds: S on the tensor
//                   cores, running maximum and sum of the kept entries -> L_i = log2 sum_j 2^(c S_ij)
//                   (c = log2 e), and D_i from dO and O; both go to the workspace.  Sweep 2: S and dP
//                   on the tensor cores, dS by the threads (P = 2^(c S - L), rounded to the tensors'
//                   16-bit type and written to shared memory in the operand layout), dQ += dS K on the
//                   tensor cores (accumulator in TMEM).
//   columns kernel  one CTA per (b, h, key tile), looping over the query tiles whose list row holds
//                   that key tile (the next one's Q and dO are copied ahead): S, dP, then P to shared
//                   memory and dV += P^T dO, then dS to the same area and dK += dS^T Q, which runs
//                   under the next query tile's S and dP.
// Every output element is written once, by the thread that owns its row: no atomics, results are
// reproducible bit for bit.  All tiles are staged by TMA with the 128-byte swizzle, one layout
// ([64-element slab][row][128 bytes]) serving as K-major and as MN-major operand; P and dS are
// written by the threads in that same layout.  Every wait is bounded.
#include <math_constants.h>

#include "ap_common.cuh"
#include "ap_sm100.cuh"

namespace ap {

namespace {

using namespace sm100;

constexpr int kThreads = 256;  // thread (half, r): row r of the tile, chunks 2 half and 2 half + 1
constexpr int kSubBytes = 128 * 128;  // one slab: 128 rows x 64 elements of 2 bytes
constexpr uint32_t kTmemCols = 512;
constexpr float kLog2e = 1.4426950408889634f;

struct Bars {
  uint64_t tma, mma, mma2;
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
__device__ __forceinline__ float2 unpack2(uint32_t pk) {
  if constexpr (kF16) {
    return __half22float2(*reinterpret_cast<const __half2 *>(&pk));
  } else {
    return make_float2(__uint_as_float(pk << 16), __uint_as_float(pk & 0xffff0000u));
  }
}

// Bounded wait of the whole CTA on one barrier phase; the outcome is the same for every thread.  (Every
// thread polls: with one polling thread and the others parked at the CTA barrier the kernels were 4 % slower.)
__device__ __forceinline__ bool cta_wait(uint64_t *bar, uint32_t parity, Bars *bars, unsigned *err,
                                         uint32_t max_polls) {
  bool ok = false;
  volatile int *abort_flag = &bars->abort_flag;
  for (uint32_t i = 0; i < max_polls; ++i) {
    if (mbar_try_wait(bar, parity)) {
      ok = true;
      break;
    }
    if (*abort_flag) break;
    if (i > 1024) __nanosleep(64);
  }
  if (!ok && !*abort_flag) {
    *abort_flag = 1;
    atomicOr(err, kDevErrTimeout);
  }
  return __syncthreads_and(ok ? 1 : 0) != 0;
}

// After a wait has given up: lets a copy that may still be in flight (the phase after the last one
// waited for) land before the CTA returns; bounded.
__device__ __forceinline__ void drain_copies(Bars *bars, uint32_t phases_waited) {
  if (threadIdx.x == 0) mbar_wait(&bars->tma, phases_waited & 1u, 1u << 16);
  __syncthreads();
}

// Non-empty 16-column groups of list tile t (all eight for a tile flagged as fully kept); loaded where
// it is written, one tile ahead of its use.
__device__ __forceinline__ uint32_t group_mask(const uint8_t *flags, const uint8_t *groups, int t) {
  const uint32_t f = ldg_now_u8(flags + t), g = ldg_now_u8(groups + t);
  return (f & 1u) ? 0xffu : g;
}

// Address of 16-byte piece `piece` (0..7) of row r in slab `slab` of a staged tile.
__device__ __forceinline__ unsigned char *piece_ptr(unsigned char *tile, int slab, int r, int piece) {
  return tile + slab * kSubBytes + r * 128 + ((piece ^ (r & 7)) << 4);
}

// One thread: copies rows [row0, row0 + 128) of (batch, head) index bh into a staged tile of D columns.
template <int D>
__device__ __forceinline__ void load_tile(unsigned char *dst, const CUtensorMap *m, uint64_t *bar, int row0, int bh) {
#pragma unroll
  for (int s = 0; s < D / 64; ++s) tma_load_3d(dst + s * kSubBytes, m, bar, 64 * s, row0, bh);
}

// One thread: C[128 x 128] = A B^T with A and B staged tiles of D columns (rows x D, D contiguous),
// restricted to the span of 16-column groups of C from the first to the last one named in `groups`
// (bit g: columns [16g, 16g+16), i.e. rows [16g, 16g+16) of B); columns outside the span are left as they
// are.  One product per step of the contraction: its cost hardly depends on the width, so the span is
// not split further.
template <int D, bool kF16>
__device__ __forceinline__ void mma_abt_span(uint32_t d_tmem, const unsigned char *a, const unsigned char *b,
                                             uint32_t groups) {
  const int first = __ffs((int)groups) - 1, last = 31 - __clz((int)groups);
  const uint32_t idesc = idesc_bf16_f32(128, 16 * (last - first + 1), false, false, kF16);
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    const int sub = ks / 4, off = (ks % 4) * 32;
    mma_ss(d_tmem + 16 * first, smem_desc_sw128(smem_u32(a + sub * kSubBytes + off), 16, 1024),
           smem_desc_sw128(smem_u32(b + sub * kSubBytes + first * 2048 + off), 16, 1024), idesc, ks > 0);
  }
}

// One thread: C[128 x D] (+)= A^T B, A a staged 128 x 128 tile (rows = contraction index), B a staged
// tile of D columns with the same rows.
template <int D>
__device__ __forceinline__ void mma_atb(uint32_t d_tmem, const unsigned char *a, const unsigned char *b, uint32_t idesc,
                                        bool accumulate) {
#pragma unroll
  for (int ks = 0; ks < 8; ++ks)  // 16 rows of the contraction per step
    mma_ss(d_tmem, smem_desc_sw128(smem_u32(a + ks * 2048), kSubBytes, 1024),
           smem_desc_sw128(smem_u32(b + ks * 2048), kSubBytes, 1024), idesc, accumulate || ks > 0);
}

// One thread: C[128 x D] (+)= A B, A a staged 128 x 128 tile (columns = contraction index), B a staged
// tile of D columns whose rows are the contraction index.
// Only the contraction steps named in `groups` are taken (bit g: columns [16g, 16g+16) of A).
template <int D>
__device__ __forceinline__ void mma_ab(uint32_t d_tmem, const unsigned char *a, const unsigned char *b, uint32_t idesc,
                                       bool accumulate, uint32_t groups) {
  bool acc = accumulate;
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    if (!((groups >> ks) & 1u)) continue;
    const int sub = ks / 4, off = (ks % 4) * 32;
    mma_ss(d_tmem, smem_desc_sw128(smem_u32(a + sub * kSubBytes + off), 16, 1024),
           smem_desc_sw128(smem_u32(b + ks * 2048), kSubBytes, 1024), idesc, acc);
    acc = true;
  }
}

struct BwdMaps {
  CUtensorMap q, k, v, o, d_o;  // boxes of 128 rows
  CUtensorMap kbox[4], vbox[4];  // boxes of 16, 32, 64, 128 rows: runs of 1, 2, 4, 8 slots of a round
};

template <int D>
struct Cfg {
  static constexpr int kTileBytes = (D / 64) * kSubBytes;  // a staged tile of D columns
  static constexpr int kSquareBytes = 2 * kSubBytes;       // a staged 128 x 128 tile (P, dS)
  // rows kernel: Q, dO, two (K, V) pairs (the next tile's pair is copied while this one is used), dS
  // (O is staged in the dS area first)
  static constexpr int kRowsSmem = 6 * kTileBytes + kSquareBytes + 1024 + 256;
  // columns kernel: K, V, two (Q, dO) pairs, one area for P and then dS, the staged lookup column
  static constexpr int kColsSmem = 6 * kTileBytes + kSquareBytes + 1024 + 256 + 1024;
};

// Thread r's 32 values of one chunk -> 16-bit pairs in row r of a staged 128 x 128 tile, columns [32c, 32c+32).
__device__ __forceinline__ void store_chunk(unsigned char *tile, int r, int c, const uint32_t pk[16]) {
#pragma unroll
  for (int q = 0; q < 4; ++q)
    *reinterpret_cast<uint4 *>(piece_ptr(tile, c >> 1, r, (c & 1) * 4 + q)) =
        make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
}

// ------------------------------------------------------------------------------------------ rows kernel

template <int D, bool kF16>
__global__ void __launch_bounds__(kThreads, 1)
bwd_rows_kernel(const __grid_constant__ BwdMaps maps, uint16_t *__restrict__ dQ, float *__restrict__ stat_l,
                float *__restrict__ stat_d, const int32_t *__restrict__ round_ptr,
                const int32_t *__restrict__ round_rows, const uint8_t *__restrict__ round_info,
                const uint32_t *__restrict__ round_bitmap, int H, int Lq, int n_qt, float scale, unsigned *err,
                uint32_t max_polls, int dbg_skip) {
  using C = Cfg<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem =
      reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char *q_s = smem, *do_s = smem + C::kTileBytes, *kv_s = smem + 2 * C::kTileBytes,
                *ds_s = smem + 6 * C::kTileBytes;
  Bars *bars = reinterpret_cast<Bars *>(smem + 6 * C::kTileBytes + C::kSquareBytes);

  // late query tiles (the longest list rows under a causal mask) first
  const int qt = n_qt - 1 - (int)(blockIdx.x / (gridDim.x / n_qt)), bh = blockIdx.x % (gridDim.x / n_qt), h = bh % H;
  const int r = threadIdx.x & 127, half = threadIdx.x >> 7, warp = threadIdx.x >> 5;
  const int i = qt * kTile + r;
  const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
  const bool leader = threadIdx.x == 0;
  // the query tile's rounds: up to eight non-empty 16-column groups (slots) each, gathered from its
  // key tiles, as the forward pass visits them
  const int t0 = round_ptr[h * n_qt + qt], t1 = round_ptr[h * n_qt + qt + 1];
  struct RoundMeta {
    uint4 lo, hi;   // first key row of slots 0..3 and 4..7
    uint32_t info;  // bits 0..3: slots; bit 7: every entry kept
  };
  auto meta_of = [&](int t) {
    RoundMeta mt;
    mt.lo = ldg_now_v4(round_rows + (size_t)t * 8);
    mt.hi = ldg_now_v4(round_rows + (size_t)t * 8 + 4);
    mt.info = ldg_now_u8(round_info + t);
    return mt;
  };
  // One thread: copies the key rows (and value rows) of a round's slots, slot q to rows [16q, 16q+16).
  // Slots whose key rows follow one another are copied together, in boxes of 8, 4, 2 or 1 slots.
  auto load_round = [&](unsigned char *kb, const RoundMeta &mt, bool with_v) {
    const int ng = (int)(mt.info & 15u);
    const int first[8] = {(int)mt.lo.x, (int)mt.lo.y, (int)mt.lo.z, (int)mt.lo.w,
                          (int)mt.hi.x, (int)mt.hi.y, (int)mt.hi.z, (int)mt.hi.w};
    mbar_arrive_expect_tx(&bars->tma, (uint32_t)((with_v ? 2 : 1) * ng * 16 * D * 2));
    int q = 0;
    while (q < ng) {
      int run = 1;
      while (q + run < ng && first[q + run] == first[q] + 16 * run) ++run;
      for (int done = 0; done < run;) {
        const int left = run - done;
        const int lg = left >= 8 ? 3 : left >= 4 ? 2 : left >= 2 ? 1 : 0;
#pragma unroll
        for (int sl = 0; sl < D / 64; ++sl) {
          unsigned char *dst = kb + sl * kSubBytes + (q + done) * 2048;
          tma_load_3d(dst, &maps.kbox[lg], &bars->tma, 64 * sl, first[q] + 16 * done, bh);
          if (with_v) tma_load_3d(dst + C::kTileBytes, &maps.vbox[lg], &bars->tma, 64 * sl, first[q] + 16 * done, bh);
        }
        done += 1 << lg;
      }
      q += run;
    }
  };
  const float c = scale * kLog2e;

  if (leader) {
    mbar_init(&bars->tma, 1);
    mbar_init(&bars->mma, 1);
    bars->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&bars->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = bars->tmem_base;
  const uint32_t tmem_s = tmem, tmem_dp = tmem + 128, tmem_dq = tmem + 256;
  uint32_t tma_n = 0, mma_n = 0;  // phases used so far
  bool ok = true;

  // Q, dO and O of the query tile; D_i = dO_i . O_i  (test hook: the copies are left out, the wait below runs out)
  if (leader && dbg_skip == 0) {
    mbar_arrive_expect_tx(&bars->tma, 3 * C::kTileBytes);
    load_tile<D>(q_s, &maps.q, &bars->tma, qt * kTile, bh);
    load_tile<D>(do_s, &maps.d_o, &bars->tma, qt * kTile, bh);
    load_tile<D>(ds_s, &maps.o, &bars->tma, qt * kTile, bh);
  }
  ok = cta_wait(&bars->tma, tma_n++ & 1u, bars, err, max_polls);
  // each of the row's two threads takes half of every 128-byte line; the halves are added in a fixed order
  float dsum = 0.f;
  float *xch = reinterpret_cast<float *>(kv_s);  // [half][row]; the K / V area is not in use yet
  if (ok) {
#pragma unroll
    for (int s = 0; s < D / 64; ++s)
#pragma unroll
      for (int p = 4 * half; p < 4 * half + 4; ++p) {
        const uint4 a = *reinterpret_cast<const uint4 *>(piece_ptr(do_s, s, r, p));
        const uint4 b = *reinterpret_cast<const uint4 *>(piece_ptr(ds_s, s, r, p));
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 x = unpack2<kF16>(aw[e]), y = unpack2<kF16>(bw[e]);
          dsum = fmaf(x.x, y.x, dsum);
          dsum = fmaf(x.y, y.y, dsum);
        }
      }
  }
  xch[half * 128 + r] = dsum;
  __syncthreads();  // O is read: its area becomes dS
  dsum = xch[r] + xch[128 + r];
  fence_proxy_async_smem();  // the area is written by the copy engine next
  __syncthreads();

  constexpr uint32_t idesc_dq = idesc_bf16_f32(128, D, false, true, kF16);

  // ---- sweep 1: row maximum and sum over the kept entries
  float m = -CUDART_INF_F, l = 0.f;
  RoundMeta cur = meta_of(t0 < t1 ? t0 : 0), nxt = meta_of(t0 + 1 < t1 ? t0 + 1 : 0);  // fetched ahead of their use
  if (leader && ok && t0 < t1) load_round(kv_s, cur, false);
  for (int t = t0; t < t1 && ok; ++t) {
    unsigned char *k_s = kv_s + ((t - t0) & 1) * 2 * C::kTileBytes;
    const RoundMeta me = cur, after = nxt;
    cur = nxt;
    if (t + 2 < t1) nxt = meta_of(t + 2);
    const uint32_t gm = (1u << (me.info & 15u)) - 1u;  // the round's slots, packed from slot 0
    ok = cta_wait(&bars->tma, tma_n++ & 1u, bars, err, max_polls);
    if (!ok) break;
    if (leader) {
      // the other pair was last read by the MMA of round t - 1, which has completed
      if (t + 1 < t1) load_round(kv_s + ((t + 1 - t0) & 1) * 2 * C::kTileBytes, after, false);
      tc_fence_after_sync();
      mma_abt_span<D, kF16>(tmem_s, q_s, k_s, gm);
      mma_commit(&bars->mma);
    }
    uint4 bw = make_uint4(0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu);
    if (!(me.info & 0x80u)) bw = *reinterpret_cast<const uint4 *>(round_bitmap + ((size_t)t * kTile + r) * 4);
    const uint32_t w[4] = {bw.x, bw.y, bw.z, bw.w};
    ok = cta_wait(&bars->mma, mma_n++ & 1u, bars, err, max_polls);
    if (!ok) break;
    tc_fence_after_sync();
#pragma unroll 1
    for (int ch = 2 * half; ch < 2 * half + 2; ++ch) {
      if (!((gm >> (2 * ch)) & 3u)) continue;  // nothing kept in these 32 columns (the same for the whole warp)
      uint32_t x[32];
      tmem_ld32(tmem_s + lane_addr + 32 * ch, x);
      tmem_wait_ld();
      float cm = -CUDART_INF_F;
#pragma unroll
      for (int e = 0; e < 32; ++e)
        if ((w[ch] >> e) & 1u) cm = fmaxf(cm, __uint_as_float(x[e]));
      if (cm > m) {
        l *= ex2_approx((m - cm) * c);  // 0 when m was -inf
        m = cm;
      }
      if (m > -CUDART_INF_F) {
        const float neg = -m * c;
#pragma unroll
        for (int e = 0; e < 32; ++e)
          if ((w[ch] >> e) & 1u) l += ex2_approx(fmaf(__uint_as_float(x[e]), c, neg));
      }
    }
    tc_fence_before_sync();
    __syncthreads();  // S and K may be overwritten
  }
  // L_i = log2 of the row's sum of 2^(c S); +inf for a row without kept entries (then P = 0 everywhere)
  {
    // the row's two partial (maximum, sum) pairs, merged the same way by both threads
    float2 *ml = reinterpret_cast<float2 *>(ds_s);  // [half][row]; the dS area is not in use yet
    ml[half * 128 + r] = make_float2(m, l);
    __syncthreads();
    const float2 a = ml[r], b = ml[128 + r];
    m = fmaxf(a.x, b.x);
    l = (a.y > 0.f ? a.y * ex2_approx((a.x - m) * c) : 0.f) + (b.y > 0.f ? b.y * ex2_approx((b.x - m) * c) : 0.f);
    __syncthreads();
  }
  const float big_l = l > 0.f ? fmaf(m, c, lg2_approx(l)) : CUDART_INF_F;
  if (ok && i < Lq && half == 0) {
    stat_l[(size_t)bh * Lq + i] = big_l;
    stat_d[(size_t)bh * Lq + i] = dsum;
  }

  // ---- sweep 2: dS and dQ
  bool started = false;
  cur = meta_of(t0 < t1 ? t0 : 0);
  nxt = meta_of(t0 + 1 < t1 ? t0 + 1 : 0);
  if (leader && ok && t0 < t1) load_round(kv_s, cur, true);
  for (int t = t0; t < t1 && ok; ++t) {
    unsigned char *k_s = kv_s + ((t - t0) & 1) * 2 * C::kTileBytes, *v_s = k_s + C::kTileBytes;
    const RoundMeta me = cur, after = nxt;
    cur = nxt;
    if (t + 2 < t1) nxt = meta_of(t + 2);
    const uint32_t gm = (1u << (me.info & 15u)) - 1u;
    ok = cta_wait(&bars->tma, tma_n++ & 1u, bars, err, max_polls);
    if (!ok) break;
    if (leader) {
      // the other pair was last read by dQ += dS K of round t - 1, which has completed
      if (t + 1 < t1) load_round(kv_s + ((t + 1 - t0) & 1) * 2 * C::kTileBytes, after, true);
      tc_fence_after_sync();
      mma_abt_span<D, kF16>(tmem_s, q_s, k_s, gm);
      mma_abt_span<D, kF16>(tmem_dp, do_s, v_s, gm);
      mma_commit(&bars->mma);
    }
    uint4 bw = make_uint4(0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu);
    if (!(me.info & 0x80u)) bw = *reinterpret_cast<const uint4 *>(round_bitmap + ((size_t)t * kTile + r) * 4);
    const uint32_t w[4] = {bw.x, bw.y, bw.z, bw.w};
    ok = cta_wait(&bars->mma, mma_n++ & 1u, bars, err, max_polls);
    if (!ok) break;
    tc_fence_after_sync();
#pragma unroll 1
    for (int ch = 2 * half; ch < 2 * half + 2; ++ch) {
      if (!((gm >> (2 * ch)) & 3u)) continue;  // dS of these columns is not read: their steps of dQ += dS K are skipped
      uint32_t x[32], y[32], pk[16];
      tmem_ld32(tmem_s + lane_addr + 32 * ch, x);
      tmem_ld32(tmem_dp + lane_addr + 32 * ch, y);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        float ds[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int col = 2 * e + u;
          const bool kept = (w[ch] >> col) & 1u;
          // columns of an empty group hold whatever an earlier tile left in S and dP: never used
          ds[u] = kept ? ex2_approx(fmaf(__uint_as_float(x[col]), c, -big_l)) * (__uint_as_float(y[col]) - dsum) : 0.f;
        }
        pk[e] = pack2<kF16>(ds[0], ds[1]);
      }
      store_chunk(ds_s, r, ch, pk);
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (leader) {
      tc_fence_after_sync();
      mma_ab<D>(tmem_dq, ds_s, k_s, idesc_dq, started, gm);
      mma_commit(&bars->mma);
    }
    started = true;
    ok = cta_wait(&bars->mma, mma_n++ & 1u, bars, err, max_polls);  // K, V, dS may be overwritten
  }

  // ---- dQ rows, scaled and rounded once (the loads are warp-wide: rows beyond Lq take part and store nothing)
  if (ok) {
    uint16_t *out = dQ + ((size_t)bh * Lq + i) * D;
    tc_fence_after_sync();
#pragma unroll 1
    for (int ch = half; ch < D / 32; ch += 2) {
      uint32_t x[32];
      if (started) {  // the same for every thread
        tmem_ld32(tmem_dq + lane_addr + 32 * ch, x);
        tmem_wait_ld();
      }
      if (i < Lq) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t pk[4];
#pragma unroll
          for (int e = 0; e < 4; ++e)
            pk[e] = started ? pack2<kF16>(__uint_as_float(x[8 * q + 2 * e]) * scale,
                                          __uint_as_float(x[8 * q + 2 * e + 1]) * scale)
                            : 0u;
          *reinterpret_cast<uint4 *>(out + 32 * ch + 8 * q) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
      }
    }
  }
  if (!ok) drain_copies(bars, tma_n);  // ok is the same for every thread
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// --------------------------------------------------------------------------------------- columns kernel

// tile_id[(h * n_qt + qt) * n_kt + kt] = position of tile (qt, kt) in head h's list, -1 if it is not
// stored: what the columns kernel walks (the list itself is ordered by query tile).
__global__ void tile_lookup_kernel(const int32_t *__restrict__ row_ptr, const int32_t *__restrict__ col_idx,
                                   int n_rows, int n_kt, int32_t *__restrict__ tile_id) {
  const int row = blockIdx.x;  // h * n_qt + qt
  if (row >= n_rows) return;
  for (int kt = threadIdx.x; kt < n_kt; kt += blockDim.x) tile_id[(size_t)row * n_kt + kt] = -1;
  __syncthreads();
  const int t0 = row_ptr[row], t1 = row_ptr[row + 1];
  for (int t = t0 + (int)threadIdx.x; t < t1; t += blockDim.x) tile_id[(size_t)row * n_kt + col_idx[t]] = t;
}

constexpr int kMaxIds = 256;  // query tiles whose lookup entries are staged in shared memory

template <int D, bool kF16>
__global__ void __launch_bounds__(kThreads, 1)
bwd_cols_kernel(const __grid_constant__ BwdMaps maps, uint16_t *__restrict__ dK, uint16_t *__restrict__ dV,
                const float *__restrict__ stat_l, const float *__restrict__ stat_d,
                const int32_t *__restrict__ tile_id, const uint8_t *__restrict__ flags,
                const uint8_t *__restrict__ groups, const uint32_t *__restrict__ bitmap, int H, int Lq, int Lk,
                int n_qt, int n_kt, float scale, unsigned *err, uint32_t max_polls, int dbg_skip) {
  using C = Cfg<D>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem =
      reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  // K, V of the key tile; two (Q, dO) pairs (the next query tile's pair is copied while this one is
  // used); one 128 x 128 area that holds P for dV += P^T dO and then dS for dK += dS^T Q
  unsigned char *k_s = smem, *v_s = smem + C::kTileBytes, *qd_s = smem + 2 * C::kTileBytes,
                *x_s = smem + 6 * C::kTileBytes;
  Bars *bars = reinterpret_cast<Bars *>(smem + 6 * C::kTileBytes + C::kSquareBytes);
  int32_t *ids = reinterpret_cast<int32_t *>(smem + 6 * C::kTileBytes + C::kSquareBytes + 256);  // [kMaxIds]

  const int kt = blockIdx.x % n_kt, bh = blockIdx.x / n_kt, h = bh % H;
  const int r = threadIdx.x & 127, half = threadIdx.x >> 7, warp = threadIdx.x >> 5;
  const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
  const bool leader = threadIdx.x == 0;
  const float c = scale * kLog2e;

  if (leader) {
    mbar_init(&bars->tma, 1);
    mbar_init(&bars->mma, 1);
    mbar_init(&bars->mma2, 1);
    bars->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&bars->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = bars->tmem_base;
  const uint32_t tmem_s = tmem, tmem_dp = tmem + 128, tmem_dv = tmem + 256, tmem_dk = tmem + 256 + D;
  uint32_t tma_n = 0, mma_n = 0, dk_n = 0;
  bool ok = true;

  // this key tile's column of the lookup table: one entry per query tile, staged once
  for (int qt = threadIdx.x; qt < n_qt && qt < kMaxIds; qt += kThreads)
    ids[qt] = tile_id[((size_t)h * n_qt + qt) * n_kt + kt];
  __syncthreads();
  // The next query tile at or after qt0 whose list row holds this key tile; n_qt if there is none.
  // The same for every thread.
  auto find_from = [&](int qt0, int &t_out) {
    for (int qt = qt0; qt < n_qt; ++qt) {
      const int t = qt < kMaxIds ? ids[qt] : tile_id[((size_t)h * n_qt + qt) * n_kt + kt];
      if (t >= 0) {
        t_out = t;
        return qt;
      }
    }
    t_out = -1;
    return n_qt;
  };

  int t_cur = -1;
  int qt_cur = find_from(0, t_cur);
  // (test hook: these copies are left out, so the first wait runs out)
  if (leader && qt_cur < n_qt && dbg_skip == 0) {  // K, V and the first query tile's Q, dO in one go
    mbar_arrive_expect_tx(&bars->tma, 4 * C::kTileBytes);
    load_tile<D>(k_s, &maps.k, &bars->tma, kt * kTile, bh);
    load_tile<D>(v_s, &maps.v, &bars->tma, kt * kTile, bh);
    load_tile<D>(qd_s, &maps.q, &bars->tma, qt_cur * kTile, bh);
    load_tile<D>(qd_s + C::kTileBytes, &maps.d_o, &bars->tma, qt_cur * kTile, bh);
  }

  constexpr uint32_t idesc_t = idesc_bf16_f32(128, D, true, true, kF16);

  bool started = false;
  uint32_t gm_next = qt_cur < n_qt ? group_mask(flags, groups, t_cur) : 0u;
  for (uint32_t n = 0; qt_cur < n_qt && ok; ++n) {
    int t_nxt = -1;
    const int qt_nxt = find_from(qt_cur + 1, t_nxt);
    unsigned char *q_s = qd_s + (n & 1u) * 2 * C::kTileBytes, *do_s = q_s + C::kTileBytes;
    const int t = t_cur;
    const uint32_t gm = gm_next;
    if (qt_nxt < n_qt) gm_next = group_mask(flags, groups, t_nxt);
    const int i = qt_cur * kTile + r;
    const float big_l = i < Lq ? stat_l[(size_t)bh * Lq + i] : CUDART_INF_F;
    const float dsum = i < Lq ? stat_d[(size_t)bh * Lq + i] : 0.f;
    const uint4 bw = *reinterpret_cast<const uint4 *>(bitmap + ((size_t)t * kTile + r) * 4);
    const uint32_t w[4] = {bw.x, bw.y, bw.z, bw.w};
    ok = cta_wait(&bars->tma, tma_n++ & 1u, bars, err, max_polls);
    if (!ok) break;
    if (leader) {
      tc_fence_after_sync();
      mma_abt_span<D, kF16>(tmem_s, q_s, k_s, gm);
      mma_abt_span<D, kF16>(tmem_dp, do_s, v_s, gm);
      mma_commit(&bars->mma);
    }
    // products complete in order: with S and dP, dK += dS^T Q of the previous query tile is over too,
    // so its (Q, dO) pair and the P / dS area are free
    ok = cta_wait(&bars->mma, mma_n++ & 1u, bars, err, max_polls);
    if (!ok) break;
    if (leader && qt_nxt < n_qt) {
      unsigned char *nq = qd_s + ((n + 1u) & 1u) * 2 * C::kTileBytes;
      mbar_arrive_expect_tx(&bars->tma, 2 * C::kTileBytes);
      load_tile<D>(nq, &maps.q, &bars->tma, qt_nxt * kTile, bh);
      load_tile<D>(nq + C::kTileBytes, &maps.d_o, &bars->tma, qt_nxt * kTile, bh);
    }
    tc_fence_after_sync();
    // this thread's two chunks of P and dS, rounded to the tensors' type; zero where nothing is kept
    // (the products below read all 128 key columns)
    uint32_t pp[2][16], pd[2][16];
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) {
      const int ch = 2 * half + cc;
      if (!((gm >> (2 * ch)) & 3u)) {  // the same for the whole warp
#pragma unroll
        for (int e = 0; e < 16; ++e) pp[cc][e] = pd[cc][e] = 0u;
        continue;
      }
      uint32_t x[32], y[32];
      tmem_ld32(tmem_s + lane_addr + 32 * ch, x);
      tmem_ld32(tmem_dp + lane_addr + 32 * ch, y);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        float p[2], ds[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int col = 2 * e + u;
          const bool kept = (w[ch] >> col) & 1u;
          // columns of an empty group hold whatever an earlier tile left in S and dP: never used
          p[u] = kept ? ex2_approx(fmaf(__uint_as_float(x[col]), c, -big_l)) : 0.f;
          ds[u] = kept ? p[u] * (__uint_as_float(y[col]) - dsum) : 0.f;
        }
        pp[cc][e] = pack2<kF16>(p[0], p[1]);
        pd[cc][e] = pack2<kF16>(ds[0], ds[1]);
      }
    }
    store_chunk(x_s, r, 2 * half, pp[0]);
    store_chunk(x_s, r, 2 * half + 1, pp[1]);
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (leader) {
      tc_fence_after_sync();
      mma_atb<D>(tmem_dv, x_s, do_s, idesc_t, started);
      mma_commit(&bars->mma);
    }
    ok = cta_wait(&bars->mma, mma_n++ & 1u, bars, err, max_polls);  // P is read: the area takes dS
    if (!ok) break;
    store_chunk(x_s, r, 2 * half, pd[0]);
    store_chunk(x_s, r, 2 * half + 1, pd[1]);
    fence_proxy_async_smem();
    __syncthreads();
    if (leader) {
      tc_fence_after_sync();
      mma_atb<D>(tmem_dk, x_s, q_s, idesc_t, started);
      mma_commit(&bars->mma2);  // waited for through the next tile's S and dP, or below
    }
    ++dk_n;
    started = true;
    qt_cur = qt_nxt;
    t_cur = t_nxt;
  }
  if (ok && started) ok = cta_wait(&bars->mma2, (dk_n - 1u) & 1u, bars, err, max_polls);

  // ---- dV and dK rows of this key tile (thread r = key row), rounded once
  const int j = kt * kTile + r;
  if (ok) {
    tc_fence_after_sync();
#pragma unroll 1
    for (int which = 0; which < 2; ++which) {
      uint16_t *out = (which ? dK : dV) + ((size_t)bh * Lk + j) * D;
      const float f = which ? scale : 1.f;
#pragma unroll 1
      for (int ch = half; ch < D / 32; ch += 2) {
        uint32_t x[32];
        if (started) {  // the same for every thread; the loads are warp-wide
          tmem_ld32((which ? tmem_dk : tmem_dv) + lane_addr + 32 * ch, x);
          tmem_wait_ld();
        }
        if (j < Lk) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e)
              pk[e] = started ? pack2<kF16>(__uint_as_float(x[8 * q + 2 * e]) * f,
                                            __uint_as_float(x[8 * q + 2 * e + 1]) * f)
                              : 0u;
            *reinterpret_cast<uint4 *>(out + 32 * ch + 8 * q) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
      }
    }
  }
  if (!ok) drain_copies(bars, tma_n);  // ok is the same for every thread
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

template <int D, bool kF16>
cudaError_t launch(const BwdMaps &maps, void *dQ, void *dK, void *dV, float *stat_l, float *stat_d, int32_t *tile_id,
                   const ap_tiles &t, int B, int H, int Lq, int Lk, float scale, unsigned *err, cudaStream_t s) {
  using C = Cfg<D>;
  const DebugKnobs knobs = debug_knobs();  // poll limit; test hook of the failure path
  auto rows = bwd_rows_kernel<D, kF16>;
  auto cols = bwd_cols_kernel<D, kF16>;
  cudaError_t e = cudaFuncSetAttribute(rows, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kRowsSmem);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(cols, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kColsSmem);
  if (e != cudaSuccess) return e;
  rows<<<B * H * t.n_qt, kThreads, C::kRowsSmem, s>>>(maps, static_cast<uint16_t *>(dQ), stat_l, stat_d, t.round_ptr,
                                                      t.round_rows, t.round_info, t.round_bitmap, H, Lq, t.n_qt,
                                                      scale, err, knobs.max_polls, knobs.skip_arrive);
  tile_lookup_kernel<<<H * t.n_qt, 128, 0, s>>>(t.row_ptr, t.col_idx, H * t.n_qt, t.n_kt, tile_id);
  count_launches(2);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  cols<<<B * H * t.n_kt, kThreads, C::kColsSmem, s>>>(maps, static_cast<uint16_t *>(dK), static_cast<uint16_t *>(dV),
                                                      stat_l, stat_d, tile_id, t.flags, t.groups, t.bitmap, H, Lq, Lk,
                                                      t.n_qt, t.n_kt, scale, err, knobs.max_polls, knobs.skip_arrive);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

// row statistics (L and D, one float each per query row) and the (query tile, key tile) -> list position table
size_t bwd_workspace_bytes(int B, int H, int Lq, int Lk) {
  const size_t stats = (2 * sizeof(float) * (size_t)B * H * Lq + 255) / 256 * 256;
  return stats + sizeof(int32_t) * (size_t)H * ceil_div(Lq, kTile) * ceil_div(Lk, kTile);
}

cudaError_t launch_bwd_tc(const void *Q, const void *K, const void *V, const void *O, const void *dO,
                          const ap_tiles &t, void *dQ, void *dK, void *dV, void *workspace, int B, int H, int Lq,
                          int Lk, int d, int f16, float scale, cudaStream_t s) {
  unsigned *err = device_error_word();
  if (!err) return cudaErrorUnknown;
  BwdMaps maps;
  if (!make_tile_map_bf16(&maps.q, Q, B * H, Lq, d) || !make_tile_map_bf16(&maps.k, K, B * H, Lk, d) ||
      !make_tile_map_bf16(&maps.v, V, B * H, Lk, d) || !make_tile_map_bf16(&maps.o, O, B * H, Lq, d) ||
      !make_tile_map_bf16(&maps.d_o, dO, B * H, Lq, d))
    return cudaErrorUnknown;
  for (int lg = 0; lg < 4; ++lg)
    if (!make_tile_map_bf16(&maps.kbox[lg], K, B * H, Lk, d, 16 << lg) ||
        !make_tile_map_bf16(&maps.vbox[lg], V, B * H, Lk, d, 16 << lg))
      return cudaErrorUnknown;
  float *stat_l = static_cast<float *>(workspace);
  float *stat_d = stat_l + (size_t)B * H * Lq;
  int32_t *tile_id = reinterpret_cast<int32_t *>(static_cast<char *>(workspace) +
                                                 (2 * sizeof(float) * (size_t)B * H * Lq + 255) / 256 * 256);
  if (d == 64)
    return f16 ? launch<64, true>(maps, dQ, dK, dV, stat_l, stat_d, tile_id, t, B, H, Lq, Lk, scale, err, s)
               : launch<64, false>(maps, dQ, dK, dV, stat_l, stat_d, tile_id, t, B, H, Lq, Lk, scale, err, s);
  return f16 ? launch<128, true>(maps, dQ, dK, dV, stat_l, stat_d, tile_id, t, B, H, Lq, Lk, scale, err, s)
             : launch<128, false>(maps, dQ, dK, dV, stat_l, stat_d, tile_id, t, B, H, Lq, Lk, scale, err, s);
}

}  // namespace ap
