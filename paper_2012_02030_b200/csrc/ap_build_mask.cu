// Eq. 2 as an exact per-head top-k selection.
//
// Order of the entries of one head: forced (diagonal) first, then larger fp32
// value, then lower linear index i*Lk + j.  The k-th entry of that order is
// found with a most-significant-digit-first radix select over order-preserving
// 32-bit keys: three digits of 11, 11 and 10 bits, one histogram pass over the
// accumulator each.  Large heads first try a shortcut that needs one pass: a
// random sample of the head brackets the threshold between two pivot keys, one
// pass counts the keys above the upper pivot and collects those between the
// pivots, and the threshold is selected among the collected keys (the same radix
// select on their offsets from the lower pivot, grid-wide); it is exact
// whenever the bracket holds the threshold and the collected keys fit their
// buffer (checked with the exact counts), else the head takes the three passes.  Entries equal to the threshold key are all kept when the
// count allows it (the usual case); otherwise they are ranked by linear index
// with per-row-segment tie counts and a prefix sum, so that exactly k entries
// are kept.  The emit pass writes the element mask and per-tile bitmaps;
// ap_tiles.cu compacts them.  Integer work throughout: no floating-point
// arithmetic decides a bit.
//
// One threshold for the whole layer (Eq. 2 as stated) is the same selection run
// once over a virtual head of H*Lq rows: row i' = h*Lq + i has the domain of row
// i, and the linear index i'*Lk + j is the layer-wide tie order.
#include "ap_common.cuh"

namespace ap {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kBins = 2048;
constexpr int kPasses = 3;

__host__ __device__ constexpr int digit_shift(int pass) { return pass == 0 ? 21 : (pass == 1 ? 10 : 0); }
__host__ __device__ constexpr uint32_t digit_mask(int pass) { return pass == 2 ? 0x3ffu : 0x7ffu; }

// Larger float <=> larger key; -0 is mapped onto +0 first.
__device__ __forceinline__ uint32_t key_of(float f) {
  uint32_t b = __float_as_uint(f);
  if (b == 0x80000000u) b = 0u;
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// The float whose key is `key`.  Keys 0 and 0xffffffff (no pivot / no threshold) give NaNs, for
// which every ordered comparison is false.  For values and pivots that are not NaN,
// key_of(f) > key <=> f > float_of_key(key), and likewise for == and <.
__device__ __forceinline__ float float_of_key(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key ^ 0x80000000u) : ~key);
}

struct SelectState {  // per selection
  uint32_t prefix;    // digits of the threshold key found so far
  uint32_t thr;       // threshold key (valid after the last digit)
  unsigned long long remaining;  // rank still to resolve inside the current prefix
  unsigned long long ties_kept;  // entries equal to thr that are kept (lowest indices first)
  uint32_t all_ties_kept;        // every entry equal to thr is kept: no ranking needed
  uint32_t done;                 // thr, ties_kept, all_ties_kept are final (set by the one-pass shortcut)
  // the shortcut's bracket and what the collecting pass found
  uint32_t lo, hi;               // pivot keys, lo <= hi; hi == 0xffffffff: no upper pivot
  unsigned long long above_hi;   // keys > hi
  uint32_t n_cand;               // keys in [lo, hi] (may exceed the buffer: then the shortcut fails)
  uint32_t use_shortcut;
  // when not all entries equal to thr are kept: those with linear index i*Lk + j <= tie_cut are
  // (valid if have_cut; otherwise the ties are ranked with tie counts and a prefix sum)
  uint32_t tie_cut, have_cut;
  // selection among the collected keys
  uint32_t cand_select;          // the bracket holds the threshold: the passes over the collected keys run
  uint32_t thr_count;            // entries equal to the threshold key
  uint32_t tie_n;                // entries gathered in the tie list
  // the classifying pass and the patch pass have written this selection's mask and tile bitmaps: the
  // emit pass has nothing left to do for it
  uint32_t emitted;
  // CTAs of the running kernel that have finished their share of this selection: the last one goes on
  // with the step that needs all of them (digit pick, tie scan, finish) and puts the count back to zero
  uint32_t ticket;
};

// Called by all threads of a CTA when its share of selection h is done (its global writes issued):
// true in exactly the CTA that finishes last, which then sees everything the others wrote.
__device__ __forceinline__ bool last_cta_of(SelectState *state, int h, uint32_t n_ctas) {
  __shared__ uint32_t last_s;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool last = atomicAdd(&state[h].ticket, 1u) == n_ctas - 1u;
    if (last) state[h].ticket = 0u;
    last_s = last ? 1u : 0u;
  }
  __syncthreads();
  if (last_s) __threadfence();
  return last_s != 0u;
}

// Selection among the keys the one-pass shortcut collected (see below).
// The bracket holds the threshold (the (k_rest - above_hi)-th largest collected key) and every key
// of the bracket was collected.  All fields are final once the collecting pass has ended.
__device__ __forceinline__ bool bracket_holds(const SelectState &st, uint32_t cand_cap, unsigned long long k_rest) {
  return st.use_shortcut && st.n_cand <= cand_cap && st.above_hi < k_rest && k_rest - st.above_hi <= st.n_cand;
}
// All offsets are at most hi - lo: a leading digit in which that span is zero is zero for every
// key and needs no pass (the pick leaves the digit at zero).
__device__ __forceinline__ bool digit_is_zero(const SelectState &st, int pass) {
  return pass < kPasses - 1 && ((st.hi - st.lo) >> digit_shift(pass)) == 0u;
}

constexpr int kMaxCutTies = 4096;  // ties with the threshold ranked inside the shortcut (more: tie counts + scan)

struct Scratch {
  uint32_t *hist;       // [H][kBins]
  SelectState *state;   // [H]
  uint32_t *tie_count;  // [H][Lq][n_kt] -> exclusive prefix after the scan
  uint32_t *tie_list;   // [H][kMaxCutTies] linear indices of the collected entries equal to the threshold
  uint2 *cand;          // [H][cand_cap] (key, linear index) of the entries collected by the shortcut
};

// The shortcut is tried for heads of at least this many selectable entries.
constexpr long long kShortcutMinEntries = 1ll << 20;
constexpr int kSamples = 16384;  // draws per head (over the Lq x Lk rectangle; draws outside the domain are dropped)
__host__ __device__ inline long long cand_capacity(long long n_rest) {
  return n_rest >= kShortcutMinEntries ? n_rest / 16 : 0;
}

__host__ __device__ inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// Loads 4 consecutive entries of a row starting at column j0 (j0 % 4 == 0).
// Entries at or beyond `jend` come back as 0 and are flagged invalid by the caller.
__device__ __forceinline__ void load4(const float *__restrict__ row, int j0, int jend, bool vec, float v[4]) {
  if (vec && j0 + 4 <= jend) {
    float4 t = *reinterpret_cast<const float4 *>(row + j0);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  } else {
#pragma unroll
    for (int c = 0; c < 4; ++c) v[c] = (j0 + c < jend) ? row[j0 + c] : 0.f;
  }
}

// n_sel selections (one per head, or one for the layer); nnz[H] starts at nnz_init.
__global__ void init_state_kernel(SelectState *state, uint32_t *hist, int n_sel, unsigned long long k_rest, int H,
                                  long long nnz_init, int64_t *nnz) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < n_sel * kBins) hist[idx] = 0u;
  if (nnz && idx < H) nnz[idx] = nnz_init;
  if (idx < n_sel) {
    state[idx].prefix = 0u;
    state[idx].thr = 0xffffffffu;
    state[idx].remaining = k_rest;
    state[idx].ties_kept = 0ull;
    state[idx].all_ties_kept = 0u;
    state[idx].done = 0u;
    state[idx].lo = 0u;
    state[idx].hi = 0xffffffffu;
    state[idx].above_hi = 0ull;
    state[idx].n_cand = 0u;
    state[idx].use_shortcut = 0u;
    state[idx].tie_cut = 0u;
    state[idx].have_cut = 0u;
    state[idx].cand_select = 0u;
    state[idx].thr_count = 0u;
    state[idx].tie_n = 0u;
    state[idx].emitted = 0u;
    state[idx].ticket = 0u;
  }
}

__device__ void pick_digit(SelectState *state, uint32_t *hist, int h, int pass, int from_cand, uint32_t cand_cap,
                           unsigned long long k_rest);

// Histogram of one digit over the non-forced domain entries whose higher digits
// equal the prefix found so far; the CTA that finishes last picks the digit.  grid = (row blocks, selections); a warp takes a row at
// a time and its lanes stride over the row, two float4 loads in flight each.
// Here and in the kernels below Lq counts the rows of the selection and row i has
// the domain of row i % period of a head (period == Lq unless heads are stacked).
// Under the causal constraint row r of a head sees the keys j <= r + (Lk - period):
// Lk - period memory keys, then its own segment; its own position r + (Lk - period)
// is the forced entry when the diagonal is kept.
__global__ void __launch_bounds__(kThreads) digit_histogram_kernel(const float *__restrict__ acc, int Lq, int Lk,
                                                                   int period, int causal, int diag, int pass,
                                                                   SelectState *state, uint32_t *hist) {
  __shared__ uint32_t sh[kBins];
  const int h = blockIdx.y;
  if (state[h].done) return;  // resolved by the shortcut
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int b = threadIdx.x; b < kBins; b += kThreads) sh[b] = 0u;
  __syncthreads();
  const int shift = digit_shift(pass);
  const uint32_t dmask = digit_mask(pass);
  const uint32_t prefix = state[h].prefix;
  const uint32_t hi_mask = pass == 0 ? 0u : ~((1u << (shift + (pass == 1 ? 11 : 10))) - 1u);
  const uint32_t want_hi = prefix & hi_mask;
  const bool vec = (Lk & 3) == 0;
  const int off = (causal || diag) ? Lk - period : 0;
  for (int i = blockIdx.x * kWarps + warp; i < Lq; i += gridDim.x * kWarps) {
    const float *row = acc + ((size_t)h * Lq + i) * Lk;
    const int own = i % period + off;  // the row's own position among the keys
    const int jend = causal ? min(Lk, own + 1) : Lk;
    for (int base = 0; base < jend; base += 256) {  // warp-uniform trip count
      float v[2][4];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int j0 = base + 128 * u + 4 * lane;
        v[u][0] = v[u][1] = v[u][2] = v[u][3] = 0.f;
        if (j0 < jend) load4(row, j0, jend, vec, v[u]);
      }
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int j0 = base + 128 * u + 4 * lane;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int j = j0 + c;
          const uint32_t key = key_of(v[u][c]);
          const bool take = j < jend && !(diag && j == own) && ((key & hi_mask) == want_hi);
          const uint32_t bin = (key >> shift) & dmask;
          // lanes that hit the same bin elect one to add their count
          const unsigned voters = __ballot_sync(0xffffffffu, take);
          if (take) {
            const unsigned peers = __match_any_sync(voters, bin);
            if (lane == __ffs(peers) - 1) atomicAdd(&sh[bin], (uint32_t)__popc(peers));
          }
        }
      }
    }
  }
  __syncthreads();
  for (int b = threadIdx.x; b < kBins; b += kThreads) {
    const uint32_t s = sh[b];
    if (s) atomicAdd(&hist[h * kBins + b], s);
  }
  if (last_cta_of(state, h, gridDim.x)) pick_digit(state, hist, h, pass, 0, 0u, 0ull);
}

// One CTA per head: picks the digit whose bin contains the wanted rank.  Thread t
// owns bins [kBins-1-8t, kBins-8-8t] (descending); a block-wide prefix over the
// threads' sums locates the owner, which then walks its eight bins.
// from_cand: the histogram came from the collected keys (offsets from the lower pivot); the first
// such pass opens the selection among them if the bracket holds the threshold.
// Run by the last CTA (256 threads) of the histogram pass that filled hist.
__device__ void pick_digit(SelectState *state, uint32_t *hist, int h, int pass, int from_cand, uint32_t cand_cap,
                           unsigned long long k_rest) {
  __shared__ uint32_t warp_sums[8];
  if (!from_cand && state[h].done) return;  // resolved by the shortcut
  if (from_cand) {
    const SelectState cur = state[h];
    if (!(pass == 0 ? bracket_holds(cur, cand_cap, k_rest) : cur.cand_select != 0u)) return;
    if (digit_is_zero(cur, pass)) {
      if (pass == 0 && threadIdx.x == 0) {
        state[h].remaining = k_rest - cur.above_hi;
        state[h].prefix = 0u;
        state[h].cand_select = 1u;
      }
      return;
    }
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t cnt[8];
  uint32_t mine = 0u;
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const int bin = kBins - 1 - (8 * (int)threadIdx.x + e);
    cnt[e] = __ldcg(hist + h * kBins + bin);
    hist[h * kBins + bin] = 0u;
    mine += cnt[e];
  }
  uint32_t incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) warp_sums[warp] = incl;
  SelectState st = state[h];  // read by everyone before the barrier, written by the owner after it
  if (from_cand && pass == 0) {
    st.remaining = k_rest - st.above_hi;
    st.prefix = 0u;
    st.cand_select = 1u;
  }
  __syncthreads();
  unsigned long long before = incl - mine;  // entries in bins above this thread's
  for (int w = 0; w < warp; ++w) before += warp_sums[w];
  // the owner: fewer than `remaining` entries above its bins, at least that many including them;
  // the last thread also takes the case of an over-long rank (cannot happen for valid k)
  const bool owner = before < st.remaining && (before + mine >= st.remaining || threadIdx.x == 255);
  if (owner) {
    unsigned long long above = before;
    int e = 0;
    for (; e < 7; ++e) {
      if (above + cnt[e] >= st.remaining) break;
      above += cnt[e];
    }
    const int bin = kBins - 1 - (8 * (int)threadIdx.x + e);
    SelectState out = st;
    out.remaining = st.remaining - above;
    out.prefix = st.prefix | ((uint32_t)bin << digit_shift(pass));
    if (pass == kPasses - 1) {
      out.thr = out.prefix;
      out.ties_kept = out.remaining;
      out.all_ties_kept = out.remaining == cnt[e] ? 1u : 0u;
      out.thr_count = cnt[e];
    }
    state[h] = out;
  }
}

// ---- the one-pass shortcut ------------------------------------------------------------------

// CTA-wide (1024 threads) radix select: the key of rank `rank` (1 = largest) among keys[0..n),
// 1 <= rank <= n.  Returns the key, how many keys equal it, and the rank inside that group of
// equals.  hist: 2048 words of shared memory; xch: 4 words.
struct Picked {
  uint32_t key, count, rank_in_ties;
};
// scan(fn) calls fn(key) once for every key, the keys spread over the CTA's threads in any way.
template <typename Scan>
__device__ Picked block_select_over(uint32_t n, uint32_t rank, uint32_t *hist, uint32_t *xch, Scan scan) {
  __shared__ uint32_t warp_sums[32];
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  uint32_t prefix = 0u, hi_mask = 0u, count = n;
  for (int pass = 0; pass < kPasses; ++pass) {
    const int shift = digit_shift(pass);
    const uint32_t dmask = digit_mask(pass);
    hist[t] = 0u;
    hist[t + 1024] = 0u;
    __syncthreads();
    scan([&](uint32_t key) {
      if ((key & hi_mask) == prefix) atomicAdd(&hist[(key >> shift) & dmask], 1u);
    });
    __syncthreads();
    // thread t owns bins 2047 - 2t and 2046 - 2t (descending order of keys)
    const uint32_t c0 = hist[kBins - 1 - 2 * t], c1 = hist[kBins - 2 - 2 * t];
    const uint32_t mine = c0 + c1;
    uint32_t incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    uint32_t before = incl - mine;
    for (int w = 0; w < warp; ++w) before += warp_sums[w];
    if (before < rank && before + mine >= rank) {  // exactly one thread
      const bool first = before + c0 >= rank;
      xch[0] = (uint32_t)(kBins - 1 - 2 * t - (first ? 0 : 1));
      xch[1] = rank - before - (first ? 0u : c0);
      xch[2] = first ? c0 : c1;
    }
    __syncthreads();
    prefix |= xch[0] << shift;
    rank = xch[1];
    count = xch[2];
    hi_mask |= dmask << shift;
    __syncthreads();
  }
  Picked p;
  p.key = prefix;
  p.count = count;
  p.rank_in_ties = rank;
  return p;
}
__device__ Picked block_select(const uint32_t *keys, uint32_t n, uint32_t rank, uint32_t *hist, uint32_t *xch) {
  return block_select_over(n, rank, hist, xch, [&](auto fn) {
    for (uint32_t idx0 = threadIdx.x; idx0 < n; idx0 += 8 * 1024) {  // eight loads in flight per thread
      uint32_t kk[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const uint32_t idx = idx0 + u * 1024;
        kk[u] = idx < n ? keys[idx] : 0xffffffffu;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u)
        if (idx0 + u * 1024 < n) fn(kk[u]);
    }
  });
}

__device__ __forceinline__ unsigned long long mix64(unsigned long long x) {
  x += 0x9e3779b97f4a7c15ull;
  x = (x ^ (x >> 30)) * 0xbf58476d1ce4e5b9ull;
  x = (x ^ (x >> 27)) * 0x94d049bb133111ebull;
  return x ^ (x >> 31);
}

// Two CTAs per selection (blockIdx.y = 0: upper pivot, 1: lower pivot), each of which samples the
// selection's entries (the same draws) and sets its end of the bracket [lo, hi] around the
// expected threshold.
__global__ void __launch_bounds__(1024) sample_pivots_kernel(const float *__restrict__ acc, int Lq, int Lk, int period,
                                                             int causal, int diag, unsigned long long k_rest,
                                                             unsigned long long n_rest, SelectState *state) {
  extern __shared__ uint32_t sm_dyn[];
  uint32_t *keys = sm_dyn;               // kSamples
  uint32_t *hist = sm_dyn + kSamples;    // kBins
  __shared__ uint32_t xch[4];
  __shared__ uint32_t n_valid_s;
  const int h = blockIdx.x, t = threadIdx.x;
  if (t == 0) n_valid_s = 0u;
  __syncthreads();
  const int off = (causal || diag) ? Lk - period : 0;
  constexpr int kDraws = kSamples / 1024;  // per thread, all loads in flight at once
  float drawn[kDraws];
  bool valid[kDraws];
#pragma unroll
  for (int u = 0; u < kDraws; ++u) {
    const int s = t + 1024 * u;
    // row and column from the two halves of one 64-bit draw, scaled by multiplication (64-bit
    // divisions, emulated in dozens of instructions each, made up most of this kernel's time)
    const unsigned long long m = mix64(((unsigned long long)h << 32) | (unsigned)s);
    const int i = (int)(((m >> 32) * (unsigned long long)Lq) >> 32);
    const int j = (int)(((m & 0xffffffffull) * (unsigned long long)Lk) >> 32);
    const int own = i % period + off;
    valid[u] = !((causal && j > own) || (diag && j == own));
    drawn[u] = valid[u] ? acc[((size_t)h * Lq + i) * Lk + j] : 0.f;
  }
#pragma unroll
  for (int u = 0; u < kDraws; ++u)
    if (valid[u]) keys[atomicAdd(&n_valid_s, 1u)] = key_of(drawn[u]);
  __syncthreads();
  const uint32_t nv = n_valid_s;
  if (nv < 1024u) return;  // too few draws landed in the domain: no shortcut for this head
  // expected rank of the threshold inside the sample and a bracket of six standard deviations
  const double frac = (double)k_rest / (double)n_rest;
  const double r = frac * nv;
  const double dev = 6.0 * sqrt(fmax(r * (1.0 - frac), 1.0)) + 16.0;
  const long long r_hi = (long long)floor(r - dev), r_lo = (long long)ceil(r + dev);
  if (blockIdx.y == 0) {
    uint32_t hi = 0xffffffffu;
    if (r_hi >= 1) hi = block_select(keys, nv, (uint32_t)r_hi, hist, xch).key;
    if (t == 0) state[h].hi = hi;
  } else {
    uint32_t lo = 0u;
    if (r_lo <= (long long)nv) lo = block_select(keys, nv, (uint32_t)r_lo, hist, xch).key;
    if (t == 0) state[h].lo = lo;
  }
  if (t == 0) state[h].use_shortcut = 1u;  // both CTAs take the same decision
}

// One pass over the selection's rows: counts the keys above the upper pivot and collects those
// inside the bracket.  grid = (row blocks, selections); a warp takes a row at a time.  Values are
// compared with the pivots as floats (the same order as their keys); the key is computed for the
// collected entries only.  Each warp stages its collected entries in shared memory and appends
// them to the selection's buffer, one reservation per flush, whenever the stage is half full at
// the end of a chunk of the row (an entry that finds the stage full goes straight to the buffer).
constexpr int kWarpStage = 512;
__global__ void __launch_bounds__(kThreads) collect_kernel(const float *__restrict__ acc, int Lq, int Lk, int period,
                                                           int causal, int diag, SelectState *state,
                                                           uint2 *__restrict__ cand, uint32_t cand_cap) {
  __shared__ uint2 stage_all[kWarps][kWarpStage];
  __shared__ uint32_t stage_n_all[kWarps];  // may run past the stage: those entries were not staged
  const int h = blockIdx.y;
  if (!state[h].use_shortcut) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint2 *stage = stage_all[warp];
  uint32_t *stage_n = &stage_n_all[warp];
  if (lane == 0) *stage_n = 0u;
  __syncwarp();
  const float lo_f = float_of_key(state[h].lo), hi_f = float_of_key(state[h].hi);
  uint2 *out = cand + (size_t)h * cand_cap;
  uint32_t *n_cand = &state[h].n_cand;
  auto push = [&](float f, uint32_t index) {  // a few per cent of the entries
    const uint2 entry = make_uint2(key_of(f), index);
    const uint32_t pos = atomicAdd(stage_n, 1u);
    if (pos < (uint32_t)kWarpStage) {
      stage[pos] = entry;
    } else {
      const uint32_t g = atomicAdd(n_cand, 1u);
      if (g < cand_cap) out[g] = entry;
    }
  };
  auto flush = [&](uint32_t at_least) {  // by the whole warp
    __syncwarp();
    const uint32_t n = min(*stage_n, (uint32_t)kWarpStage);
    if (n >= at_least && n > 0u) {
      uint32_t dst = 0u;
      if (lane == 0) dst = atomicAdd(n_cand, n);
      dst = __shfl_sync(0xffffffffu, dst, 0);
      for (uint32_t e = lane; e < n; e += 32)
        if (dst + e < cand_cap) out[dst + e] = stage[e];
      __syncwarp();
      if (lane == 0) *stage_n = 0u;
      __syncwarp();
    }
  };
  const bool vec = (Lk & 3) == 0;
  uint32_t above = 0u;  // per thread: fewer than 2^32 entries
  const int off = (causal || diag) ? Lk - period : 0;
  for (int i = blockIdx.x * kWarps + warp; i < Lq; i += gridDim.x * kWarps) {
    const float *row = acc + ((size_t)h * Lq + i) * Lk;
    const int own = i % period + off;  // the row's own position among the keys
    const int jend = causal ? min(Lk, own + 1) : Lk;
    const uint32_t row_index = (uint32_t)i * (uint32_t)Lk;
    for (int base = 0; base < jend; base += 512) {  // warp-uniform trip count
      float v[4][4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int j0 = base + 128 * u + 4 * lane;
        v[u][0] = v[u][1] = v[u][2] = v[u][3] = 0.f;
        if (j0 < jend) load4(row, j0, jend, vec, v[u]);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int j0 = base + 128 * u + 4 * lane;
        if (j0 + 4 <= jend && !(diag && own >= j0 && own < j0 + 4)) {
          // four entries of the domain: nothing to check per entry, and nothing to do at all where all
          // four lie below the bracket (most pieces of a row: the bracket sits near the top of the values)
          if (v[u][0] < lo_f && v[u][1] < lo_f && v[u][2] < lo_f && v[u][3] < lo_f) continue;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const float f = v[u][c];
            const bool gt = f > hi_f;
            above += gt ? 1u : 0u;
            if (!(f < lo_f) && !gt) push(f, row_index + (uint32_t)(j0 + c));
          }
        } else if (j0 < jend) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int j = j0 + c;
            const float f = v[u][c];
            const bool in = j < jend && !(diag && j == own);
            const bool gt = in && f > hi_f;
            above += gt ? 1u : 0u;
            if (in && !(f < lo_f) && !gt) push(f, row_index + (uint32_t)j);
          }
        }
      }
      flush(kWarpStage / 2);
    }
  }
  flush(1u);
  unsigned long long above_warp = above;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) above_warp += __shfl_xor_sync(0xffffffffu, above_warp, o);
  if (lane == 0 && above_warp) atomicAdd(&state[h].above_hi, above_warp);
}

// ---- selection among the collected keys: the radix select on their offsets from the lower pivot ----


// grid = (CTAs, selections)
__global__ void __launch_bounds__(kThreads) cand_histogram_kernel(SelectState *state, const uint2 *__restrict__ cand,
                                                                  uint32_t cand_cap, unsigned long long k_rest,
                                                                  int pass, uint32_t *hist) {
  __shared__ uint32_t sh[kBins];
  const int h = blockIdx.y;
  const SelectState st = state[h];
  if (!(pass == 0 ? bracket_holds(st, cand_cap, k_rest) : st.cand_select != 0u)) return;
  if (digit_is_zero(st, pass)) {  // no pass needed; the first CTA lets the pick open the selection
    if (blockIdx.x == 0) pick_digit(state, hist, h, pass, 1, cand_cap, k_rest);
    return;
  }
  const int lane = threadIdx.x & 31;
  for (int b = threadIdx.x; b < kBins; b += kThreads) sh[b] = 0u;
  __syncthreads();
  const int shift = digit_shift(pass);
  const uint32_t dmask = digit_mask(pass);
  const uint32_t hi_mask = pass == 0 ? 0u : ~((1u << (shift + (pass == 1 ? 11 : 10))) - 1u);
  const uint32_t want_hi = (pass == 0 ? 0u : st.prefix) & hi_mask;
  const uint32_t n = st.n_cand, lo = st.lo;
  const uint2 *mine = cand + (size_t)h * cand_cap;
  for (uint32_t base = blockIdx.x * (4 * kThreads); base < n; base += gridDim.x * (4 * kThreads)) {  // warp-uniform
    uint32_t key[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {  // four loads in flight
      const uint32_t idx = base + u * kThreads + threadIdx.x;
      key[u] = idx < n ? mine[idx].x - lo : 0u;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t idx = base + u * kThreads + threadIdx.x;
      const bool take = idx < n && (key[u] & hi_mask) == want_hi;
      const uint32_t bin = (key[u] >> shift) & dmask;
      const unsigned voters = __ballot_sync(0xffffffffu, take);
      if (take) {
        const unsigned peers = __match_any_sync(voters, bin);
        if (lane == __ffs(peers) - 1) atomicAdd(&sh[bin], (uint32_t)__popc(peers));
      }
    }
  }
  __syncthreads();
  for (int b = threadIdx.x; b < kBins; b += kThreads) {
    const uint32_t s = sh[b];
    if (s) atomicAdd(&hist[h * kBins + b], s);
  }
  if (last_cta_of(state, h, gridDim.x)) pick_digit(state, hist, h, pass, 1, cand_cap, k_rest);
}

// Ranks `count` <= kMaxCutTies distinct linear indices: returns (in *cut_s, after a barrier) the one
// with exactly rank - 1 smaller ones.  By all threads of a CTA.
__device__ void rank_ties(const uint32_t *tie_idx, uint32_t count, uint32_t rank, uint32_t *cut_s) {
  for (uint32_t e = threadIdx.x; e < count; e += blockDim.x) {
    const uint32_t me = tie_idx[e];
    uint32_t smaller = 0u;
    for (uint32_t f = 0; f < count; ++f) smaller += tie_idx[f] < me ? 1u : 0u;
    if (smaller == rank - 1u) *cut_s = me;
  }
  __syncthreads();
}

// Closes the selection among the collected keys.  grid = (CTAs, selections).  First the linear indices
// of the collected entries equal to the threshold are gathered, when they must be ranked and are few
// enough; the CTA that finishes last then turns the digits found among the collected keys into the
// threshold, ranks those ties (the lowest linear indices are kept) and marks the selection as done.
__global__ void __launch_bounds__(kThreads) cand_finish_kernel(SelectState *state, const uint2 *__restrict__ cand,
                                                               uint32_t cand_cap, uint32_t *tie_list,
                                                               int classified) {
  __shared__ uint32_t tie_idx[kMaxCutTies];
  __shared__ uint32_t cut_s;
  const int h = blockIdx.y;
  const SelectState st = state[h];
  if (!st.cand_select) return;
  const bool rank_them = !st.all_ties_kept && st.thr_count <= (uint32_t)kMaxCutTies;
  if (rank_them) {
    const uint32_t want = st.prefix + st.lo;
    const uint2 *mine = cand + (size_t)h * cand_cap;
    for (uint32_t idx = blockIdx.x * kThreads + threadIdx.x; idx < st.n_cand; idx += gridDim.x * kThreads) {
      const uint2 c = mine[idx];
      if (c.x == want) {
        const uint32_t pos = atomicAdd(&state[h].tie_n, 1u);
        if (pos < (uint32_t)kMaxCutTies) tie_list[(size_t)h * kMaxCutTies + pos] = c.y;
      }
    }
  }
  if (!last_cta_of(state, h, gridDim.x)) return;
  if (rank_them) {
    for (uint32_t e = threadIdx.x; e < st.thr_count; e += kThreads)
      tie_idx[e] = __ldcg(tie_list + (size_t)h * kMaxCutTies + e);
    __syncthreads();
    rank_ties(tie_idx, st.thr_count, (uint32_t)st.ties_kept, &cut_s);
  }
  if (threadIdx.x == 0) {
    state[h].tie_cut = rank_them ? cut_s : 0u;
    state[h].have_cut = rank_them ? 1u : 0u;
    state[h].thr = st.prefix + st.lo;
    state[h].prefix = st.prefix + st.lo;
    state[h].done = 1u;
    // with the classifying pass before it, the patch pass can finish the mask unless the ties would
    // have to be ranked by their counts per row segment
    state[h].emitted = (classified && (st.all_ties_kept || rank_them)) ? 1u : 0u;
  }
}

// ---- small selections: everything in one CTA ----------------------------------------------------

constexpr long long kSelectSmallEntries = 1ll << 15;  // rows x Lk of a selection, at most

// One CTA of 1024 threads per selection of at most kSelectSmallEntries entries: sets up the
// selection's state (and nnz), finds the threshold with the CTA-wide radix select straight over
// the selection's domain, and where only some of the entries equal to the threshold are kept, the
// linear index of the last kept one (tie_cut): by ranking the ties when there are at most
// kMaxCutTies of them, else by bisection on the index (each probe counts the ties up to it).  Such a
// selection needs no other kernel before the emit pass.
__global__ void __launch_bounds__(1024) select_small_kernel(const float *__restrict__ acc, int rows, int Lk,
                                                            int period, int causal, int diag,
                                                            unsigned long long k_rest, SelectState *state, int H,
                                                            long long nnz_init, int64_t *nnz) {
  __shared__ uint32_t hist[kBins];
  __shared__ uint32_t xch[4];
  __shared__ uint32_t tie_idx[kMaxCutTies];
  __shared__ uint32_t tie_n_s, cut_s;
  const int h = blockIdx.x;
  if (nnz && h == 0)
    for (int x = threadIdx.x; x < H; x += 1024) nnz[x] = nnz_init;
  SelectState st;
  st.prefix = 0u, st.thr = 0xffffffffu, st.remaining = k_rest, st.ties_kept = 0ull, st.all_ties_kept = 0u;
  st.done = 1u, st.lo = 0u, st.hi = 0xffffffffu, st.above_hi = 0ull, st.n_cand = 0u, st.use_shortcut = 0u;
  st.tie_cut = 0u, st.have_cut = 0u, st.cand_select = 0u, st.thr_count = 0u, st.tie_n = 0u, st.ticket = 0u;
  st.emitted = 0u;
  if (k_rest == 0ull) {  // nothing but the forced entries is kept
    if (threadIdx.x == 0) state[h] = st;
    return;
  }
  const float *base = acc + (size_t)h * rows * Lk;
  const int off = (causal || diag) ? Lk - period : 0;
  const uint32_t n = (uint32_t)rows * (uint32_t)Lk;
  const bool vec = (Lk & 3) == 0;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // fn(key, linear index) for every selectable entry of rows [0, row_end): a warp takes a row at a time,
  // its lanes four consecutive entries each, two loads in flight
  auto scan_rows = [&](int row_end, auto fn) {
    for (int i = warp; i < row_end; i += 32) {
      const float *row = base + (size_t)i * Lk;
      const int own = i % period + off;  // the row's own position among the keys
      const int jend = causal ? min(Lk, own + 1) : Lk;
      for (int j00 = 0; j00 < jend; j00 += 256) {
        float v[2][4];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int j0 = j00 + 128 * u + 4 * lane;
          v[u][0] = v[u][1] = v[u][2] = v[u][3] = 0.f;
          if (j0 < jend) load4(row, j0, jend, vec, v[u]);
        }
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int j = j00 + 128 * u + 4 * lane + c;
            if (j < jend && !(diag && j == own)) fn(key_of(v[u][c]), (uint32_t)i * (uint32_t)Lk + (uint32_t)j);
          }
      }
    }
  };
  const Picked p = block_select_over(n, (uint32_t)k_rest, hist, xch, [&](auto fn) {
    scan_rows(rows, [&](uint32_t key, uint32_t) { fn(key); });
  });
  st.prefix = st.thr = p.key;
  st.remaining = st.ties_kept = p.rank_in_ties;
  st.thr_count = p.count;
  st.all_ties_kept = p.rank_in_ties == p.count ? 1u : 0u;
  if (!st.all_ties_kept) {
    if (p.count <= (uint32_t)kMaxCutTies) {
      if (threadIdx.x == 0) tie_n_s = 0u;
      __syncthreads();
      scan_rows(rows, [&](uint32_t key, uint32_t idx) {
        if (key == p.key) tie_idx[atomicAdd(&tie_n_s, 1u)] = idx;
      });
      __syncthreads();
      rank_ties(tie_idx, p.count, p.rank_in_ties, &cut_s);
    } else {
      // the smallest index L with rank_in_ties ties at indices <= L
      uint32_t lo = 0u, hi = n - 1u;
      while (lo < hi) {  // the same for every thread
        const uint32_t mid = lo + (hi - lo) / 2u;
        uint32_t mine = 0u;
        scan_rows((int)(mid / (uint32_t)Lk) + 1, [&](uint32_t key, uint32_t idx) {
          mine += (key == p.key && idx <= mid) ? 1u : 0u;
        });
        if (threadIdx.x == 0) tie_n_s = 0u;
        __syncthreads();
        mine = __reduce_add_sync(0xffffffffu, mine);
        if (lane == 0 && mine) atomicAdd(&tie_n_s, mine);
        __syncthreads();
        const uint32_t upto = tie_n_s;
        __syncthreads();
        if (upto >= p.rank_in_ties) hi = mid; else lo = mid + 1u;
      }
      if (threadIdx.x == 0) cut_s = lo;
      __syncthreads();
    }
    st.tie_cut = cut_s;
    st.have_cut = 1u;
  }
  if (threadIdx.x == 0) state[h] = st;
}

// Entries equal to the threshold key per (row, 128-column segment); only for heads
// where the ties must be ranked.  grid = (row blocks, H); a warp takes a row.  The CTA that finishes
// last turns the head's counts into their exclusive prefix sum, in place.
__global__ void __launch_bounds__(kThreads) tie_count_kernel(const float *__restrict__ acc, int Lq, int Lk, int period,
                                                             int n_kt, int causal, int diag, SelectState *state,
                                                             uint32_t *tie_count) {
  const int h = blockIdx.y;
  if (state[h].all_ties_kept || state[h].have_cut) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t thr = state[h].thr;
  const bool vec = (Lk & 3) == 0;
  const int off = (causal || diag) ? Lk - period : 0;
  for (int i = blockIdx.x * kWarps + warp; i < Lq; i += gridDim.x * kWarps) {
    const float *row = acc + ((size_t)h * Lq + i) * Lk;
    const int own = i % period + off;  // the row's own position among the keys
    const int jend = causal ? min(Lk, own + 1) : Lk;
    for (int kt = 0; kt < n_kt; ++kt) {
      const int j0 = kt * kTile + 4 * lane;
      int ties = 0;
      if (j0 < jend) {
        float v[4];
        load4(row, j0, jend, vec, v);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int j = j0 + c;
          ties += (j < jend && !(diag && j == own) && key_of(v[c]) == thr) ? 1 : 0;
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ties += __shfl_xor_sync(0xffffffffu, ties, o);
      if (lane == 0) tie_count[((size_t)h * Lq + i) * n_kt + kt] = (uint32_t)ties;
    }
  }
  if (!last_cta_of(state, h, gridDim.x)) return;
  __shared__ uint32_t warp_sums[kWarps];
  __shared__ uint32_t carry_s;
  const int n_per_head = Lq * n_kt;
  uint32_t *a = tie_count + (size_t)h * n_per_head;
  if (threadIdx.x == 0) carry_s = 0u;
  __syncthreads();
  for (int base = 0; base < n_per_head; base += kThreads) {
    const int idx = base + threadIdx.x;
    const uint32_t x = idx < n_per_head ? __ldcg(a + idx) : 0u;
    uint32_t incl = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    uint32_t before = 0u, total = 0u;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      if (w < warp) before += warp_sums[w];
      total += warp_sums[w];
    }
    const uint32_t carry = carry_s;
    if (idx < n_per_head) a[idx] = carry + before + incl - x;
    __syncthreads();
    if (threadIdx.x == 0) carry_s = carry + total;
    __syncthreads();
  }
}

// A warp's way into a selection's buffer of collected entries: staged in shared memory and appended
// with one reservation per flush (an entry that finds the stage full goes straight to the buffer).
struct Collector {
  uint2 *stage;        // this warp's kWarpStage entries of shared memory
  uint32_t *stage_n;   // entries pushed since the last flush (may run past the stage)
  uint2 *out;          // the selection's buffer
  uint32_t *n_cand;    // entries reserved in it so far (may exceed the capacity: then the shortcut fails)
  uint32_t cap;
  __device__ __forceinline__ void push(float f, uint32_t index) {
    const uint2 entry = make_uint2(key_of(f), index);
    const uint32_t pos = atomicAdd(stage_n, 1u);
    if (pos < (uint32_t)kWarpStage) {
      stage[pos] = entry;
    } else {
      const uint32_t g = atomicAdd(n_cand, 1u);
      if (g < cap) out[g] = entry;
    }
  }
  __device__ __forceinline__ void flush(uint32_t at_least, int lane) {  // by the whole warp
    __syncwarp();
    const uint32_t n = min(*stage_n, (uint32_t)kWarpStage);
    if (n >= at_least && n > 0u) {
      uint32_t dst = 0u;
      if (lane == 0) dst = atomicAdd(n_cand, n);
      dst = __shfl_sync(0xffffffffu, dst, 0);
      for (uint32_t e = lane; e < n; e += 32)
        if (dst + e < cap) out[dst + e] = stage[e];
      __syncwarp();
      if (lane == 0) *stage_n = 0u;
      __syncwarp();
    }
  }
};

// What the emit pass needs of a selection.
struct EmitSel {
  float thr_f;  // the threshold as a float (NaN when nothing but the forced entries is kept)
  float lo_f;   // classifying pass: thr_f is the bracket's upper pivot, lo_f its lower one
  unsigned long long ties_kept;
  bool all_ties, have_cut;
  uint32_t tie_cut;
  uint32_t first_row;  // of this head in the tie order
};

// The rows of one tile; returns this lane's share of the tile's popcount (lanes 0, 8, 16, 24).
// kInterior: every row and column of the tile exists and lies in the domain and none is forced,
// so nothing is checked per entry.
// kClassify: the classifying pass of the one-pass shortcut instead of the emit pass proper.  Entries
// above the bracket are kept, entries inside it are collected (col) and left out for the patch pass
// to decide, entries above the bracket are counted (above).
template <bool kInterior, bool kClassify>
__device__ __forceinline__ int emit_tile_rows(const float *__restrict__ acc, int Lq, int Lk, int n_kt, int h, int qt,
                                              int kt, int tile, int causal, int diag, const EmitSel &sel,
                                              const uint32_t *__restrict__ tie_prefix, uint8_t *__restrict__ mask,
                                              uint32_t *__restrict__ stage_bitmap, Collector &col, uint32_t &above) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool vec = (Lk & 3) == 0;
  const int j0 = kt * kTile + 4 * lane;
  const float thr_f = sel.thr_f;
  const int off = (causal || diag) ? Lk - Lq : 0;  // row i's own position is key i + off
  int count = 0;
  for (int r0 = warp; r0 < kTile; r0 += 16) {
    float v[4][4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {  // rows r0, r0+4, r0+8, r0+12: four loads in flight
      const int i = qt * kTile + r0 + 4 * u;
      if (kInterior) {
        const float4 t = *reinterpret_cast<const float4 *>(acc + ((size_t)h * Lq + i) * Lk + j0);
        v[u][0] = t.x; v[u][1] = t.y; v[u][2] = t.z; v[u][3] = t.w;
      } else {
        v[u][0] = v[u][1] = v[u][2] = v[u][3] = 0.f;
        if (i < Lq) {
          const int jend = causal ? min(Lk, i + 1 + off) : Lk;
          if (j0 < jend) load4(acc + ((size_t)h * Lq + i) * Lk, j0, jend, vec, v[u]);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int r = r0 + 4 * u;
      const int i = qt * kTile + r;
      uint32_t nib = 0u;
      if (kInterior || i < Lq) {  // warp-uniform
        uint32_t tie_bits = 0u, gt_bits = 0u;
        // the lowest value that needs a closer look: the threshold, or the bracket's lower pivot
        const float floor_f = kClassify ? sel.lo_f : thr_f;
        uint32_t forced_bits = 0u;
        if (kInterior) {
          // (most pieces of a row lie wholly below it: one test instead of eight)
          if (!(v[u][0] < floor_f && v[u][1] < floor_f && v[u][2] < floor_f && v[u][3] < floor_f)) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              gt_bits |= (v[u][c] > thr_f ? 1u : 0u) << c;
              tie_bits |= ((kClassify ? !(v[u][c] < floor_f) && !(v[u][c] > thr_f) : v[u][c] == thr_f) ? 1u : 0u) << c;
            }
          }
        } else {
          const int jend = causal ? min(Lk, i + 1 + off) : Lk;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const int j = j0 + c;
            if (j < jend) {
              if (diag && j == i + off) {
                forced_bits |= 1u << c;
              } else {
                gt_bits |= (v[u][c] > thr_f ? 1u : 0u) << c;
                tie_bits |= ((kClassify ? !(v[u][c] < floor_f) && !(v[u][c] > thr_f) : v[u][c] == thr_f) ? 1u : 0u) << c;
              }
            }
          }
        }
        nib = gt_bits | forced_bits;
        if (kClassify) {
          above += (uint32_t)__popc(gt_bits);
          if (tie_bits) {
#pragma unroll
            for (int c = 0; c < 4; ++c)
              if (tie_bits & (1u << c))
                col.push(v[u][c], (sel.first_row + (uint32_t)i) * (uint32_t)Lk + (uint32_t)(j0 + c));
          }
        } else if (sel.all_ties) {
          nib |= tie_bits;
        } else if (sel.have_cut) {
          if (tie_bits) {
#pragma unroll
            for (int c = 0; c < 4; ++c)
              if ((tie_bits & (1u << c)) &&
                  (sel.first_row + (uint32_t)i) * (uint32_t)Lk + (uint32_t)(j0 + c) <= sel.tie_cut)
                nib |= 1u << c;
          }
        } else if (__any_sync(0xffffffffu, tie_bits != 0u)) {
          // rank of each tie in linear-index order = ties before this row segment
          // + ties in lower lanes + ties in lower columns of this lane
          int before = __popc(tie_bits);
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, before, o);
            if (lane >= o) before += t;
          }
          before -= __popc(tie_bits);
          unsigned long long rank = (unsigned long long)tie_prefix[((size_t)h * Lq + i) * n_kt + kt] + before;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            if (tie_bits & (1u << c)) {
              if (rank < sel.ties_kept) nib |= 1u << c;
              ++rank;
            }
          }
        }
        if (mask) {
          uint8_t *mrow = mask + ((size_t)h * Lq + i) * Lk;
          if (kInterior || (vec && j0 + 4 <= Lk)) {
            *reinterpret_cast<uchar4 *>(mrow + j0) =
                make_uchar4(nib & 1u, (nib >> 1) & 1u, (nib >> 2) & 1u, (nib >> 3) & 1u);
          } else {
#pragma unroll
            for (int c = 0; c < 4; ++c)
              if (j0 + c < Lk) mrow[j0 + c] = (nib >> c) & 1u;
          }
        }
      }
      // 8 lanes x 4 bits -> one bitmap word, complete in the first lane of each group of eight
      uint32_t w = nib << (4 * (lane & 7));
      w |= __shfl_xor_sync(0xffffffffu, w, 1);
      w |= __shfl_xor_sync(0xffffffffu, w, 2);
      w |= __shfl_xor_sync(0xffffffffu, w, 4);
      if ((lane & 7) == 0) {
        count += __popc(w);
        if (stage_bitmap) stage_bitmap[(size_t)tile * kBitmapWords + 4 * r + (lane >> 3)] = w;
      }
    }
    if (kClassify) col.flush(kWarpStage / 2, lane);
  }
  if (kClassify) col.flush(1u, lane);
  return count;
}

// One CTA per tile of the (h, qt, kt) grid; warp w takes tile rows w, w+4, ...
// (four rows loaded ahead) and each lane four consecutive columns.  Writes the
// element mask, the tile's bitmap and popcount into the staging area.  Values are
// compared with the threshold as floats (the same order as their keys).  per_layer:
// all heads share selection 0, ties are ordered by (h*Lq + i)*Lk + j, and the
// tiles' popcounts are added up into nnz[h].  keep_ties: every entry equal to the threshold is
// kept (no ranking), and the popcounts are added up as well (the count is not known beforehand).
// kClassify: the shortcut's one pass over the accumulator, which does the collecting pass's work
// (entries above the upper pivot counted, entries inside the bracket appended to the selection's
// buffer) and most of the emit pass's at once: everything above the bracket is kept, everything else
// left out, and patch_kernel adds the collected entries that turn out to be kept.  Only for exact
// per-head selections (the kept count is known beforehand, nothing is counted here).
template <bool kClassify>
__global__ void __launch_bounds__(128) emit_kernel(const float *__restrict__ acc, int Lq, int Lk, int n_qt, int n_kt,
                                                   int causal, int diag, int per_layer, int keep_ties,
                                                   SelectState *state, const uint32_t *__restrict__ tie_prefix,
                                                   uint8_t *__restrict__ mask, uint32_t *__restrict__ stage_bitmap,
                                                   int32_t *__restrict__ stage_count, int64_t *__restrict__ nnz,
                                                   uint2 *__restrict__ cand, uint32_t cand_cap) {
  const int tile = blockIdx.x;
  const int kt = tile % n_kt;
  const int qt = (tile / n_kt) % n_qt;
  const int h = tile / (n_kt * n_qt);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __shared__ int warp_count[4];
  __shared__ uint2 stage_all[kClassify ? 4 : 1][kClassify ? kWarpStage : 1];
  __shared__ uint32_t stage_n_all[4];
  SelectState &st = state[per_layer ? 0 : h];
  if (kClassify ? !st.use_shortcut : st.emitted != 0u) return;  // not this pass's selection
  // own positions of the tile's rows among the keys: columns own_lo .. own_hi
  const int own_lo = qt * kTile + ((causal || diag) ? Lk - Lq : 0), own_hi = own_lo + kTile - 1;
  if (causal && kt * kTile > own_hi) {
    // the whole tile lies above the diagonal: nothing is kept, nothing needs to be read
    const bool vec = (Lk & 3) == 0;
    const int j0 = kt * kTile + 4 * lane;
    for (int r = warp; r < kTile; r += 4) {
      const int i = qt * kTile + r;
      if (i < Lq && mask) {
        uint8_t *mrow = mask + ((size_t)h * Lq + i) * Lk;
        if (vec && j0 + 4 <= Lk) {
          *reinterpret_cast<uchar4 *>(mrow + j0) = make_uchar4(0, 0, 0, 0);
        } else {
          for (int c = 0; c < 4; ++c)
            if (j0 + c < Lk) mrow[j0 + c] = 0;
        }
      }
      if (stage_bitmap && lane == 0)
        reinterpret_cast<uint4 *>(stage_bitmap + (size_t)tile * kBitmapWords)[r] = make_uint4(0u, 0u, 0u, 0u);
    }
    if (stage_count && threadIdx.x == 0) stage_count[tile] = 0;
    return;
  }
  EmitSel sel;
  sel.thr_f = float_of_key(kClassify ? st.hi : st.thr);
  sel.lo_f = float_of_key(st.lo);
  sel.ties_kept = st.ties_kept;
  sel.all_ties = st.all_ties_kept != 0u || keep_ties != 0;
  sel.have_cut = st.have_cut != 0u;
  sel.tie_cut = st.tie_cut;
  sel.first_row = per_layer ? (uint32_t)h * (uint32_t)Lq : 0u;
  Collector col;
  col.stage = stage_all[kClassify ? warp : 0];
  col.stage_n = &stage_n_all[warp];
  col.out = cand + (size_t)(per_layer ? 0 : h) * cand_cap;
  col.n_cand = &st.n_cand;
  col.cap = cand_cap;
  if (lane == 0) stage_n_all[warp] = 0u;
  __syncwarp();
  uint32_t above = 0u;
  const bool below = !causal || kt * kTile + kTile - 1 <= own_lo;  // every column in every row's domain
  const bool has_diag = diag && own_lo <= kt * kTile + kTile - 1 && own_hi >= kt * kTile;
  const bool interior = (qt + 1) * kTile <= Lq && (kt + 1) * kTile <= Lk && (Lk & 3) == 0 && below && !has_diag;
  int count = interior ? emit_tile_rows<true, kClassify>(acc, Lq, Lk, n_kt, h, qt, kt, tile, causal, diag, sel,
                                                         tie_prefix, mask, stage_bitmap, col, above)
                       : emit_tile_rows<false, kClassify>(acc, Lq, Lk, n_kt, h, qt, kt, tile, causal, diag, sel,
                                                          tie_prefix, mask, stage_bitmap, col, above);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) count += __shfl_xor_sync(0xffffffffu, count, o);
  if (kClassify) {
    above = __reduce_add_sync(0xffffffffu, above);
    if (lane == 0 && above) atomicAdd(&st.above_hi, (unsigned long long)above);
  }
  if (lane == 0) warp_count[warp] = count;
  __syncthreads();
  if (threadIdx.x == 0) {
    const int total = warp_count[0] + warp_count[1] + warp_count[2] + warp_count[3];
    if (stage_count) stage_count[tile] = total;
    if (!kClassify && (per_layer || keep_ties) && nnz && total)
      atomicAdd(reinterpret_cast<unsigned long long *>(nnz + h), (unsigned long long)total);
  }
}

// The collected entries of a selection that the classifying pass left out and that are kept after all:
// above the threshold, or equal to it and within the ties that are kept.  grid = (CTAs, selections).
__global__ void __launch_bounds__(kThreads) patch_kernel(const SelectState *__restrict__ state,
                                                         const uint2 *__restrict__ cand, uint32_t cand_cap, int Lq,
                                                         int Lk, int n_qt, int n_kt, uint8_t *__restrict__ mask,
                                                         uint32_t *__restrict__ stage_bitmap,
                                                         int32_t *__restrict__ stage_count) {
  const int h = blockIdx.y;
  const SelectState st = state[h];
  if (!st.emitted) return;
  const uint2 *mine = cand + (size_t)h * cand_cap;
  const int lane = threadIdx.x & 31;
  const uint32_t n = st.n_cand;
  // (warp-uniform trip count; entries that follow one another in the buffer were collected by one warp
  // from one stretch of a tile, so lanes that hit the same bitmap word or tile combine their updates)
  for (uint32_t base = blockIdx.x * kThreads; base < n; base += gridDim.x * kThreads) {
    const uint32_t idx = base + threadIdx.x;
    uint2 c = make_uint2(0u, 0u);
    if (idx < n) c = mine[idx];
    const bool keep = idx < n && (c.x > st.thr || (c.x == st.thr && (st.all_ties_kept != 0u || c.y <= st.tie_cut)));
    const uint32_t i = c.y / (uint32_t)Lk, j = c.y - i * (uint32_t)Lk;
    if (keep && mask) mask[((size_t)h * Lq + i) * Lk + j] = 1;
    if (stage_bitmap) {
      const uint32_t tile = (uint32_t)((h * n_qt + (int)(i >> 7)) * n_kt + (int)(j >> 7));
      const uint32_t word = tile * (uint32_t)kBitmapWords + 4u * (i & 127u) + ((j & 127u) >> 5);
      const unsigned voters = __ballot_sync(0xffffffffu, keep);
      if (keep) {
        const unsigned same_word = __match_any_sync(voters, word);
        const uint32_t all_bits = __reduce_or_sync(same_word, 1u << (j & 31u));
        if (lane == __ffs((int)same_word) - 1) atomicOr(stage_bitmap + word, all_bits);
        const unsigned same_tile = __match_any_sync(voters, tile);
        if (lane == __ffs((int)same_tile) - 1) atomicAdd(stage_count + tile, __popc(same_tile));
      }
    }
  }
}

Scratch carve(void *scratch, int H, int Lq, int Lk) {
  char *p = static_cast<char *>(scratch);
  Scratch s;
  s.hist = reinterpret_cast<uint32_t *>(p);
  p += align256((size_t)H * kBins * sizeof(uint32_t));
  s.state = reinterpret_cast<SelectState *>(p);
  p += align256((size_t)H * sizeof(SelectState));
  s.tie_count = reinterpret_cast<uint32_t *>(p);
  p += align256((size_t)H * Lq * ceil_div(Lk, kTile) * sizeof(uint32_t));
  s.tie_list = reinterpret_cast<uint32_t *>(p);
  p += align256((size_t)H * kMaxCutTies * sizeof(uint32_t));
  s.cand = reinterpret_cast<uint2 *>(p);
  return s;
}

}  // namespace

size_t select_scratch_bytes(int H, int Lq, int Lk) {
  // the candidate buffer is sized for the larger of the causal and the full domain, and for one
  // selection over all heads (never smaller than H selections of one head each)
  return align256((size_t)H * kBins * sizeof(uint32_t)) + align256((size_t)H * sizeof(SelectState)) +
         align256((size_t)H * Lq * ceil_div(Lk, kTile) * sizeof(uint32_t)) +
         align256((size_t)H * kMaxCutTies * sizeof(uint32_t)) +
         align256((size_t)cand_capacity((long long)H * Lq * Lk) * sizeof(uint2));
}

cudaError_t launch_build_mask(const BuildMaskArgs &a, cudaStream_t s) {
  const int n_qt = ceil_div(a.Lq, kTile), n_kt = ceil_div(a.Lk, kTile);
  const int diag = (a.keep_diag && (a.Lq == a.Lk || a.causal)) ? 1 : 0;
  Scratch sc = carve(a.scratch, a.H, a.Lq, a.Lk);
  // the selections: one per head over Lq rows, or one over the H*Lq rows of the layer
  const int n_sel = a.per_layer ? 1 : a.H;
  const int rows = a.per_layer ? a.H * a.Lq : a.Lq;
  const int period = a.Lq;
  cudaError_t e;
  // per head nnz = k; per layer, or with all ties kept, the emit pass counts it
  const bool count_nnz = a.per_layer || a.keep_ties;
  {
    // very small selections: one kernel instead of the passes below (measured: one CTA per selection
    // beats the ten launches of the passes up to about 2^15 entries per selection: 0.085 -> 0.065 ms on
    // B32 H12 L128; at 2^17 and more it loses, the passes spread a selection over many CTAs)
    if ((long long)rows * a.Lk <= kSelectSmallEntries) {
      select_small_kernel<<<n_sel, 1024, 0, s>>>(a.acc, rows, a.Lk, period, a.causal, diag,
                                                 (unsigned long long)a.k_rest, sc.state, a.H,
                                                 count_nnz ? 0ll : (long long)a.k, a.nnz);
      count_launches(1);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
      emit_kernel<false><<<a.H * n_qt * n_kt, 128, 0, s>>>(a.acc, a.Lq, a.Lk, n_qt, n_kt, a.causal, diag,
                                                           a.per_layer, a.keep_ties, sc.state, sc.tie_count, a.mask,
                                                           a.stage_bitmap, a.stage_count, a.nnz, nullptr, 0u);
      count_launches(1);
      return cudaGetLastError();
    }
  }
  init_state_kernel<<<ceil_div(max(n_sel * kBins, a.H), 256), 256, 0, s>>>(
      sc.state, sc.hist, n_sel, (unsigned long long)a.k_rest, a.H, count_nnz ? 0ll : (long long)a.k, a.nnz);
  count_launches(1);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  // enough CTAs per selection to fill the GPU, at most one warp-row each
  int row_blocks = ceil_div(rows, kWarps);
  const int want = ceil_div(148 * 8, n_sel);
  if (row_blocks > want) row_blocks = want;
  dim3 grid(row_blocks, n_sel);
  if (a.k_rest > 0) {
    // large selections: the one-pass shortcut first (those it resolves skip the three passes below)
    const long long n_valid = domain_size(a.Lq, a.Lk, a.causal);
    const long long n_rest = (n_valid - (diag ? a.Lq : 0)) * (a.per_layer ? a.H : 1);
    const long long cap = cand_capacity(n_rest);
    if (cap > 0) {
      const size_t smem = (kSamples + kBins) * sizeof(uint32_t);
      e = cudaFuncSetAttribute(sample_pivots_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      sample_pivots_kernel<<<dim3(n_sel, 2), 1024, smem, s>>>(a.acc, rows, a.Lk, period, a.causal, diag,
                                                     (unsigned long long)a.k_rest, (unsigned long long)n_rest, sc.state);
      // Exact per-head selections: the one pass over the accumulator also writes what is certain of the
      // mask and the tile bitmaps (the patch pass below adds the collected entries that are kept), so
      // the emit pass at the end has nothing to read for the selections the shortcut resolves.  Other
      // selections count what they keep in the emit pass, which therefore has to see every entry.
      const bool classify = !a.per_layer && !a.keep_ties;
      if (classify) {
        emit_kernel<true><<<a.H * n_qt * n_kt, 128, 0, s>>>(a.acc, a.Lq, a.Lk, n_qt, n_kt, a.causal, diag, 0, 0,
                                                            sc.state, sc.tie_count, a.mask, a.stage_bitmap,
                                                            a.stage_count, a.nnz, sc.cand, (uint32_t)cap);
      } else {
        // one wave of CTAs (five fit an SM), so that no SM idles while a second, partial wave runs
        int collect_blocks = ceil_div(rows, kWarps);
        if (collect_blocks > 148 * 5 / n_sel) collect_blocks = max(148 * 5 / n_sel, 1);
        collect_kernel<<<dim3(collect_blocks, n_sel), kThreads, 0, s>>>(a.acc, rows, a.Lk, period, a.causal, diag,
                                                                       sc.state, sc.cand, (uint32_t)cap);
      }
      // the threshold among the collected keys: the same three digits, on offsets from the lower pivot
      const dim3 cand_grid(ceil_div(148 * 8, n_sel), n_sel);
      for (int pass = 0; pass < kPasses; ++pass) {
        cand_histogram_kernel<<<cand_grid, kThreads, 0, s>>>(sc.state, sc.cand, (uint32_t)cap,
                                                             (unsigned long long)a.k_rest, pass, sc.hist);
      }
      cand_finish_kernel<<<cand_grid, kThreads, 0, s>>>(sc.state, sc.cand, (uint32_t)cap, sc.tie_list,
                                                        classify ? 1 : 0);
      count_launches(3 + kPasses);
      if (classify) {
        patch_kernel<<<cand_grid, kThreads, 0, s>>>(sc.state, sc.cand, (uint32_t)cap, a.Lq, a.Lk, n_qt, n_kt, a.mask,
                                                    a.stage_bitmap, a.stage_count);
        count_launches(1);
      }
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    for (int pass = 0; pass < kPasses; ++pass) {
      digit_histogram_kernel<<<grid, kThreads, 0, s>>>(a.acc, rows, a.Lk, period, a.causal, diag, pass, sc.state,
                                                       sc.hist);
      count_launches(1);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    if (!a.keep_ties) {  // the ties' ranks are needed only where some of them are pruned
      // both return at once for selections whose ties with the threshold are all kept
      tie_count_kernel<<<grid, kThreads, 0, s>>>(a.acc, rows, a.Lk, period, n_kt, a.causal, diag, sc.state,
                                                 sc.tie_count);
      count_launches(1);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
  }
  emit_kernel<false><<<a.H * n_qt * n_kt, 128, 0, s>>>(a.acc, a.Lq, a.Lk, n_qt, n_kt, a.causal, diag, a.per_layer,
                                                       a.keep_ties, sc.state, sc.tie_count, a.mask, a.stage_bitmap,
                                                       a.stage_count, a.nnz, nullptr, 0u);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace ap
