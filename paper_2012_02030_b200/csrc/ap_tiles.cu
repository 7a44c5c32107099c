// Tile lists: element mask -> per-tile bitmaps -> compacted CSR of non-empty tiles.
//
// The tile list is an encoding of the pruning mask of Eq. 2 (the paper itself
// only states the element mask).  Bitmaps are first written for every tile of
// the grid into a staging area ordered (h, qt, kt); a single-CTA scan then
// assigns list positions to the non-empty ones in that order, and a copy
// kernel moves their bitmaps to the compacted list.
#include "ap_common.cuh"

namespace ap {

size_t stage_bytes(int H, int Lq, int Lk) {
  size_t n = (size_t)H * ceil_div(Lq, kTile) * ceil_div(Lk, kTile);
  // bitmaps, popcounts, list positions
  return n * (kBitmapWords * sizeof(uint32_t)) + 2 * ((n * sizeof(int32_t) + 255) / 256 * 256);
}

namespace {

// One CTA per tile; warp w takes rows w, w+4, ...; a ballot over 32 consecutive
// mask bytes yields one bitmap word.
__global__ void __launch_bounds__(128) stage_from_mask_kernel(const uint8_t *__restrict__ mask, int Lq,
                                                              int Lk, int n_qt, int n_kt,
                                                              uint32_t *__restrict__ stage_bitmap,
                                                              int32_t *__restrict__ stage_count) {
  const int tile = blockIdx.x;
  const int kt = tile % n_kt;
  const int qt = (tile / n_kt) % n_qt;
  const int h = tile / (n_kt * n_qt);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __shared__ int warp_count[4];
  int count = 0;
  uint4 *out = reinterpret_cast<uint4 *>(stage_bitmap + (size_t)tile * kBitmapWords);
  for (int r = warp; r < kTile; r += 4) {
    const int i = qt * kTile + r;
    uint32_t w[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int j = kt * kTile + 32 * c + lane;
      bool keep = false;
      if (i < Lq && j < Lk) keep = mask[((size_t)h * Lq + i) * Lk + j] != 0;
      w[c] = __ballot_sync(0xffffffffu, keep);
      count += __popc(w[c]);
    }
    if (lane == 0) out[r] = make_uint4(w[0], w[1], w[2], w[3]);
  }
  // every lane of a warp holds the same count
  if (lane == 0) warp_count[warp] = count;
  __syncthreads();
  if (threadIdx.x == 0)
    stage_count[tile] = warp_count[0] + warp_count[1] + warp_count[2] + warp_count[3];
}

// Single CTA: exclusive scan of "tile is non-empty" over the (h, qt, kt) order.  A thread takes
// sixteen consecutive tiles at a time (all loads in flight), the CTA scans the threads' sums.
__global__ void __launch_bounds__(1024) scan_tiles_kernel(const int32_t *__restrict__ stage_count,
                                                          int32_t *__restrict__ stage_pos, int n_tiles,
                                                          int n_kt, int cap, int32_t *__restrict__ row_ptr,
                                                          unsigned *err) {
  constexpr int kPer = 16;
  __shared__ int warp_sums[32];
  __shared__ int carry_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) {
    carry_s = 0;
    row_ptr[0] = 0;
  }
  __syncthreads();
  for (int base = 0; base < n_tiles; base += 1024 * kPer) {
    const int idx0 = base + (int)threadIdx.x * kPer;
    int cnt[kPer];
    const bool vec = idx0 + kPer <= n_tiles && (reinterpret_cast<uintptr_t>(stage_count) & 15u) == 0 &&
                     (reinterpret_cast<uintptr_t>(stage_pos) & 15u) == 0;
    if (vec) {  // four 16-byte loads instead of sixteen strided 4-byte ones
#pragma unroll
      for (int q = 0; q < kPer / 4; ++q) {
        const int4 c4 = reinterpret_cast<const int4 *>(stage_count + idx0)[q];
        cnt[4 * q] = c4.x, cnt[4 * q + 1] = c4.y, cnt[4 * q + 2] = c4.z, cnt[4 * q + 3] = c4.w;
      }
    } else {
#pragma unroll
      for (int e = 0; e < kPer; ++e) cnt[e] = idx0 + e < n_tiles ? stage_count[idx0 + e] : 0;
    }
    int mine = 0;
#pragma unroll
    for (int e = 0; e < kPer; ++e) mine += cnt[e] > 0 ? 1 : 0;
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int v = warp_sums[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += u;
      }
      warp_sums[lane] = v;  // inclusive over warps
    }
    __syncthreads();
    const int carry = carry_s;
    int before = carry + (warp ? warp_sums[warp - 1] : 0) + incl - mine;
    int row = idx0 / n_kt, kt = idx0 - row * n_kt;  // list row and key tile of the tile, stepped below
    int pos[kPer];
#pragma unroll
    for (int e = 0; e < kPer; ++e) {
      const int idx = idx0 + e;
      const int flag = cnt[e] > 0 ? 1 : 0;
      pos[e] = flag ? before : -1;
      if (idx < n_tiles) {
        if (!vec) stage_pos[idx] = pos[e];
        if (kt == n_kt - 1) row_ptr[row + 1] = min(before + flag, cap);
      }
      before += flag;
      if (++kt == n_kt) {
        kt = 0;
        ++row;
      }
    }
    if (vec) {
#pragma unroll
      for (int q = 0; q < kPer / 4; ++q)
        reinterpret_cast<int4 *>(stage_pos + idx0)[q] = make_int4(pos[4 * q], pos[4 * q + 1], pos[4 * q + 2], pos[4 * q + 3]);
    }
    __syncthreads();
    if (threadIdx.x == 1023) carry_s = carry + warp_sums[31];
    __syncthreads();
  }
  if (threadIdx.x == 0 && carry_s > cap) atomicOr(err, kDevErrCapacity);
}

// Called by all 128 threads of a CTA, thread r holding bitmap row r of one tile: bit g of the
// result says whether any row keeps an entry among columns [16g, 16g+16).
__device__ __forceinline__ uint32_t group_mask_of_tile(uint4 row) {
  __shared__ uint32_t warp_or[4][4];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t w0 = __reduce_or_sync(0xffffffffu, row.x), w1 = __reduce_or_sync(0xffffffffu, row.y),
                 w2 = __reduce_or_sync(0xffffffffu, row.z), w3 = __reduce_or_sync(0xffffffffu, row.w);
  if (lane == 0) {
    warp_or[warp][0] = w0;
    warp_or[warp][1] = w1;
    warp_or[warp][2] = w2;
    warp_or[warp][3] = w3;
  }
  __syncthreads();
  uint32_t gm = 0u;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const uint32_t w = warp_or[0][c] | warp_or[1][c] | warp_or[2][c] | warp_or[3][c];
    gm |= ((w & 0xffffu) ? 1u : 0u) << (2 * c);
    gm |= ((w >> 16) ? 1u : 0u) << (2 * c + 1);
  }
  return gm;
}

// One CTA per grid tile: non-empty tiles copy their bitmap to their list slot.
__global__ void __launch_bounds__(128) gather_tiles_kernel(const uint32_t *__restrict__ stage_bitmap,
                                                           const int32_t *__restrict__ stage_count,
                                                           const int32_t *__restrict__ stage_pos, int n_kt,
                                                           int cap, int32_t *__restrict__ col_idx,
                                                           uint8_t *__restrict__ flags,
                                                           uint32_t *__restrict__ bitmap,
                                                           uint8_t *__restrict__ groups) {
  const int tile = blockIdx.x;
  const int pos = stage_pos[tile];
  if (pos < 0 || pos >= cap) return;
  const uint4 *src = reinterpret_cast<const uint4 *>(stage_bitmap + (size_t)tile * kBitmapWords);
  uint4 *dst = reinterpret_cast<uint4 *>(bitmap + (size_t)pos * kBitmapWords);
  const uint4 row = src[threadIdx.x];
  dst[threadIdx.x] = row;
  const uint32_t gm = group_mask_of_tile(row);
  if (threadIdx.x == 0) {
    col_idx[pos] = tile % n_kt;
    flags[pos] = stage_count[tile] == kTile * kTile ? 1 : 0;
    groups[pos] = (uint8_t)gm;
  }
}

// One CTA per grid tile, thread r = tile row r: writes the list of the full
// (optionally causal) domain in closed form, rounds included: in such a list only the last tile of
// a list row can have fewer than eight non-empty groups (the others lie inside the domain of the
// tile's last row), and its groups are the first ones of the tile, so round k of a list row is its
// k-th tile - same key rows, same bitmap.
__global__ void __launch_bounds__(128) dense_tiles_kernel(int H, int Lq, int Lk, int n_qt, int n_kt, int causal,
                                                          int cap, int32_t *__restrict__ row_ptr,
                                                          int32_t *__restrict__ col_idx,
                                                          uint8_t *__restrict__ flags,
                                                          uint32_t *__restrict__ bitmap,
                                                          uint8_t *__restrict__ groups,
                                                          int32_t *__restrict__ round_ptr,
                                                          int32_t *__restrict__ round_rows,
                                                          uint8_t *__restrict__ round_info,
                                                          uint32_t *__restrict__ round_bitmap, unsigned *err) {
  const int tile = blockIdx.x;
  const int kt = tile % n_kt;
  const int qt = (tile / n_kt) % n_qt;
  const int h = tile / (n_kt * n_qt);
  const int per_head = (int)dense_row_start(n_qt, n_kt, Lq, Lk, causal);
  const int row_start = h * per_head + (int)dense_row_start(qt, n_kt, Lq, Lk, causal);
  if (threadIdx.x == 0 && kt == 0) {
    row_ptr[h * n_qt + qt] = round_ptr[h * n_qt + qt] = min(row_start, cap);
    if (h == H - 1 && qt == n_qt - 1) {
      row_ptr[H * n_qt] = round_ptr[H * n_qt] = min(H * per_head, cap);
      if (H * per_head > cap) atomicOr(err, kDevErrCapacity);
    }
  }
  if (kt >= dense_row_tiles(qt, n_kt, Lq, Lk, causal)) return;
  const int pos = row_start + kt;
  if (pos >= cap) return;
  const int r = threadIdx.x;
  const int i = qt * kTile + r;
  uint32_t w[4] = {0u, 0u, 0u, 0u};
  if (i < Lq) {
    int jend = causal ? min(Lk, i + 1 + (Lk - Lq)) : Lk;  // first column not kept
    int n = jend - kt * kTile;                // kept columns of this tile row
    n = max(0, min(kTile, n));
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      int m = n - 32 * c;
      w[c] = m >= 32 ? 0xffffffffu : (m > 0 ? ((1u << m) - 1u) : 0u);
    }
  }
  reinterpret_cast<uint4 *>(bitmap + (size_t)pos * kBitmapWords)[r] = make_uint4(w[0], w[1], w[2], w[3]);
  reinterpret_cast<uint4 *>(round_bitmap + (size_t)pos * kBitmapWords)[r] = make_uint4(w[0], w[1], w[2], w[3]);
  const int full = __syncthreads_and(w[0] == 0xffffffffu && w[1] == 0xffffffffu &&
                                     w[2] == 0xffffffffu && w[3] == 0xffffffffu);
  const uint32_t gm = group_mask_of_tile(make_uint4(w[0], w[1], w[2], w[3]));
  const int ng = __popc(gm);  // the tile's first ng groups
  if (r < 8) round_rows[(size_t)pos * 8 + r] = r < ng ? kt * kTile + 16 * r : -1;
  if (r == 0) {
    col_idx[pos] = kt;
    flags[pos] = full ? 1 : 0;
    groups[pos] = (uint8_t)gm;
    round_info[pos] = (uint8_t)(ng | ((full && ng == 8) ? 0x80 : 0));
  }
}

// ---- rounds: the forward pass's schedule (slots = non-empty 16-column groups in list order, eight per round)

__device__ __forceinline__ uint32_t group_mask_of(const uint8_t *flags, const uint8_t *groups, int t) {
  return (flags[t] & 1) ? 0xffu : (uint32_t)groups[t];
}

// One warp per list row: round_ptr[row + 1] = number of rounds of the row (scanned afterwards).
__global__ void __launch_bounds__(128) count_rounds_kernel(const int32_t *__restrict__ row_ptr,
                                                           const uint8_t *__restrict__ flags,
                                                           const uint8_t *__restrict__ groups, int n_rows,
                                                           int32_t *__restrict__ round_ptr) {
  const int row = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= n_rows) return;
  int slots = 0;
  for (int t = row_ptr[row] + lane; t < row_ptr[row + 1]; t += 32) slots += __popc(group_mask_of(flags, groups, t));
  slots = __reduce_add_sync(0xffffffffu, slots);
  if (lane == 0) {
    round_ptr[row + 1] = (slots + 7) / 8;
    if (row == 0) round_ptr[0] = 0;
  }
}

// Single CTA: inclusive scan in place over round_ptr[1 .. n_rows].
__global__ void __launch_bounds__(1024) scan_rounds_kernel(int32_t *__restrict__ round_ptr, int n_rows) {
  __shared__ int warp_sums[32];
  __shared__ int carry_s;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base < n_rows; base += 1024) {
    const int idx = base + threadIdx.x;
    const int x = idx < n_rows ? round_ptr[idx + 1] : 0;
    int incl = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int v = warp_sums[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += u;
      }
      warp_sums[lane] = v;
    }
    __syncthreads();
    const int carry = carry_s;
    if (idx < n_rows) round_ptr[idx + 1] = carry + (warp ? warp_sums[warp - 1] : 0) + incl;
    __syncthreads();
    if (threadIdx.x == 1023) carry_s = carry + warp_sums[31];
    __syncthreads();
  }
}

// One CTA per list row, thread r = bitmap row r.  The row's tiles are taken 128 at a time: their
// slots are listed in shared memory, and every complete group of eight slots (plus the remainder
// at the end of the list row) is written out as a round.
__global__ void __launch_bounds__(128) fill_rounds_kernel(const int32_t *__restrict__ row_ptr,
                                                          const int32_t *__restrict__ col_idx,
                                                          const uint8_t *__restrict__ flags,
                                                          const uint8_t *__restrict__ groups,
                                                          const uint32_t *__restrict__ bitmap,
                                                          const int32_t *__restrict__ round_ptr, int cap,
                                                          int32_t *__restrict__ round_rows,
                                                          uint8_t *__restrict__ round_info,
                                                          uint32_t *__restrict__ round_bitmap) {
  constexpr int kSeg = 128;                      // tiles per pass
  __shared__ uint32_t slot_src[kSeg * 8 + 8];    // tile index << 4 | group << 1 | tile fully kept
  __shared__ int32_t slot_row[kSeg * 8 + 8];     // first key row of the slot
  __shared__ int warp_sums[4];
  const int row = blockIdx.x, r = threadIdx.x, lane = r & 31, warp = r >> 5;
  const int t_begin = row_ptr[row], t_end = row_ptr[row + 1];
  int rho = round_ptr[row];
  int pending = 0;  // slots carried over from the previous pass (fewer than eight)
  for (int base = t_begin; base < t_end; base += kSeg) {
    const int t = base + r;
    uint32_t gm = 0u;
    int kt = 0;
    bool full = false;
    if (t < t_end) {
      full = flags[t] & 1;
      gm = full ? 0xffu : (uint32_t)groups[t];
      kt = col_idx[t];
    }
    const int cnt = __popc(gm);
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    int before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      if (w < warp) before += warp_sums[w];
      total += warp_sums[w];
    }
    int s = pending + before + incl - cnt;
    while (gm) {
      const int g = __ffs((int)gm) - 1;
      gm &= gm - 1u;
      slot_src[s] = ((uint32_t)t << 4) | ((uint32_t)g << 1) | (full ? 1u : 0u);
      slot_row[s] = kt * kTile + 16 * g;
      ++s;
    }
    __syncthreads();
    const int avail = pending + total;
    const bool last_pass = base + kSeg >= t_end;
    const int n_emit = last_pass ? (avail + 7) / 8 : avail / 8;
    for (int k = 0; k < n_emit; ++k) {
      const int ng = min(8, avail - 8 * k);
      uint32_t w[4] = {0u, 0u, 0u, 0u};
      bool all_full = true;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        if (q >= ng) continue;
        const uint32_t src = slot_src[8 * k + q];
        uint32_t field = 0xffffu;
        if (!(src & 1u)) {
          const uint32_t g = (src >> 1) & 7u;
          field = (bitmap[(size_t)(src >> 4) * kBitmapWords + r * 4 + (g >> 1)] >> (16u * (g & 1u))) & 0xffffu;
          all_full = false;
        }
        w[q >> 1] |= field << (16 * (q & 1));
      }
      const int out = rho + k;
      if (out < cap) {
        reinterpret_cast<uint4 *>(round_bitmap + (size_t)out * kBitmapWords)[r] = make_uint4(w[0], w[1], w[2], w[3]);
        if (r < 8) round_rows[(size_t)out * 8 + r] = r < ng ? slot_row[8 * k + r] : -1;
        if (r == 0) round_info[out] = (uint8_t)(ng | ((all_full && ng == 8) ? 0x80 : 0));
      }
    }
    rho += n_emit;
    __syncthreads();
    // fewer than eight slots are left over; they move to the front (no overlap: they start at or
    // beyond index 8 unless nothing was written out, in which case they are in place already)
    const int left = avail - 8 * n_emit;
    if (!last_pass && n_emit > 0 && r < left) {
      const uint32_t a = slot_src[8 * n_emit + r];
      const int32_t b = slot_row[8 * n_emit + r];
      slot_src[r] = a;
      slot_row[r] = b;
    }
    pending = last_pass ? 0 : left;
    __syncthreads();
  }
}

// ---- gathered rounds: a list row's active key columns, 128 per round ----------------------------

// The 128-bit column summary of one stored tile (bit c: some row keeps column c), by one warp:
// lane l ORs rows l, l + 32, l + 64, l + 96.  Every lane returns the four words.
__device__ __forceinline__ uint4 column_summary(const uint32_t *__restrict__ bitmap, int t, int lane) {
  uint4 m = make_uint4(0u, 0u, 0u, 0u);
  const uint4 *rows = reinterpret_cast<const uint4 *>(bitmap + (size_t)t * kBitmapWords);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const uint4 w = rows[lane + 32 * k];
    m.x |= w.x, m.y |= w.y, m.z |= w.z, m.w |= w.w;
  }
  m.x = __reduce_or_sync(0xffffffffu, m.x);
  m.y = __reduce_or_sync(0xffffffffu, m.y);
  m.z = __reduce_or_sync(0xffffffffu, m.z);
  m.w = __reduce_or_sync(0xffffffffu, m.w);
  return m;
}

// How many of a summary word's two 16-column groups have every column active.
__device__ __forceinline__ int whole_groups(uint32_t m) {
  return ((m & 0xffffu) == 0xffffu ? 1 : 0) + ((m >> 16) == 0xffffu ? 1 : 0);
}

// One warp per list row: ground_ptr[row + 1] = ceil(active columns / 128) (scanned afterwards), or 0
// where gathered rounds would not pay.  Measured on the forward: a gathered round takes 1.1 to 1.3
// times a round of the same width (the copy warp has more to do), a slot whose 16 key rows are
// fetched one by one costs a quarter of a round and more on top, and the kernel that can follow
// gathered rounds is some 10 % slower on every round; so a list row of r rounds gets its g gathered
// rounds, s of whose slots are of that kind, only where they halve the work: r > 2 g + s / 2.
__global__ void __launch_bounds__(128) count_grounds_kernel(const int32_t *__restrict__ row_ptr,
                                                            const uint32_t *__restrict__ bitmap,
                                                            const int32_t *__restrict__ round_ptr, int n_rows,
                                                            int always, int32_t *__restrict__ ground_ptr) {
  const int row = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= n_rows) return;
  int cols = 0, whole = 0;
  for (int t = row_ptr[row]; t < row_ptr[row + 1]; ++t) {
    const uint4 m = column_summary(bitmap, t, lane);
    cols += __popc(m.x) + __popc(m.y) + __popc(m.z) + __popc(m.w);
    whole += whole_groups(m.x) + whole_groups(m.y) + whole_groups(m.z) + whole_groups(m.w);
  }
  if (lane == 0) {
    const int r = round_ptr[row + 1] - round_ptr[row];
    const int g = (cols + kTile - 1) / kTile;
    const int s = (cols - 16 * whole + 15) / 16;
    ground_ptr[row + 1] = (always || 2 * r > 4 * g + s) ? g : 0;
    if (row == 0) ground_ptr[0] = 0;
  }
}

// One CTA per list row, thread r = bitmap row r (and column p of the round being written).  The
// row's tiles are taken 32 at a time, twice: first the 16-column groups in which every column is
// active are listed in shared memory (a slot of such a group is 16 key rows that follow one another
// from a multiple of 16 on, which the forward fetches as one box), then the active columns of the
// other groups, each time in ascending key order; every complete set of 128 listed columns (plus
// the remainder at the end) is written out as a gathered round.
__global__ void __launch_bounds__(128) fill_grounds_kernel(const int32_t *__restrict__ row_ptr,
                                                           const int32_t *__restrict__ col_idx,
                                                           const uint32_t *__restrict__ bitmap,
                                                           const int32_t *__restrict__ ground_ptr, int cap,
                                                           int32_t *__restrict__ ground_keys,
                                                           uint8_t *__restrict__ ground_info,
                                                           uint32_t *__restrict__ ground_bitmap) {
  constexpr int kSeg = 32;                         // tiles per pass
  __shared__ uint32_t summary[kSeg * 4];           // column summaries of the pass's tiles
  __shared__ int32_t tile_kt[kSeg];
  __shared__ int32_t col_key[kSeg * kTile + kTile];  // key index of each listed column
  __shared__ uint32_t col_src[kSeg * kTile + kTile]; // tile index << 7 | column inside the tile
  __shared__ int warp_sums[4];
  const int row = blockIdx.x, r = threadIdx.x, lane = r & 31, warp = r >> 5;
  const int t_begin = row_ptr[row], t_end = row_ptr[row + 1];
  int rho = ground_ptr[row];
  if (ground_ptr[row + 1] == rho) return;  // no gathered rounds for this list row
  int pending = 0;  // columns carried over from the previous pass (fewer than 128)
  for (int phase = 0; phase < 2; ++phase)
  for (int base = t_begin; base < t_end; base += kSeg) {
    const int n_here = min(kSeg, t_end - base);
    for (int k = warp; k < kSeg; k += 4) {  // warp w summarises tiles w, w + 4, ...
      uint4 m = make_uint4(0u, 0u, 0u, 0u);
      if (k < n_here) m = column_summary(bitmap, base + k, lane);
      if (lane == 0) {
        summary[4 * k] = m.x, summary[4 * k + 1] = m.y, summary[4 * k + 2] = m.z, summary[4 * k + 3] = m.w;
        tile_kt[k] = k < n_here ? col_idx[base + k] : 0;
      }
    }
    __syncthreads();
    // thread r owns summary word r (tile r / 4, columns 32 (r % 4) ...), of which this phase takes the
    // halves that are all ones, or the others: exclusive prefix of the popcounts
    uint32_t m = summary[r];
    const uint32_t whole = ((m & 0xffffu) == 0xffffu ? 0xffffu : 0u) | ((m >> 16) == 0xffffu ? 0xffff0000u : 0u);
    m = phase == 0 ? whole : m & ~whole;
    const int cnt = __popc(m);
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    int before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      if (w < warp) before += warp_sums[w];
      total += warp_sums[w];
    }
    int s = pending + before + incl - cnt;
    const int tile = base + (r >> 2), kt = tile_kt[r >> 2];
    while (m) {
      const int c = 32 * (r & 3) + __ffs((int)m) - 1;
      m &= m - 1u;
      col_key[s] = kt * kTile + c;
      col_src[s] = ((uint32_t)tile << 7) | (uint32_t)c;
      ++s;
    }
    __syncthreads();
    const int avail = pending + total;
    const bool last_pass = phase == 1 && base + kSeg >= t_end;
    const int n_emit = last_pass ? (avail + kTile - 1) / kTile : avail / kTile;
    for (int k = 0; k < n_emit; ++k) {
      const int nc = min(kTile, avail - kTile * k);  // columns of this round
      // row r of the round's bitmap: bit p = bit (column of p) of row r of (tile of p)
      uint32_t w[4] = {0u, 0u, 0u, 0u};
      uint32_t cur_word_id = 0xffffffffu, cur_word = 0u;
      for (int p = 0; p < nc; ++p) {
        const uint32_t src = col_src[kTile * k + p];
        const uint32_t word_id = ((src >> 7) << 2) | ((src & 127u) >> 5);  // (tile, word of the row)
        if (word_id != cur_word_id) {
          cur_word_id = word_id;
          cur_word = bitmap[(size_t)(src >> 7) * kBitmapWords + r * 4 + ((src & 127u) >> 5)];
        }
        w[p >> 5] |= ((cur_word >> (src & 31u)) & 1u) << (p & 31);
      }
      const bool mine_full = (w[0] & w[1] & w[2] & w[3]) == 0xffffffffu;
      const int all_full = __syncthreads_and(mine_full ? 1 : 0);
      const int out = rho + k;
      if (out < cap) {
        reinterpret_cast<uint4 *>(ground_bitmap + (size_t)out * kBitmapWords)[r] = make_uint4(w[0], w[1], w[2], w[3]);
        ground_keys[(size_t)out * kTile + r] = col_key[kTile * k + min(r, nc - 1)];
        if (r == 0) ground_info[out] = (uint8_t)(((nc + 15) / 16) | ((all_full && nc == kTile) ? 0x80 : 0));
      }
    }
    rho += n_emit;
    __syncthreads();
    // fewer than 128 columns are left over; they move to the front (no overlap: they start at or
    // beyond index 128 unless nothing was written out, in which case they are in place already)
    const int left = avail - kTile * n_emit;
    int32_t a = 0;
    uint32_t b = 0u;
    const bool move = !last_pass && n_emit > 0 && r < left;
    if (move) a = col_key[kTile * n_emit + r], b = col_src[kTile * n_emit + r];
    __syncthreads();
    if (move) col_key[r] = a, col_src[r] = b;
    pending = last_pass ? 0 : left;
    __syncthreads();
  }
}

// ---- units of work of the forward: balanced pairs of a head's query tiles ------------------------

// One CTA per head.  The head's list rows are ranked by their number of rounds (more first, ties by
// lower index); unit j pairs rank j with rank n_qt - 1 - j.  Heads of more than kMaxPairTiles query
// tiles keep the plain pairing (n_qt - 1 - j, j).
constexpr int kMaxPairTiles = 2048;
__global__ void __launch_bounds__(256) pair_units_kernel(const int32_t *__restrict__ round_ptr, int n_qt,
                                                         int32_t *__restrict__ unit_qt) {
  __shared__ int32_t rounds[kMaxPairTiles];
  __shared__ int32_t sorted[kMaxPairTiles];
  const int h = blockIdx.x, n_half = (n_qt + 1) / 2;
  int32_t *out = unit_qt + (size_t)h * n_half * 2;
  if (n_qt > kMaxPairTiles) {
    for (int j = threadIdx.x; j < n_half; j += blockDim.x) {
      out[2 * j] = n_qt - 1 - j;
      out[2 * j + 1] = j != n_qt - 1 - j ? j : -1;
    }
    return;
  }
  for (int q = threadIdx.x; q < n_qt; q += blockDim.x)
    rounds[q] = round_ptr[h * n_qt + q + 1] - round_ptr[h * n_qt + q];
  __syncthreads();
  for (int q = threadIdx.x; q < n_qt; q += blockDim.x) {
    const int32_t mine = rounds[q];
    int rank = 0;
    for (int p = 0; p < n_qt; ++p) rank += (rounds[p] > mine || (rounds[p] == mine && p < q)) ? 1 : 0;
    sorted[rank] = q;
  }
  __syncthreads();
  for (int j = threadIdx.x; j < n_half; j += blockDim.x) {
    out[2 * j] = sorted[j];
    out[2 * j + 1] = j != n_qt - 1 - j ? sorted[n_qt - 1 - j] : -1;
  }
}

// No gathered schedule (dense lists): every list row has zero gathered rounds.
__global__ void clear_grounds_kernel(int32_t *__restrict__ ground_ptr, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) ground_ptr[i] = 0;
}

}  // namespace

// Writes the round arrays of a finished tile list (row_ptr, col_idx, flags, groups, bitmap), and the
// gathered rounds where the list has room for them (gathered == false: an empty gathered schedule).
cudaError_t launch_build_rounds(const ap_tiles &t, cudaStream_t s, bool gathered) {
  const int n_rows = t.H * t.n_qt;
  count_rounds_kernel<<<ceil_div(n_rows, 4), 128, 0, s>>>(t.row_ptr, t.flags, t.groups, n_rows, t.round_ptr);
  scan_rounds_kernel<<<1, 1024, 0, s>>>(t.round_ptr, n_rows);
  fill_rounds_kernel<<<n_rows, 128, 0, s>>>(t.row_ptr, t.col_idx, t.flags, t.groups, t.bitmap, t.round_ptr, t.cap,
                                            t.round_rows, t.round_info, t.round_bitmap);
  count_launches(3);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (t.unit_qt) {
    pair_units_kernel<<<t.H, 256, 0, s>>>(t.round_ptr, t.n_qt, t.unit_qt);
    count_launches(1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  if (!t.ground_ptr) return e;
  if (!gathered) {
    clear_grounds_kernel<<<ceil_div(n_rows + 1, 256), 256, 0, s>>>(t.ground_ptr, n_rows + 1);
    count_launches(1);
    return cudaGetLastError();
  }
  // (test hook: every list row gets its gathered rounds, see ap_debug_schedule)
  count_grounds_kernel<<<ceil_div(n_rows, 4), 128, 0, s>>>(t.row_ptr, t.bitmap, t.round_ptr, n_rows,
                                                           debug_knobs().schedule == 2 ? 1 : 0, t.ground_ptr);
  scan_rounds_kernel<<<1, 1024, 0, s>>>(t.ground_ptr, n_rows);
  fill_grounds_kernel<<<n_rows, 128, 0, s>>>(t.row_ptr, t.col_idx, t.bitmap, t.ground_ptr, t.cap, t.ground_keys,
                                             t.ground_info, t.ground_bitmap);
  count_launches(3);
  return cudaGetLastError();
}

cudaError_t launch_stage_from_mask(const uint8_t *mask, int H, int Lq, int Lk, uint32_t *stage_bitmap,
                                   int32_t *stage_count, cudaStream_t s) {
  const int n_qt = ceil_div(Lq, kTile), n_kt = ceil_div(Lk, kTile);
  stage_from_mask_kernel<<<H * n_qt * n_kt, 128, 0, s>>>(mask, Lq, Lk, n_qt, n_kt, stage_bitmap,
                                                       stage_count);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_compact_tiles(const uint32_t *stage_bitmap, const int32_t *stage_count,
                                 const ap_tiles &t, cudaStream_t s) {
  const int n_tiles = t.H * t.n_qt * t.n_kt;
  unsigned *err = device_error_word();
  if (!err) return cudaErrorUnknown;
  // list positions live right behind the popcounts in the staging area
  int32_t *stage_pos = const_cast<int32_t *>(stage_count) + ((size_t)n_tiles * 4 + 255) / 256 * 64;
  scan_tiles_kernel<<<1, 1024, 0, s>>>(stage_count, stage_pos, n_tiles, t.n_kt, t.cap, t.row_ptr, err);
  count_launches(1);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  gather_tiles_kernel<<<n_tiles, 128, 0, s>>>(stage_bitmap, stage_count, stage_pos, t.n_kt, t.cap,
                                              t.col_idx, t.flags, t.bitmap, t.groups);
  count_launches(1);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  return launch_build_rounds(t, s, true);
}

cudaError_t launch_dense_tiles(const ap_tiles &t, int causal, cudaStream_t s) {
  unsigned *err = device_error_word();
  if (!err) return cudaErrorUnknown;
  dense_tiles_kernel<<<t.H * t.n_qt * t.n_kt, 128, 0, s>>>(t.H, t.Lq, t.Lk, t.n_qt, t.n_kt, causal, t.cap,
                                                         t.row_ptr, t.col_idx, t.flags, t.bitmap, t.groups,
                                                         t.round_ptr, t.round_rows, t.round_info, t.round_bitmap, err);
  count_launches(1);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (t.unit_qt) {
    pair_units_kernel<<<t.H, 256, 0, s>>>(t.round_ptr, t.n_qt, t.unit_qt);
    count_launches(1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  if (!t.ground_ptr) return e;
  // no gathered schedule for a dense list
  const int n_rows = t.H * t.n_qt;
  clear_grounds_kernel<<<ceil_div(n_rows + 1, 256), 256, 0, s>>>(t.ground_ptr, n_rows + 1);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace ap
