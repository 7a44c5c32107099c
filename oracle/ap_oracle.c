/*
 * CPU oracle for Attention Pruning's compute path.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, fp64 restatement of what the CUDA library computes, written from
 * the paper's equations.  It shares no code with the CUDA path and must never be
 * called from it: only the test-suite, the smoke check and the CPU-baseline leg
 * of the benchmark may load this file.
 *
 *   oracle_accumulate      Eq. 1 (the element-wise sum of softmax attention
 *                          matrices over samples; the 1/n factor is left to the
 *                          caller, see below) with the attention matrix of
 *                          Section 3.1, softmax(Q K^T / sqrt(d_k)).
 *   oracle_build_mask      Eq. 2 read as an exact top-k selection per head.
 *   oracle_build_mask_layer  Eq. 2 with one threshold for all heads of the layer.
 *   oracle_build_mask_ties   Eq. 2 with its strict inequality: ties with the threshold all stay.
 *   oracle_mask_to_tiles   the 128x128 tile list + bitmaps (an encoding of the
 *                          mask of Eq. 2; no counterpart in the paper).
 *   oracle_attention_fwd   the masked attention equation of Section 3.2,
 *                          softmax((Q K^T + M_p)/sqrt(d_k)) V with M_p = -inf
 *                          on pruned entries.
 *   oracle_attention_bwd   its derivative with respect to Q, K and V (what step 4 of
 *                          the procedure, retraining under the mask, needs).
 *   oracle_entmax15, oracle_accumulate_entmax15, oracle_attention_entmax15_fwd
 *                          the same average and masked attention with 1.5-entmax as the
 *                          normaliser (the section on sparse normalisation).
 *
 * Parity status: every function here is pinned by tests that do not go through
 * this file's own formulas (library SDPA, closed forms, brute force, invariants,
 * a hand-computed 4x4 example).  The one thing that cannot be pinned is whether
 * the synthetic masks look like masks of the paper's trained models: parity
 * unpinned for mask realism (no weights, no datasets).
 *
 * Inputs are float arrays holding the exact values the GPU receives (bf16 or
 * fp32 values widened to float); all arithmetic below is double.
 * OpenMP is used over independent (batch, head) units only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define AP_TILE 128

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void oracle_set_num_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

/*
 * Row domain: all keys, or, under the causal constraint, keys j <= i + (Lk - Lq).
 * With Lq == Lk that is j <= i.  With Lk = mem + Lq it is the mask of a model that
 * attends to `mem` cached positions of earlier segments, all visible, followed by
 * the current segment under its autoregressive mask (the Transformer-XL masks of
 * the language-modelling section: memory in the left half, causal right half).
 * Query i's own position is key i + (Lk - Lq).  Needs Lk >= Lq.
 */
static int row_domain_end(int i, int Lq, int Lk, int causal) {
  if (!causal) return Lk;
  int end = i + 1 + (Lk - Lq);
  if (end < 0) end = 0;
  return end < Lk ? end : Lk;
}

/* Forced entries of Eq. 2's selection: each query's own position, when asked for. */
static int is_forced(int i, int j, int Lq, int Lk, int causal, int keep_diag) {
  return keep_diag && (Lq == Lk || causal) && j == i + (Lk - Lq);
}

/*
 * Eq. 1 without the 1/n factor, one row (h, i) of the accumulator.  For every
 * sample b:
 *   s_j = (q_i . k_j) * scale + bias[h,i,j]       for j in the row's domain
 *   p_j = exp(s_j - max_j s) / sum_j exp(s_j - max_j s)
 *   arow[j] += p_j
 * Entries outside the domain are never touched.  `bias` may be NULL.
 * Samples are added in ascending b.  The raw sum is kept: dividing by n would
 * not change which entries are largest.
 */
static void accumulate_row(double *arow, const float *Q, const float *K, const float *bias, int h,
                           int i, int B, int H, int Lq, int Lk, int d, int causal, double scale) {
  int jend = row_domain_end(i, Lq, Lk, causal);
  double *s = (double *)malloc(sizeof(double) * (size_t)(jend > 0 ? jend : 1));
  for (int b = 0; b < B; ++b) {
    const float *q = Q + (((size_t)b * H + h) * Lq + i) * d;
    const float *Kh = K + ((size_t)b * H + h) * (size_t)Lk * d;
    double m = -INFINITY;
    for (int j = 0; j < jend; ++j) {
      double dot = 0.0;
      for (int t = 0; t < d; ++t) dot += (double)q[t] * (double)Kh[(size_t)j * d + t];
      double v = dot * scale;
      if (bias) v += (double)bias[((size_t)h * Lq + i) * Lk + j];
      s[j] = v;
      if (v > m) m = v;
    }
    double z = 0.0;
    for (int j = 0; j < jend; ++j) {
      s[j] = exp(s[j] - m);
      z += s[j];
    }
    for (int j = 0; j < jend; ++j) arow[j] += s[j] / z;
  }
  free(s);
}

/* Eq. 1 (sum form) for every head and row: acc[H,Lq,Lk] += sum_b softmax rows. */
void oracle_accumulate(double *acc, const float *Q, const float *K, const float *bias, int B,
                       int H, int Lq, int Lk, int d, int causal, double scale) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int hi = 0; hi < H * Lq; ++hi) {
    int h = hi / Lq, i = hi % Lq;
    accumulate_row(acc + ((size_t)h * Lq + i) * Lk, Q, K, bias, h, i, B, H, Lq, Lk, d, causal,
                   scale);
  }
}

/*
 * The same for a sample of rows, for sizes where all rows take too long:
 * rows[r] = (h, i) pairs, out[r, 0..Lk) += the row's sum (out is not cleared).
 */
void oracle_accumulate_rows(double *out, const int32_t *rows, int n_rows, const float *Q,
                            const float *K, const float *bias, int B, int H, int Lq, int Lk, int d,
                            int causal, double scale) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int r = 0; r < n_rows; ++r)
    accumulate_row(out + (size_t)r * Lk, Q, K, bias, rows[2 * r], rows[2 * r + 1], B, H, Lq, Lk, d,
                   causal, scale);
}

/* One candidate of the selection in Eq. 2. */
typedef struct {
  float value;
  int32_t forced;
  int64_t index; /* i * Lk + j */
} ap_entry;

/* forced first, then larger value first (compared as fp32), then lower index. */
static int entry_before(const void *pa, const void *pb) {
  const ap_entry *a = (const ap_entry *)pa, *b = (const ap_entry *)pb;
  if (a->forced != b->forced) return b->forced - a->forced;
  if (a->value > b->value) return -1;
  if (a->value < b->value) return 1;
  if (a->index < b->index) return -1;
  if (a->index > b->index) return 1;
  return 0;
}

/* Number of entries to keep out of n_valid, rounded half up in double. */
int64_t oracle_keep_count(int64_t n_valid, int64_t n_forced, double keep_frac) {
  int64_t k = (int64_t)floor(keep_frac * (double)n_valid + 0.5);
  if (k > n_valid) k = n_valid;
  if (k < n_forced) k = n_forced;
  return k;
}

/*
 * Block-structured pruning (the hardware section applies the method with sparseness
 * patterns "structured around blocks", block size 16, without saying how entries are
 * grouped).  Reading: a block's score is the mean of the averaged attention over the
 * block's entries inside the domain; Eq. 2's selection then runs over blocks
 * (oracle_build_mask on the pooled array, which has the same causal structure at block
 * level when Lq and Lk are multiples of the block size), and a kept block keeps all
 * of its entries inside the domain.
 *   pooled[h,I,J] = mean of acc[h,i,j] over I*bs <= i < (I+1)*bs, J*bs <= j < (J+1)*bs,
 *                   (i,j) in the domain; 0 for blocks without such entries
 * Needs Lq % bs == 0 and Lk % bs == 0.
 */
void oracle_pool_scores(const float *acc, int H, int Lq, int Lk, int bs, int causal, double *pooled) {
  int nI = Lq / bs, nJ = Lk / bs;
  for (int h = 0; h < H; ++h)
    for (int I = 0; I < nI; ++I)
      for (int J = 0; J < nJ; ++J) {
        double sum = 0.0;
        int64_t count = 0;
        for (int i = I * bs; i < (I + 1) * bs; ++i) {
          int jend = row_domain_end(i, Lq, Lk, causal);
          for (int j = J * bs; j < (J + 1) * bs && j < jend; ++j) {
            sum += (double)acc[((size_t)h * Lq + i) * Lk + j];
            ++count;
          }
        }
        pooled[((size_t)h * nI + I) * nJ + J] = count ? sum / (double)count : 0.0;
      }
}

/* A kept block keeps its entries inside the domain: mask[h,i,j] = block_mask[h,i/bs,j/bs] there, else 0. */
void oracle_expand_block_mask(const uint8_t *block_mask, int H, int Lq, int Lk, int bs, int causal,
                              uint8_t *mask) {
  int nI = Lq / bs, nJ = Lk / bs;
  for (int h = 0; h < H; ++h)
    for (int i = 0; i < Lq; ++i) {
      int jend = row_domain_end(i, Lq, Lk, causal);
      for (int j = 0; j < Lk; ++j)
        mask[((size_t)h * Lq + i) * Lk + j] =
            (j < jend && block_mask[((size_t)h * nI + i / bs) * nJ + j / bs]) ? 1 : 0;
    }
}

/*
 * Scores for the random-pruning control (the section that compares tailored masks
 * with pruning random entries): score n, n = (h*Lq + i)*Lk + j, is the top 24 bits
 * of the (n+1)-th output of the SplitMix64 generator seeded with `seed`, scaled to
 * [0, 1).  Passed through Eq. 2's selection they give a random mask with exactly
 * the count of a tailored one, inside the same domain and with the same forced
 * entries.  The generator (Steele, Lea, Flood: "Fast splittable pseudorandom number
 * generators", 2014) advances a 64-bit state by the odd constant below and scrambles
 * it with two multiply-xorshift steps; output n+1 depends only on seed and n.
 */
void oracle_random_scores(float *out, int64_t count, uint64_t seed) {
  uint64_t state = seed;
  for (int64_t n = 0; n < count; ++n) {
    state += 0x9E3779B97F4A7C15ull;
    uint64_t z = state;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z = z ^ (z >> 31);
    out[n] = (float)(z >> 40) * (1.0f / 16777216.0f);
  }
}

/*
 * Eq. 2 as an exact per-head top-k: an entry is pruned (M_p = -inf) iff it does
 * not belong to the k largest entries of the head's average attention matrix.
 *   domain   all (i,j), or j <= i + (Lk - Lq) when causal
 *   forced   each query's own position j = i + (Lk - Lq), when keep_diag and
 *            (Lq == Lk or causal)
 *   k        max(|forced|, min(n_valid, floor(keep_frac * n_valid + 0.5)))
 *   order    forced first, value descending (as fp32), index i*Lk+j ascending
 * mask[h,i,j] = 1 for the first k entries in that order, 0 elsewhere;
 * nnz[h] = k.  Returns 0, or -1 when an allocation fails.
 */
int oracle_build_mask(const float *acc, int H, int Lq, int Lk, double keep_frac, int causal,
                      int keep_diag, uint8_t *mask, int64_t *nnz) {
  int failed = 0;
  memset(mask, 0, (size_t)H * Lq * Lk);
#pragma omp parallel for schedule(dynamic, 1)
  for (int h = 0; h < H; ++h) {
    int64_t n_valid = 0;
    for (int i = 0; i < Lq; ++i) n_valid += row_domain_end(i, Lq, Lk, causal);
    ap_entry *e = (ap_entry *)malloc(sizeof(ap_entry) * (size_t)(n_valid > 0 ? n_valid : 1));
    if (!e) {
      failed = 1;
      continue;
    }
    int64_t n = 0, n_forced = 0;
    for (int i = 0; i < Lq; ++i) {
      int jend = row_domain_end(i, Lq, Lk, causal);
      for (int j = 0; j < jend; ++j) {
        e[n].value = acc[((size_t)h * Lq + i) * Lk + j];
        e[n].forced = is_forced(i, j, Lq, Lk, causal, keep_diag);
        e[n].index = (int64_t)i * Lk + j;
        n_forced += e[n].forced;
        ++n;
      }
    }
    int64_t k = oracle_keep_count(n_valid, n_forced, keep_frac);
    qsort(e, (size_t)n, sizeof(ap_entry), entry_before);
    for (int64_t r = 0; r < k; ++r) mask[(size_t)h * Lq * Lk + (size_t)e[r].index] = 1;
    nnz[h] = k;
    free(e);
  }
  return failed ? -1 : 0;
}

/*
 * Eq. 2 with one threshold for the whole layer, as the paper states it: the
 * percentile is taken over the averaged attention matrices of ALL heads of the
 * layer together, so heads keep unequal numbers of entries.  Read, like the
 * per-head variant, as an exact top-k: the population is the union of the
 * heads' domains (N = H * n_valid entries), the diagonals of all heads are
 * forced (under the per-head rule's condition) and counted inside
 *   k = max(#forced, min(N, floor(keep_frac * N + 0.5))),
 * and the order is: forced first, then larger value, then lower global index
 * (h * Lq + i) * Lk + j.  mask[h,i,j] = 1 for the first k entries; nnz[h] =
 * entries kept in head h.  Returns 0, or -1 when an allocation fails.
 */
int oracle_build_mask_layer(const float *acc, int H, int Lq, int Lk, double keep_frac, int causal,
                            int keep_diag, uint8_t *mask, int64_t *nnz) {
  memset(mask, 0, (size_t)H * Lq * Lk);
  int64_t n_valid = 0;
  for (int i = 0; i < Lq; ++i) n_valid += row_domain_end(i, Lq, Lk, causal);
  int64_t N = n_valid * H;
  ap_entry *e = (ap_entry *)malloc(sizeof(ap_entry) * (size_t)(N > 0 ? N : 1));
  if (!e) return -1;
  int64_t n = 0, n_forced = 0;
  for (int h = 0; h < H; ++h) {
    nnz[h] = 0;
    for (int i = 0; i < Lq; ++i) {
      int jend = row_domain_end(i, Lq, Lk, causal);
      for (int j = 0; j < jend; ++j) {
        e[n].value = acc[((size_t)h * Lq + i) * Lk + j];
        e[n].forced = is_forced(i, j, Lq, Lk, causal, keep_diag);
        e[n].index = ((int64_t)h * Lq + i) * Lk + j;
        n_forced += e[n].forced;
        ++n;
      }
    }
  }
  int64_t k = oracle_keep_count(N, n_forced, keep_frac);
  qsort(e, (size_t)n, sizeof(ap_entry), entry_before);
  for (int64_t r = 0; r < k; ++r) {
    mask[(size_t)e[r].index] = 1;
    nnz[e[r].index / ((int64_t)Lq * Lk)] += 1;
  }
  free(e);
  return 0;
}

/*
 * Eq. 2 with its strict inequality taken literally: an entry is pruned iff its average lies
 * strictly BELOW the threshold, so every entry equal to the threshold stays and the kept count
 * can exceed k.  The threshold tau is the value of the last entry the exact top-k above would
 * keep (the k-th in the order forced first, value descending); when the forced entries alone
 * fill k there is no threshold and only they are kept.
 *   mask[h,i,j] = 1  iff  (i,j) is forced, or in the domain with acc[h,i,j] >= tau (as fp32)
 * per_layer = 0: one population, k and tau per head; per_layer = 1: one for all heads together
 * (the layer rule above).  nnz[h] = entries kept in head h.  Returns 0, or -1 on a failed allocation.
 */
int oracle_build_mask_ties(const float *acc, int H, int Lq, int Lk, double keep_frac, int causal,
                           int keep_diag, int per_layer, uint8_t *mask, int64_t *nnz) {
  memset(mask, 0, (size_t)H * Lq * Lk);
  int64_t n_valid = 0;
  for (int i = 0; i < Lq; ++i) n_valid += row_domain_end(i, Lq, Lk, causal);
  int heads_per_pop = per_layer ? H : 1, n_pop = per_layer ? 1 : H;
  int64_t N = n_valid * heads_per_pop;
  ap_entry *e = (ap_entry *)malloc(sizeof(ap_entry) * (size_t)(N > 0 ? N : 1));
  if (!e) return -1;
  for (int h = 0; h < H; ++h) nnz[h] = 0;
  for (int pop = 0; pop < n_pop; ++pop) {
    int64_t n = 0, n_forced = 0;
    for (int hh = 0; hh < heads_per_pop; ++hh) {
      int h = pop * heads_per_pop + hh;
      for (int i = 0; i < Lq; ++i) {
        int jend = row_domain_end(i, Lq, Lk, causal);
        for (int j = 0; j < jend; ++j) {
          e[n].value = acc[((size_t)h * Lq + i) * Lk + j];
          e[n].forced = is_forced(i, j, Lq, Lk, causal, keep_diag);
          e[n].index = ((int64_t)h * Lq + i) * Lk + j;
          n_forced += e[n].forced;
          ++n;
        }
      }
    }
    int64_t k = oracle_keep_count(N, n_forced, keep_frac);
    qsort(e, (size_t)n, sizeof(ap_entry), entry_before);
    int64_t kept = k;
    if (k > n_forced) {
      float tau = e[k - 1].value;
      while (kept < n && e[kept].value >= tau) ++kept; /* sorted: the rest of the ties follow */
    }
    for (int64_t r = 0; r < kept; ++r) {
      mask[(size_t)e[r].index] = 1;
      nnz[e[r].index / ((int64_t)Lq * Lk)] += 1;
    }
  }
  free(e);
  return 0;
}

/*
 * Tile encoding of a mask.  Rows of the list are (h, qt) in ascending order;
 * inside a row the key tiles kt are ascending and only tiles with at least one
 * kept entry appear.  bitmap[t][r][w] bit c (LSB first) is entry
 * (128*qt + r, 128*kt + 32*w + c); flags[t] bit 0 says all 128*128 bits are set.
 * Returns the number of tiles, or -1 if it exceeds `cap`.
 */
int64_t oracle_mask_to_tiles(const uint8_t *mask, int H, int Lq, int Lk, int32_t *row_ptr,
                             int32_t *col_idx, uint8_t *flags, uint32_t *bitmap, int64_t cap) {
  int n_qt = (Lq + AP_TILE - 1) / AP_TILE, n_kt = (Lk + AP_TILE - 1) / AP_TILE;
  int64_t t = 0;
  row_ptr[0] = 0;
  for (int h = 0; h < H; ++h) {
    for (int qt = 0; qt < n_qt; ++qt) {
      for (int kt = 0; kt < n_kt; ++kt) {
        uint32_t words[AP_TILE][4];
        int64_t count = 0;
        memset(words, 0, sizeof(words));
        for (int r = 0; r < AP_TILE; ++r) {
          int i = qt * AP_TILE + r;
          if (i >= Lq) break;
          for (int c = 0; c < AP_TILE; ++c) {
            int j = kt * AP_TILE + c;
            if (j >= Lk) break;
            if (mask[((size_t)h * Lq + i) * Lk + j]) {
              words[r][c >> 5] |= 1u << (c & 31);
              ++count;
            }
          }
        }
        if (count == 0) continue;
        if (t >= cap) return -1;
        col_idx[t] = kt;
        flags[t] = (count == (int64_t)AP_TILE * AP_TILE) ? 1 : 0;
        memcpy(bitmap + (size_t)t * AP_TILE * 4, words, sizeof(words));
        ++t;
      }
      row_ptr[h * n_qt + qt + 1] = (int32_t)t;
    }
  }
  return t;
}

/*
 * Masked attention (Section 3.2), one output row.  With M_p = -inf on pruned
 * entries, row i of the output is the softmax-weighted mean of v_j over the
 * kept keys j only:
 *   J = { j : mrow[j] = 1 },  s_j = (q . k_j) * scale,  w_j = exp(s_j - max_J s)
 *   o = sum_J w_j v_j / sum_J w_j,   and exactly 0 when J is empty.
 */
static void attention_row(double *o, const float *q, const float *Kh, const float *Vh,
                          const uint8_t *mrow, int Lk, int d, double scale) {
  double *s = (double *)malloc(sizeof(double) * (size_t)Lk);
  double m = -INFINITY, z = 0.0;
  int any = 0;
  for (int t = 0; t < d; ++t) o[t] = 0.0;
  for (int j = 0; j < Lk; ++j) {
    if (!mrow[j]) continue;
    double dot = 0.0;
    for (int t = 0; t < d; ++t) dot += (double)q[t] * (double)Kh[(size_t)j * d + t];
    s[j] = dot * scale;
    if (s[j] > m) m = s[j];
    any = 1;
  }
  if (any) {
    for (int j = 0; j < Lk; ++j) {
      if (!mrow[j]) continue;
      double w = exp(s[j] - m);
      z += w;
      for (int t = 0; t < d; ++t) o[t] += w * (double)Vh[(size_t)j * d + t];
    }
    for (int t = 0; t < d; ++t) o[t] /= z;
  }
  free(s);
}

/* Masked attention for all rows: Q[B,H,Lq,d], K,V[B,H,Lk,d], mask[H,Lq,Lk] -> O[B,H,Lq,d]. */
void oracle_attention_fwd(const float *Q, const float *K, const float *V, const uint8_t *mask,
                          double *O, int B, int H, int Lq, int Lk, int d, double scale) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int bh = 0; bh < B * H; ++bh) {
    int h = bh % H;
    for (int i = 0; i < Lq; ++i)
      attention_row(O + ((size_t)bh * Lq + i) * d, Q + ((size_t)bh * Lq + i) * d,
                    K + (size_t)bh * Lk * d, V + (size_t)bh * Lk * d,
                    mask + ((size_t)h * Lq + i) * Lk, Lk, d, scale);
  }
}

/*
 * The same for a sample of output rows, for sizes where all rows take too long:
 * rows[r] = (b, h, i) triples, out[r, 0..d).
 */
void oracle_attention_rows(const float *Q, const float *K, const float *V, const uint8_t *mask,
                           double *out, const int32_t *rows, int n_rows, int B, int H, int Lq,
                           int Lk, int d, double scale) {
  (void)B;
#pragma omp parallel for schedule(dynamic, 8)
  for (int r = 0; r < n_rows; ++r) {
    int b = rows[3 * r], h = rows[3 * r + 1], i = rows[3 * r + 2];
    size_t bh = (size_t)b * H + h;
    attention_row(out + (size_t)r * d, Q + (bh * Lq + i) * d, K + bh * (size_t)Lk * d,
                  V + bh * (size_t)Lk * d, mask + ((size_t)h * Lq + i) * Lk, Lk, d, scale);
  }
}

/*
 * Derivative of the masked attention of Section 3.2 (step 4 of the procedure retrains the
 * model under the mask, so gradients flow through exactly this function).  For one query
 * row i with kept keys j:
 *   s_j = scale * q_i.k_j,  p = softmax over the kept j,  o_i = sum_j p_j v_j
 * and an incoming gradient g = dL/do_i:
 *   dL/dv_j += p_j g
 *   dL/dp_j  = g.v_j
 *   dL/ds_j  = p_j (dL/dp_j - sum_k p_k dL/dp_k)          (softmax Jacobian)
 *   dL/dq_i += scale * sum_j dL/ds_j k_j,   dL/dk_j += scale * dL/ds_j q_i
 * Pruned entries have p = 0 and receive no gradient; a row without kept entries outputs 0
 * and passes no gradient.  dQ[B,H,Lq,d], dK,dV[B,H,Lk,d] are overwritten.
 */
void oracle_attention_bwd(const float *Q, const float *K, const float *V, const float *dO,
                          const uint8_t *mask, double *dQ, double *dK, double *dV, int B, int H,
                          int Lq, int Lk, int d, double scale) {
  memset(dQ, 0, sizeof(double) * (size_t)B * H * Lq * d);
  memset(dK, 0, sizeof(double) * (size_t)B * H * Lk * d);
  memset(dV, 0, sizeof(double) * (size_t)B * H * Lk * d);
#pragma omp parallel for schedule(dynamic, 1)
  for (int bh = 0; bh < B * H; ++bh) {
    int h = bh % H;
    const float *Kh = K + (size_t)bh * Lk * d, *Vh = V + (size_t)bh * Lk * d;
    double *dKh = dK + (size_t)bh * Lk * d, *dVh = dV + (size_t)bh * Lk * d;
    double *p = (double *)malloc(sizeof(double) * (size_t)Lk);
    double *dp = (double *)malloc(sizeof(double) * (size_t)Lk);
    for (int i = 0; i < Lq; ++i) {
      const float *q = Q + ((size_t)bh * Lq + i) * d, *g = dO + ((size_t)bh * Lq + i) * d;
      const uint8_t *mrow = mask + ((size_t)h * Lq + i) * Lk;
      double *dq = dQ + ((size_t)bh * Lq + i) * d;
      double m = -INFINITY;
      int kept = 0;
      for (int j = 0; j < Lk; ++j) {
        if (!mrow[j]) continue;
        double dot = 0.0;
        for (int t = 0; t < d; ++t) dot += (double)q[t] * (double)Kh[(size_t)j * d + t];
        p[j] = dot * scale;
        if (p[j] > m) m = p[j];
        ++kept;
      }
      if (!kept) continue;
      double z = 0.0;
      for (int j = 0; j < Lk; ++j)
        if (mrow[j]) {
          p[j] = exp(p[j] - m);
          z += p[j];
        }
      double pdp = 0.0;
      for (int j = 0; j < Lk; ++j)
        if (mrow[j]) {
          p[j] /= z;
          double a = 0.0;
          for (int t = 0; t < d; ++t) a += (double)g[t] * (double)Vh[(size_t)j * d + t];
          dp[j] = a;
          pdp += p[j] * a;
        }
      for (int j = 0; j < Lk; ++j)
        if (mrow[j]) {
          double ds = p[j] * (dp[j] - pdp);
          for (int t = 0; t < d; ++t) {
            dVh[(size_t)j * d + t] += p[j] * (double)g[t];
            dq[t] += scale * ds * (double)Kh[(size_t)j * d + t];
            dKh[(size_t)j * d + t] += scale * ds * (double)q[t];
          }
        }
    }
    free(p);
    free(dp);
  }
}

/* ------------------------------------------------------------------------------------------
 * Sparse normalisation: 1.5-entmax in place of the softmax (the section on sparse
 * normalisation runs the whole procedure with alpha-entmax, alpha = 1.5, as the normaliser).
 *
 * alpha-entmax maps a score vector z to the point p of the probability simplex that maximises
 * p.z + H_alpha(p), H_alpha the Tsallis entropy sum_j (p_j - p_j^alpha) / (alpha (alpha - 1)).
 * Stationarity on the support and complementary slackness off it give, for alpha = 1.5,
 *   p_j = max(z_j / 2 - tau, 0)^2      with tau the one number for which sum_j p_j = 1.
 * (alpha -> 1 is the softmax, alpha = 2 the Euclidean projection onto the simplex.)
 *
 * Solved exactly here: with x = z / 2 sorted in descending order, if the support is the k
 * largest entries then tau solves sum_{j<=k} (x_(j) - tau)^2 = 1 below x_(k), i.e.
 *   tau_k = mean_k - sqrt((1 - k var_k) / k),  mean_k, var_k = mean and variance of x_(1..k),
 * and the support is the largest k for which that number exists and lies below x_(k).
 * Values are taken relative to the largest one (p is invariant to a shift of z).
 * ------------------------------------------------------------------------------------------ */
static int descending(const void *a, const void *b) {
  double x = *(const double *)a, y = *(const double *)b;
  return (x < y) - (x > y);
}

/* p[0..n) = 1.5-entmax(z[0..n)); n >= 1; p may alias z. */
void oracle_entmax15(const double *z, int n, double *p) {
  double *x = (double *)malloc(sizeof(double) * (size_t)n);
  double top = -INFINITY;
  for (int j = 0; j < n; ++j)
    if (z[j] > top) top = z[j];
  for (int j = 0; j < n; ++j) x[j] = (z[j] - top) / 2.0; /* <= 0, the largest is 0 */
  qsort(x, (size_t)n, sizeof(double), descending);
  double sum = 0.0, sumsq = 0.0, tau = -1.0; /* k = 1: (0 - tau)^2 = 1 */
  for (int k = 1; k <= n; ++k) {
    sum += x[k - 1];
    sumsq += x[k - 1] * x[k - 1];
    double mean = sum / k, var = sumsq / k - mean * mean;
    double disc = (1.0 - k * var) / k;
    if (disc < 0.0) continue;
    double t = mean - sqrt(disc);
    if (t < x[k - 1]) tau = t;
  }
  for (int j = 0; j < n; ++j) {
    double u = (z[j] - top) / 2.0 - tau;
    p[j] = u > 0.0 ? u * u : 0.0;
  }
  free(x);
}

/* Eq. 1 (sum form) with the 1.5-entmax attention matrix: one row (h, i), as accumulate_row. */
static void accumulate_row_entmax15(double *arow, const float *Q, const float *K, const float *bias,
                                    int h, int i, int B, int H, int Lq, int Lk, int d, int causal,
                                    double scale) {
  int jend = row_domain_end(i, Lq, Lk, causal);
  if (jend <= 0) return;
  double *s = (double *)malloc(sizeof(double) * (size_t)jend);
  for (int b = 0; b < B; ++b) {
    const float *q = Q + (((size_t)b * H + h) * Lq + i) * d;
    const float *Kh = K + ((size_t)b * H + h) * (size_t)Lk * d;
    for (int j = 0; j < jend; ++j) {
      double dot = 0.0;
      for (int t = 0; t < d; ++t) dot += (double)q[t] * (double)Kh[(size_t)j * d + t];
      s[j] = dot * scale;
      if (bias) s[j] += (double)bias[((size_t)h * Lq + i) * Lk + j];
    }
    oracle_entmax15(s, jend, s);
    for (int j = 0; j < jend; ++j) arow[j] += s[j];
  }
  free(s);
}

/* acc[H,Lq,Lk] += sum_b entmax15 rows of (Q_b K_b^T * scale + bias) over each row's domain. */
void oracle_accumulate_entmax15(double *acc, const float *Q, const float *K, const float *bias, int B,
                                int H, int Lq, int Lk, int d, int causal, double scale) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int hi = 0; hi < H * Lq; ++hi) {
    int h = hi / Lq, i = hi % Lq;
    accumulate_row_entmax15(acc + ((size_t)h * Lq + i) * Lk, Q, K, bias, h, i, B, H, Lq, Lk, d,
                            causal, scale);
  }
}

/* The same for sampled rows: rows[r] = (h, i), out[r, 0..Lk) += the row's sum. */
void oracle_accumulate_entmax15_rows(double *out, const int32_t *rows, int n_rows, const float *Q,
                                     const float *K, const float *bias, int B, int H, int Lq, int Lk,
                                     int d, int causal, double scale) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int r = 0; r < n_rows; ++r)
    accumulate_row_entmax15(out + (size_t)r * Lk, Q, K, bias, rows[2 * r], rows[2 * r + 1], B, H, Lq,
                            Lk, d, causal, scale);
}

/*
 * Masked attention of Section 3.2 with the 1.5-entmax normaliser, one output row: pruned
 * entries are at -inf before the normaliser, so they are outside its argument;
 *   J = { j : mrow[j] = 1 },  p = entmax15((q . k_j) * scale, j in J),  o = sum_J p_j v_j,
 * and exactly 0 when J is empty.
 */
static void attention_row_entmax15(double *o, const float *q, const float *Kh, const float *Vh,
                                   const uint8_t *mrow, int Lk, int d, double scale) {
  double *s = (double *)malloc(sizeof(double) * (size_t)(Lk > 0 ? Lk : 1));
  int *idx = (int *)malloc(sizeof(int) * (size_t)(Lk > 0 ? Lk : 1));
  int n = 0;
  for (int t = 0; t < d; ++t) o[t] = 0.0;
  for (int j = 0; j < Lk; ++j) {
    if (!mrow[j]) continue;
    double dot = 0.0;
    for (int t = 0; t < d; ++t) dot += (double)q[t] * (double)Kh[(size_t)j * d + t];
    s[n] = dot * scale;
    idx[n++] = j;
  }
  if (n > 0) {
    oracle_entmax15(s, n, s);
    for (int c = 0; c < n; ++c)
      for (int t = 0; t < d; ++t) o[t] += s[c] * (double)Vh[(size_t)idx[c] * d + t];
  }
  free(s);
  free(idx);
}

/* All rows: Q[B,H,Lq,d], K,V[B,H,Lk,d], mask[H,Lq,Lk] -> O[B,H,Lq,d]. */
void oracle_attention_entmax15_fwd(const float *Q, const float *K, const float *V,
                                   const uint8_t *mask, double *O, int B, int H, int Lq, int Lk,
                                   int d, double scale) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int bh = 0; bh < B * H; ++bh) {
    int h = bh % H;
    for (int i = 0; i < Lq; ++i)
      attention_row_entmax15(O + ((size_t)bh * Lq + i) * d, Q + ((size_t)bh * Lq + i) * d,
                             K + (size_t)bh * Lk * d, V + (size_t)bh * Lk * d,
                             mask + ((size_t)h * Lq + i) * Lk, Lk, d, scale);
  }
}

/* Sampled rows: rows[r] = (b, h, i), out[r, 0..d). */
void oracle_attention_entmax15_rows(const float *Q, const float *K, const float *V,
                                    const uint8_t *mask, double *out, const int32_t *rows,
                                    int n_rows, int B, int H, int Lq, int Lk, int d, double scale) {
  (void)B;
#pragma omp parallel for schedule(dynamic, 8)
  for (int r = 0; r < n_rows; ++r) {
    int b = rows[3 * r], h = rows[3 * r + 1], i = rows[3 * r + 2];
    size_t bh = (size_t)b * H + h;
    attention_row_entmax15(out + (size_t)r * d, Q + (bh * Lq + i) * d, K + bh * (size_t)Lk * d,
                           V + bh * (size_t)Lk * d, mask + ((size_t)h * Lq + i) * Lk, Lk, d, scale);
  }
}
