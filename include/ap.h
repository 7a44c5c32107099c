/*
 * ap.h - C ABI of the Attention Pruning library for NVIDIA B200 (sm_100a).
 *
 * Attention Pruning (AP) observes, for every attention head, the average
 * softmax attention matrix over a calibration set (Eq. 1), prunes the entries
 * whose average falls below a percentile threshold (Eq. 2) and then runs every
 * later forward pass with the pruned entries forced to -infinity before the
 * softmax (the masked attention equation of Section 3.2).  This library holds
 * the three device-side steps of that procedure and nothing else:
 *
 *   ap_accumulate_attention   Eq. 1: running element-wise sum of softmax(QK^T/sqrt(d))
 *   ap_build_mask             Eq. 2: per-head top-fraction selection -> mask + tile list
 *   ap_sparse_attention_fwd   Section 3.2: masked attention that visits only kept tiles
 *
 * Conventions that hold for every entry point
 *   - Tensors are contiguous, innermost dimension last: Q[B,H,Lq,d],
 *     K,V[B,H,Lk,d], O[B,H,Lq,d], acc/bias/mask[H,Lq,Lk].
 *   - Unless a parameter says "host", every pointer is DEVICE memory owned by
 *     the caller and 16-byte aligned.  The library allocates no memory; scratch
 *     space is passed in as a workspace whose size the *_workspace_bytes
 *     functions report.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Work is enqueued on it and the call returns without synchronising.
 *   - Argument errors are detected on the host and returned BEFORE anything is
 *     enqueued.  Nothing throws, aborts or traps.  Conditions only the device
 *     can see (a tile list that outgrew its capacity, a bounded wait that
 *     expired) set a sticky device word that ap_device_status() returns.
 *   - d is 64 or 128.  Any Lq, Lk >= 1 is accepted by the 16-bit paths; the fp32
 *     accumulate keeps a row of Lk scores in shared memory and returns
 *     AP_ERR_UNSUPPORTED beyond roughly Lk = 45 000.  ap_build_mask (one
 *     selection per head) takes at most 65 535 heads.
 *   - `causal` != 0 restricts query i to the keys j <= i + (Lk - Lq) and needs
 *     Lk >= Lq.  With Lq == Lk that is the usual autoregressive mask; with
 *     Lk = mem + Lq the first `mem` keys are cached positions of earlier segments,
 *     visible to every query, followed by the current segment under its
 *     autoregressive mask (the Transformer-XL masks of the paper's language-
 *     modelling section).  Query i's own position is key i + (Lk - Lq).
 *   - There is no CPU fallback: without a CUDA device the compute calls return
 *     AP_ERR_CUDA.
 */
#ifndef AP_H_
#define AP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AP_TILE 128 /* edge of the square tiles of the tile list */

typedef enum {
  AP_OK = 0,
  AP_ERR_INVALID_ARG = 1, /* null/misaligned pointer, size or fraction out of range */
  AP_ERR_UNSUPPORTED = 2, /* d or dtype the kernels are not built for              */
  AP_ERR_WORKSPACE = 3,   /* workspace or tile capacity too small                   */
  AP_ERR_CUDA = 4,        /* a CUDA runtime call failed (no device, launch error)   */
  AP_ERR_TIMEOUT = 5      /* a bounded device-side wait gave up                     */
} ap_status;

typedef enum { AP_F32 = 0, AP_BF16 = 1, AP_F16 = 2 } ap_dtype; /* AP_F16: IEEE half precision */

/*
 * Tile list: the mask of Eq. 2 for H heads, cut into 128x128 tiles, with only
 * the tiles that contain at least one kept entry stored (CSR over tile rows).
 * The struct itself lives in host memory; its pointers are device memory.
 *
 *   row_ptr[H*n_qt + 1]  offsets into col_idx; list row r = h*n_qt + qt
 *   col_idx[cap]         key-tile index kt of each stored tile, strictly
 *                        ascending inside a list row
 *   flags[cap]           bit 0: every one of the 128*128 entries is kept
 *   bitmap[cap][128][4]  entry (r, c) of a tile is bit (c & 31) of word
 *                        [r][c >> 5], least significant bit first; bits of
 *                        rows >= Lq or columns >= Lk are 0 (also written, all
 *                        ones, for tiles flagged as fully kept)
 *   groups[cap]          summary of the bitmap: bit g is set iff some row keeps
 *                        an entry among key columns [16g, 16g+16) of the tile.
 *                        The forward pass plans from it which 16-column groups
 *                        to visit, so it must agree with the bitmap; every
 *                        builder of this library writes it.
 *
 * Rounds: the schedule the forward pass follows, derived from the fields above.
 * The non-empty groups of a list row (eight per tile flagged as fully kept),
 * taken in list order, are numbered as SLOTS 0, 1, ...; round k of the list row
 * consists of its slots [8k, 8k+8), so a round covers 16..128 key columns that
 * may come from several key tiles.  A list row with s slots has ceil(s/8) rounds;
 * there are never more rounds than stored tiles.
 *   round_ptr[H*n_qt + 1]      offsets into the round arrays, per list row
 *   round_rows[cap][8]         first key row (kt*128 + 16*group) of each slot of a
 *                              round; -1 for the unused slots of a row's last round
 *   round_info[cap]            bits 0..3: slots of the round (1..8); bit 7: all
 *                              128*128 entries of the round are kept
 *   round_bitmap[cap][128][4]  the round's bitmap: the 16 columns of slot q are
 *                              bits [16q, 16q+16) of row r (bit 16q + c of the
 *                              128-bit row, words LSB first); 0 for unused slots
 * Every builder of this library (ap_build_mask, ap_mask_to_tiles[_static],
 * ap_dense_tiles) writes groups and the round arrays along with the tile list; a
 * list assembled by hand must provide them too for ap_sparse_attention_fwd.
 *
 * Gathered rounds: an optional second schedule (all four pointers null, or all four
 * set; the CSR arrays and the rounds above do not depend on it).  A list row's ACTIVE
 * KEY COLUMNS - the keys that at least one of the 128 query rows keeps - are put in
 * this order: first the columns of the 16-column groups [16g, 16g+16) in which every
 * column is active, then all other active columns, ascending in each part; gathered
 * round k of the list row consists of columns [128k, 128k+128) of that order, whatever
 * key tiles they come from, so a list row with c active columns has ceil(c/128)
 * gathered rounds (never more than its rounds above).  The builders give a list row
 * gathered rounds only where the forward is expected to gain from them: with r rounds,
 * g = ceil(c/128) and s = ceil((c - 16 w)/16), w the number of those whole groups, if
 * 2 r > 4 g + s; other list rows have none.
 *   ground_ptr[H*n_qt + 1]      offsets into the gathered-round arrays, per list row;
 *                               all zero: no gathered schedule (ap_dense_tiles)
 *   ground_keys[cap][128]       key index of each column of a gathered round; the unused
 *                               tail of a row's last round repeats its last key
 *   ground_info[cap]            bits 0..3: ceil(columns / 16), 1..8 (the forward computes
 *                               that many 16-column slots); bit 7: 128 columns, all kept
 *   ground_bitmap[cap][128][4]  bit p of the 128-bit row r: query row r keeps column p
 *                               of the round; 0 for unused columns
 * Work units: optional (null: the forward pairs query tile n_qt-1-j with query tile j).
 *   unit_qt[H][ceil(n_qt/2)][2]  the two query tiles of each unit of work of a head; every query
 *                               tile of the head appears exactly once, the second entry of at most
 *                               one unit is -1 (odd n_qt).  The builders pair the list row with the
 *                               most rounds with the one with the fewest, the second with the
 *                               second fewest, and so on (ties by lower index first), so that a
 *                               head's units weigh about the same; ap_sparse_attention_fwd hands
 *                               whole units to its thread blocks.
 *
 * ap_sparse_attention_fwd follows the gathered rounds of a list row that has some (a
 * slot of 16 keys that follow one another from a multiple of 8 on is fetched as one box,
 * the rows of other slots one by one), the rounds otherwise; the result is the same
 * masked attention either way.
 *
 * cap is the capacity in tiles; ap_tiles_capacity() always suffices.
 */
typedef struct ap_tiles {
  int32_t H, Lq, Lk;
  int32_t n_qt, n_kt; /* ceil(Lq/128), ceil(Lk/128) */
  int32_t cap;
  int32_t *row_ptr;
  int32_t *col_idx;
  uint8_t *flags;
  uint32_t *bitmap;
  uint8_t *groups;
  int32_t *round_ptr;
  int32_t *round_rows;
  uint8_t *round_info;
  uint32_t *round_bitmap;
  int32_t *ground_ptr;
  int32_t *ground_keys;
  uint8_t *ground_info;
  uint32_t *ground_bitmap;
  int32_t *unit_qt;
} ap_tiles;

/* Library version (major*10000 + minor*100 + patch). */
int ap_version(void);

/* Kernels this library has launched so far in this process (a diagnostic counter). */
uint64_t ap_launch_count(void);

/*
 * Test hook for the failure path (no counterpart in the paper).  Every wait inside the tensor-core
 * kernels polls a bounded number of times; when a wait runs out the kernel raises the device status
 * word, every role leaves its loop, copies in flight are waited for (bounded), tensor memory is
 * freed and the kernel returns, after which ap_device_status() reports AP_ERR_TIMEOUT once.
 * With on != 0, the following launches of ap_sparse_attention_fwd, ap_accumulate_attention and
 * ap_sparse_attention_bwd (16-bit types) poll a few thousand times only and leave out the first
 * copies of a thread block (forward and accumulate: on a grid of ONE thread block), so that this path
 * runs within milliseconds without faulting or hanging anything; their output is undefined.
 * on == 0 restores normal operation.  Process-wide; not for production use.
 */
void ap_debug_expire_waits(int on);

/*
 * Test and measurement hook (no counterpart in the paper) for the two schedules of a tile list.
 * 0 (the default): the builders give a list row gathered rounds where they are expected to pay, and
 * ap_sparse_attention_fwd (16-bit types) follows them where a list row has some.  1: the forward
 * follows the rounds only.  2: the builders give every list row with a kept entry its gathered
 * rounds (and the forward follows them).  The forward's output is the same masked attention in
 * every mode (the exponentials are summed in a different order, so the last bit may differ).
 * Process-wide.
 */
void ap_debug_schedule(int mode);

/* Static, human-readable name of a status code. */
const char *ap_status_string(ap_status s);

/* Upper bound on the tiles of any mask of this shape: H * ceil(Lq/128) * ceil(Lk/128). */
int64_t ap_tiles_capacity(int H, int Lq, int Lk);

/* Workspace sizes in bytes (0 if the shape is invalid). */
size_t ap_build_mask_workspace_bytes(int H, int Lq, int Lk);
size_t ap_mask_to_tiles_workspace_bytes(int H, int Lq, int Lk);

/*
 * Eq. 1 (with the attention matrix of Section 3.1), as a running sum:
 *   acc[h,i,j] += sum_{b<B} softmax_j( Q[b,h,i,:].K[b,h,j,:] * scale + bias[h,i,j] )
 * over the row's domain (all j, or the causal domain above); entries outside the
 * domain are not touched.  The 1/n of Eq. 1 is left to the caller, who counts
 * the samples: the selection of Eq. 2 does not depend on it.
 *   acc    [H,Lq,Lk] fp32, in/out.  The samples are summed in ascending b inside the kernel,
 *          in chunks whose size depends only on the shape and the device's SM count (all B
 *          samples at once for shapes with many (head, query tile) pairs), and every chunk's
 *          sum is added to acc in ascending order of the chunks, so results are reproducible
 *          bit for bit on a given device.
 *   Q, K   [B,H,Lq,d], [B,H,Lk,d] of type dt (AP_BF16 and AP_F16 run on the tensor cores)
 *   bias   [H,Lq,Lk] fp32 added after scaling, or NULL
 *   scale  multiplier of Q.K^T; 0 selects 1/sqrt(d)
 */
ap_status ap_accumulate_attention(float *acc, const void *Q, const void *K, const float *bias,
                                  int B, int H, int Lq, int Lk, int d, ap_dtype dt, int causal,
                                  float scale, void *stream);

/*
 * Eq. 1 for a model whose normaliser is 1.5-entmax instead of the softmax (the section on
 * sparse normalisation): the same running sum with
 *   p = entmax15_j( Q[b,h,i,:].K[b,h,j,:] * scale + bias[h,i,j] ),
 *   entmax15(z)_j = max(z_j / 2 - tau, 0)^2,  tau such that the row sums to 1,
 * over the row's domain.  Entries outside the domain, and entries inside it that no sample
 * gives weight, keep their value.  tau is found in fp32 by solving the row's equation on the
 * support of a trial threshold and repeating until the step falls under 2e-6 max(1, |tau|).
 * (5e-7 for fp32 tensors, which run on the CUDA cores).
 * Arguments, layout, ordering of the sum and error behaviour as ap_accumulate_attention.
 */
ap_status ap_accumulate_attention_entmax15(float *acc, const void *Q, const void *K, const float *bias,
                                           int B, int H, int Lq, int Lk, int d, ap_dtype dt, int causal,
                                           float scale, void *stream);

/*
 * Eq. 2 with one threshold per head, as an exact top-k: an entry is pruned
 * unless it is among the k largest of its head.
 *   domain  all (i,j), or the causal domain; n_valid = its size
 *   forced  when keep_diag != 0 and (Lq == Lk or causal): every query's own
 *           position j = i + (Lk - Lq) (counted inside k)
 *   k       max(#forced, min(n_valid, floor(keep_frac*n_valid + 0.5))), in double
 *   order   forced first, then larger fp32 value, then lower index i*Lk + j
 * Outputs (any of mask / tiles / nnz_per_head may be NULL):
 *   mask          [H,Lq,Lk] uint8, 1 = kept
 *   tiles         tile list of the same mask; tiles->H/Lq/Lk/n_qt/n_kt are
 *                 written by this call, pointers and cap are read
 *   nnz_per_head  [H] int64, entries kept per head (= k)
 * acc must not contain NaN; -0 is treated as +0.  keep_frac must be in (0, 1].
 * More stored tiles than tiles->cap sets AP_ERR_WORKSPACE in the device status
 * and leaves a truncated list.
 */
ap_status ap_build_mask(const float *acc, int H, int Lq, int Lk, double keep_frac, int causal,
                        int keep_diag, uint8_t *mask, ap_tiles *tiles, int64_t *nnz_per_head,
                        void *workspace, size_t workspace_bytes, void *stream);

/*
 * Eq. 2 as the paper states it: ONE threshold for all H heads passed in (the heads of one
 * layer), i.e. an exact top-k over the union of the heads' domains, so that heads keep unequal
 * numbers of entries.  Same arguments, outputs and conventions as ap_build_mask with
 *   domain  the union over h of head h's domain; N = H * n_valid entries
 *   forced  every head's forced entries under the per-head rule (counted inside k)
 *   k       max(#forced, min(N, floor(keep_frac*N + 0.5))), in double
 *   order   forced first, then larger fp32 value, then lower index (h*Lq + i)*Lk + j
 *   nnz_per_head[h]  entries kept in head h (they sum to k)
 * Needs H*Lq*Lk < 2^32 (AP_ERR_UNSUPPORTED otherwise).
 */
ap_status ap_build_mask_layer(const float *acc, int H, int Lq, int Lk, double keep_frac, int causal,
                              int keep_diag, uint8_t *mask, ap_tiles *tiles, int64_t *nnz_per_head,
                              void *workspace, size_t workspace_bytes, void *stream);

/*
 * Both rules with Eq. 2's strict inequality taken literally.  flags is a sum of
 *   AP_MASK_PER_LAYER  one selection over all heads (ap_build_mask_layer) instead of one per head
 *   AP_MASK_KEEP_TIES  an entry is pruned iff its average lies strictly below the threshold, the
 *                      value of the last entry the exact top-k would keep: every entry equal to
 *                      it stays, so a head (the layer) may keep more than k entries.  Where the
 *                      forced entries alone fill k there is no threshold and only they are kept.
 * With flags = 0 this is ap_build_mask.  nnz_per_head[h] = entries kept in head h.  Other
 * arguments, outputs and errors as above; unknown flag bits are AP_ERR_INVALID_ARG.
 */
#define AP_MASK_PER_LAYER 1
#define AP_MASK_KEEP_TIES 2
ap_status ap_build_mask_ex(const float *acc, int H, int Lq, int Lk, double keep_frac, int causal,
                           int keep_diag, int flags, uint8_t *mask, ap_tiles *tiles,
                           int64_t *nnz_per_head, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Derivative of ap_sparse_attention_fwd with respect to Q, K and V (retraining under the
 * mask, step 4 of the paper's procedure, differentiates exactly this function).  With
 * S = scale*Q.K^T, P = softmax of S over the kept entries of a row, O = P.V and dO given:
 *   dV = P^T.dO,  dP = dO.V^T,  dS = P o (dP - rowsum(dO o O)),  dQ = scale*dS.K,  dK = scale*dS^T.Q
 * Pruned entries receive no gradient; a row without kept entries passes none.
 *   Q, O, dO, dQ  [B,H,Lq,d];  K, V, dK, dV  [B,H,Lk,d], all of type dt (AP_BF16 or AP_F16;
 *   AP_F32 is AP_ERR_UNSUPPORTED); O is the forward's output for the same inputs and tiles.
 *   dQ, dK, dV are overwritten (every element written once: reproducible bit for bit).
 *   workspace     ap_sparse_attention_bwd_workspace_bytes(B, H, Lq, Lk) bytes (row statistics and a
 *                 table from (query tile, key tile) to the tile's position in the list)
 */
size_t ap_sparse_attention_bwd_workspace_bytes(int B, int H, int Lq, int Lk);
ap_status ap_sparse_attention_bwd(const void *Q, const void *K, const void *V, const void *O, const void *dO,
                                  const ap_tiles *tiles, void *dQ, void *dK, void *dV, int B, int H,
                                  int Lq, int Lk, int d, ap_dtype dt, float scale, void *workspace,
                                  size_t workspace_bytes, void *stream);

/*
 * Block-structured pruning (the paper's hardware section uses sparseness patterns made of
 * blocks of 16; how entries are grouped is not stated).  Three steps:
 *   ap_pool_scores         pooled[h,I,J] = mean of acc over the entries of block (I,J) that lie
 *                          inside the domain (0 if none), [H, Lq/block, Lk/block] fp32
 *   ap_build_mask[_layer]  on the pooled array with the same causal / keep_diag arguments:
 *                          Eq. 2 over blocks (the pooled array has the element domain's shape
 *                          at block level)
 *   ap_expand_block_mask   mask[h,i,j] = block_mask[h, i/block, j/block] inside the domain,
 *                          0 outside; then ap_mask_to_tiles for the forward pass
 * block is 16, 32, 64 or 128 and must divide Lq and Lk (AP_ERR_UNSUPPORTED otherwise).  With
 * block = 128 every stored tile is fully kept, except where the causal boundary cuts it.
 */
ap_status ap_pool_scores(const float *acc, int H, int Lq, int Lk, int block, int causal, float *pooled,
                         void *stream);
ap_status ap_expand_block_mask(const uint8_t *block_mask, int H, int Lq, int Lk, int block, int causal,
                               uint8_t *mask, void *stream);

/*
 * Scores for the random-pruning control (the paper's comparison of tailored masks with
 * pruning random entries): scores[n], n = (h*Lq + i)*Lk + j, is the top 24 bits of the
 * (n+1)-th output of the SplitMix64 generator seeded with `seed`, scaled to [0, 1).
 * ap_build_mask[_layer] on these scores gives a random mask with exactly the count, the
 * domain and the forced entries of a tailored mask of the same keep_frac.
 *   scores  [H,Lq,Lk] fp32, written
 */
ap_status ap_random_scores(float *scores, int H, int Lq, int Lk, uint64_t seed, void *stream);

/*
 * Tile list of an arbitrary element mask (uint8 [H,Lq,Lk], non-zero = kept):
 * the same encoding ap_build_mask emits, for masks made elsewhere (random
 * masks as in the paper's control experiment, all-ones, hand-made).
 */
ap_status ap_mask_to_tiles(const uint8_t *mask, int H, int Lq, int Lk, ap_tiles *tiles,
                           void *workspace, size_t workspace_bytes, void *stream);

/*
 * ap_mask_to_tiles for callers that cannot allocate device memory (the paper has
 * no counterpart for this entry point; it exists for the library's users only).
 * Who needs it: code that runs where cudaMalloc is off limits - a plugin living
 * inside another framework's memory pool, a latency-critical loop that must not
 * enter the allocator, a process whose memory budget is fixed at start-up.
 * Instead of a caller-provided workspace the staging area is a fixed array in
 * device global memory that is part of the library image: every GPU that loads
 * the library holds AP_STATIC_SCRATCH_BYTES (about 2.1 MB) of it until exit.
 *   - Inputs and outputs are the caller's, exactly as for ap_mask_to_tiles, and
 *     the resulting tile list is identical bit for bit.
 *   - Limit: H * ceil(Lq/128) * ceil(Lk/128) <= AP_STATIC_MAX_TILES; larger shapes
 *     return AP_ERR_WORKSPACE before anything is enqueued.
 *   - The call itself allocates nothing (no cudaMalloc/cudaFree, no allocating
 *     library routine).  The first call on each device looks up the array's
 *     device address (cudaGetSymbolAddress, with that device current); make that
 *     first call before starting any stream capture.
 *   - All calls share the one array and it keeps the previous call's contents.
 *     Each call overwrites everything it later reads, so a stale array is
 *     harmless, but two calls that overlap on the GPU (different streams, no
 *     ordering between them) race on it: serialise them.
 */
#define AP_STATIC_MAX_TILES 1024
#define AP_STATIC_SCRATCH_BYTES (AP_STATIC_MAX_TILES * (128 * 4 * 4 + 8))
ap_status ap_mask_to_tiles_static(const uint8_t *mask, int H, int Lq, int Lk, ap_tiles *tiles,
                                  void *stream);

/*
 * Tile list of the unpruned attention (the zero mask matrix of Section 3.2):
 * every tile of the domain, written without reading any mask.  This is the
 * library's dense path and the baseline the sparse path is compared with.
 * Needs tiles->cap >= the number of domain tiles (ap_tiles_capacity suffices).
 */
ap_status ap_dense_tiles(int H, int Lq, int Lk, int causal, ap_tiles *tiles, void *stream);

/*
 * Masked attention of Section 3.2.  For every b, h and query row i, with
 * J = { j : entry (i,j) of head h is kept }:
 *   O[b,h,i,:] = sum_{j in J} w_j V[b,h,j,:] / sum_{j in J} w_j,
 *   w_j = exp( (Q[b,h,i,:].K[b,h,j,:]) * scale - max_J(...) ),
 * and exactly 0 when J is empty.  Pruned entries get weight exactly 0.  Only the
 * tiles stored in `tiles` are visited; causality is whatever the mask says.
 *   Q, K, V, O  of type dt (O is rounded once, from fp32)
 *   tiles       list for H heads and this Lq, Lk, shared by all b
 *   scale       0 selects 1/sqrt(d)
 */
ap_status ap_sparse_attention_fwd(const void *Q, const void *K, const void *V,
                                  const ap_tiles *tiles, void *O, int B, int H, int Lq, int Lk,
                                  int d, ap_dtype dt, float scale, void *stream);

/*
 * The same masked attention for a model whose normaliser is 1.5-entmax (the section on sparse
 * normalisation): pruned entries are outside the normaliser's argument,
 *   O[b,h,i,:] = sum_j p_j V[b,h,j,:],  p = entmax15( scale * Q[b,h,i,:].K[b,h,j,:] : j kept ),
 *   entmax15(z)_j = max(z_j / 2 - tau, 0)^2,  tau such that the row sums to 1
 * (found in fp32 as in ap_accumulate_attention_entmax15, to a step under 2e-6 max(1, |tau|)); a row
 * without kept entries outputs exactly 0.  The weights are rounded to dt before they multiply V
 * and the row is divided by the sum of the rounded weights.  Follows the tile list's rounds
 * (round_ptr, round_rows, round_info, round_bitmap); fp32 tensors run on the CUDA cores over
 * the stored tiles (row_ptr, col_idx, flags, bitmap), with fp32 weights and a step bound of
 * 5e-7.  Arguments and error behaviour as ap_sparse_attention_fwd.
 */
ap_status ap_sparse_attention_entmax15_fwd(const void *Q, const void *K, const void *V, const ap_tiles *tiles,
                                           void *O, int B, int H, int Lq, int Lk, int d, ap_dtype dt,
                                           float scale, void *stream);

/*
 * The same call for HOST tensors (pinned memory, or the copies are not asynchronous): copies
 * Q, K, V to the caller's device staging buffers, runs ap_sparse_attention_fwd and copies O
 * back.  dQ..dO are device buffers of the tensors' sizes.  The batch is cut into up to 8 chunks
 * of batch elements that are copied in, computed and copied out as a pipeline, so that the two
 * directions of the host link work at the same time: the kernels run on `stream`, the copies on
 * two streams the library keeps per device (created on the first call, with 18 events, and never
 * destroyed), ordered after the work already in `stream`; when the call returns, `stream` is
 * ordered after the last output copy, so synchronising `stream` is enough.  Calls on one device
 * share those streams and events: issue them from one host thread at a time.
 */
ap_status ap_sparse_attention_fwd_host(const void *hQ, const void *hK, const void *hV,
                                       const ap_tiles *tiles, void *hO, void *dQ, void *dK,
                                       void *dV, void *dO, int B, int H, int Lq, int Lk, int d,
                                       ap_dtype dt, float scale, void *stream);

/*
 * Synchronises `stream`, then returns and clears the sticky device status of
 * the current device: AP_OK, AP_ERR_WORKSPACE (tile capacity exceeded),
 * AP_ERR_TIMEOUT (a bounded wait expired; outputs of that call are invalid) or
 * AP_ERR_CUDA (the stream reported an error).
 */
ap_status ap_device_status(void *stream);

#ifdef __cplusplus
}
#endif
#endif /* AP_H_ */
