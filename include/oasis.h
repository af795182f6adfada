/*
 * oasis.h -- C ABI of the B200 (sm_100a) implementation of the OasisKV per-decode-step
 * hot path: lookahead scoring of KV blocks, per-head top-k selection, host->HBM block
 * gather, and sparse paged decode attention (OasisKV, Sec. 4.2-4.3, 5.1-5.2).
 *
 * Conventions shared by every call
 *   - Every buffer is caller-owned.  Unless a parameter says "host", a pointer must be
 *     dereferenceable by the GPU: device memory, or pinned host memory mapped into the
 *     device address space (unified addressing).  The library allocates nothing, keeps
 *     no state besides the last-error string, never synchronises and never blocks: each
 *     call validates its scalar arguments on the host, enqueues its kernels on `stream`
 *     (a cudaStream_t passed as void*; NULL = the legacy default stream) and returns.
 *   - Return value: OASIS_OK or an oasis_status_t error.  On error nothing was enqueued
 *     and oasis_last_error() describes the problem.  Contents of device arrays are not
 *     validated on the host; out-of-range block ids or slots are the caller's error.
 *   - bf16 tensors are raw 16-bit patterns, dense and row-major with the innermost index
 *     last, and their base addresses must be 16-byte aligned (OASIS_ERR_INVALID_ARG
 *     otherwise).  head_dim must be 128 and block_size 16 (OASIS_ERR_UNSUPPORTED
 *     otherwise); n_q_heads must be a multiple of n_kv_heads.
 *   - One "entry" is the K part then the V part of one (block, KV head):
 *     [2][16][128] bf16 = 8192 contiguous bytes.  The full-KV pool is
 *     [n_phys_blocks][n_kv_heads] entries (the paper's Head-Token-Dimension order,
 *     Sec. 4.3); the HBM working-set pool is [n_slots] entries.
 *   - Query head a reads KV head a / (n_q_heads / n_kv_heads).
 */
#ifndef OASIS_H
#define OASIS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    OASIS_OK = 0,
    OASIS_ERR_INVALID_ARG = 1, /* null pointer, misaligned buffer, inconsistent sizes   */
    OASIS_ERR_UNSUPPORTED = 2, /* a shape this build has no kernel for                   */
    OASIS_ERR_CUDA = 3,        /* a CUDA runtime call or kernel launch failed            */
    OASIS_ERR_WORKSPACE = 4    /* workspace missing or smaller than required             */
} oasis_status_t;

typedef enum { OASIS_REDUCE_MAX = 0, OASIS_REDUCE_SUM = 1 } oasis_reduce_t;

typedef struct {
    int32_t batch;      /* B: requests in the step                                  */
    int32_t n_q_heads;  /* Hq                                                        */
    int32_t n_kv_heads; /* Hkv                                                       */
    int32_t head_dim;   /* 128                                                       */
    int32_t block_size; /* 16 tokens per KV block                                    */
    int32_t max_blocks; /* row stride of every per-request block array               */
} oasis_dims_t;

#define OASIS_ENTRY_BYTES 8192
#define OASIS_MAX_K 2048 /* largest k accepted by oasis_select_topk */

/*
 * Step 0 -- block summaries (Sec. 4.2.1: the coordinate-wise minimum and maximum of the
 * keys of each logical block; Sec. 5.2: two summary rows per block, 1/16 of the KV size).
 * For request b and every KV head h, (re)builds the summaries of logical blocks
 * j = first_block[b] .. first_block[b] + n_blocks[b] - 1 from the K part of entry
 * (block_table[b][j], h) of kv_pool.
 *   kv_pool        full-KV pool (device memory, or mapped pinned host memory)
 *   block_table    [B][max_blocks] int32, logical -> physical block
 *   first_block, n_blocks   [B] int32 (device)
 *   max_new_blocks host-side upper bound of n_blocks[b]; sizes the launch (blocks past
 *                  n_blocks[b] are skipped on the device)
 *   summaries      [B][Hkv][max_blocks][2][128] bf16, row 0 = min, row 1 = max; only the
 *                  requested blocks are written
 */
int oasis_build_summaries(const oasis_dims_t *dims, const void *kv_pool,
                          const int32_t *block_table, const int32_t *first_block,
                          const int32_t *n_blocks, int32_t max_new_blocks, void *summaries,
                          void *stream);

/*
 * Step 0 for several layers in one launch: the same as one oasis_build_summaries call per layer with that
 * layer's pool, block table and summaries (host arrays of n_layers device pointers; first_block, n_blocks
 * and max_new_blocks are shared, as a decode step appends the same positions to every layer's cache).
 * n_layers may not exceed OASIS_MAX_LAYERS.
 */
#define OASIS_MAX_LAYERS 128
int oasis_build_summaries_layers(const oasis_dims_t *dims, int32_t n_layers, const void *const *kv_pools,
                                 const int32_t *const *block_tables, const int32_t *first_block,
                                 const int32_t *n_blocks, int32_t max_new_blocks, void *const *summaries,
                                 void *stream);

/*
 * Dense -> sparse hand-over (Sec. 4.3: a request prefills and decodes densely; once its context
 * exceeds the sparsification threshold the full KV cache is copied to CPU memory and only the
 * selected blocks and a local window stay on the GPU; both pools keep their blocks in
 * Head-Token-Dimension order, each behind its own page table).
 * For request b and logical blocks j = first_block[b] .. first_block[b] + n_blocks[b] - 1 (those
 * below max_blocks) and every KV head h:
 *   host_kv entry (block_table[b][j], h) = [ dense_k block (gpu_table[b][j], h) |
 *                                            dense_v block (gpu_table[b][j], h) ]
 * and, when summaries is not NULL, summaries[b][h][j] is built from the copied keys as in step 0
 * (pass NULL for a partially filled block, which has no final summary yet).
 *   dense_k, dense_v   [P_gpu][Hkv][16][128] bf16 (device): the dense pool's key / value blocks
 *   gpu_table          [B][max_blocks] int32 (device): logical -> physical block of the dense pool
 *   block_table        [B][max_blocks] int32 (device): logical -> physical block of host_kv
 *   max_new_blocks     host-side upper bound of n_blocks[b]; sizes the launch
 *   host_kv            full-KV pool of 8192-byte entries: mapped pinned host memory (or device memory)
 * The working set of the first sparse step is then selected and gathered by steps 1-3 as usual.
 */
int oasis_offload_blocks(const oasis_dims_t *dims, const void *dense_k, const void *dense_v,
                         const int32_t *gpu_table, const int32_t *block_table,
                         const int32_t *first_block, const int32_t *n_blocks, int32_t max_new_blocks,
                         void *host_kv, void *summaries, void *stream);

/*
 * Step 1 -- block scores from the lookahead (draft) queries (Sec. 4.2.1: each draft query
 * scans the summaries and ranks all logical blocks independently for every KV head).
 * For one query row q and block j the estimate is the upper bound that min/max summaries
 * admit, U(q, j) = sum_x max(q_x * min_jx, q_x * max_jx), accumulated in fp32.  The
 * n_draft * (Hq/Hkv) rows that share KV head h are reduced with max (OASIS_REDUCE_MAX) or
 * sum (OASIS_REDUCE_SUM).
 *   q_draft        draft queries, bf16, element (b, t, a, x) at
 *                  q_draft[b * q_batch_stride + (t * Hq + a) * 128 + x]; q_batch_stride is
 *                  in elements, a multiple of 8 (n_draft*Hq*128 when dense; larger when
 *                  the drafts are a view into the stacked verify-step queries)
 *   n_full_blocks  [B] int32 (device): blocks j < n_full_blocks[b] are candidates
 *   scores         [B][Hkv][max_blocks] fp32; -inf for j >= n_full_blocks[b]
 * n_draft * (Hq/Hkv) may not exceed 128.
 */
int oasis_score_blocks(const oasis_dims_t *dims, const void *q_draft, int64_t q_batch_stride,
                       int32_t n_draft, const void *summaries, const int32_t *n_full_blocks,
                       int32_t reduce_mode, float *scores, void *stream);

/*
 * Step 2 -- top-k blocks per (request, KV head) plus the always-kept local blocks
 * (Sec. 5.2: K selected blocks and the active local block; no sink tokens).
 * With K_eff = min(k, n_full_blocks[b]):
 *   sel[b][h][0 .. K_eff)   block ids by descending score, equal scores by ascending id
 *   sel[b][h][K_eff .. k)   -1
 *   sel[b][h][k], [k+1]     the local blocks n_full_blocks[b] .. ceil((seq_len[b] +
 *                           n_q_tokens) / 16) - 1 (at most two), else -1
 * Scores are compared as fp32; -0 equals +0; NaN is not supported.
 * Optional gather lists (both NULL, or both given), one request per sel column:
 *   stage_idx   [B][Hkv][k+2] int64: block_table[b][sel] * Hkv + h, or -1 for a -1 column
 *   stage_slots [B][Hkv][k+2] int32: (b * Hkv + h) * (k + 2) + column
 *   seq_len     [B] int32 (device): history tokens before this step
 * 1 <= k <= OASIS_MAX_K; max_blocks <= 49152.
 */
int oasis_select_topk(const oasis_dims_t *dims, const float *scores,
                      const int32_t *n_full_blocks, const int32_t *seq_len,
                      int32_t n_q_tokens, int32_t k, const int32_t *block_table, int32_t *sel,
                      int64_t *stage_idx, int32_t *stage_slots, void *stream);

/*
 * Step 3 -- gather of selected entries from the host-resident full KV cache into HBM
 * slots (Sec. 5.1: a gather kernel reads the selected block-head entries from the pinned
 * CPU cache through unified addressing and writes them into the resident GPU pages).
 *   hbm_pool[slots[i]] = host_kv[idx[i]]   for i < n, 8192-byte entries; idx[i] < 0: skip
 *   host_kv   full-KV pool: pinned host memory mapped for the device (or device memory)
 *   idx       [n] int64 (device), slots [n] int32 (device); two requests must not name
 *             the same slot
 * Typically enqueued on a side stream so that it overlaps other layers' compute.
 */
int oasis_stage_blocks(const void *host_kv, const int64_t *idx, const int32_t *slots,
                       int32_t n, void *hbm_pool, void *stream);

/*
 * Step 3 for several layers in one launch: the same as one oasis_stage_blocks call per layer with that layer's
 * pool, lists (each of length n) and working-set pool (host arrays of n_layers <= OASIS_MAX_STAGE_LAYERS device
 * pointers).  A few large gathers keep the host link busier than many small ones.
 *   max_ctas   thread blocks of the launch (each keeps 64 KiB of reads in flight); 0 = the library's default of
 *              64, which is what the host link of a B200 takes before its rate drops.  A small value makes a
 *              low-intensity copy that can run beside another gather (e.g. the upload of a step's queries).
 */
#define OASIS_MAX_STAGE_LAYERS 64
int oasis_stage_blocks_layers(int32_t n_layers, const void *const *host_kvs, const int64_t *const *idx,
                              const int32_t *const *slots, int32_t n, void *const *hbm_pools, int32_t max_ctas,
                              void *stream);

/*
 * Step 3 for several layers in one launch, through the copy unit: the same result as oasis_stage_blocks_layers, but the
 * entries move as 8 KiB bulk copies (CPU pool -> shared memory -> working-set pool) issued by one thread of a
 * small thread block per entry stream, so that the gather runs beside kernels that fill the SMs (the fused
 * attention + scoring launch) without competing for their issue slots.  Faster than the warp-per-entry gather where
 * the host link bounds the decode step and also carries the step's query uploads; no better otherwise.  A copy that does not complete within
 * the library's bounded wait records code 71 in the error word.
 *   max_streams   entry streams (thread blocks) of the launch, shared among the layers, each with one 8 KiB copy
 *                 in flight; 0 = the library's default of 128 (1 MiB in flight).
 */
int oasis_stage_blocks_bulk(int32_t n_layers, const void *const *host_kvs, const int64_t *const *idx,
                            const int32_t *const *slots, int32_t n, void *const *hbm_pools,
                            int32_t max_streams, void *stream);

/*
 * Step 4 -- sparse paged decode attention over the staged working set (Sec. 4.2.1: the
 * stacked normal and draft queries run over one resident KV working set in one call;
 * Sec. 4.3: the selected key and value blocks share one ordering).
 * Query token t of request b sits at position seq_len[b] + t.  For KV head h the keys are
 * the tokens i of every column c with blk_tbl[b][h][c] = j >= 0 whose position
 * j * 16 + i <= seq_len[b] + t, read from entry slot_tbl[b][h][c] of hbm_pool.
 * out = softmax(scale * q K^T) V with bf16 tensor-core products and fp32 accumulation.
 *   q, out      [B][n_q_tokens][Hq][128] bf16
 *   slot_tbl, blk_tbl   [B][Hkv][n_cols] int32 (device)
 *   lse         optional [B][n_q_tokens][Hq] fp32: natural-log sum of exponentials
 *   workspace   device scratch of at least oasis_attn_workspace_bytes() bytes, 16-byte
 *               aligned; its contents need no initialisation and are undefined afterwards.
 *               May be NULL when that function returns 0.
 * n_q_tokens * (Hq/Hkv) may not exceed 128.  A query row that sees no key yields zeros
 * (lse = -inf).
 * Every byte of an entry named by a column with blk_tbl >= 0 must be a finite bf16 pattern, also the
 * token rows that lie past the visible positions (the unwritten tail of the local block): masked keys
 * enter the P V product with weight zero, and 0 x NaN or 0 x Inf is NaN.  A pool that was zeroed
 * once and only ever receives real keys and values satisfies this.
 */
int oasis_sparse_attn(const oasis_dims_t *dims, const void *q, int32_t n_q_tokens,
                      const void *hbm_pool, const int32_t *slot_tbl, const int32_t *blk_tbl,
                      int32_t n_cols, const int32_t *seq_len, float scale, void *out,
                      float *lse, void *workspace, size_t workspace_bytes, void *stream);

/* Scratch bytes oasis_sparse_attn needs for these shapes on the current device. */
size_t oasis_attn_workspace_bytes(const oasis_dims_t *dims, int32_t n_q_tokens,
                                  int32_t n_cols);

/*
 * Steps 4 and 1 of one layer in a single launch (Sec. 4.2.2: a layer's attention over the working set
 * staged by the previous step and its look-ahead scoring for the next step are independent).  Same
 * arguments, arithmetic and results as oasis_sparse_attn (q .. lse) followed by oasis_score_blocks
 * (q_draft .. scores).  One persistent thread block per SM scores its share of the layer's blocks and
 * attends (request, KV head) rows c, c + SMs, c + 2 SMs, ... over the same shared-memory ring, the
 * shares sized so that every SM moves the same number of bytes.  With B * Hkv <= SMs / 2 and rows too
 * long to be attended whole, the column lists are split as oasis_sparse_attn splits them, each split a
 * work item, and a second, small launch merges the parts: pass a `workspace` of
 * oasis_attn_workspace_bytes() bytes (16-byte aligned, contents undefined before and after; may be
 * NULL where that is 0).
 * Only shapes with  n_q_tokens * (Hq/Hkv) <= 128,  n_draft * (Hq/Hkv) <= 64  and a shared-memory
 * footprint within 227 KiB are taken (oasis_attn_and_score_supported tells); others
 * return OASIS_ERR_UNSUPPORTED: make the two calls.
 *   q_batch_stride   elements between consecutive requests of q_draft (0 = dense)
 * Stream ordering.  The kernel is launched with programmatic stream serialization and its scoring phase
 * runs before it waits for the previous launch of `stream`: q_draft, summaries, n_full_blocks and seq_len
 * are read, and scores written, while that previous launch may still be running, and the launch after this
 * one may start as soon as this one has begun.  So the previous launch on `stream` must neither produce
 * those inputs nor still use `scores` (an oasis_attn_and_score of another layer is the intended
 * predecessor; it, oasis_sparse_attn and their merge launches are the launches of this library that let
 * a successor start early); separate such producers and consumers from this call by an event on another
 * stream or by another launch in between.  Everything the attention phase touches (q,
 * hbm_pool, the tables, out, lse, workspace) is ordered as usual.
 */
int oasis_attn_and_score(const oasis_dims_t *dims, const void *q, int32_t n_q_tokens, const void *hbm_pool,
                         const int32_t *slot_tbl, const int32_t *blk_tbl, int32_t n_cols,
                         const int32_t *seq_len, float scale, void *out, float *lse, const void *q_draft,
                         int64_t q_batch_stride, int32_t n_draft, const void *summaries,
                         const int32_t *n_full_blocks, int32_t reduce_mode, float *scores, void *workspace,
                         size_t workspace_bytes, void *stream);

/* 1 if oasis_attn_and_score takes these shapes on the current device, else 0. */
int oasis_attn_and_score_supported(const oasis_dims_t *dims, int32_t n_q_tokens, int32_t n_cols,
                                   int32_t n_draft);

/*
 * Sparse attention with built-in scratch memory.  (This entry point has no counterpart in the
 * paper: it is a packaging variant of step 4.)
 * Same computation, arguments and results as oasis_sparse_attn, but the caller passes no
 * workspace: the split-KV partials go to a fixed array of oasis_static_scratch_bytes() bytes
 * (4 MiB) that is part of the library image, so every GPU that loads the library holds that
 * much memory until the process exits.  It is meant for callers that cannot provide scratch
 * memory themselves -- an engine that gave all free device memory to its KV-cache pool at
 * start-up, or a decode loop that must not call cudaMalloc (it can fail at that point and it
 * synchronises the device).  The call allocates and frees nothing.
 *   - Shapes whose partials need more than the array holds are rejected with
 *     OASIS_ERR_WORKSPACE (the message states both sizes); use oasis_sparse_attn for those.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call before any stream capture begins.
 *   - All calls share the one array.  It keeps whatever the previous call left in it, which is
 *     harmless (every partial is written before it is read), but two calls whose kernels
 *     overlap on the GPU (different streams) race on it: serialise them.
 */
int oasis_sparse_attn_static_scratch(const oasis_dims_t *dims, const void *q, int32_t n_q_tokens,
                                     const void *hbm_pool, const int32_t *slot_tbl,
                                     const int32_t *blk_tbl, int32_t n_cols,
                                     const int32_t *seq_len, float scale, void *out, float *lse,
                                     void *stream);

/* Size in bytes of the built-in scratch array used by oasis_sparse_attn_static_scratch. */
size_t oasis_static_scratch_bytes(void);

/*
 * KV selection stage -- delta selection with capped eviction (Sec. 4.2.3; the cap is a
 * fraction of K, Sec. 5.5.1: cap = floor(ratio * K)).  Each (b, h) row owns n_res resident
 * columns: resident[b][h][c] is the logical block held in column c (-1 = empty) and
 * stamp[b][h][c] the step at which it was last selected.  With pred = sel[b][h][0..k):
 *   1. a resident block that is in pred stays in place; its stamp becomes `step`;
 *   2. the predicted blocks that are not resident are the candidates, in rank order;
 *   3. the columns whose block is not in pred are eviction targets, least recently
 *      selected first (empty columns first; equal stamps by ascending column);
 *   4. candidate i replaces target i for i < min(cap, #candidates, #targets): the column
 *      takes the block and stamp `step`, and a gather request is emitted:
 *      plan_idx = block_table[b][block] * Hkv + h, plan_slots = row * slot_stride + column
 *      with row = b * Hkv + h.  All other columns are left unchanged.
 *   5. the n_local (0..2) always-kept local blocks sel[b][h][k .. k+n_local) (Sec. 4.3:
 *      the selected blocks and a local window stay in GPU memory) are copied to columns
 *      n_res .. n_res+n_local-1 of the row, stamps untouched, and requested unconditionally.
 *   sel         [B][Hkv][sel_cols] int32, k + n_local <= sel_cols
 *   resident, stamp   [B][Hkv][res_stride] int32, updated in place, res_stride >= n_res +
 *               n_local; with res_stride = n_res + n_local, resident is directly the blk_tbl
 *               of oasis_sparse_attn
 *   plan_idx [B][Hkv][cap + n_local] int64, plan_slots (same shape) int32: the pairs first,
 *               then the local blocks; unused requests have idx = -1
 *   n_admitted  [B][Hkv] int32 number of pairs (may be NULL)
 * 1 <= k <= OASIS_MAX_K, 1 <= n_res <= OASIS_MAX_K, 0 <= cap <= k, slot_stride >= n_res +
 * n_local, max_blocks <= 524288.
 */
int oasis_plan_delta(const oasis_dims_t *dims, const int32_t *sel, int32_t sel_cols, int32_t k,
                     const int32_t *block_table, int32_t *resident, int32_t *stamp,
                     int32_t n_res, int32_t res_stride, int32_t n_local, int32_t slot_stride,
                     int32_t cap, int32_t step, int64_t *plan_idx, int32_t *plan_slots,
                     int32_t *n_admitted, void *stream);

/*
 * Local window (Sec. 4.3: the selected blocks and a local window stay in GPU memory; Sec. 5.2: the active
 * local block is kept on top of the K selected blocks).  With L = seq_len[b] and T = n_q_tokens (1..16),
 * the step's tokens sit at positions L .. L+T-1, in the local blocks lo = L / 16 .. hi = (L+T-1) / 16 (at
 * most two).  Local block j lives in column local_col + (j & 1) of its (request, KV head) row, so a block
 * keeps its column, and with it its slot, for as long as it is local.
 * oasis_local_window sets   blk_tbl[b][h][local_col + (lo & 1)] = lo   and the other local column to hi
 * (if hi > lo) or -1, and leaves every other column alone.  Optionally (both lists, or both NULL) it emits
 * two gather requests per row that load the local blocks from the CPU pool with oasis_stage_blocks -- used
 * once, when a request enters sparse decoding with a partially filled block:
 *   stage_idx   [B][Hkv][2] int64: block_table[b][j] * Hkv + h for the block j of column local_col + r, or -1
 *   stage_slots [B][Hkv][2] int32: (b * Hkv + h) * slot_stride + local_col + r
 */
int oasis_local_window(const oasis_dims_t *dims, const int32_t *seq_len, int32_t n_q_tokens,
                       const int32_t *block_table, int32_t *blk_tbl, int32_t n_cols, int32_t local_col,
                       int32_t slot_stride, int64_t *stage_idx, int32_t *stage_slots, void *stream);

/*
 * KV append of one decode step.  The paper keeps the newest tokens in the GPU-resident local window (Sec. 4.3,
 * 5.2) and does not say how they reach the CPU pool; this library writes them through: the step's tokens are
 * produced on the GPU and go straight into the local window, and the tokens the step commits are also stored
 * into the CPU full-KV pool, so that a block that fills up is complete there and is summarised, selected and
 * gathered like any other.  The local blocks therefore never cross the host link towards the GPU.
 *   1. the local columns of blk_tbl are set as by oasis_local_window;
 *   2. token t < n_q_tokens of request b, KV head h (key row, then value row, of new_kv) is written to row
 *      (L + t) % 16 of the K part and of the V part of entry slot_tbl[b][h][local_col + (j & 1)] of hbm_pool,
 *      j = (L + t) / 16;
 *   3. the first n_commit tokens are also written to the same rows of entry (block_table[b][j], h) of host_kv.
 *   new_kv      [B][n_q_tokens][Hkv][2][128] bf16 (device)
 *   slot_tbl    [B][Hkv][n_cols] int32 (device), blk_tbl the same shape, updated in place
 *   host_kv     the CPU full-KV pool (mapped pinned memory, or device memory); may be NULL when n_commit = 0
 * Rows of a local entry that earlier steps wrote are left as they are.  1 <= n_q_tokens <= 16,
 * 0 <= n_commit <= n_q_tokens, local_col + 2 <= n_cols.
 * oasis_append_kv_layers does the same for n_layers <= OASIS_MAX_APPEND_LAYERS layers in one launch (host
 * arrays of per-layer device pointers; seq_len is shared, as a step appends the same positions in every layer).
 */
int oasis_append_kv(const oasis_dims_t *dims, const void *new_kv, int32_t n_q_tokens, int32_t n_commit,
                    const int32_t *seq_len, const int32_t *block_table, const int32_t *slot_tbl,
                    int32_t *blk_tbl, int32_t n_cols, int32_t local_col, void *hbm_pool, void *host_kv,
                    void *stream);

#define OASIS_MAX_APPEND_LAYERS 64
int oasis_append_kv_layers(const oasis_dims_t *dims, int32_t n_layers, const void *const *new_kv,
                           int32_t n_q_tokens, int32_t n_commit, const int32_t *seq_len,
                           const int32_t *const *block_tables, const int32_t *const *slot_tbls,
                           int32_t *const *blk_tbls, int32_t n_cols, int32_t local_col,
                           void *const *hbm_pools, void *const *host_kvs, void *stream);

/*
 * Head-union block set (Sec. 4.4.1, partial transfer: per layer the per-head selected sets are
 * united at block granularity -- a block is included if at least one KV head selected it -- and
 * the index of every included block is sent with its data).
 *   sel         [B][Hkv][sel_cols] int32; columns [0, k) of every head take part, negative = none
 *   union_idx   [B][max_union] int32: the distinct block ids of request b in ascending order,
 *               then -1; ids beyond max_union are dropped
 *   n_union     [B] int32: size of the union (also when it exceeds max_union)
 * 1 <= k <= sel_cols, max_union >= 1, max_blocks <= 1048576.
 */
int oasis_union_blocks(const oasis_dims_t *dims, const int32_t *sel, int32_t sel_cols, int32_t k,
                       int32_t max_union, int32_t *union_idx, int32_t *n_union, void *stream);

/*
 * Registers a device word (int32, zero-initialised by the caller, or NULL to unregister) in
 * which kernels record a non-zero code if one of their internal waits (on a shared-memory
 * barrier of an asynchronous copy or tensor-core operation) runs out of its iteration bound.
 * Such a kernel stops working and returns; its outputs are then undefined.  The word is
 * process-wide and is only ever written with a compare-and-swap from zero.
 */
int oasis_set_error_word(int32_t *device_word);

/*
 * Bounds-check build (no counterpart in the paper: a debugging aid of this library).  The library also builds
 * with -DOASIS_BOUNDS_CHECK (liboasis_checked.so).  In that build every index that a kernel reads from a device
 * array is range-checked on the device before use: entries of the full-KV pool (block_table[..] * Hkv + h, idx[])
 * against n_host_entries, slots (slots[], slot_tbl[..], computed plan slots) against n_slots, logical block ids
 * against dims->max_blocks, per-request block counts and ranges against dims->max_blocks.  A violation writes
 * its code into the error word registered with oasis_set_error_word (the first violation wins: 201 host entry,
 * 202 slot, 203 block id, 204 block count) and the access is skipped -- the request is dropped, the column is
 * treated as missing, the count is clamped; nothing traps or asserts.  The attention's tensor map then also
 * declares the pool's real extent.  oasis_set_extents declares the two extents (process-wide, like the error
 * word; 0 = unknown = unchecked); in the regular build it is accepted and has no effect.
 * oasis_bounds_checked() tells which build is loaded (1 = checked).
 */
int oasis_set_extents(int64_t n_host_entries, int64_t n_slots);
int oasis_bounds_checked(void);

/*
 * Self-test of the bounded waits behind oasis_set_error_word (no counterpart in the paper).  One small
 * launch waits, with a bound of `probes` polls (1 .. 2^20), on a barrier that nothing ever completes; the
 * wait gives up, the kernel records code 99 in the registered error word (if one is registered and still
 * zero), releases what it holds and returns -- the path the real kernels take when a copy or tensor-core
 * operation never signals.  result (device, int32[2], may be NULL) receives {1 if the wait gave up else 0,
 * the code}.  Nothing is left in flight; later calls work as usual.
 */
int oasis_selftest_wait_timeout(uint32_t probes, int32_t *result, void *stream);

/* Description of the calling thread's most recent error ("" if none). Static storage. */
const char *oasis_last_error(void);

/* Library version, "major.minor". */
const char *oasis_version(void);

#ifdef __cplusplus
}
#endif
#endif /* OASIS_H */
