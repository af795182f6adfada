/*
 * oasis_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded CPU statement of the per-decode-step hot path of
 * OasisKV (lookahead sparse KV prefetching): block summaries, block scoring with the
 * draft queries, per-head top-k selection, the host->HBM block gather, sparse paged
 * attention, and the delta/capped-eviction transfer plan.  It exists so that the CUDA
 * library can be checked against something written independently from the paper; it
 * shares no code, header or table with the CUDA path and must never be called from
 * the product path.  Only tests, the smoke check and the benchmark's CPU-baseline leg
 * may use it.
 *
 * Arithmetic: floating point is done in fp32 with contraction disabled
 * (-ffp-contract=off), in the order written below, with an optional fp64 shadow of
 * every score and attention output that the tests use for adjudication.  bf16 values
 * travel as raw uint16 bit patterns.
 *
 * Layouts (all row-major, innermost index last; bs = tokens per block, d = head dim):
 *   KV pool      [n_phys_blocks][Hkv][2][bs][d] bf16  -- "Head-Token-Dimension" order
 *                (Sec. 4.3); index 2 = {K part, V part}; one (block, head) "entry" is
 *                2*bs*d contiguous elements.
 *   block_table  [B][max_blocks] int32   logical block -> physical block (Sec. 4.3)
 *   summaries    [B][Hkv][max_blocks][2][d] bf16, row 0 = min, row 1 = max (Sec. 4.2.1)
 *   scores       [B][Hkv][max_blocks] fp32
 *   sel          [B][Hkv][k+2] int32
 *   q            [B][T][Hq][d] bf16; query head a uses KV head a / (Hq/Hkv)
 *
 * Parity pins: every function here is pinned by tests/test_oracle_pins.py (brute
 * force on tiny inputs, invariants, closed forms, library cross-checks).  The CHOICE
 * of estimator in oasis_oracle_score_blocks (the Quest upper bound) and of the
 * reduction over the query rows sharing a KV head is a reading of Sec. 4.2.1, which
 * names the summaries but prints no formula: beyond its invariants that choice is
 * "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---------------------------------------------------------------- bf16 helpers */

static float bf16_to_f32(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* round-to-nearest-even; inputs are finite in every use below */
static uint16_t f32_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u); /* NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

void oasis_oracle_f32_to_bf16(const float *src, uint16_t *dst, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) dst[i] = f32_to_bf16(src[i]);
}

void oasis_oracle_bf16_to_f32(const uint16_t *src, float *dst, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) dst[i] = bf16_to_f32(src[i]);
}

/* ---------------------------------------------------------------- step 0: summaries
 * Sec. 4.2.1 (per logical block and KV head, one summary row holds the smallest and one
 * the largest value of every key coordinate), Fig. "Look-ahead attention" (min/max pooling),
 * Sec. 5.2 (two summary rows per block = 1/16 of the KV size, hence bf16 like the KV).
 * For request b, logical blocks first_block[b] .. first_block[b]+n_blocks[b]-1.
 */
void oasis_oracle_build_summaries(int32_t B, int32_t Hkv, int32_t d, int32_t bs,
                                  int32_t max_blocks, const uint16_t *kv_pool,
                                  const int32_t *block_table, const int32_t *first_block,
                                  const int32_t *n_blocks, uint16_t *summaries)
{
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t j = first_block[b]; j < first_block[b] + n_blocks[b]; ++j) {
            int64_t phys = block_table[(int64_t)b * max_blocks + j];
            for (int32_t h = 0; h < Hkv; ++h) {
                const uint16_t *kpart = kv_pool + ((phys * Hkv + h) * 2 + 0) * (int64_t)bs * d;
                uint16_t *row_min = summaries + ((((int64_t)b * Hkv + h) * max_blocks + j) * 2 + 0) * d;
                uint16_t *row_max = row_min + d;
                for (int32_t x = 0; x < d; ++x) {
                    uint16_t lo = kpart[x], hi = kpart[x];
                    for (int32_t i = 1; i < bs; ++i) {
                        uint16_t v = kpart[(int64_t)i * d + x];
                        if (bf16_to_f32(v) < bf16_to_f32(lo)) lo = v;
                        if (bf16_to_f32(v) > bf16_to_f32(hi)) hi = v;
                    }
                    row_min[x] = lo;
                    row_max[x] = hi;
                }
            }
        }
    }
}

/* ---------------------------------------------------------------- step 1: scores
 * Sec. 4.2.1: the draft queries are compared with every block's summary, separately for
 * each KV head, and the blocks are ranked by the result.  The estimate for one query row q and block j is
 * the Quest upper bound  U(q, j) = sum_x max(q_x * min_jx, q_x * max_jx), summed over
 * x ascending.  The Td draft tokens and the G = Hq/Hkv query heads that share KV head
 * h give R = Td*G rows; they are reduced with max (reduce_mode 0) or sum (1), rows
 * visited in (t, g) order.  Candidate blocks are the full ones, j < n_full[b]; every
 * other j gets -inf.  scores64 (optional) is the same in double precision.
 */
void oasis_oracle_score_blocks(int32_t B, int32_t Hq, int32_t Hkv, int32_t d,
                               int32_t max_blocks, const uint16_t *q_draft, int32_t Td,
                               const uint16_t *summaries, const int32_t *n_full,
                               int32_t reduce_mode, float *scores, double *scores64)
{
    const int32_t G = Hq / Hkv;
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t h = 0; h < Hkv; ++h) {
            for (int32_t j = 0; j < max_blocks; ++j) {
                int64_t o = ((int64_t)b * Hkv + h) * max_blocks + j;
                if (j >= n_full[b]) {
                    scores[o] = -INFINITY;
                    if (scores64) scores64[o] = -INFINITY;
                    continue;
                }
                const uint16_t *row_min = summaries + (o * 2 + 0) * d;
                const uint16_t *row_max = row_min + d;
                float s = 0.0f;
                double s64 = 0.0;
                for (int32_t t = 0; t < Td; ++t) {
                    for (int32_t g = 0; g < G; ++g) {
                        const uint16_t *q = q_draft + (((int64_t)b * Td + t) * Hq + (h * G + g)) * d;
                        float u = 0.0f;
                        double u64 = 0.0;
                        for (int32_t x = 0; x < d; ++x) {
                            float qx = bf16_to_f32(q[x]);
                            float a = qx * bf16_to_f32(row_min[x]);
                            float c = qx * bf16_to_f32(row_max[x]);
                            float m = a > c ? a : c;
                            u = u + m;
                            u64 = u64 + (double)m; /* products of two bf16 are exact in fp32 */
                        }
                        if (t == 0 && g == 0) {
                            s = u;
                            s64 = u64;
                        } else if (reduce_mode == 0) {
                            if (u > s) s = u;
                            if (u64 > s64) s64 = u64;
                        } else {
                            s = s + u;
                            s64 = s64 + u64;
                        }
                    }
                }
                scores[o] = s;
                if (scores64) scores64[o] = s64;
            }
        }
    }
}

/* ---------------------------------------------------------------- step 2: top-k
 * Sec. 5.2: K blocks are selected per KV head and the active local block is kept on
 * top of them (K + 1 blocks, no sink tokens, no dense layer).  For each (b, h):
 * K_eff = min(k, n_full[b]); rank r takes the largest score not yet taken, the lowest
 * block index among equals; then the local block ids n_full[b] .. ceil((L+T)/bs)-1
 * (at most two) fill columns k and k+1; every unused column is -1.  When stage_idx /
 * stage_slots are given, column c of row (b,h) is also written as a gather request:
 * source entry block_table[b][j]*Hkv + h, destination slot (b*Hkv+h)*(k+2)+c, and -1
 * as the source of an unused column.
 */
void oasis_oracle_select_topk(int32_t B, int32_t Hkv, int32_t max_blocks, int32_t bs,
                              const float *scores, const int32_t *n_full,
                              const int32_t *seq_len, int32_t n_q_tokens, int32_t k,
                              const int32_t *block_table, int32_t *sel,
                              int64_t *stage_idx, int32_t *stage_slots)
{
    const int32_t cols = k + 2;
    uint8_t *taken = (uint8_t *)malloc((size_t)(max_blocks > 0 ? max_blocks : 1));
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t h = 0; h < Hkv; ++h) {
            const float *s = scores + ((int64_t)b * Hkv + h) * max_blocks;
            int32_t *row = sel + ((int64_t)b * Hkv + h) * cols;
            int32_t nf = n_full[b];
            int32_t k_eff = k < nf ? k : nf;
            memset(taken, 0, (size_t)(max_blocks > 0 ? max_blocks : 1));
            for (int32_t c = 0; c < cols; ++c) row[c] = -1;
            for (int32_t r = 0; r < k_eff; ++r) {
                int32_t best = -1;
                for (int32_t j = 0; j < nf; ++j) {
                    if (taken[j]) continue;
                    if (best < 0 || s[j] > s[best]) best = j;
                }
                taken[best] = 1;
                row[r] = best;
            }
            int32_t end_block = (seq_len[b] + n_q_tokens + bs - 1) / bs; /* exclusive */
            int32_t c = k;
            for (int32_t j = nf; j < end_block && c < cols; ++j) row[c++] = j;
            if (stage_idx && stage_slots) {
                for (int32_t cc = 0; cc < cols; ++cc) {
                    int64_t o = ((int64_t)b * Hkv + h) * cols + cc;
                    stage_slots[o] = (int32_t)o;
                    stage_idx[o] = row[cc] < 0
                                       ? -1
                                       : (int64_t)block_table[(int64_t)b * max_blocks + row[cc]] * Hkv + h;
                }
            }
        }
    }
    free(taken);
}

/* ---------------------------------------------------------------- step 3: gather
 * Sec. 5.1: the gather reads the selected block-head entries from the pinned host
 * cache and writes them into the resident GPU pages.  pool[slots[i]] = host_kv[idx[i]]
 * for i < n, entries of entry_bytes bytes; idx[i] < 0 is skipped.
 */
void oasis_oracle_stage_blocks(const uint8_t *host_kv, const int64_t *idx,
                               const int32_t *slots, int32_t n, int64_t entry_bytes,
                               uint8_t *pool)
{
    for (int32_t i = 0; i < n; ++i) {
        if (idx[i] < 0) continue;
        memcpy(pool + (int64_t)slots[i] * entry_bytes, host_kv + idx[i] * entry_bytes,
               (size_t)entry_bytes);
    }
}

/* ---------------------------------------------------------------- step 4: attention
 * Sec. 4.2.1: the attention takes the stacked normal and draft queries over one
 * resident working set and returns all outputs in one call; Sec. 4.3: the selected
 * key and value blocks share one ordering, so it is ordinary softmax attention over
 * the working set.  For request b, query token t (position seq_len[b] + t) and query
 * head a (KV head h = a / G): the keys are the tokens i of every column c with
 * blk_tbl[b][h][c] = j >= 0 whose position j*bs + i is <= seq_len[b] + t, read from
 * pool slot slot_tbl[b][h][c].  Logit = (q . k) * scale, dot product over x ascending;
 * two-pass softmax (max, then exp and sum); out = sum_p softmax_p * v_p.
 * out32 [B][T][Hq][d] fp32, out64 the same in double, out_bf16 = RNE(out32),
 * lse [B][T][Hq] = max + log(sum) (natural log).  Any output pointer may be NULL.
 * A row that sees no key gets zeros and lse = -inf.
 * out_abs [B][T][Hq][d] (optional, double) = sum_p softmax_p * |v_p|: the scale of the terms behind each
 * output element.  It is not part of the method; the parity tests use it to bound what rounding the
 * softmax weights to 8 significant bits (a tensor-core operand format) can do to an output element.
 */
void oasis_oracle_sparse_attn_abs(int32_t B, int32_t T, int32_t Hq, int32_t Hkv, int32_t d,
                                  int32_t bs, const uint16_t *q, const uint16_t *pool,
                                  const int32_t *slot_tbl, const int32_t *blk_tbl,
                                  int32_t n_cols, const int32_t *seq_len, float scale,
                                  float *out32, double *out64, uint16_t *out_bf16, float *lse,
                                  double *out_abs);

void oasis_oracle_sparse_attn(int32_t B, int32_t T, int32_t Hq, int32_t Hkv, int32_t d,
                              int32_t bs, const uint16_t *q, const uint16_t *pool,
                              const int32_t *slot_tbl, const int32_t *blk_tbl,
                              int32_t n_cols, const int32_t *seq_len, float scale,
                              float *out32, double *out64, uint16_t *out_bf16, float *lse)
{
    oasis_oracle_sparse_attn_abs(B, T, Hq, Hkv, d, bs, q, pool, slot_tbl, blk_tbl, n_cols, seq_len, scale,
                                 out32, out64, out_bf16, lse, NULL);
}

void oasis_oracle_sparse_attn_abs(int32_t B, int32_t T, int32_t Hq, int32_t Hkv, int32_t d,
                                  int32_t bs, const uint16_t *q, const uint16_t *pool,
                                  const int32_t *slot_tbl, const int32_t *blk_tbl,
                                  int32_t n_cols, const int32_t *seq_len, float scale,
                                  float *out32, double *out64, uint16_t *out_bf16, float *lse,
                                  double *out_abs)
{
    const int32_t G = Hq / Hkv;
    const int64_t max_keys = (int64_t)n_cols * bs;
    float *logit = (float *)malloc(sizeof(float) * (size_t)(max_keys > 0 ? max_keys : 1));
    double *logit64 = (double *)malloc(sizeof(double) * (size_t)(max_keys > 0 ? max_keys : 1));
    const uint16_t **vrow = (const uint16_t **)malloc(sizeof(void *) * (size_t)(max_keys > 0 ? max_keys : 1));
    float *acc = (float *)malloc(sizeof(float) * (size_t)d);
    double *acc64 = (double *)malloc(sizeof(double) * (size_t)d);
    double *accabs = (double *)malloc(sizeof(double) * (size_t)d);

    for (int32_t b = 0; b < B; ++b) {
        for (int32_t t = 0; t < T; ++t) {
            for (int32_t a = 0; a < Hq; ++a) {
                const int32_t h = a / G;
                const uint16_t *qv = q + (((int64_t)b * T + t) * Hq + a) * d;
                const int32_t *slots = slot_tbl + ((int64_t)b * Hkv + h) * n_cols;
                const int32_t *blks = blk_tbl + ((int64_t)b * Hkv + h) * n_cols;
                const int64_t limit = (int64_t)seq_len[b] + t; /* last visible position */
                int64_t nk = 0;
                for (int32_t c = 0; c < n_cols; ++c) {
                    if (blks[c] < 0) continue;
                    const uint16_t *entry = pool + (int64_t)slots[c] * 2 * bs * d;
                    for (int32_t i = 0; i < bs; ++i) {
                        if ((int64_t)blks[c] * bs + i > limit) continue;
                        const uint16_t *kv = entry + (int64_t)i * d;
                        float s = 0.0f;
                        double s64 = 0.0;
                        for (int32_t x = 0; x < d; ++x) {
                            float p = bf16_to_f32(qv[x]) * bf16_to_f32(kv[x]);
                            s = s + p;
                            s64 = s64 + (double)p;
                        }
                        logit[nk] = s * scale;
                        logit64[nk] = s64 * (double)scale;
                        vrow[nk] = entry + (int64_t)bs * d + (int64_t)i * d;
                        ++nk;
                    }
                }
                const int64_t o = (((int64_t)b * T + t) * Hq + a);
                if (nk == 0) {
                    for (int32_t x = 0; x < d; ++x) {
                        if (out32) out32[o * d + x] = 0.0f;
                        if (out64) out64[o * d + x] = 0.0;
                        if (out_bf16) out_bf16[o * d + x] = 0;
                        if (out_abs) out_abs[o * d + x] = 0.0;
                    }
                    if (lse) lse[o] = -INFINITY;
                    continue;
                }
                float mx = logit[0];
                double mx64 = logit64[0];
                for (int64_t p = 1; p < nk; ++p) {
                    if (logit[p] > mx) mx = logit[p];
                    if (logit64[p] > mx64) mx64 = logit64[p];
                }
                float den = 0.0f;
                double den64 = 0.0;
                for (int32_t x = 0; x < d; ++x) {
                    acc[x] = 0.0f;
                    acc64[x] = 0.0;
                    accabs[x] = 0.0;
                }
                for (int64_t p = 0; p < nk; ++p) {
                    float w = expf(logit[p] - mx);
                    double w64 = exp(logit64[p] - mx64);
                    den = den + w;
                    den64 = den64 + w64;
                    for (int32_t x = 0; x < d; ++x) {
                        float v = bf16_to_f32(vrow[p][x]);
                        acc[x] = acc[x] + w * v;
                        acc64[x] = acc64[x] + w64 * (double)v;
                        accabs[x] = accabs[x] + w64 * fabs((double)v);
                    }
                }
                for (int32_t x = 0; x < d; ++x) {
                    float r = acc[x] / den;
                    if (out32) out32[o * d + x] = r;
                    if (out64) out64[o * d + x] = acc64[x] / den64;
                    if (out_bf16) out_bf16[o * d + x] = f32_to_bf16(r);
                    if (out_abs) out_abs[o * d + x] = accabs[x] / den64;
                }
                if (lse) lse[o] = mx + logf(den);
            }
        }
    }
    free(logit);
    free(logit64);
    free(vrow);
    free(acc);
    free(acc64);
    free(accabs);
}

/* ---------------------------------------------------------------- lookahead recall
 * Stand-in for the per-layer agreement figure of Sec. 4.2.1: the share of the top-k
 * set chosen with the draft queries that is also in the set chosen with the true
 * next-step queries, averaged over the (b, h) rows that select at least one block.
 * Both inputs are sel arrays [rows][cols]; only their first k columns are compared.
 */
double oasis_oracle_topk_recall(int32_t rows, int32_t cols, int32_t k,
                                const int32_t *sel_draft, const int32_t *sel_true)
{
    double total = 0.0;
    int32_t counted = 0;
    for (int32_t r = 0; r < rows; ++r) {
        const int32_t *a = sel_draft + (int64_t)r * cols;
        const int32_t *t = sel_true + (int64_t)r * cols;
        int32_t n_true = 0, hit = 0;
        for (int32_t i = 0; i < k; ++i) {
            if (t[i] < 0) continue;
            ++n_true;
            for (int32_t j = 0; j < k; ++j) {
                if (a[j] == t[i]) {
                    ++hit;
                    break;
                }
            }
        }
        if (n_true > 0) {
            total += (double)hit / (double)n_true;
            ++counted;
        }
    }
    return counted > 0 ? total / counted : 1.0;
}

/* ---------------------------------------------------------------- delta selection
 * Sec. 4.2.3 (delta selection and capped eviction) and Sec. 5.5.1 (the cap is a
 * fraction of K).  One (b, h) row owns n_res resident columns.  resident[c] is the
 * logical block held in column c (or -1 = empty), stamp[c] the step at which it was
 * last selected.  pred[0..k) is this step's predicted top-k in rank order (-1 = none).
 *   1. every resident block that is in pred stays in place and gets stamp = step;
 *   2. the predicted blocks that are not resident are the candidates, in rank order;
 *   3. the columns whose block is not in pred are the eviction targets, ordered by
 *      stamp ascending (least recently selected first), empty columns before any
 *      occupied one, column index ascending among equals;
 *   4. candidate i is paired with target i for i < min(cap, #candidates, #targets):
 *      resident[target] = candidate, stamp[target] = step, and the pair is emitted as
 *      a gather request (source entry block_table[b][cand]*Hkv + h, destination slot
 *      row*slot_stride + target); every other column is left unchanged.
 *   5. Sec. 4.3 keeps a local window next to the selected blocks: the n_local always-kept
 *      local block ids sel[row][k .. k+n_local) are copied to columns n_res .. n_res+n_local-1
 *      of the row (their stamps untouched) and requested unconditionally.
 * resident / stamp rows are res_stride apart (res_stride >= n_res + n_local).
 * plan_idx / plan_slots hold cap + n_local requests per row (pairs first, then the local
 * blocks), unused ones with idx = -1.  n_admitted[row] receives the number of pairs.
 */
void oasis_oracle_plan_delta(int32_t B, int32_t Hkv, int32_t max_blocks, int32_t k,
                             int32_t sel_cols, int32_t n_res, int32_t res_stride,
                             int32_t n_local, int32_t slot_stride,
                             int32_t cap, int32_t step, const int32_t *sel,
                             const int32_t *block_table, int32_t *resident,
                             int32_t *stamp, int64_t *plan_idx, int32_t *plan_slots,
                             int32_t *n_admitted)
{
    int32_t *cand = (int32_t *)malloc(sizeof(int32_t) * (size_t)(k > 0 ? k : 1));
    int32_t *target = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n_res > 0 ? n_res : 1));
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t h = 0; h < Hkv; ++h) {
            const int64_t row = (int64_t)b * Hkv + h;
            const int32_t *pred = sel + row * sel_cols;
            int32_t *res = resident + row * res_stride;
            int32_t *stp = stamp + row * res_stride;
            const int32_t plan_cols = cap + n_local;
            int32_t n_cand = 0, n_target = 0;
            /* 1 + 3a: hits keep their column; the others are eviction targets */
            for (int32_t c = 0; c < n_res; ++c) {
                int hit = 0;
                if (res[c] >= 0)
                    for (int32_t r = 0; r < k; ++r)
                        if (pred[r] == res[c]) hit = 1;
                if (hit) stp[c] = step;
                else target[n_target++] = c;
            }
            /* 3b: stable insertion sort of the targets by (empty first, stamp, column) */
            for (int32_t i = 1; i < n_target; ++i) {
                int32_t c = target[i];
                int32_t j = i - 1;
                while (j >= 0) {
                    int32_t o = target[j];
                    int64_t key_o = res[o] < 0 ? INT64_MIN : (int64_t)stp[o];
                    int64_t key_c = res[c] < 0 ? INT64_MIN : (int64_t)stp[c];
                    if (key_o > key_c) {
                        target[j + 1] = o;
                        --j;
                    } else break;
                }
                target[j + 1] = c;
            }
            /* 2: candidates in rank order */
            for (int32_t r = 0; r < k; ++r) {
                if (pred[r] < 0) continue;
                int resident_already = 0;
                for (int32_t c = 0; c < n_res; ++c)
                    if (res[c] == pred[r]) resident_already = 1;
                if (!resident_already) cand[n_cand++] = pred[r];
            }
            /* 4: pair up */
            int32_t n_pair = cap;
            if (n_cand < n_pair) n_pair = n_cand;
            if (n_target < n_pair) n_pair = n_target;
            for (int32_t i = 0; i < plan_cols; ++i) {
                plan_idx[row * plan_cols + i] = -1;
                plan_slots[row * plan_cols + i] = 0;
            }
            for (int32_t i = 0; i < n_pair; ++i) {
                int32_t c = target[i];
                res[c] = cand[i];
                stp[c] = step;
                plan_idx[row * plan_cols + i] =
                    (int64_t)block_table[(int64_t)b * max_blocks + cand[i]] * Hkv + h;
                plan_slots[row * plan_cols + i] = (int32_t)(row * slot_stride + c);
            }
            n_admitted[row] = n_pair;
            /* 5: the local window */
            for (int32_t i = 0; i < n_local; ++i) {
                int32_t j = pred[k + i];
                res[n_res + i] = j;
                plan_slots[row * plan_cols + cap + i] = (int32_t)(row * slot_stride + n_res + i);
                if (j >= 0)
                    plan_idx[row * plan_cols + cap + i] =
                        (int64_t)block_table[(int64_t)b * max_blocks + j] * Hkv + h;
            }
        }
    }
    free(cand);
    free(target);
}

/* ---------------------------------------------------------------- head-union set
 * Sec. 4.4.1 (partial transfer): per layer, the union over the KV heads of a request's
 * selected sets at block granularity -- a block is included if at least one head selected
 * it -- and the index of every included block travels with its data.
 * For request b: the distinct ids among sel[b][h][0..k) over all h (negative = none), in
 * ascending order, written to union_idx[b][0..n) and padded with -1 up to max_union;
 * n_union[b] = n (the ids beyond max_union, if any, are dropped but still counted).
 */
void oasis_oracle_union_blocks(int32_t B, int32_t Hkv, int32_t max_blocks, int32_t sel_cols,
                               int32_t k, const int32_t *sel, int32_t max_union,
                               int32_t *union_idx, int32_t *n_union)
{
    uint8_t *seen = (uint8_t *)malloc((size_t)(max_blocks > 0 ? max_blocks : 1));
    for (int32_t b = 0; b < B; ++b) {
        memset(seen, 0, (size_t)(max_blocks > 0 ? max_blocks : 1));
        for (int32_t h = 0; h < Hkv; ++h)
            for (int32_t r = 0; r < k; ++r) {
                int32_t j = sel[((int64_t)b * Hkv + h) * sel_cols + r];
                if (j >= 0 && j < max_blocks) seen[j] = 1;
            }
        int32_t n = 0;
        for (int32_t j = 0; j < max_blocks; ++j) {
            if (!seen[j]) continue;
            if (n < max_union) union_idx[(int64_t)b * max_union + n] = j;
            ++n;
        }
        for (int32_t i = n; i < max_union; ++i) union_idx[(int64_t)b * max_union + i] = -1;
        n_union[b] = n;
    }
    free(seen);
}

/* ---------------------------------------------------------------- dense -> sparse hand-over
 * Sec. 4.3: a request starts out dense (prefill and the first decode steps); when its context
 * grows past the sparsification threshold its whole KV cache is moved to the CPU pool;
 * both pools keep their blocks in Head-Token-Dimension order and each has its own page table.
 * The dense GPU pool holds keys and values separately, dense_k / dense_v [P_gpu][Hkv][bs][d];
 * the CPU pool holds one entry [K part | V part] per (block, head).  For request b and logical
 * blocks j = first_block[b] .. first_block[b] + n_blocks[b] - 1 (those below max_blocks):
 *   host_kv[(block_table[b][j] * Hkv + h)] = [ dense_k[(gpu_table[b][j] * Hkv + h)] |
 *                                              dense_v[(gpu_table[b][j] * Hkv + h)] ]
 * and, when summaries is given, the block's min / max rows are taken from the copied keys
 * exactly as in step 0.
 */
void oasis_oracle_offload_blocks(int32_t B, int32_t Hkv, int32_t d, int32_t bs, int32_t max_blocks,
                                 const uint16_t *dense_k, const uint16_t *dense_v,
                                 const int32_t *gpu_table, const int32_t *block_table,
                                 const int32_t *first_block, const int32_t *n_blocks,
                                 uint16_t *host_kv, uint16_t *summaries)
{
    const int64_t part = (int64_t)bs * d;
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t j = first_block[b]; j < first_block[b] + n_blocks[b]; ++j) {
            if (j < 0 || j >= max_blocks) continue;
            int64_t src = gpu_table[(int64_t)b * max_blocks + j];
            int64_t dst = block_table[(int64_t)b * max_blocks + j];
            for (int32_t h = 0; h < Hkv; ++h) {
                const uint16_t *k = dense_k + (src * Hkv + h) * part;
                const uint16_t *v = dense_v + (src * Hkv + h) * part;
                uint16_t *entry = host_kv + (dst * Hkv + h) * 2 * part;
                memcpy(entry, k, (size_t)part * sizeof(uint16_t));
                memcpy(entry + part, v, (size_t)part * sizeof(uint16_t));
                if (!summaries) continue;
                uint16_t *row_min = summaries + ((((int64_t)b * Hkv + h) * max_blocks + j) * 2 + 0) * d;
                uint16_t *row_max = row_min + d;
                for (int32_t x = 0; x < d; ++x) {
                    uint16_t lo = k[x], hi = k[x];
                    for (int32_t i = 1; i < bs; ++i) {
                        uint16_t t = k[(int64_t)i * d + x];
                        if (bf16_to_f32(t) < bf16_to_f32(lo)) lo = t;
                        if (bf16_to_f32(t) > bf16_to_f32(hi)) hi = t;
                    }
                    row_min[x] = lo;
                    row_max[x] = hi;
                }
            }
        }
    }
}

/* ---------------------------------------------------------------- local window and KV append
 * Sec. 4.3 keeps, next to the selected blocks, a local window in GPU memory; Sec. 5.2 calls it the
 * active local block (the block being written), kept on top of the K selected ones.  The paper does
 * not say how the newest tokens reach the CPU pool; the reading taken here is write-through: the
 * tokens a step produces are written into the local window of the GPU working set (they are produced
 * on the GPU and never cross the host link in that direction), and the ones the step commits are
 * also written to the CPU full-KV pool, so that a block that fills up is complete there and can be
 * summarised, selected and gathered like any other.
 *
 * Geometry.  With L = seq_len[b] history tokens and T verify-step tokens, token t sits at position
 * L + t, i.e. row (L + t) % bs of logical block (L + t) / bs.  The local blocks are lo = L / bs ..
 * hi = (L + T - 1) / bs (T <= bs, so at most two).  Local block j lives in column local_col + (j & 1)
 * of its (b, h) row: a block keeps its column, hence its slot, for as long as it is local, and the
 * column of the other parity is free again by the time block j + 2 needs it.
 *
 * oasis_oracle_local_window: blk_tbl[b][h][local_col + (lo & 1)] = lo; the other local column = hi
 * if hi > lo else -1.  When stage_idx / stage_slots are given ([B][Hkv][2]) request r of a row
 * (re)loads the block of column local_col + r from the CPU pool: idx = block_table[b][j] * Hkv + h
 * (-1 for an empty column), slot = row * slot_stride + local_col + r.
 */
void oasis_oracle_local_window(int32_t B, int32_t Hkv, int32_t bs, int32_t max_blocks,
                               const int32_t *seq_len, int32_t n_q_tokens,
                               const int32_t *block_table, int32_t *blk_tbl, int32_t n_cols,
                               int32_t local_col, int32_t slot_stride, int64_t *stage_idx,
                               int32_t *stage_slots)
{
    for (int32_t b = 0; b < B; ++b) {
        int32_t lo = seq_len[b] / bs;
        int32_t hi = (seq_len[b] + n_q_tokens - 1) / bs;
        for (int32_t h = 0; h < Hkv; ++h) {
            int64_t row = (int64_t)b * Hkv + h;
            int32_t *cols = blk_tbl + row * n_cols + local_col;
            cols[lo & 1] = lo;
            cols[(lo & 1) ^ 1] = hi > lo ? hi : -1;
            if (stage_idx && stage_slots) {
                for (int32_t r = 0; r < 2; ++r) {
                    int32_t j = cols[r];
                    stage_slots[row * 2 + r] = (int32_t)(row * slot_stride + local_col + r);
                    stage_idx[row * 2 + r] =
                        j < 0 ? -1 : (int64_t)block_table[(int64_t)b * max_blocks + j] * Hkv + h;
                }
            }
        }
    }
}

/* oasis_oracle_append_kv: the KV append of one decode step.
 * new_kv [B][T][Hkv][2][d] bf16: key row then value row of token t for KV head h.
 *   1. the local columns of blk_tbl are set as in oasis_oracle_local_window;
 *   2. every token t < T is written to row (L + t) % bs of the K part and of the V part of the pool
 *      entry slot_tbl[b][h][local_col + (j & 1)], j = (L + t) / bs;
 *   3. the first n_commit tokens are also written to the same rows of entry
 *      (block_table[b][j], h) of the CPU pool host_kv (skipped when host_kv is NULL).
 * Nothing else is touched: the rows of a local entry that earlier steps wrote stay as they are.
 */
void oasis_oracle_append_kv(int32_t B, int32_t T, int32_t Hkv, int32_t d, int32_t bs,
                            int32_t max_blocks, int32_t n_commit, const uint16_t *new_kv,
                            const int32_t *seq_len, const int32_t *block_table,
                            const int32_t *slot_tbl, int32_t *blk_tbl, int32_t n_cols,
                            int32_t local_col, uint16_t *pool, uint16_t *host_kv)
{
    const int64_t part = (int64_t)bs * d;
    oasis_oracle_local_window(B, Hkv, bs, max_blocks, seq_len, T, block_table, blk_tbl, n_cols,
                              local_col, 0, NULL, NULL);
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t t = 0; t < T; ++t) {
            int32_t pos = seq_len[b] + t;
            int32_t j = pos / bs, i = pos % bs;
            for (int32_t h = 0; h < Hkv; ++h) {
                int64_t row = (int64_t)b * Hkv + h;
                const uint16_t *src = new_kv + ((((int64_t)b * T + t) * Hkv + h) * 2) * d;
                int64_t slot = slot_tbl[row * n_cols + local_col + (j & 1)];
                uint16_t *entry = pool + slot * 2 * part;
                memcpy(entry + (int64_t)i * d, src, sizeof(uint16_t) * (size_t)d);
                memcpy(entry + part + (int64_t)i * d, src + d, sizeof(uint16_t) * (size_t)d);
                if (host_kv && t < n_commit) {
                    int64_t phys = block_table[(int64_t)b * max_blocks + j];
                    uint16_t *he = host_kv + (phys * Hkv + h) * 2 * part;
                    memcpy(he + (int64_t)i * d, src, sizeof(uint16_t) * (size_t)d);
                    memcpy(he + part + (int64_t)i * d, src + d, sizeof(uint16_t) * (size_t)d);
                }
            }
        }
    }
}

/* ---------------------------------------------------------------- attention mass per block
 * Second reading of "the exact set of the true next-token query" in the agreement figures of Sec. 3 and
 * Sec. 4.2.1: the blocks that matter are those that receive the attention of the true query.  For
 * request b and every query row (t, a) of q_true [B][Tq][Hq][d] -- row t sits at position seq_len[b] + t
 * and sees every position <= its own -- dense causal softmax attention over the WHOLE context read from
 * the full-KV pool (two passes, double precision) gives a probability per key; the probabilities of
 * a block's keys are added up, and the rows that share KV head h are reduced with max:
 *   mass[b][h][j] = max_{t, a in head group h}  sum_{i : j*bs+i visible} softmax_{t,a}(j*bs + i)
 * for every logical block j that holds a visible key (0 for the others).
 */
void oasis_oracle_block_mass(int32_t B, int32_t Tq, int32_t Hq, int32_t Hkv, int32_t d, int32_t bs,
                             int32_t max_blocks, const uint16_t *q_true, const uint16_t *kv_pool,
                             const int32_t *block_table, const int32_t *seq_len, float scale,
                             double *mass)
{
    const int32_t G = Hq / Hkv;
    const int64_t part = (int64_t)bs * d;
    double *logit = (double *)malloc(sizeof(double) * (size_t)max_blocks * (size_t)bs);
    for (int64_t o = 0; o < (int64_t)B * Hkv * max_blocks; ++o) mass[o] = 0.0;
    for (int32_t b = 0; b < B; ++b) {
        for (int32_t t = 0; t < Tq; ++t) {
            int64_t n_vis = (int64_t)seq_len[b] + t + 1;
            if (n_vis > (int64_t)max_blocks * bs) n_vis = (int64_t)max_blocks * bs;
            for (int32_t a = 0; a < Hq; ++a) {
                const int32_t h = a / G;
                const uint16_t *qv = q_true + (((int64_t)b * Tq + t) * Hq + a) * d;
                double mx = -INFINITY;
                for (int64_t p = 0; p < n_vis; ++p) {
                    int64_t phys = block_table[(int64_t)b * max_blocks + p / bs];
                    const uint16_t *kr = kv_pool + (phys * Hkv + h) * 2 * part + (p % bs) * d;
                    double s = 0.0;
                    for (int32_t x = 0; x < d; ++x)
                        s = s + (double)bf16_to_f32(qv[x]) * (double)bf16_to_f32(kr[x]);
                    logit[p] = s * (double)scale;
                    if (logit[p] > mx) mx = logit[p];
                }
                double den = 0.0;
                for (int64_t p = 0; p < n_vis; ++p) {
                    logit[p] = exp(logit[p] - mx);
                    den = den + logit[p];
                }
                for (int64_t j = 0; j * bs < n_vis; ++j) {
                    double m = 0.0;
                    for (int64_t p = j * bs; p < (j + 1) * bs && p < n_vis; ++p) m = m + logit[p];
                    m = m / den;
                    double *dst = mass + ((int64_t)b * Hkv + h) * max_blocks + j;
                    if (m > *dst) *dst = m;
                }
            }
        }
    }
    free(logit);
}
