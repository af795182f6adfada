// Steps 1 + 4 of one layer in a single launch (Sec. 4.2.2: the look-ahead scoring for the next step and
// the attention over the working set staged by the previous step are independent pieces of work of
// the same layer).  Run as two kernels they each need every SM -- one CTA per SM with almost all of
// its shared memory -- so they can only alternate, and every alternation costs a CTA launch, a
// set-up, a pipeline fill and a drain per SM, while the 20 SMs that get no attention row wait.  Here
// one persistent CTA per SM does both over one ring of shared memory:
//   scoring phase    (every CTA)         a contiguous range of the layer's scoring tiles, exactly as in
//                    score_tc.cu (2-D TMA tiles of 128 summaries, swap-AB contraction against (q^- | q^+));
//   attention phase  (CTA c: work items c, c + grid, c + 2 grid, ...)  the sparse attention of whole
//                    (request, KV head) rows, one after the other, exactly as in attn_tc.cu (5-D TMA entry
//                    copies, Q K^T and P V issued by two warps, one softmax thread per MMA row with row
//                    copies).  Tiles are counted through all rows of the CTA, so the ring and the S buffers
//                    never drain between rows; Q of the next row goes to tensor memory while the row before
//                    it is written out.  With fewer rows than half the SMs and rows too long to attend
//                    whole, a work item is one split of a row's column list (split as attn.cu splits) and
//                    writes a normalised partial; the merge launch follows on the stream.
//                    The row copies of a CTA's last work item meet in the ring, idle by then, in one round.
// The ring's six 32 KiB stages serve the scoring phase as three 64 KiB stages; the producer starts the
// attention copies into a stage as soon as the scoring tiles that last used its pair have been
// consumed, so the stream of bytes into the SM never stops between the phases.  (With 64 scoring rows the two
// 32 KiB operand buffers leave room for four stages only; they become stages 4 and 5 of the attention phase once the
// last scoring MMA has completed.)  The scoring ranges
// are sized so that every SM moves the same number of bytes: a CTA with one more attention row of n
// tiles (32 KiB each) gets n / 2 fewer scoring tiles (64 KiB each) than the others.
// Scoring comes first because it needs nothing from the previous layer (draft queries and summaries
// exist before the step), whereas the attention's queries do: the kernel is launched with programmatic
// stream serialization, so behind another launch of itself its CTAs start as soon as an SM has room
// (griddepcontrol.launch_dependents at the top), score, and only then wait for the predecessor
// (griddepcontrol.wait) before touching the attention inputs.  SMs are thus handed from one layer to
// the next one by one, without the idle time around a kernel boundary.
//   warp 0     TMA producer of both phases
//   warp 1     issues the scoring MMAs, then Q K^T  (both issuing warps run converged, elect.sync picks the lane)
//   warp 2     issues P V
//   warps 3-6  scoring epilogue, then Q into tensor memory, softmax and write-out of the attention row
//   warp 7     builds the (q^- | q^+) operands of the CTA's scoring range ahead of time
//   warps 8-11 only with 65 to 128 query rows: the second set of softmax warps (alternate tiles, own O accumulator;
//              see attn_tc.cu); idle in the scoring phase
// Every wait is bounded; a time-out records a code in the error word and the CTA winds down.
// Algorithmic traffic: 8 KiB per (request, KV head, column) + Q / O, and 512 B + 4 B per scored block.
#include <cuda.h>
#include <math_constants.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace oasis {

constexpr int kLyThreads = 256;                             // (128 more with two softmax sets: warps 8-11)
__host__ __device__ constexpr int ly_threads(int mma_m, int copies) { return kLyThreads + (at_softmax_sets(mma_m, copies) - 1) * 128; }
constexpr int kLyMaxStages = 6;                             // 32 KiB stages (attention) = three 64 KiB pairs (scoring)
constexpr int kLyTileBlocks = 128;                          // summaries per scoring tile
constexpr int kLyATileBytes = kLyTileBlocks * kSummaryBytes;   // 64 KiB
constexpr int kLySubTileBytes = kLyTileBlocks * 128;        // one 64-element K chunk of a scoring tile: 16 KiB
constexpr int kLyTmemCols = 512;                            // S [0,256), O [256,384), Q [384,448), narrow scoring accumulators [448,512)

struct LayerTcParams {
    // attention phase
    const uint8_t *q;
    const int32_t *slot_tbl;
    const int32_t *blk_tbl;
    const int32_t *seq_len;
    uint8_t *out;
    float *lse;
    float scale_log2;
    int T, Hq, Hkv, G, n_cols, R;
    int items;                  // attention work items: (request, KV head) rows x splits of their column lists
    int n_splits, cols_per_split;
    float *part_o, *part_lse;   // split runs: normalised partial outputs [items][R][128] and their log2 sum-exps [items][R]
    int n_more;                 // CTAs 0 .. n_more-1 attend one row more than the others
    // scoring phase
    const uint8_t *q_draft;
    long long q_batch_stride;
    const int32_t *n_full;
    float *scores;
    int Rs, N, max_blocks, tiles_per_bh, reduce_sum;
    int acc_col;                // first tensor-memory column of the two scoring accumulators
    int total_tiles;            // rows * tiles_per_bh (the host checks that summaries rows fit 31 bits)
    double w_row, w_free;       // scoring tiles of a CTA with the larger / the smaller number of attention rows
    int32_t *err;
    long long n_slots;          // bounds-check build: slots of the working-set pool (else unused)
};

// MODE: 0 = at most one whole row per thread block; 1 = more rows than thread blocks, several whole rows per block;
// 2 = fewer rows than half the SMs, their column lists split into one work item per thread block.  Separate
// instantiations because the kernel is sensitive to every instruction its issuing threads execute (the row loop
// costs mode 0 1.5 us at 128 rows, the split arithmetic 0.5 us).  STAGES: 32 KiB stages of the ring (6, or 4 where
// the scoring operands or the copy-merge staging need the room); ASTAGES: stages in the attention phase.
template <int MMA_M, int COPIES, int MODE, int STAGES, int ASTAGES>
__global__ void __launch_bounds__(ly_threads(MMA_M, COPIES), 1)
layer_tc_kernel(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ CUtensorMap tmap_summ,
                const LayerTcParams p)
{
    constexpr bool MULTI = MODE == 1, SPLIT = MODE == 2;
    // ASTAGES: stages of the ring in the attention phase.  Where 64 scoring rows leave room for only four stages beside
    // the two 32 KiB operand buffers, those buffers, idle once the last scoring MMA has completed, are stages 4 and 5.
    constexpr int kLyStages = ASTAGES, kLyPairs = STAGES / 2;
    constexpr int RPC = MMA_M / COPIES;                     // MMA rows per copy of the query rows
    constexpr int LANES = MMA_M / 4;                        // lanes of each softmax warp that hold an MMA row
    constexpr int BPC = kAtTileCols / COPIES;               // blocks of a tile each copy handles
    constexpr int KPC = BPC * kBlock;                       // keys of a tile each copy handles
    constexpr int kStageF = COPIES > 1 ? 20 : 0;            // floats per MMA row of the copy-merge staging (16 + pad)
    constexpr int SETS = at_softmax_sets(MMA_M, COPIES);    // softmax warp sets, taking alternate tiles of a row
    constexpr int SBUFS = at_s_bufs(SETS);                  // S / P buffers in tensor memory
    constexpr int THREADS = ly_threads(MMA_M, COPIES);
    constexpr int kAtQBytes = 0;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t kv_u32 = base;                                    // [STAGES][32 KiB] = [STAGES / 2][64 KiB]
    const uint32_t b_bytes = (uint32_t)p.N * kSummaryBytes;
    const uint32_t b_u32 = kv_u32 + STAGES * kAtStageBytes;          // [2][N][512 B] as 4 sub-tiles of N x 128 B
    uint8_t *b_ptr = base_ptr + (size_t)STAGES * kAtStageBytes;
    float *o_sm = reinterpret_cast<float *>(b_ptr + 2 * b_bytes);    // [MMA_M][kStageF]
    float *m_sm = o_sm + MMA_M * kStageF;                            // [SETS][MMA_M]
    float *l_sm = m_sm + MMA_M * SETS;                               // [SETS][MMA_M]
    uint8_t *misc = reinterpret_cast<uint8_t *>(l_sm + MMA_M * SETS);
    const uint32_t bar_u32 = smem_u32(misc);
    // attention-phase barriers
    auto bar_full = [&](int s) { return bar_u32 + 8u * s; };
    auto bar_empty = [&](int s) { return bar_u32 + 8u * (kLyStages + s); };
    auto bar_s_full = [&](int a) { return bar_u32 + 8u * (2 * kLyStages + a); };
    auto bar_p_full = [&](int a) { return bar_u32 + 8u * (2 * kLyStages + kAtSBufs + a); };
    // scoring-phase barriers
    constexpr int kB0 = 2 * kLyStages + 2 * kAtSBufs;
    auto sbar_full = [&](int s) { return bar_u32 + 8u * (kB0 + s); };
    auto sbar_empty = [&](int s) { return bar_u32 + 8u * (kB0 + kLyPairs + s); };
    auto bar_acc_full = [&](int a) { return bar_u32 + 8u * (kB0 + 2 * kLyPairs + a); };
    auto bar_acc_empty = [&](int a) { return bar_u32 + 8u * (kB0 + 2 * kLyPairs + 2 + a); };
    auto bar_b_full = [&](int a) { return bar_u32 + 8u * (kB0 + 2 * kLyPairs + 4 + a); };
    auto bar_b_empty = [&](int a) { return bar_u32 + 8u * (kB0 + 2 * kLyPairs + 6 + a); };
    const uint32_t bar_q = bar_u32 + 8u * (kB0 + 2 * kLyPairs + 8);  // Q is in tensor memory
    const uint32_t bar_score_done = bar_u32 + 8u * (kB0 + 2 * kLyPairs + 9);   // every scoring MMA has completed
    constexpr int kNBars = kB0 + 2 * kLyPairs + 10;                  // 36 with six stages
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(misc + 8 * kNBars);
    int32_t *tile_blk = reinterpret_cast<int32_t *>(misc + 8 * kNBars + 16);   // [stages][4]
    int32_t *win = reinterpret_cast<int32_t *>(misc + 512);                    // two table windows

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // ---- attention geometry: CTA c < rows owns row c ------------------------------------------------------
    // An attention work item is one (request, KV head) row, or one split of its column list where there are fewer
    // rows than half the SMs (items of a row are consecutive: item = row * n_splits + split).
    const int n_my_rows = (int)blockIdx.x < p.items ? (MULTI ? (p.items - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 1) : 0;
    const bool cta_has_row = n_my_rows > 0;
    auto my_row = [&](int k) { return (int)blockIdx.x + k * (int)gridDim.x; };     // k-th item of this CTA
    auto row_of = [&](int item) { return SPLIT ? item / p.n_splits : item; };
    auto first_col = [&](int item) { return SPLIT ? (item % p.n_splits) * p.cols_per_split : 0; };
    auto end_col = [&](int item) { return SPLIT ? min(first_col(item) + p.cols_per_split, p.n_cols) : p.n_cols; };
    // tiles of 4 columns an item covers: the same for every whole row; a split item is its thread block's only one
    const int tiles_first = ((SPLIT && cta_has_row ? end_col((int)blockIdx.x) - first_col((int)blockIdx.x) : p.n_cols) +
                             kAtTileCols - 1) / kAtTileCols;
    auto tiles_of = [&](int) { return tiles_first; };
    const int L0 = p.seq_len[(cta_has_row ? row_of((int)blockIdx.x) : 0) / p.Hkv];   // length of the request of the first item
    // ---- scoring geometry: tiles [t0, t1) ---------------------------------------------------------
    auto tiles_before = [&](int c) {
        const double w = c <= p.n_more ? c * p.w_row : p.n_more * p.w_row + (c - p.n_more) * p.w_free;
        int t = (int)w;
        return t < p.total_tiles ? t : p.total_tiles;
    };
    const int t0 = tiles_before(blockIdx.x);
    const int t1 = blockIdx.x + 1 == gridDim.x ? p.total_tiles : tiles_before(blockIdx.x + 1);

    // First tile at or after t (and before t1) that has candidate blocks; t1 if there is none.
    auto next_active = [&](int t) {
#pragma unroll 1
        for (; t < t1; ++t) {
            const int sbh = t / p.tiles_per_bh;
            const int j0 = (int)(t % p.tiles_per_bh) * kLyTileBlocks;
            if (j0 < p.n_full[(int)(sbh / p.Hkv)]) break;
        }
        return t;
    };
    // (q^- | q^+) rows of one (request, KV head), K-major, 128-byte swizzle: element k of row n
    // lives in sub-tile k / 64.  `nthr` threads (index `me`) share the work; loads are issued
    // eight at a time so their latencies overlap.
    auto build_b = [&](int bh, int buf, int me, int nthr) {
        build_qpm_operand(b_ptr + (size_t)buf * b_bytes, p.q_draft, p.q_batch_stride, bh / p.Hkv, bh % p.Hkv, p.Rs, p.G, p.Hq, p.N,
                          p.reduce_sum, me, nthr);
    };

    // The next launch on the stream may start as soon as an SM has room for one of its thread blocks (its scoring
    // phase needs nothing from this one); it waits for this grid before its attention phase.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // the first scoring tile with candidates: asked for now, so that the look-up's trip to global memory overlaps the set-up
    const int t_first = next_active(t0);
    // ---- set-up: barriers (one thread each), tensor memory ---------------------------------------------------
    if (tid < kNBars) {
        // arrival counts: the four softmax / epilogue warps arrive on P-written, accumulator-read and Q-written
        const bool four = (tid >= 2 * kLyStages + kAtSBufs && tid < kB0) ||
                          (tid >= kB0 + 2 * kLyPairs + 2 && tid < kB0 + 2 * kLyPairs + 4) || tid == kB0 + 2 * kLyPairs + 8;
        mbar_init(bar_u32 + 8u * tid, four ? 4 : 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();                             // the barriers exist; the producer starts copying right away
    uint32_t tmem_base = 0, tmem_o = 0, tmem_q = 0;
    if (warp != 0) {
        // Meanwhile warp 1 allocates the tensor memory.
        if (warp == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)kLyTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
        tc_fence_before();
        asm volatile("bar.sync 2, %0;" ::"n"(THREADS - 32) : "memory");
        tc_fence_after();
        tmem_base = *tmem_slot;
        tmem_o = tmem_base + SBUFS * kAtTileKeys;
        tmem_q = tmem_o + SETS * kHeadDim;                                // Q as the A operand: 128 rows x 64 packed columns
    }
    if (warp == 0) {
        bool alive = true;
        int it = 0;                                                  // scoring tiles issued
        {
            // ---------------------------------------------------------------- scoring phase: tiles
            int t = t_first;
            while (t < t1 && alive) {
                const int bh = t / p.tiles_per_bh;
                const int j0 = (int)(t % p.tiles_per_bh) * kLyTileBlocks;
                if (lane == 0) {
                    const int s = it % kLyPairs;
                    alive = alive && mbar_wait(sbar_empty(s), ((it / kLyPairs) & 1) ^ 1, p.err, 12);
                    if (alive) {
                        mbar_arrive_expect_tx(sbar_full(s), kLyATileBytes);
                        const int y = bh * p.max_blocks + j0;
                        load_score_tile(kv_u32 + s * kLyATileBytes, &tmap_summ, y, kLySubTileBytes, sbar_full(s));
                    }
                }
                alive = __shfl_sync(0xffffffffu, (int)alive, 0) != 0;
                ++it;
                const int tn = next_active(t + 1);
                t = tn;
            }
        }
        // ---------------------------------------------------------------- producer
        // Table entries come 32 columns (eight tiles) at a time through two window buffers, one window ahead.
        // the attention phase reads what the previous layer may have produced: wait for it (no-op without a programmatic launch)
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const uint32_t win_u32 = smem_u32(win);
        int s = 0, gi = 0;                                           // ring stage and index of the tile among all rows
        uint32_t ph = 1;                                             // parity of the "empty" phase to wait for
#pragma unroll 1
        for (int k = 0; k < n_my_rows && alive; ++k) {
        const int item = my_row(k), tpr = tiles_of(item);
        const int32_t *slot_row = p.slot_tbl + (long long)row_of(item) * p.n_cols;
        const int32_t *blk_row = p.blk_tbl + (long long)row_of(item) * p.n_cols;
        const int c0 = first_col(item), c1 = end_col(item);          // column range of the item
        __syncwarp();                                                // the previous row's window reads are over
        window_request(win_u32, lane, blk_row, slot_row, c0 + lane, c1);
#pragma unroll 1
        for (int i = 0; i < tpr && alive; ++i, ++gi, ph ^= (s + 1 == kLyStages), s = (s + 1 == kLyStages) ? 0 : s + 1) {
            if ((i & 7) == 0) {
                window_wait();
                window_request(win_u32 + (((i >> 3) + 1) & 1) * kWinBytes, lane, blk_row, slot_row, c0 + (i + 8) * kAtTileCols + lane, c1);
            }
            int blk, slot;
            window_read(win, i, lane, blk, slot);
            if (kBoundsCheck && blk >= 0 && !in_range(slot, p.n_slots, Bounds{0, 0, p.err}, kErrSlot)) blk = -1;
            if (lane == 0 && gi < kLyStages) {
                if (s < STAGES) {
                    // first use of this stage: the scoring tiles that last used its 64 KiB pair must have been consumed
                    const int pr = s >> 1;
                    const int uses = it > pr ? (it - pr + kLyPairs - 1) / kLyPairs : 0;
                    if (uses > 0) alive = mbar_wait(sbar_empty(pr), (uses - 1) & 1, p.err, 14);
                } else {
                    // a stage in the place of the scoring operands: every scoring MMA must have completed
                    alive = mbar_wait(bar_score_done, 0, p.err, 15);
                }
            }
            if (lane == 0) alive = alive && mbar_wait(bar_empty(s), ph, p.err, 41);
            alive = __shfl_sync(0xffffffffu, (int)alive, 0) != 0;
            if (!alive) break;
            stage_attn_tile(lane, blk, slot, tile_blk + s * kAtTileCols, base_ptr + kAtQBytes + (size_t)s * kAtStageBytes,
                            kv_u32 + s * kAtStageBytes, &tmap, bar_full(s));
        }
        }
    } else if (warp == 1) {
        {
            // ---------------------------------------------------------------- scoring phase: MMAs (the whole warp, converged)
            {
                const uint32_t idesc = idesc_score(p.N, kLyTileBlocks);
                int it = 0, bo = -1;
                int cur_bh = -1;
                bool alive = true;
#pragma unroll 1
                for (int t = t0; t < t1 && alive; ++t) {
                    const int bh = t / p.tiles_per_bh;
                    const int j0 = (int)(t % p.tiles_per_bh) * kLyTileBlocks;
                    const int b = (int)(bh / p.Hkv);
                    if (j0 >= p.n_full[b]) continue;
                    if (bh != cur_bh) {
                        if (bo >= 0) tc_commit(bar_b_empty(bo % 2));   // earlier MMAs no longer read that operand
                        cur_bh = bh;
                        ++bo;
                        alive = mbar_wait_warp(bar_b_full(bo % 2), (bo / 2) & 1, p.err, 21);
                        if (!alive) break;
                    }
                    const int acc = it & 1, s = it % kLyPairs;
                    alive = mbar_wait_warp(bar_acc_empty(acc), ((it >> 1) & 1) ^ 1, p.err, 22) &&
                            mbar_wait_warp(sbar_full(s), (it / kLyPairs) & 1, p.err, 23);
                    if (!alive) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)p.acc_col + (uint32_t)(acc * p.N);
                    const uint32_t a_tile = kv_u32 + s * kLyATileBytes;
                    const uint32_t b_tile = b_u32 + (bo % 2) * b_bytes;
                    issue_score_tile(d_tmem, a_tile, b_tile, p.N, kLySubTileBytes, idesc);
                    tc_commit(sbar_empty(s));         // the stage may be refilled once these MMAs have read it
                    tc_commit(bar_acc_full(acc));    // the accumulator is complete
                    ++it;
                }
                if (ASTAGES > STAGES) tc_commit(bar_score_done);     // (arrives at once if this thread block scored nothing)
            }
        }
        // ---------------------------------------------------------------- Q K^T issuer (the whole warp, converged)
        {
            const uint32_t idesc = idesc_qk(MMA_M);
            // descriptors: the operand start address occupies the low 14 bits (16-byte units), so offsets are added there
            const uint64_t k_desc0 = smem_desc_sw128_k(kv_u32, kImgGroup);
            bool alive = true;
            int s = 0, sb = 0, s_old = 0;                            // stage and S buffer of tile i; stage of tile i - SBUFS
            uint32_t ph = 0, ph_old = 0;
            int i = 0;                                               // index of the tile among all rows of this CTA
#pragma unroll 1
            for (int k = 0; k < n_my_rows && alive; ++k) {
            const int tpr = tiles_of(my_row(k));
            alive = mbar_wait_warp(bar_q, (uint32_t)(k & 1), p.err, 55);  // the row's Q is in tensor memory
            tc_fence_after();
#pragma unroll 1
            for (int it = 0; it < tpr && alive; ++it, ++i) {
                // the S buffer also held P of tile i - SBUFS: its P V must have completed
                if (i >= SBUFS) {
                    alive = mbar_wait_warp(bar_empty(s_old), ph_old, p.err, 51);
                    ph_old ^= (s_old + 1 == kLyStages);
                    s_old = (s_old + 1 == kLyStages) ? 0 : s_old + 1;
                }
                alive = alive && mbar_wait_warp(bar_full(s), ph, p.err, 52);
                if (!alive) break;
                tc_fence_after();
                const uint64_t k_desc = k_desc0 + (uint64_t)((s * kAtStageBytes) >> 4);
                const uint32_t d_tmem = tmem_base + (uint32_t)(sb * kAtTileKeys);
                issue_qk_tile(d_tmem, tmem_q, k_desc, idesc);
                tc_commit(bar_s_full(sb));
                ph ^= (s + 1 == kLyStages);
                s = (s + 1 == kLyStages) ? 0 : s + 1;
                sb = (sb + 1 == SBUFS) ? 0 : sb + 1;
            }
            }
        }
    } else if (warp == 2) {
        // ---------------------------------------------------------------- P V issuer (the whole warp, converged)
        {
            const uint32_t idesc = idesc_pv(MMA_M);
            const uint64_t v_desc0 = smem_desc_sw128_mn(kv_u32 + kImgPart, kImgHalf, kImgGroup);
            bool alive = true;
            int s = 0, sb = 0;
            uint32_t ph_p = 0;
#pragma unroll 1
            for (int k = 0; k < n_my_rows && alive; ++k) {
            const int tpr = tiles_of(my_row(k));
#pragma unroll 1
            for (int it = 0; it < tpr && alive; ++it) {
                alive = mbar_wait_warp(bar_p_full(sb), ph_p, p.err, 53);
                if (!alive) break;
                tc_fence_after();
                const uint64_t v_desc = v_desc0 + (uint64_t)((s * kAtStageBytes) >> 4);
                const uint32_t p_tmem = tmem_base + (uint32_t)(sb * kAtTileKeys);
                // O starts afresh with every row (two softmax sets: even tiles of the row go to the first O, odd ones to the second)
                issue_pv_tile(tmem_o + (uint32_t)((it % SETS) * kHeadDim), p_tmem, v_desc, idesc, it < SETS);
                tc_commit(bar_empty(s));                             // stage free, and O complete up to this tile
                s = (s + 1 == kLyStages) ? 0 : s + 1;
                sb = (sb + 1 == SBUFS) ? 0 : sb + 1;
                ph_p ^= (sb == 0);
            }
            }
        }
    } else if (warp == 7) {
        // ---------------------------------------------------------------- operand builder
        // Walks the CTA's scoring tiles ahead of everyone else and builds (q^- | q^+) of every (request, KV head)
        // as soon as an operand buffer is free.
        int bo = -1;
        bool alive = true;
        int cur_bh = -1;
#pragma unroll 1
        for (int t = t_first; t < t1 && alive; t = next_active(t + 1)) {
            const int bh = t / p.tiles_per_bh;
            if (bh == cur_bh) continue;
            cur_bh = bh;
            ++bo;
            const int buf = bo % 2;
            if (lane == 0) alive = mbar_wait(bar_b_empty(buf), ((bo / 2) & 1) ^ 1, p.err, 11);
            alive = __shfl_sync(0xffffffffu, (int)alive, 0) != 0;
            if (!alive) break;
            build_b(bh, buf, lane, 32);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_b_full(buf));
        }
    } else {
        // ---------------------------------------------------------------- softmax, one thread per MMA row (two sets: warps
        // 3-6 take the even tiles of a row, warps 8-11 the odd ones; the first set alone has a part in the scoring phase)
        const int set = SETS == 2 ? (warp >= 8 ? 1 : 0) : 0;
        const int quarter = warp & 3;
        const int m_row = quarter * LANES + (lane % LANES);         // MMA row held by this tensor-memory lane
        const int copy = m_row / RPC, row = m_row % RPC;            // which copy of the rows, which query row
        const bool has_row = lane < LANES;
        const bool live_row = has_row && row < p.R;
        const bool live_warp = (quarter * LANES) % RPC < p.R;       // some lane of this warp holds a query row
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        if (set == 0) {
            // ---------------------------------------------------------------- scoring phase: epilogue
            int it = 0;
            bool alive = true;
#pragma unroll 1
            for (int t = t0; t < t1 && alive; ++t) {
                const int bh = t / p.tiles_per_bh;
                const int j0 = (int)(t % p.tiles_per_bh) * kLyTileBlocks;
                const int b = (int)(bh / p.Hkv);
                const int nf = p.n_full[b];
                if (kBoundsCheck && lane == 0 && nf > p.max_blocks) in_range(nf, p.max_blocks + 1, Bounds{0, 0, p.err}, kErrBlockCount);
                const int j = j0 + quarter * 32 + lane;
                float *out = p.scores + (long long)bh * p.max_blocks;
                if (j0 >= nf) {
                    if (j < p.max_blocks) out[j] = -CUDART_INF_F;
                    continue;
                }
                const int acc = it & 1;
                alive = mbar_wait(bar_acc_full(acc), (it >> 1) & 1, p.err, 31);
                if (!alive) break;
                tc_fence_after();
                const uint32_t taddr = tmem_base + (uint32_t)p.acc_col + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * p.N);
                const float res = reduce_score_row(taddr, p.N, p.reduce_sum);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acc_empty(acc));
                if (j < p.max_blocks) out[j] = j < nf ? res : -CUDART_INF_F;
                ++it;
            }
        }
        // ---- attention phase: this thread's Q row goes to its tensor-memory lane (rows are replicated across the copies, rows
        // past R are zero); q may come from the previous layer: wait for it (no-op without a programmatic launch)
        asm volatile("griddepcontrol.wait;" ::: "memory");
        auto load_q = [&](int bh) {
            const int b = bh / p.Hkv, h = bh % p.Hkv;
            uint4 v[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) v[c] = make_uint4(0, 0, 0, 0);
            if (live_row) {
                const int tq = row / p.G, a = h * p.G + row % p.G;
                const uint4 *src = reinterpret_cast<const uint4 *>(p.q + ((((long long)b * p.T + tq) * p.Hq + a) * kHeadDim) * 2);
#pragma unroll
                for (int c = 0; c < 16; ++c) v[c] = src[c];
            }
            q_row_to_tmem(tmem_q + lane_base, v);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_q);
        };
        if (set == 0 && cta_has_row) load_q(row_of(my_row(0)));
        bool alive = true;
        int i0 = 0;                                                 // index of the row's first tile among all tiles of this CTA
        const uint32_t my_o = tmem_o + (uint32_t)(set * kHeadDim) + lane_base;   // this thread's O row
#pragma unroll 1
        for (int k = 0; k < n_my_rows; ++k) {
        const int item = my_row(k), tpr = tiles_of(item);
        const int bh = row_of(item), b = bh / p.Hkv, h = bh % p.Hkv;
        // last visible position of this row; MMA rows past R hold zero queries and need no masking (masking them would
        // send their whole warp down the masked path on every tile), lanes without an MMA row see nothing
        const int limit = live_row ? (k == 0 ? L0 : p.seq_len[b]) + row / p.G : (has_row ? 0x3fffffff : -1);
        float m_ref = -CUDART_INF_F, l_sum = 0.f;
        // Tile g of the CTA (counted through all its rows) lives in ring stage g % stages and S buffer g % SBUFS; the
        // barriers of its stage / buffer complete for it with parity (g / stages) & 1, (g / SBUFS) & 1.
#pragma unroll 1
        for (int it = set; it < tpr && alive; it += SETS) {
            const int g = i0 + it, sb = g % SBUFS, s = g % kLyStages;
            alive = mbar_wait(bar_s_full(sb), (uint32_t)((g / SBUFS) & 1), p.err, 61);
            if (!alive) break;
            tc_fence_after();
            const uint32_t s_tmem = tmem_base + lane_base + (uint32_t)(sb * kAtTileKeys);
            if (live_warp)
                alive = softmax_tile<COPIES>(s_tmem, my_o, tile_blk + s * kAtTileCols, copy, limit, has_row,
                                             p.scale_log2, m_ref, l_sum, it >= SETS,
                                             // the P V of this set's previous tile of the row
                                             [&] { return mbar_wait(bar_empty((g - SETS) % kLyStages), (uint32_t)(((g - SETS) / kLyStages) & 1), p.err, 62); });
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_p_full(sb));
        }
        // ---- Q of the CTA's next row goes to tensor memory first (this warp has seen S of the row's last tile, so
        // every Q K^T of the row has completed), then the row is written out: merge the copies, normalise.  The
        // next row's first P V, which overwrites O, needs P of that tile from these warps, so it comes later.
        {
            // (with two softmax sets the first one has not seen the row's odd tiles: it loads Q after the last P V instead)
            if (SETS == 1 && MULTI && alive && k + 1 < n_my_rows) load_q(my_row(k + 1));
            if (alive && tpr > 0) {                                  // the row's last P V has completed
                const int g = i0 + tpr - 1;
                alive = mbar_wait(bar_empty(g % kLyStages), (uint32_t)((g / kLyStages) & 1), p.err, 63);
            }
            tc_fence_after();
            if (SETS == 2 && MULTI && alive && set == 0 && k + 1 < n_my_rows) load_q(my_row(k + 1));
            i0 += tpr;
            // From here on the four softmax warps meet at named barriers, which have no time-out: go on only if
            // none of them has given up (every thread gets here, because all its waits above are bounded).
            alive = softmax_warps_all<128 * SETS>(alive);
            const int t_task = quarter * 32 + lane;
            // writes 16 output dims [d0, d0 + 16) of query row `orow`
            auto emit = [&](int orow, int d0, const float (&acc)[16], float mx, float den) {
                const float inv = den > 0.f ? 1.f / den : 0.f;
                if (SPLIT) {
                    // one split of the row: normalised partial and its log2 sum-exp, merged by the combine launch
                    float4 *dstp = reinterpret_cast<float4 *>(p.part_o + ((long long)item * p.R + orow) * kHeadDim + d0);
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        dstp[e] = make_float4(acc[4 * e] * inv, acc[4 * e + 1] * inv, acc[4 * e + 2] * inv, acc[4 * e + 3] * inv);
                    if (d0 == 0) p.part_lse[(long long)item * p.R + orow] = den > 0.f ? mx + log2f(den) : -CUDART_INF_F;
                    return;
                }
                const int tq = orow / p.G, a = h * p.G + orow % p.G;
                const long long o_row = ((long long)b * p.T + tq) * p.Hq + a;
                uint4 *dst = reinterpret_cast<uint4 *>(p.out + (o_row * kHeadDim + d0) * 2);
#pragma unroll
                for (int e = 0; e < 2; ++e)
                    dst[e] = make_uint4(pack_bf16x2(acc[8 * e] * inv, acc[8 * e + 1] * inv),
                                        pack_bf16x2(acc[8 * e + 2] * inv, acc[8 * e + 3] * inv),
                                        pack_bf16x2(acc[8 * e + 4] * inv, acc[8 * e + 5] * inv),
                                        pack_bf16x2(acc[8 * e + 6] * inv, acc[8 * e + 7] * inv));
                if (p.lse && d0 == 0) p.lse[o_row] = den > 0.f ? (mx + log2f(den)) * kAtLn2 : -CUDART_INF_F;
            };
            if (alive && SETS == 2) {
                // the two threads of a row exchange maximum and sum; each then merges and writes one half of the output dims,
                // reading both O accumulators at its own tensor-memory lane
                m_sm[set * MMA_M + m_row] = m_ref;
                l_sm[set * MMA_M + m_row] = l_sum;
                asm volatile("bar.sync 1, 256;" ::: "memory");      // the eight softmax warps
                const float m_o = m_sm[(set ^ 1) * MMA_M + m_row], l_o = l_sm[(set ^ 1) * MMA_M + m_row];
                const float mx = fmaxf(m_ref, m_o);
                const float w_me = mx == -CUDART_INF_F ? 0.f : fast_exp2(m_ref - mx), w_ot = mx == -CUDART_INF_F ? 0.f : fast_exp2(m_o - mx);
                const float den = w_me * l_sum + w_ot * l_o;
                const float w_a = set == 0 ? w_me : w_ot, w_b = set == 0 ? w_ot : w_me;   // weights of the first and second accumulator
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    const int d0 = set * 64 + c * 16;
                    uint32_t va[16], vb[16];
                    if (live_warp) {
                        tc_ld16(tmem_o + lane_base + d0, va);
                        tc_ld16(tmem_o + kHeadDim + lane_base + d0, vb);
                    }
                    float acc[16];
                    // an accumulator whose set saw no key (weight 0) was never written: its contents do not enter
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        acc[e] = live_warp ? (w_a != 0.f ? w_a * __uint_as_float(va[e]) : 0.f) + (w_b != 0.f ? w_b * __uint_as_float(vb[e]) : 0.f) : 0.f;
                    if (live_row) emit(row, d0, acc, mx, den);
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");      // the exchange area is rewritten for the next row
            } else if (alive && COPIES > 1) {
                // with several rows per thread block the ring already holds the next row's tiles: the copies meet in a
                // small staging area, 16 dims at a time (small enough that the selection kernels of other streams still
                // fit beside this CTA)
                if (lane < LANES) {
                    m_sm[m_row] = m_ref;
                    l_sm[m_row] = l_sum;
                }
                float mx = -CUDART_INF_F, den = 0.f, wt[COPIES];
                if (!MULTI || k + 1 == n_my_rows) {
                    // the thread block's only (or last) work item: the ring is idle, so whole O rows meet there in one round
                    // ([MMA_M][132] floats) and the (row, slice of the dims) tasks go to the first MMA_M threads
                    float *o_big = reinterpret_cast<float *>(base_ptr + kAtQBytes);
                    if (live_warp) {
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            uint32_t v[16];
                            tc_ld16(tmem_o + lane_base + c * 16, v);
                            float4 *dst = reinterpret_cast<float4 *>(o_big + m_row * 132 + c * 16);
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if (lane < LANES) dst[e] = make_float4(__uint_as_float(v[4 * e]), __uint_as_float(v[4 * e + 1]),
                                                                       __uint_as_float(v[4 * e + 2]), __uint_as_float(v[4 * e + 3]));
                        }
                    }
                    asm volatile("bar.sync 1, 128;" ::: "memory");  // the four softmax warps
                    constexpr int DLEN = kHeadDim / COPIES;
                    const int orow = t_task % RPC, d_first = (t_task / RPC) * DLEN;
                    if (t_task < MMA_M && orow < p.R) {
#pragma unroll
                        for (int c = 0; c < COPIES; ++c) mx = fmaxf(mx, m_sm[c * RPC + orow]);
#pragma unroll
                        for (int c = 0; c < COPIES; ++c) {
                            wt[c] = mx == -CUDART_INF_F ? 0.f : fast_exp2(m_sm[c * RPC + orow] - mx);
                            den += wt[c] * l_sm[c * RPC + orow];
                        }
#pragma unroll 1
                        for (int d0 = d_first; d0 < d_first + DLEN; d0 += 16) {
                            float acc[16];
#pragma unroll
                            for (int e = 0; e < 16; ++e) acc[e] = 0.f;
#pragma unroll
                            for (int c = 0; c < COPIES; ++c) {
                                if (wt[c] == 0.f) continue;         // a copy that saw no key holds no O row
                                const float4 *src = reinterpret_cast<const float4 *>(o_big + (c * RPC + orow) * 132 + d0);
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const float4 v4 = src[e];
                                    acc[4 * e] += wt[c] * v4.x; acc[4 * e + 1] += wt[c] * v4.y;
                                    acc[4 * e + 2] += wt[c] * v4.z; acc[4 * e + 3] += wt[c] * v4.w;
                                }
                            }
                            emit(orow, d0, acc, mx, den);
                        }
                    }
                } else
#pragma unroll 1
                for (int rd = 0; rd < 8; ++rd) {
                    if (live_warp) {
                        uint32_t v[16];
                        tc_ld16(tmem_o + lane_base + rd * 16, v);
                        float4 *dst = reinterpret_cast<float4 *>(o_sm + m_row * kStageF);
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (lane < LANES) dst[e] = make_float4(__uint_as_float(v[4 * e]), __uint_as_float(v[4 * e + 1]),
                                                                   __uint_as_float(v[4 * e + 2]), __uint_as_float(v[4 * e + 3]));
                    }
                    asm volatile("bar.sync 1, 128;" ::: "memory");  // the four softmax warps
                    if (t_task < RPC && t_task < p.R) {
                        if (rd == 0) {
#pragma unroll
                            for (int c = 0; c < COPIES; ++c) mx = fmaxf(mx, m_sm[c * RPC + t_task]);
#pragma unroll
                            for (int c = 0; c < COPIES; ++c) {
                                wt[c] = mx == -CUDART_INF_F ? 0.f : fast_exp2(m_sm[c * RPC + t_task] - mx);
                                den += wt[c] * l_sm[c * RPC + t_task];
                            }
                        }
                        float acc[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) acc[e] = 0.f;
#pragma unroll
                        for (int c = 0; c < COPIES; ++c) {
                            if (wt[c] == 0.f) continue;             // a copy that saw no key holds no O row
                            const float4 *src = reinterpret_cast<const float4 *>(o_sm + (c * RPC + t_task) * kStageF);
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float4 v4 = src[e];
                                acc[4 * e] += wt[c] * v4.x; acc[4 * e + 1] += wt[c] * v4.y;
                                acc[4 * e + 2] += wt[c] * v4.z; acc[4 * e + 3] += wt[c] * v4.w;
                            }
                        }
                        emit(t_task, rd * 16, acc, mx, den);
                    }
                    asm volatile("bar.sync 1, 128;" ::: "memory");  // the staging rows are rewritten next round
                }
            } else if (alive) {
#pragma unroll 1
                for (int rd = 0; rd < 8; ++rd) {                    // the thread's own O row, read by the whole warp
                    float acc[16];
                    uint32_t v[16];
                    if (live_warp) tc_ld16(tmem_o + lane_base + rd * 16, v);
#pragma unroll
                    for (int e = 0; e < 16; ++e) acc[e] = live_warp ? __uint_as_float(v[e]) : 0.f;
                    if (live_row) emit(row, rd * 16, acc, m_ref, l_sum);
                }
            }
            if (!alive) break;
        }
        }
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kLyTmemCols)
                     : "memory");
    }
}

// ---- host side -----------------------------------------------------------------------------------------

static size_t layer_tc_smem_bytes(int mma_m, int copies, int N, int stages)
{
    return 1024 + (size_t)stages * kAtStageBytes + 2 * (size_t)N * kSummaryBytes +
           (size_t)mma_m * ((copies > 1 ? 20 : 0) + 2 * at_softmax_sets(mma_m, copies)) * sizeof(float) + 512 + 2 * kWinBytes;
}

struct LayerTcPlan {
    int R, Rs, N, mma_m, copies, stages, astages;
    int n_splits, cols_per_split;       // of every row's column list (1 = rows are attended whole)
    size_t smem, workspace;
};

void attn_split_plan(const oasis_dims_t *dims, int T, int n_cols, int *n_splits, int *cols_per_split, size_t *workspace);
int launch_attn_combine_after(const oasis_dims_t *dims, int T, void *out, float *lse, float *part_o, float *part_lse,
                              int n_splits, cudaStream_t st, const char *who);                       // attn.cu

// Whether the fused launch takes these shapes, and with which variant.  Wanted: at most 128 attention rows and 64
// scoring rows per KV head (two accumulators of up to 32 columns fit beside the attention's tensor memory, wider
// ones take the place of the S buffers, which the attention phase only touches after the last scoring epilogue)
// and a footprint within 227 KiB with six ring stages, or with four for the 128-row variants.
// With more rows than SMs a CTA attends rows c, c + grid, c + 2 grid, ...; with fewer rows than half the SMs, and
// rows too long to be attended whole without making stragglers, the column lists are split exactly as
// oasis_sparse_attn splits them, each split a work item of its own, and a combine launch merges the parts.
static bool layer_tc_plan(const oasis_dims_t *dims, int n_q_tokens, int n_cols, int n_draft, LayerTcPlan *out)
{
    LayerTcPlan pl;
    const int G = dims->n_q_heads / dims->n_kv_heads;
    pl.R = n_q_tokens * G;
    pl.Rs = n_draft * G;
    const long long rows = (long long)dims->batch * dims->n_kv_heads;
    const int sms = sm_count();
    pl.N = (pl.Rs + 15) / 16 * 16;
    pl.mma_m = pl.R <= 32 ? 64 : 128;
    pl.copies = pl.R <= 16 ? 4 : (pl.R <= 64 ? 2 : 1);
    pl.stages = kLyMaxStages;
    pl.smem = layer_tc_smem_bytes(pl.mma_m, pl.copies, pl.N, pl.stages);
    if (pl.smem > 227 * 1024 && pl.mma_m == 128) {
        pl.stages = 4;
        pl.smem = layer_tc_smem_bytes(pl.mma_m, pl.copies, pl.N, pl.stages);
    }
    // attention-phase stages: with four stages the two operand buffers (2 x N x 512 B: 64 KiB at 64 scoring rows, 32 KiB
    // at 32) are one or two more
    pl.astages = pl.stages;
    if (pl.stages == 4) {
        const int extra = (int)(2 * (size_t)pl.N * kSummaryBytes / kAtStageBytes);
        pl.astages = 4 + (extra > 2 ? 2 : extra);
    }
    pl.n_splits = 1;
    pl.cols_per_split = n_cols;
    pl.workspace = 0;
    if (rows * 2 <= sms && rows >= 1 && pl.R >= 1 && pl.R <= 128 && n_cols >= 1) {
        // Few rows.  Whole rows are still fine while a row's tiles stay within 1.25 times an SM's equal share of the
        // launch (the thread blocks without a row score instead); longer rows would be stragglers and are split.
        const double nt_a = (n_cols + kAtTileCols - 1) / kAtTileCols;
        const double tiles_s = (double)rows * ((dims->max_blocks + kLyTileBlocks - 1) / kLyTileBlocks);
        const double share = ((double)rows * nt_a + 2.0 * tiles_s) / sms;     // 32 KiB units per SM
        if (nt_a > 1.25 * share)
            attn_split_plan(dims, n_q_tokens, n_cols, &pl.n_splits, &pl.cols_per_split, &pl.workspace);
    }
    if (out) *out = pl;
    if (pl.R < 1 || pl.R > 128 || pl.Rs < 1 || pl.Rs > 64 || n_cols < 1 || rows < 1 ||
        rows * (long long)dims->max_blocks > 0x7fffffffLL || pl.smem > 227 * 1024)      // summary rows are indexed with 31 bits
        return false;
    return rows * (long long)pl.n_splits <= 0x7fffffffLL;
}

}  // namespace oasis

extern "C" int oasis_attn_and_score_supported(const oasis_dims_t *dims, int32_t n_q_tokens, int32_t n_cols, int32_t n_draft)
{
    using namespace oasis;
    if (check_dims(dims) != OASIS_OK || n_q_tokens < 1 || n_cols < 1 || n_draft < 1 || dims->batch == 0) return 0;
    return layer_tc_plan(dims, n_q_tokens, n_cols, n_draft, nullptr) ? 1 : 0;
}

extern "C" int oasis_attn_and_score(const oasis_dims_t *dims, const void *q, int32_t n_q_tokens, const void *hbm_pool,
                                    const int32_t *slot_tbl, const int32_t *blk_tbl, int32_t n_cols,
                                    const int32_t *seq_len, float scale, void *out, float *lse, const void *q_draft,
                                    int64_t q_batch_stride, int32_t n_draft, const void *summaries,
                                    const int32_t *n_full_blocks, int32_t reduce_mode, float *scores, void *workspace,
                                    size_t workspace_bytes, void *stream)
{
    using namespace oasis;
    const char *who = "oasis_attn_and_score";
    if (int rc = check_dims(dims)) return rc;
    if (!q || !hbm_pool || !slot_tbl || !blk_tbl || !seq_len || !out || !q_draft || !summaries || !n_full_blocks || !scores)
        return fail(OASIS_ERR_INVALID_ARG, "%s: NULL pointer argument", who);
    if (!aligned16(q) || !aligned16(hbm_pool) || !aligned16(out) || !aligned16(q_draft) || !aligned16(summaries))
        return fail(OASIS_ERR_INVALID_ARG, "%s: q, hbm_pool, out, q_draft and summaries must be 16-byte aligned", who);
    if (n_q_tokens < 1 || n_cols < 1 || n_draft < 1)
        return fail(OASIS_ERR_INVALID_ARG, "%s: n_q_tokens %d, n_cols %d, n_draft %d", who, n_q_tokens, n_cols, n_draft);
    if (reduce_mode != OASIS_REDUCE_MAX && reduce_mode != OASIS_REDUCE_SUM)
        return fail(OASIS_ERR_INVALID_ARG, "%s: reduce_mode %d", who, reduce_mode);
    const int G = dims->n_q_heads / dims->n_kv_heads;
    if (q_batch_stride == 0) q_batch_stride = (int64_t)n_draft * dims->n_q_heads * kHeadDim;
    if ((q_batch_stride * 2) % 16 != 0) return fail(OASIS_ERR_INVALID_ARG, "%s: q_batch_stride %lld", who, (long long)q_batch_stride);
    if (dims->batch == 0) return OASIS_OK;
    // Shapes outside the fused launch (see layer_tc_plan) take the two separate calls.
    const long long rows = (long long)dims->batch * dims->n_kv_heads;
    const int sms = sm_count();
    LayerTcPlan pl;
    if (!layer_tc_plan(dims, n_q_tokens, n_cols, n_draft, &pl))
        return fail(OASIS_ERR_UNSUPPORTED,
                    "%s: %lld rows of %d columns on %d SMs, %d attention rows and %d scoring rows per KV head are outside "
                    "the fused launch; call oasis_sparse_attn and oasis_score_blocks", who, rows, n_cols, sms, pl.R, pl.Rs);
    const int R = pl.R, Rs = pl.Rs, N = pl.N;
    const size_t smem = pl.smem;
    if (pl.workspace > 0) {
        if (!workspace || workspace_bytes < pl.workspace)
            return fail(OASIS_ERR_WORKSPACE, "%s: workspace of %zu bytes required, %zu given", who, pl.workspace, workspace_bytes);
        if (!aligned16(workspace)) return fail(OASIS_ERR_INVALID_ARG, "%s: workspace must be 16-byte aligned", who);
    }
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return fail(OASIS_ERR_CUDA, "%s: cuTensorMapEncodeTiled is not available", who);
    CUtensorMap tmap_kv, tmap_summ;
    {
        // the pool as 8 KiB entries (see attn_tc.cu): one box = one entry, landing as [group][half][part][8 rows][128 B]
        // (bounds-check build with declared extents: the map covers exactly the pool's slots, so a copy by a slot id
        // outside them would read the fill value instead of foreign memory -- and such ids are dropped before that)
        const cuuint64_t pool_parts = (kBoundsCheck && bounds().n_slots < (1ll << 30)) ? (cuuint64_t)(2 * bounds().n_slots)
                                                                                       : (cuuint64_t)1 << 31;
        const cuuint64_t gdim[5] = {64, 8, pool_parts, 2, 2};
        const cuuint64_t gstride[4] = {256, 4096, 128, 2048};
        const cuuint32_t box[5] = {64, 8, 2, 2, 2};
        const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
        CUresult cr = encode(&tmap_kv, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(hbm_pool), gdim, gstride, box,
                             estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (cr != CUDA_SUCCESS) return fail(OASIS_ERR_CUDA, "%s: cuTensorMapEncodeTiled failed (%d)", who, (int)cr);
    }
    {
        // the summaries as rows of 256 bf16 (see score_tc.cu): one box = 64 elements of 128 consecutive blocks
        const cuuint64_t gdim[2] = {256, (cuuint64_t)(rows * dims->max_blocks)};
        const cuuint64_t gstride[1] = {(cuuint64_t)kSummaryBytes};
        const cuuint32_t box[2] = {64, (cuuint32_t)kLyTileBlocks};
        const cuuint32_t estr[2] = {1, 1};
        CUresult cr = encode(&tmap_summ, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(summaries), gdim, gstride,
                             box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (cr != CUDA_SUCCESS) return fail(OASIS_ERR_CUDA, "%s: cuTensorMapEncodeTiled failed (%d)", who, (int)cr);
    }
    LayerTcParams p;
    p.q = (const uint8_t *)q; p.slot_tbl = slot_tbl; p.blk_tbl = blk_tbl; p.seq_len = seq_len;
    p.out = (uint8_t *)out; p.lse = lse;
    p.scale_log2 = scale * kAtLog2e;
    p.T = n_q_tokens; p.Hq = dims->n_q_heads; p.Hkv = dims->n_kv_heads; p.G = G;
    p.n_cols = n_cols; p.R = R; p.items = (int)(rows * pl.n_splits);
    p.n_splits = pl.n_splits; p.cols_per_split = pl.cols_per_split;
    p.part_o = (float *)workspace;
    p.part_lse = p.part_o ? p.part_o + (size_t)p.items * R * kHeadDim : nullptr;
    p.q_draft = (const uint8_t *)q_draft; p.q_batch_stride = q_batch_stride; p.n_full = n_full_blocks; p.scores = scores;
    p.Rs = Rs; p.N = N; p.max_blocks = dims->max_blocks;
    // two accumulators of up to 32 columns fit behind Q; wider ones, and all with two softmax sets (whose second O takes that
    // place), use the S buffers' columns, which the attention phase only touches after the last scoring epilogue
    p.acc_col = (N <= 32 && at_softmax_sets(pl.mma_m, pl.copies) == 1) ? 448 : 0;
    p.tiles_per_bh = (dims->max_blocks + kLyTileBlocks - 1) / kLyTileBlocks;
    p.reduce_sum = reduce_mode == OASIS_REDUCE_SUM;
    p.total_tiles = (int)(rows * p.tiles_per_bh);
    p.err = error_word();
    p.n_slots = bounds().n_slots;
    // Equal bytes per SM: an attention tile is 32 KiB, a scoring tile 64 KiB.  The first `n_more` CTAs attend
    // one row more than the others and take correspondingly fewer scoring tiles.
    const int grid = sms;
    const long long items = p.items;
    long long row_tiles = 0;                                   // attention tiles of one row, over its splits
    for (int c0 = 0; c0 < n_cols; c0 += pl.cols_per_split)
        row_tiles += ((c0 + pl.cols_per_split < n_cols ? pl.cols_per_split : n_cols - c0) + kAtTileCols - 1) / kAtTileCols;
    const double nt_a = (double)row_tiles / pl.n_splits;        // per work item
    const long long m_rows = items / grid;
    const int rem = (int)(items % grid);
    if (rem == 0) {
        p.n_more = grid;
        p.w_row = (double)p.total_tiles / (double)grid;
        p.w_free = 0.0;
    } else {
        const double units = ((double)items * nt_a + 2.0 * (double)p.total_tiles) / grid;
        double w_more = (units - (double)(m_rows + 1) * nt_a) / 2.0;
        if (w_more < 0.0) w_more = 0.0;
        p.n_more = rem;
        p.w_row = w_more;
        p.w_free = ((double)p.total_tiles - (double)rem * w_more) / (double)(grid - rem);
    }
    cudaError_t e;
    cudaStream_t st = (cudaStream_t)stream;
    // Programmatic dependent launch: behind another launch of this kernel on the same stream the thread blocks start
    // as soon as an SM has room (their scoring phase depends on nothing the predecessor writes) and wait for the
    // predecessor only before their attention phase (griddepcontrol.wait in the kernel).
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kLyThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
#define OASIS_LAYER_TC_LAUNCH_2(M, C, MU, ST, AST)                                                                            \
    do {                                                                                                                      \
        cfg.blockDim = dim3(ly_threads(M, C));                                                                                \
        e = cudaFuncSetAttribute(layer_tc_kernel<M, C, MU, ST, AST>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  \
        if (e == cudaSuccess) prefer_max_shared_carveout(layer_tc_kernel<M, C, MU, ST, AST>);                                 \
        if (e == cudaSuccess) e = cudaLaunchKernelEx(&cfg, layer_tc_kernel<M, C, MU, ST, AST>, tmap_kv, tmap_summ, p);         \
    } while (0)
#define OASIS_LAYER_TC_LAUNCH(M, C, ST, AST)                          \
    do {                                                              \
        if (pl.n_splits > 1) OASIS_LAYER_TC_LAUNCH_2(M, C, 2, ST, AST);  \
        else if (items > grid) OASIS_LAYER_TC_LAUNCH_2(M, C, 1, ST, AST); \
        else OASIS_LAYER_TC_LAUNCH_2(M, C, 0, ST, AST);               \
    } while (0)
    if (R <= 16) OASIS_LAYER_TC_LAUNCH(64, 4, 6, 6);
    else if (R <= 32) OASIS_LAYER_TC_LAUNCH(64, 2, 6, 6);
    else if (R <= 64 && pl.stages == 6) OASIS_LAYER_TC_LAUNCH(128, 2, 6, 6);
    else if (R <= 64 && pl.astages == 6) OASIS_LAYER_TC_LAUNCH(128, 2, 4, 6);
    else if (R <= 64 && pl.astages == 5) OASIS_LAYER_TC_LAUNCH(128, 2, 4, 5);
    else if (R <= 64) OASIS_LAYER_TC_LAUNCH(128, 2, 4, 4);
    else if (pl.stages == 6) OASIS_LAYER_TC_LAUNCH(128, 1, 6, 6);
    else if (pl.astages == 6) OASIS_LAYER_TC_LAUNCH(128, 1, 4, 6);
    else if (pl.astages == 5) OASIS_LAYER_TC_LAUNCH(128, 1, 4, 5);
    else OASIS_LAYER_TC_LAUNCH(128, 1, 4, 4);
#undef OASIS_LAYER_TC_LAUNCH
#undef OASIS_LAYER_TC_LAUNCH_2
    if (e != cudaSuccess) return fail(OASIS_ERR_CUDA, "%s: launch with %zu B of shared memory: %s", who, smem, cudaGetErrorString(e));
    if (int rc = check_launch(who)) return rc;
    if (pl.n_splits > 1)
        return launch_attn_combine_after(dims, n_q_tokens, out, lse, p.part_o, p.part_lse, pl.n_splits, st, who);
    return OASIS_OK;
}
