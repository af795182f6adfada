// Step 4 on the 5th-generation tensor cores: sparse paged decode attention (Sec. 4.2.1, 4.3).
//
// Work item = (request, KV head, split of the column list).  All query rows that share the KV
// head (G heads x T verify-step tokens, at most 128) are the M rows of every MMA (M = 64 for up to
// 32 rows, else 128), so each staged K/V block is read from HBM once.  A tile is four columns
// = 64 keys (32 KiB of K and V); one CTA per SM keeps a ring of seven such stages in flight.
//
//   warp 0     TMA producer: one 5-D tensor copy per block brings its whole 8 KiB entry (gathered
//              by slot id) as [row group][dim half][K, V][8 rows][128 B] with the 128-byte swizzle,
//              so that the 8-row groups of consecutive blocks are uniformly 4 KiB apart and both
//              the K operand (K-major) and the V operand (key-major) can be described to the MMA.
//              Slot / block tables come 32 columns at a time, one window ahead, by asynchronous
//              copies into two small shared-memory buffers.
//   warp 1     issues S = Q K^T (8 x tcgen05.mma M x 64 x 16, Q read from tensor memory, K from
//              shared memory) into one of four S buffers as soon as a tile has landed and the
//              buffer's previous P V has completed.
//   warp 2     issues O += P V (4 x tcgen05.mma M x 128 x 16, P read from tensor memory, V from
//              shared memory) as soon as the tile's P is written; the commit after P V releases
//              the stage.  Both warps run converged and elect.sync picks the issuing lane: from
//              inside an `if (lane == 0)` branch every tcgen05.mma cost its thread about 60 cycles
//              whatever its shape, from a converged warp the tensor core's own time.
//   warps 3-6  softmax, one thread per MMA row: tcgen05.ld of the row's logits, masking on local
//              blocks only, exp2 against a running reference maximum that is raised lazily (only
//              when a logit exceeds it by 2^8; the O row is then rescaled in tensor memory),
//              running sum in a register, P rounded to bf16 and written back over S with
//              tcgen05.st.  No cross-thread reduction exists anywhere in the softmax.
//              A warp only reaches its own quarter of the tensor-memory lanes and a single warp's
//              instruction rate bounds the softmax, so when the query rows fit several times into
//              the M rows they are replicated (2 or 4 copies) and each copy takes its share of the
//              tile's four blocks, writing P = 0 for the others.  The copies' partial (max, sum, O)
//              are merged through shared memory after the last tile.
//   warps 7-10 only with 65 to 128 query rows (one copy of the rows in 128 MMA rows): a second set of
//              softmax warps.  The two sets take alternate tiles, each with a running maximum, sum
//              and O accumulator of its own (P V of even tiles goes to the first O, of odd tiles to
//              the second; three S buffers), so that one set's waits and tensor-memory traffic
//              overlap the other's exponentials; the two threads of a row merge when it is written.
// After the merge the rows are normalised and written as bf16 (or, when the column list is
// split, as a normalised partial plus its log-sum-exp to the workspace).
// Every wait is bounded; a timeout records a code in the error word and the CTA winds down.
// Algorithmic traffic: 8 KiB per (request, KV head, column) plus Q and O.
#include <cuda.h>
#include <math_constants.h>

#include <cstdlib>

#include "common.cuh"
#include "tc_common.cuh"

namespace oasis {

constexpr int kAtThreads = 224;                             // producer, Q K^T issuer, P V issuer, four softmax warps
// (four more with two softmax sets)
__host__ __device__ constexpr int at_threads(int mma_m, int copies) { return kAtThreads + (at_softmax_sets(mma_m, copies) - 1) * 128; }
struct AttnTcParams {
    const uint8_t *q;
    const int32_t *slot_tbl;
    const int32_t *blk_tbl;
    const int32_t *seq_len;
    uint8_t *out;
    float *lse;
    float *part_o;
    float *part_lse;
    int32_t *err;
    float scale_log2;
    int T, Hq, Hkv, G, n_cols, R, n_splits, cols_per_split, stages;
    long long n_slots;          // bounds-check build: slots of the working-set pool (else unused)
};

// MMA_M = 64 halves the tensor work when the query rows fit; its rows live in tensor-memory lanes
// (m % 16) + 32 * (m / 16), i.e. sixteen per softmax warp.
template <int MMA_M, int COPIES>
__global__ void __launch_bounds__(at_threads(MMA_M, COPIES), 1)
sparse_attn_tc_kernel(const __grid_constant__ CUtensorMap tmap, const AttnTcParams p)
{
    constexpr int RPC = MMA_M / COPIES;                     // MMA rows per copy of the query rows
    constexpr int LANES = MMA_M / 4;                        // lanes of each softmax warp that hold an MMA row
    constexpr int BPC = kAtTileCols / COPIES;               // blocks of a tile each copy handles
    constexpr int SETS = at_softmax_sets(MMA_M, COPIES);    // softmax warp sets, taking alternate tiles
    constexpr int SBUFS = at_s_bufs(SETS);                  // S / P buffers in tensor memory
    constexpr int THREADS = at_threads(MMA_M, COPIES);
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t kv_u32 = base + kAtQBytes;                        // [stages][32 KiB]
    uint8_t *misc = base_ptr + kAtQBytes + (size_t)p.stages * kAtStageBytes;
    const uint32_t bar_u32 = smem_u32(misc);
    auto bar_full = [&](int s) { return bar_u32 + 8u * s; };
    auto bar_empty = [&](int s) { return bar_u32 + 8u * (kAtMaxStages + s); };
    auto bar_s_full = [&](int a) { return bar_u32 + 8u * (2 * kAtMaxStages + a); };
    auto bar_p_full = [&](int a) { return bar_u32 + 8u * (2 * kAtMaxStages + kAtSBufs + a); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(misc + 8 * (2 * kAtMaxStages + 2 * kAtSBufs + 2));
    int32_t *tile_blk = reinterpret_cast<int32_t *>(misc + 8 * (2 * kAtMaxStages + 2 * kAtSBufs + 4));   // [stages][4]
    int32_t *win = reinterpret_cast<int32_t *>(misc + 512);                                             // two table windows

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // a merge launch behind this one (split runs) may bring its thread blocks onto the SMs already; it waits for the partials
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int split = blockIdx.x % p.n_splits;
    const int bh = blockIdx.x / p.n_splits;
    const int b = bh / p.Hkv, h = bh % p.Hkv;
    const int c0 = split * p.cols_per_split;
    const int c1 = min(c0 + p.cols_per_split, p.n_cols);
    const int n_tiles = (c1 - c0 + kAtTileCols - 1) / kAtTileCols;
    const int L = p.seq_len[b];
    const int32_t *slot_row = p.slot_tbl + (long long)bh * p.n_cols;
    const int32_t *blk_row = p.blk_tbl + (long long)bh * p.n_cols;

    // ---- set-up: barriers, tensor memory, Q operand, zeroed stages ------------------------------------
    if (tid == 0) {
        for (int s = 0; s < kAtMaxStages; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
        for (int a = 0; a < kAtSBufs; ++a) { mbar_init(bar_s_full(a), 1); mbar_init(bar_p_full(a), 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();                             // the barriers exist; the producer starts copying right away
    uint32_t tmem_base = 0, tmem_o = 0, tmem_q = 0;
    if (warp != 0) {
        // Meanwhile: warp 1 allocates the tensor memory, and every softmax thread, owner of one MMA row, loads
        // that row of Q (rows are replicated across the copies, rows past R are zero) and then stores it to its
        // tensor-memory lane.
        if (warp == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)kAtTmemCols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
        uint4 v[16];
        if (warp >= 3 && warp < 7) {
            const int m_row = (warp & 3) * LANES + lane;
            const int r = m_row % RPC;
#pragma unroll
            for (int c = 0; c < 16; ++c) v[c] = make_uint4(0, 0, 0, 0);
            if (lane < LANES && r < p.R) {
                const int tq = r / p.G, a = h * p.G + r % p.G;
                const uint4 *src = reinterpret_cast<const uint4 *>(p.q + ((((long long)b * p.T + tq) * p.Hq + a) * kHeadDim) * 2);
#pragma unroll
                for (int c = 0; c < 16; ++c) v[c] = src[c];
            }
        }
        tc_fence_before();
        asm volatile("bar.sync 2, %0;" ::"n"(THREADS - 32) : "memory");
        tc_fence_after();
        tmem_base = *tmem_slot;
        tmem_o = tmem_base + SBUFS * kAtTileKeys;
        tmem_q = tmem_o + SETS * kHeadDim;                           // Q as the A operand: 128 rows x 64 packed columns
        if (warp >= 3 && warp < 7) {
            q_row_to_tmem(tmem_q + ((uint32_t)((warp & 3) * 32) << 16), v);
        }
        tc_fence_before();
        asm volatile("bar.sync 2, %0;" ::"n"(THREADS - 32) : "memory");
        tc_fence_after();
    }

    if (warp == 0) {
        // ---------------------------------------------------------------- producer
        bool alive = true;
        // Table entries come 32 columns (eight tiles) at a time through two window buffers, one window ahead.
        const uint32_t win_u32 = smem_u32(win);
        window_request(win_u32, lane, blk_row, slot_row, c0 + lane, c1);
        int s = 0;
        uint32_t ph = 1;                                             // parity of the "empty" phase to wait for
        for (int i = 0; i < n_tiles && alive; ++i, ph ^= (s + 1 == p.stages), s = (s + 1 == p.stages) ? 0 : s + 1) {
            if ((i & 7) == 0) {
                window_wait();
                window_request(win_u32 + (((i >> 3) + 1) & 1) * kWinBytes, lane, blk_row, slot_row, c0 + (i + 8) * kAtTileCols + lane, c1);
            }
            int blk, slot;
            window_read(win, i, lane, blk, slot);
            if (kBoundsCheck && blk >= 0 && !in_range(slot, p.n_slots, Bounds{0, 0, p.err}, kErrSlot)) blk = -1;
            if (lane == 0) alive = mbar_wait(bar_empty(s), ph, p.err, 41);
            alive = __shfl_sync(0xffffffffu, (int)alive, 0) != 0;
            if (!alive) break;
            stage_attn_tile(lane, blk, slot, tile_blk + s * kAtTileCols, base_ptr + kAtQBytes + (size_t)s * kAtStageBytes,
                            kv_u32 + s * kAtStageBytes, &tmap, bar_full(s));
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- Q K^T issuer (the whole warp, converged)
        {
            const uint32_t idesc = idesc_qk(MMA_M);
            // descriptors: the operand start address occupies the low 14 bits (16-byte units), so offsets are added there
            const uint64_t k_desc0 = smem_desc_sw128_k(kv_u32, kImgGroup);
            bool alive = true;
            int s = 0, sb = 0, s_old = 0;                            // stage and S buffer of tile i; stage of tile i - SBUFS
            uint32_t ph = 0, ph_old = 0;
            for (int i = 0; i < n_tiles && alive; ++i) {
                // the S buffer also held P of tile i - SBUFS: its P V must have completed
                if (i >= SBUFS) {
                    alive = mbar_wait_warp(bar_empty(s_old), ph_old, p.err, 51);
                    ph_old ^= (s_old + 1 == p.stages);
                    s_old = (s_old + 1 == p.stages) ? 0 : s_old + 1;
                }
                alive = alive && mbar_wait_warp(bar_full(s), ph, p.err, 52);
                if (!alive) break;
                tc_fence_after();
                const uint64_t k_desc = k_desc0 + (uint64_t)((s * kAtStageBytes) >> 4);
                const uint32_t d_tmem = tmem_base + (uint32_t)(sb * kAtTileKeys);
                issue_qk_tile(d_tmem, tmem_q, k_desc, idesc);
                tc_commit(bar_s_full(sb));
                ph ^= (s + 1 == p.stages);
                s = (s + 1 == p.stages) ? 0 : s + 1;
                sb = (sb + 1 == SBUFS) ? 0 : sb + 1;
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
            for (int i = 0; i < n_tiles && alive; ++i) {
                alive = mbar_wait_warp(bar_p_full(sb), ph_p, p.err, 53);
                if (!alive) break;
                tc_fence_after();
                const uint64_t v_desc = v_desc0 + (uint64_t)((s * kAtStageBytes) >> 4);
                const uint32_t p_tmem = tmem_base + (uint32_t)(sb * kAtTileKeys);
                // (two softmax sets: even tiles accumulate into the first O, odd tiles into the second)
                issue_pv_tile(tmem_o + (uint32_t)((i % SETS) * kHeadDim), p_tmem, v_desc, idesc, i < SETS);
                tc_commit(bar_empty(s));                             // stage free, and O complete up to this tile
                s = (s + 1 == p.stages) ? 0 : s + 1;
                sb = (sb + 1 == SBUFS) ? 0 : sb + 1;
                ph_p ^= (sb == 0);
            }
        }
    } else {
        // ---------------------------------------------------------------- softmax, one thread per MMA row (two sets: warps
        // 3-6 take the even tiles, warps 7-10 the odd ones)
        const int set = SETS == 2 ? (warp - 3) >> 2 : 0;
        const int quarter = warp & 3;
        const int m_row = quarter * LANES + (lane % LANES);         // MMA row held by this tensor-memory lane
        const int copy = m_row / RPC, row = m_row % RPC;            // which copy of the rows, which query row
        const bool has_row = lane < LANES;
        const bool live_row = has_row && row < p.R;
        const bool live_warp = (quarter * LANES) % RPC < p.R;       // some lane of this warp holds a query row
        // last visible position of this row; MMA rows past R hold zero queries and need no masking (masking them would
        // send their whole warp down the masked path on every tile), lanes without an MMA row see nothing
        const int limit = live_row ? L + row / p.G : (has_row ? 0x3fffffff : -1);
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        float m_ref = -CUDART_INF_F, l_sum = 0.f;
        bool alive = true;
        int s = 0, s_prev = 0;                                      // ring stage of tile i and of this set's previous tile
        uint32_t ph = 0, ph_prev = 0;                               // parities of the "empty" phases that end those tiles
        int sb = set;                                               // S buffer of tile i (SETS < SBUFS)
        uint32_t ph_s = 0;
        ring_advance(s, ph, set, p.stages);
        const uint32_t my_o = tmem_o + (uint32_t)(set * kHeadDim) + lane_base;   // this thread's O row
        for (int i = set; i < n_tiles && alive; i += SETS) {
            alive = mbar_wait(bar_s_full(sb), ph_s, p.err, 61);
            if (!alive) break;
            tc_fence_after();
            const uint32_t s_tmem = tmem_base + lane_base + (uint32_t)(sb * kAtTileKeys);
            if (live_warp)
                alive = softmax_tile<COPIES>(s_tmem, my_o, tile_blk + s * kAtTileCols, copy, limit, has_row,
                                             p.scale_log2, m_ref, l_sum, i >= SETS,
                                             // (the stage of this set's previous tile is released by the commit that follows its
                                             // P V; with at least four stages in the ring the phase parity is unambiguous)
                                             [&] { return mbar_wait(bar_empty(s_prev), ph_prev, p.err, 62); });
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_p_full(sb));
            s_prev = s;
            ph_prev = ph;
            ring_advance(s, ph, SETS, p.stages);
#pragma unroll
            for (int k = 0; k < SETS; ++k) {
                sb = (sb + 1 == SBUFS) ? 0 : sb + 1;
                ph_s ^= (sb == 0);
            }
        }
        // ---- epilogue: merge the copies, normalise, write out ----------------------------------------------
        if (alive && n_tiles > 0)
            alive = mbar_wait(bar_empty((n_tiles - 1) % p.stages), ((n_tiles - 1) / p.stages) & 1, p.err, 63);
        tc_fence_after();
        // the K/V ring is idle now: stage the O rows there.  [128 MMA rows][132 floats], then max and sum.
        float *o_sm = reinterpret_cast<float *>(base_ptr + kAtQBytes);
        float *m_sm = o_sm + 128 * 132;
        float *l_sm = m_sm + 128 * SETS;
        if (SETS == 2) {
            // the two threads of a row exchange maximum and sum; each then merges and writes one half of the output dims,
            // reading both O accumulators at its own tensor-memory lane
            m_sm[set * 128 + m_row] = m_ref;
            l_sm[set * 128 + m_row] = l_sum;
            asm volatile("bar.sync 1, 256;" ::: "memory");          // the eight softmax warps
            const float m_o = m_sm[(set ^ 1) * 128 + m_row], l_o = l_sm[(set ^ 1) * 128 + m_row];
            const float mx = fmaxf(m_ref, m_o);
            const float w_me = mx == -CUDART_INF_F ? 0.f : fast_exp2(m_ref - mx), w_ot = mx == -CUDART_INF_F ? 0.f : fast_exp2(m_o - mx);
            const float den = w_me * l_sum + w_ot * l_o;
            const float inv = den > 0.f ? 1.f / den : 0.f;
            const float lse2 = den > 0.f ? mx + log2f(den) : -CUDART_INF_F;
            const float w_a = set == 0 ? w_me : w_ot, w_b = set == 0 ? w_ot : w_me;   // weights of the first and second accumulator
            const int tq = row / p.G, a = h * p.G + row % p.G;
            const long long orow = ((long long)b * p.T + tq) * p.Hq + a;
            const bool run = n_tiles > 0 && live_warp && alive;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                const int d0 = set * 64 + c * 16;
                uint32_t va[16], vb[16];
                if (run) {
                    tc_ld16(tmem_o + lane_base + d0, va);
                    tc_ld16(tmem_o + kHeadDim + lane_base + d0, vb);
                }
                if (!(live_row && alive)) continue;
                float acc[16];
                // an accumulator whose set saw no key (weight 0) was never written: its contents do not enter
#pragma unroll
                for (int e = 0; e < 16; ++e)
                    acc[e] = ((w_a != 0.f ? w_a * __uint_as_float(va[e]) : 0.f) + (w_b != 0.f ? w_b * __uint_as_float(vb[e]) : 0.f)) * inv;
                if (p.n_splits == 1) {
                    uint4 *dst = reinterpret_cast<uint4 *>(p.out + (orow * kHeadDim + d0) * 2);
#pragma unroll
                    for (int e = 0; e < 2; ++e)
                        dst[e] = make_uint4(pack_bf16x2(acc[8 * e], acc[8 * e + 1]), pack_bf16x2(acc[8 * e + 2], acc[8 * e + 3]),
                                            pack_bf16x2(acc[8 * e + 4], acc[8 * e + 5]), pack_bf16x2(acc[8 * e + 6], acc[8 * e + 7]));
                } else {
                    float4 *dst = reinterpret_cast<float4 *>(p.part_o + ((long long)blockIdx.x * p.R + row) * kHeadDim + d0);
#pragma unroll
                    for (int e = 0; e < 4; ++e) dst[e] = make_float4(acc[4 * e], acc[4 * e + 1], acc[4 * e + 2], acc[4 * e + 3]);
                }
            }
            if (live_row && alive && set == 0) {
                if (p.n_splits == 1) { if (p.lse) p.lse[orow] = lse2 * kAtLn2; }
                else p.part_lse[(long long)blockIdx.x * p.R + row] = lse2;
            }
        } else if (COPIES > 1) {
            if (live_warp && alive && n_tiles > 0) {
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint32_t v[16];
                    tc_ld16(tmem_o + lane_base + c * 16, v);
                    float4 *dst = reinterpret_cast<float4 *>(o_sm + m_row * 132 + c * 16);
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (has_row) dst[e] = make_float4(__uint_as_float(v[4 * e]), __uint_as_float(v[4 * e + 1]),
                                             __uint_as_float(v[4 * e + 2]), __uint_as_float(v[4 * e + 3]));
                }
            }
            if (has_row) {
                m_sm[m_row] = m_ref;
                l_sm[m_row] = l_sum;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");          // the four softmax warps
        }
        if (SETS == 1) {
            // thread -> (query row, slice of the 128 output dims)
            // one copy: the thread that holds a row writes it; several copies: the MMA_M (row, slice) tasks go to
            // the first MMA_M softmax threads
            const int t = COPIES == 1 ? (has_row ? m_row : MMA_M) : quarter * 32 + lane;
            const int orow_idx = t % RPC, dpart = t / RPC;
            constexpr int DLEN = kHeadDim / COPIES;
            const int d0 = dpart * DLEN;
            float acc[DLEN];
            if (COPIES == 1) {                                       // the thread's own O row, read by the whole warp
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint32_t v[16];
                    if (n_tiles > 0 && live_warp && alive) tc_ld16(tmem_o + lane_base + c * 16, v);
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        acc[(c * 16 + e) % DLEN] = (n_tiles > 0 && live_warp && alive) ? __uint_as_float(v[e]) : 0.f;
                }
            }
            if (t < MMA_M && orow_idx < p.R && alive) {
                float mx = -CUDART_INF_F, den = 0.f;
                if (COPIES == 1) {
                    mx = m_ref;
                    den = l_sum;
                } else {
                    float mw[COPIES], wt[COPIES];
#pragma unroll
                    for (int c = 0; c < COPIES; ++c) {
                        mw[c] = m_sm[c * RPC + orow_idx];
                        mx = fmaxf(mx, mw[c]);
                    }
#pragma unroll
                    for (int c = 0; c < COPIES; ++c) {
                        wt[c] = mx == -CUDART_INF_F ? 0.f : fast_exp2(mw[c] - mx);
                        den += wt[c] * l_sm[c * RPC + orow_idx];
                    }
#pragma unroll
                    for (int e = 0; e < DLEN; ++e) acc[e] = 0.f;
                    if (n_tiles > 0) {
#pragma unroll
                        for (int c = 0; c < COPIES; ++c) {
                            if (wt[c] == 0.f) continue;                  // a copy that saw no key holds no O row
                            const float4 *src = reinterpret_cast<const float4 *>(o_sm + (c * RPC + orow_idx) * 132 + d0);
#pragma unroll
                            for (int e = 0; e < DLEN / 4; ++e) {
                                const float4 f = src[e];
                                acc[4 * e] += wt[c] * f.x; acc[4 * e + 1] += wt[c] * f.y;
                                acc[4 * e + 2] += wt[c] * f.z; acc[4 * e + 3] += wt[c] * f.w;
                            }
                        }
                    }
                }
                const float inv = den > 0.f ? 1.f / den : 0.f;
                const float lse2 = den > 0.f ? mx + log2f(den) : -CUDART_INF_F;
                const int tq = orow_idx / p.G, a = h * p.G + orow_idx % p.G;
                const long long orow = ((long long)b * p.T + tq) * p.Hq + a;
                if (p.n_splits == 1) {
                    uint4 *dst = reinterpret_cast<uint4 *>(p.out + (orow * kHeadDim + d0) * 2);
#pragma unroll
                    for (int e = 0; e < DLEN / 8; ++e)
                        dst[e] = make_uint4(pack_bf16x2(acc[8 * e] * inv, acc[8 * e + 1] * inv),
                                            pack_bf16x2(acc[8 * e + 2] * inv, acc[8 * e + 3] * inv),
                                            pack_bf16x2(acc[8 * e + 4] * inv, acc[8 * e + 5] * inv),
                                            pack_bf16x2(acc[8 * e + 6] * inv, acc[8 * e + 7] * inv));
                    if (p.lse && dpart == 0) p.lse[orow] = lse2 * kAtLn2;
                } else {
                    float4 *dst = reinterpret_cast<float4 *>(p.part_o + ((long long)blockIdx.x * p.R + orow_idx) * kHeadDim + d0);
#pragma unroll
                    for (int e = 0; e < DLEN / 4; ++e)
                        dst[e] = make_float4(acc[4 * e] * inv, acc[4 * e + 1] * inv, acc[4 * e + 2] * inv, acc[4 * e + 3] * inv);
                    if (dpart == 0) p.part_lse[(long long)blockIdx.x * p.R + orow_idx] = lse2;
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kAtTmemCols)
                     : "memory");
    }
}

// ---- host side -----------------------------------------------------------------------------------------

size_t attn_tc_smem_bytes(int stages) { return 1024 + kAtQBytes + (size_t)stages * kAtStageBytes + 512 + 2 * kWinBytes; }

int launch_attn_tc(const oasis_dims_t *dims, const void *q, int n_q_tokens, const void *hbm_pool,
                   const int32_t *slot_tbl, const int32_t *blk_tbl, int n_cols, const int32_t *seq_len, float scale,
                   void *out, float *lse, float *part_o, float *part_lse, int n_splits, int cols_per_split,
                   int stages, int32_t *err_word, cudaStream_t st, const char *who)
{
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return fail(OASIS_ERR_CUDA, "%s: cuTensorMapEncodeTiled is not available", who);
    // The pool is seen as rows of 256 bytes, 32 per entry.  Its size is not an argument of the call:
    // the extent only bounds the coordinates, and slot ids always stay inside the caller's pool.
    // dims (innermost first): 64 elements of a row half | 8 rows of a row group | 4 KiB parts (K, V) of all entries |
    // the two 64-dim halves of a row | the two 8-row groups of a part.  One box = one whole 8 KiB entry, landing as
    // [group][half][part][8 rows][128 B], so that 8-row groups of consecutive blocks are uniformly 4096 bytes apart.
    CUtensorMap tmap;
    // (bounds-check build with declared extents: the map covers exactly the pool's slots, so a copy by a slot id
    // outside them would read the fill value instead of foreign memory -- and such ids are dropped before that)
    const cuuint64_t pool_parts = (kBoundsCheck && bounds().n_slots < (1ll << 30)) ? (cuuint64_t)(2 * bounds().n_slots)
                                               : (cuuint64_t)1 << 31;
    const cuuint64_t gdim[5] = {64, 8, pool_parts, 2, 2};
    const cuuint64_t gstride[4] = {256, 4096, 128, 2048};
    const cuuint32_t box[5] = {64, 8, 2, 2, 2};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult cr = encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(hbm_pool), gdim, gstride, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return fail(OASIS_ERR_CUDA, "%s: cuTensorMapEncodeTiled failed (%d)", who, (int)cr);

    AttnTcParams p;
    p.q = (const uint8_t *)q; p.slot_tbl = slot_tbl; p.blk_tbl = blk_tbl; p.seq_len = seq_len;
    p.out = (uint8_t *)out; p.lse = lse; p.part_o = part_o; p.part_lse = part_lse; p.err = err_word;
    p.scale_log2 = scale * kAtLog2e;
    p.T = n_q_tokens; p.Hq = dims->n_q_heads; p.Hkv = dims->n_kv_heads; p.G = p.Hq / p.Hkv;
    p.n_cols = n_cols; p.R = n_q_tokens * p.G; p.n_splits = n_splits; p.cols_per_split = cols_per_split;
    p.stages = stages;
    p.n_slots = bounds().n_slots;
    const size_t smem = attn_tc_smem_bytes(stages);
    const long long grid = (long long)dims->batch * dims->n_kv_heads * n_splits;
    cudaError_t e;
#define OASIS_ATTN_TC_LAUNCH(M, C)                                                                                     \
    do {                                                                                                               \
        e = cudaFuncSetAttribute(sparse_attn_tc_kernel<M, C>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);  \
        if (e == cudaSuccess) prefer_max_shared_carveout(sparse_attn_tc_kernel<M, C>);                                \
        if (e == cudaSuccess) sparse_attn_tc_kernel<M, C><<<(unsigned)grid, at_threads(M, C), smem, st>>>(tmap, p);          \
    } while (0)
    if (p.R <= 16) OASIS_ATTN_TC_LAUNCH(64, 4);          // four copies of <= 16 rows, one block of a tile each
    else if (p.R <= 32) OASIS_ATTN_TC_LAUNCH(64, 2);     // two copies of <= 32 rows, two blocks each
    else if (p.R <= 64) OASIS_ATTN_TC_LAUNCH(128, 2);    // two copies of <= 64 rows: half the softmax work per thread
    else OASIS_ATTN_TC_LAUNCH(128, 1);
#undef OASIS_ATTN_TC_LAUNCH
    if (e != cudaSuccess) return fail(OASIS_ERR_CUDA, "%s: shared memory %zu B: %s", who, smem, cudaGetErrorString(e));
    return check_launch(who);
}

}  // namespace oasis
