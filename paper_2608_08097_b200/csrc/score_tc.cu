// Step 1 on the 5th-generation tensor cores: block scores from the draft queries (Sec. 4.2.1).
//
// Since max(q_x * min_jx, q_x * max_jx) = q_x^- * min_jx + q_x^+ * max_jx with q^- = min(q, 0) and q^+ = max(q, 0),
// U(q, j) = q^- . min_j + q^+ . max_j, so the scores of the R query rows that
// share a KV head against a run of blocks are one small dense contraction.  Here the blocks
// are the M dimension (swap-AB): for a tile of 128 consecutive blocks
//     D[128 blocks x N] = A[128 x 256] (summaries, [min | max], K-major)  x  B[256 x N] (q^- | q^+)
// with N = R rounded up to 16, followed by a max (or sum) over the N columns of every row.
//
// A persistent CTA per SM walks a contiguous range of tiles with four warp roles:
//   warp 0     TMA producer: four 2-D tensor copies (128 rows x 128 B, 128-byte swizzle) per tile
//              into a ring of 64 KiB stages, completion on mbarriers.  It starts right after the
//              barrier set-up, while the other warps allocate the tensor memory and build the
//              (q^- | q^+) operand of the first (request, KV head) in the same swizzled layout.
//   warp 1     issues 16 tcgen05.mma (128 x N x 16, bf16 -> fp32) per tile into one of two TMEM
//              accumulators and commits to the stage's "empty" and the accumulator's "full"
//              barrier.  The warp runs converged, elect.sync picks the issuing lane, and its two
//              waits per tile are one predicated probe by two lanes and a ballot.
//   warps 2-5  epilogue: tcgen05.ld of the thread's TMEM lane (= one block), max / sum over its N
//              columns, one coalesced fp32 store per block.
//   warp 6     builds the (q^- | q^+) operand of every further (request, KV head) of the CTA's range
//              ahead of time, into whichever of the two operand buffers is free.
// Bytes in flight are bounded by shared memory (up to three 64 KiB stages per SM), not by
// registers; the tensor work per tile is tiny, so the kernel is HBM bound.
// Every wait is bounded: on a timeout the thread records a code in the error word (if one was
// registered), stops working and the CTA releases its TMEM and returns.
// Algorithmic traffic: 512 B read + 4 B written per (request, KV head, block).
#include <cuda.h>
#include <math_constants.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace oasis {

constexpr int kTcThreads = 224;
constexpr int kTileBlocks = 128;
constexpr int kATileBytes = kTileBlocks * kSummaryBytes;   // 64 KiB
constexpr int kSubTileBytes = kTileBlocks * 128;           // one 64-element K chunk of the tile: 16 KiB
constexpr int kMaxStages = 3;

struct ScoreTcParams {
    const uint8_t *q;
    long long q_batch_stride;
    const int32_t *n_full;
    float *scores;
    int32_t *err;
    int Hq, Hkv, G, R, N, max_blocks, tiles_per_bh, reduce_sum, stages, tmem_cols, n_bbuf;
    long long total_tiles;
};

__global__ void __launch_bounds__(kTcThreads, 1)
score_tc_kernel(const __grid_constant__ CUtensorMap tmap, const ScoreTcParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t a_u32 = base;                                        // [stages][64 KiB]
    const uint32_t b_bytes = (uint32_t)p.N * kSummaryBytes;
    const uint32_t b_u32 = a_u32 + (uint32_t)p.stages * kATileBytes;     // [2][N][512 B] as 4 sub-tiles of N x 128 B
    uint8_t *b_ptr = base_ptr + (size_t)p.stages * kATileBytes;
    const uint32_t bar_u32 = b_u32 + p.n_bbuf * b_bytes;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(b_ptr + p.n_bbuf * b_bytes + 128);
    auto bar_full = [&](int s) { return bar_u32 + 8u * s; };
    auto bar_empty = [&](int s) { return bar_u32 + 8u * (kMaxStages + s); };
    auto bar_acc_full = [&](int a) { return bar_u32 + 8u * (2 * kMaxStages + a); };
    auto bar_acc_empty = [&](int a) { return bar_u32 + 8u * (2 * kMaxStages + 2 + a); };
    auto bar_b_full = [&](int a) { return bar_u32 + 8u * (2 * kMaxStages + 4 + a); };
    auto bar_b_empty = [&](int a) { return bar_u32 + 8u * (2 * kMaxStages + 6 + a); };

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    const long long t0 = p.total_tiles * blockIdx.x / gridDim.x;
    const long long t1 = p.total_tiles * (blockIdx.x + 1) / gridDim.x;

    // First tile at or after t (and before t1) that has candidate blocks; t1 if there is none.
    auto next_active = [&](long long t) {
#pragma unroll 1
        for (; t < t1; ++t) {
            const long long bh = t / p.tiles_per_bh;
            const int j0 = (int)(t % p.tiles_per_bh) * kTileBlocks;
            if (j0 < p.n_full[(int)(bh / p.Hkv)]) break;
        }
        return t;
    };
    // (q^- | q^+) rows of one (request, KV head), K-major, 128-byte swizzle: element k of row n
    // lives in sub-tile k / 64.  `nthr` threads (index `me`) share the work; loads are issued
    // eight at a time so their latencies overlap.
    auto build_b = [&](long long bh, int buf, int me, int nthr) {
        build_qpm_operand(b_ptr + (size_t)buf * b_bytes, p.q, p.q_batch_stride, (int)(bh / p.Hkv), (int)(bh % p.Hkv), p.R, p.G, p.Hq,
                          p.N, p.reduce_sum, me, nthr);
    };

    if (tid == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_acc_full(a), 1);
            mbar_init(bar_acc_empty(a), 4);
            mbar_init(bar_b_full(a), 1);
            mbar_init(bar_b_empty(a), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();                             // the barriers exist; the producer starts copying right away
    const long long t_first = next_active(t0);
    uint32_t tmem_base = 0;
    if (warp != 0) {
        // Meanwhile the other five warps allocate the tensor memory and build the operand of the first
        // (request, KV head).
        if (warp == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)p.tmem_cols) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
        if (t_first < t1) build_b(t_first / p.tiles_per_bh, 0, tid - 32, kTcThreads - 32);
        tc_fence_before();
        asm volatile("bar.sync 1, %0;" ::"n"(kTcThreads - 32) : "memory");
        tc_fence_after();
        tmem_base = *tmem_slot;
        if (tid == 32 && t_first < t1) mbar_arrive(bar_b_full(0));
    }

    if (warp == 0) {
        // ---------------------------------------------------------------- producer
        int it = 0;
        bool alive = true;
        long long t = t_first;
#pragma unroll 1
        while (t < t1 && alive) {
            const long long bh = t / p.tiles_per_bh;
            const int j0 = (int)(t % p.tiles_per_bh) * kTileBlocks;
            if (lane == 0) {
                const int s = it % p.stages;
                alive = mbar_wait(bar_empty(s), ((it / p.stages) & 1) ^ 1, p.err, 12);
                if (alive) {
                    mbar_arrive_expect_tx(bar_full(s), kATileBytes);
                    const int y = (int)(bh * p.max_blocks + j0);
                    load_score_tile(a_u32 + s * kATileBytes, &tmap, y, kSubTileBytes, bar_full(s));
                }
            }
            alive = __shfl_sync(0xffffffffu, (int)alive, 0) != 0;
            ++it;
            const long long tn = next_active(t + 1);
            t = tn;
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer (the whole warp, converged)
        {
            const uint32_t idesc = idesc_score(p.N, kTileBlocks);
            int it = 0, bo = -1;
            long long cur_bh = -1;
            bool alive = true;
#pragma unroll 1
            for (long long t = t0; t < t1 && alive; ++t) {
                const long long bh = t / p.tiles_per_bh;
                const int j0 = (int)(t % p.tiles_per_bh) * kTileBlocks;
                const int b = (int)(bh / p.Hkv);
                if (j0 >= p.n_full[b]) continue;
                if (bh != cur_bh) {
                    if (bo >= 0) tc_commit(bar_b_empty(bo % p.n_bbuf));   // earlier MMAs no longer read that operand
                    cur_bh = bh;
                    ++bo;
                    alive = mbar_wait_warp(bar_b_full(bo % p.n_bbuf), (bo / p.n_bbuf) & 1, p.err, 21);
                    if (!alive) break;
                }
                const int acc = it & 1, s = it % p.stages;
alive = mbar_wait_warp2(bar_acc_empty(acc), ((it >> 1) & 1) ^ 1, bar_full(s), (it / p.stages) & 1, p.err, 23);
                if (!alive) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * p.N);
                const uint32_t a_tile = a_u32 + s * kATileBytes;
                const uint32_t b_tile = b_u32 + (bo % p.n_bbuf) * b_bytes;
                issue_score_tile(d_tmem, a_tile, b_tile, p.N, kSubTileBytes, idesc);
                tc_commit(bar_empty(s));         // the stage may be refilled once these MMAs have read it
                tc_commit(bar_acc_full(acc));    // the accumulator is complete
                ++it;
            }
        }
    } else if (warp == 6) {
        // ---------------------------------------------------------------- operand builder
        // Walks the CTA's tiles ahead of everyone else and builds (q^- | q^+) of every further (request, KV head)
        // as soon as an operand buffer is free, so neither the copies nor the MMAs ever wait for it.
        int bo = 0;
        bool alive = true;
        long long cur_bh = t_first < t1 ? t_first / p.tiles_per_bh : -1;
#pragma unroll 1
        for (long long t = t_first < t1 ? next_active(t_first + 1) : t1; t < t1 && alive; t = next_active(t + 1)) {
            const long long bh = t / p.tiles_per_bh;
            if (bh == cur_bh) continue;
            cur_bh = bh;
            ++bo;
            const int buf = bo % p.n_bbuf;
            if (lane == 0) alive = mbar_wait(bar_b_empty(buf), ((bo / p.n_bbuf) & 1) ^ 1, p.err, 11);
            alive = __shfl_sync(0xffffffffu, (int)alive, 0) != 0;
            if (!alive) break;
            build_b(bh, buf, lane, 32);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_b_full(buf));
        }
    } else {
        // ---------------------------------------------------------------- epilogue (warps 2..5)
        const int quarter = warp & 3;            // TMEM lanes [32 * quarter, +32) belong to this warp
        int it = 0;
        bool alive = true;
#pragma unroll 1
        for (long long t = t0; t < t1 && alive; ++t) {
            const long long bh = t / p.tiles_per_bh;
            const int j0 = (int)(t % p.tiles_per_bh) * kTileBlocks;
            const int b = (int)(bh / p.Hkv);
            const int nf = p.n_full[b];
            if (kBoundsCheck && lane == 0 && nf > p.max_blocks) in_range(nf, p.max_blocks + 1, Bounds{0, 0, p.err}, kErrBlockCount);
            const int j = j0 + quarter * 32 + lane;
            float *out = p.scores + bh * p.max_blocks;
            if (j0 >= nf) {
                if (j < p.max_blocks) out[j] = -CUDART_INF_F;
                continue;
            }
            const int acc = it & 1;
            alive = mbar_wait(bar_acc_full(acc), (it >> 1) & 1, p.err, 31);
            if (!alive) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * p.N);
            const float res = reduce_score_row(taddr, p.N, p.reduce_sum);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty(acc));
            if (j < p.max_blocks) out[j] = j < nf ? res : -CUDART_INF_F;
            ++it;
        }
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols)
                     : "memory");
    }
}

// ---- host side -----------------------------------------------------------------------------------------

int score_blocks_tc(const oasis_dims_t *dims, const void *q_draft, int64_t q_batch_stride, int32_t n_draft,
                    const void *summaries, const int32_t *n_full_blocks, int32_t reduce_mode, float *scores,
                    int32_t *err_word, cudaStream_t st)
{
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return fail(OASIS_ERR_CUDA, "oasis_score_blocks: cuTensorMapEncodeTiled is not available");
    const int G = dims->n_q_heads / dims->n_kv_heads;
    const int R = n_draft * G;
    const int N = (R + 15) / 16 * 16;
    const long long rows = (long long)dims->batch * dims->n_kv_heads * dims->max_blocks;

    CUtensorMap tmap;
    const cuuint64_t gdim[2] = {256, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)kSummaryBytes};
    const cuuint32_t box[2] = {64, (cuuint32_t)kTileBlocks};
    const cuuint32_t estr[2] = {1, 1};
    CUresult cr = encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(summaries), gdim, gstride, box,
                         estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return fail(OASIS_ERR_CUDA, "oasis_score_blocks: cuTensorMapEncodeTiled failed (%d)", (int)cr);

    ScoreTcParams p;
    p.q = (const uint8_t *)q_draft;
    p.q_batch_stride = q_batch_stride;
    p.n_full = n_full_blocks;
    p.scores = scores;
    p.err = err_word;
    p.Hq = dims->n_q_heads; p.Hkv = dims->n_kv_heads; p.G = G; p.R = R; p.N = N;
    p.max_blocks = dims->max_blocks;
    p.tiles_per_bh = (dims->max_blocks + kTileBlocks - 1) / kTileBlocks;
    p.reduce_sum = reduce_mode == OASIS_REDUCE_SUM;
    p.stages = N <= 32 ? 3 : 2;
    p.n_bbuf = N <= 64 ? 2 : 1;          // 2 x 64 KiB of tiles + the operand(s) must fit in 227 KiB
    int cols = 32;
    while (cols < 2 * N) cols <<= 1;
    p.tmem_cols = cols;
    p.total_tiles = (long long)dims->batch * dims->n_kv_heads * p.tiles_per_bh;
    const size_t smem = 1024 + (size_t)p.stages * kATileBytes + (size_t)p.n_bbuf * N * kSummaryBytes + 256;
    cudaError_t e = cudaFuncSetAttribute(score_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return fail(OASIS_ERR_CUDA, "oasis_score_blocks: shared memory %zu B: %s", smem, cudaGetErrorString(e));
    prefer_max_shared_carveout(score_tc_kernel);
    long long grid = p.total_tiles < sm_count() ? p.total_tiles : sm_count();
    score_tc_kernel<<<(unsigned)grid, kTcThreads, smem, st>>>(tmap, p);
    return check_launch("oasis_score_blocks");
}

}  // namespace oasis
