// Step 1: block scores from the draft queries (Sec. 4.2.1).
//
// U(q, j) = sum_x max(q_x * min_jx, q_x * max_jx) equals  q^- . min_j + q^+ . max_j  with
// q^- = min(q, 0), q^+ = max(q, 0), because min_j <= max_j coordinate-wise.  A summary is
// stored as [min row | max row] = 256 consecutive bf16, so the scores of the R = Td * G
// query rows that share a KV head against a run of blocks are the small dense contraction
//     [R x 256] ( q^- | q^+ )  x  [256 x blocks] (summaries, one column per block)
// followed by a max (or sum) over the R rows.  Every product of two bf16 values is exact in
// fp32, so only the order of the fp32 additions differs from a scalar evaluation.
//
// Kernel: one CTA per (request, KV head, chunk of blocks).  The summaries are streamed
// exactly once, straight from global memory into the B fragments of mma.sync.m16n8k16:
// lane (g = lane / 4, t = lane % 4) reads, for block g of an 8-block tile, the 16 bytes at
// element offset 32 * c + 8 * t (c = 0..7).  The contraction index is permuted accordingly
// when the A fragments (q^- | q^+) are built, which is legal because a dot product does not
// care about the order of its terms.  A warp-wide load therefore touches 8 blocks x 64
// contiguous bytes, all sectors fully used.  With at most 16 rows the A fragments live in
// registers for the whole chunk; with more rows they are re-read from shared memory.
// Algorithmic traffic: 512 B read + 4 B written per (request, KV head, block).
#include <math_constants.h>

#include <cstdlib>

#include "common.cuh"

namespace oasis {

constexpr int kScoreWarps = 4;
constexpr int kScoreTilesPerIter = 2;                           // 8-block MMA tiles per warp iteration
constexpr int kScoreBlocksPerIter = 8 * kScoreTilesPerIter;     // blocks per warp iteration
constexpr int kScoreCtaBlocksPerIter = kScoreWarps * kScoreBlocksPerIter;
constexpr int kQRowBytes = 512 + 16;                            // (q^- | q^+) row, padded against bank conflicts

struct ScoreParams {
    const uint8_t *q;          // draft queries
    long long q_batch_stride;  // elements
    const uint8_t *summaries;
    const int32_t *n_full;
    float *scores;
    int Hq, Hkv, G, Td, R, max_blocks, blocks_per_cta, chunks_per_row, reduce_sum;
};

template <int N_MT>
__global__ void __launch_bounds__(kScoreWarps * 32)
score_blocks_kernel(const ScoreParams p)
{
    extern __shared__ __align__(16) uint8_t smem[];   // [N_MT*16][kQRowBytes]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int chunk = blockIdx.x % p.chunks_per_row;
    const int bh = blockIdx.x / p.chunks_per_row;
    const int b = bh / p.Hkv, h = bh % p.Hkv;
    const int n_full = p.n_full[b];
    const int blk_begin = chunk * p.blocks_per_cta;
    const int blk_end = min(blk_begin + p.blocks_per_cta, p.max_blocks);
    float *out = p.scores + (long long)bh * p.max_blocks;

    if (blk_begin >= n_full) {           // nothing to score in this chunk
        for (int j = blk_begin + tid; j < blk_end; j += blockDim.x) out[j] = -CUDART_INF_F;
        return;
    }

    // ---- build ( q^- | q^+ ) rows in shared memory ------------------------------------
    // row r < R is query (token r / G, head h*G + r % G); rows past R repeat earlier rows
    // (max mode: does not change the max) or are zero (sum mode).
    constexpr int ROWS = N_MT * 16;
    for (int i = tid; i < ROWS * 16; i += blockDim.x) {
        const int row = i >> 4, c16 = i & 15;              // 16-byte chunk of the 256-byte query row
        uint4 v = make_uint4(0, 0, 0, 0);
        const bool live = row < p.R || !p.reduce_sum;
        if (live) {
            const int r = row % p.R;
            const int tq = r / p.G, a = h * p.G + r % p.G;
            const uint8_t *src = p.q + ((long long)b * p.q_batch_stride + ((long long)tq * p.Hq + a) * kHeadDim) * 2 + c16 * 16;
            v = *reinterpret_cast<const uint4 *>(src);
        }
        const __nv_bfloat162 zero2 = __floats2bfloat162_rn(0.f, 0.f);
        uint4 neg, pos;
        const __nv_bfloat162 *f = reinterpret_cast<const __nv_bfloat162 *>(&v);
        __nv_bfloat162 *n2 = reinterpret_cast<__nv_bfloat162 *>(&neg);
        __nv_bfloat162 *p2 = reinterpret_cast<__nv_bfloat162 *>(&pos);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            n2[e] = __hmin2(f[e], zero2);
            p2[e] = __hmax2(f[e], zero2);
        }
        *reinterpret_cast<uint4 *>(smem + row * kQRowBytes + c16 * 16) = neg;         // pairs with the min row
        *reinterpret_cast<uint4 *>(smem + row * kQRowBytes + 256 + c16 * 16) = pos;   // pairs with the max row
    }
    __syncthreads();

    // A fragments of k-step s = 2c + u: rows g and g+8, elements 32c + 8t + 4u + {0,1} (a0/a1)
    // and + 2 (a2/a3) of the (q^- | q^+) row -- the same elements the B loads below deliver.
    uint32_t afrag[N_MT == 1 ? 16 : 1][4];
    if constexpr (N_MT == 1) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint4 lo = *reinterpret_cast<const uint4 *>(smem + g * kQRowBytes + (32 * c + 8 * t) * 2);
            const uint4 hi = *reinterpret_cast<const uint4 *>(smem + (g + 8) * kQRowBytes + (32 * c + 8 * t) * 2);
            afrag[2 * c][0] = lo.x; afrag[2 * c][1] = hi.x; afrag[2 * c][2] = lo.y; afrag[2 * c][3] = hi.y;
            afrag[2 * c + 1][0] = lo.z; afrag[2 * c + 1][1] = hi.z; afrag[2 * c + 1][2] = lo.w; afrag[2 * c + 1][3] = hi.w;
        }
    }

    const uint8_t *summ = p.summaries + (long long)bh * p.max_blocks * kSummaryBytes;
    const int last_blk = p.max_blocks - 1;

    for (int j0 = blk_begin + warp * kScoreBlocksPerIter; j0 < blk_end; j0 += kScoreCtaBlocksPerIter) {
        if (j0 >= n_full) {              // whole warp tile past the candidates
            if (lane < kScoreBlocksPerIter && j0 + lane < blk_end) out[j0 + lane] = -CUDART_INF_F;
            continue;
        }
        // ---- stream 16 summaries: 16 independent 16-byte loads per lane ----------------
        uint4 bv[kScoreTilesPerIter][8];
#pragma unroll
        for (int nt = 0; nt < kScoreTilesPerIter; ++nt) {
            const int j = min(j0 + nt * 8 + g, last_blk);
            const uint8_t *src = summ + (long long)j * kSummaryBytes + t * 16;
#pragma unroll
            for (int c = 0; c < 8; ++c) bv[nt][c] = ld_stream_v4(src + c * 64);
        }
        float res[kScoreTilesPerIter][2];
#pragma unroll
        for (int nt = 0; nt < kScoreTilesPerIter; ++nt) {
            res[nt][0] = res[nt][1] = p.reduce_sum ? 0.f : -CUDART_INF_F;
        }
#pragma unroll
        for (int mt = 0; mt < N_MT; ++mt) {
            float acc[kScoreTilesPerIter][4];
#pragma unroll
            for (int nt = 0; nt < kScoreTilesPerIter; ++nt)
                acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                uint32_t a0[4], a1[4];
                if constexpr (N_MT == 1) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) { a0[e] = afrag[2 * c][e]; a1[e] = afrag[2 * c + 1][e]; }
                } else {
                    const uint4 lo = *reinterpret_cast<const uint4 *>(smem + (mt * 16 + g) * kQRowBytes + (32 * c + 8 * t) * 2);
                    const uint4 hi = *reinterpret_cast<const uint4 *>(smem + (mt * 16 + g + 8) * kQRowBytes + (32 * c + 8 * t) * 2);
                    a0[0] = lo.x; a0[1] = hi.x; a0[2] = lo.y; a0[3] = hi.y;
                    a1[0] = lo.z; a1[1] = hi.z; a1[2] = lo.w; a1[3] = hi.w;
                }
#pragma unroll
                for (int nt = 0; nt < kScoreTilesPerIter; ++nt) {
                    mma_bf16_16816(acc[nt], a0, bv[nt][c].x, bv[nt][c].y);
                    mma_bf16_16816(acc[nt], a1, bv[nt][c].z, bv[nt][c].w);
                }
            }
            // acc[nt]: rows g (c0,c1) and g+8 (c2,c3) of this m-tile, blocks 2t, 2t+1 of the tile
#pragma unroll
            for (int nt = 0; nt < kScoreTilesPerIter; ++nt) {
                if (p.reduce_sum) {
                    res[nt][0] += acc[nt][0] + acc[nt][2];
                    res[nt][1] += acc[nt][1] + acc[nt][3];
                } else {
                    res[nt][0] = fmaxf(res[nt][0], fmaxf(acc[nt][0], acc[nt][2]));
                    res[nt][1] = fmaxf(res[nt][1], fmaxf(acc[nt][1], acc[nt][3]));
                }
            }
        }
        // ---- reduce over the 8 row groups (lane bits 2..4) and store ---------------------
#pragma unroll
        for (int nt = 0; nt < kScoreTilesPerIter; ++nt) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float v = res[nt][e];
#pragma unroll
                for (int m = 4; m < 32; m <<= 1) {
                    const float o = __shfl_xor_sync(0xffffffffu, v, m);
                    v = p.reduce_sum ? v + o : fmaxf(v, o);
                }
                res[nt][e] = v;
            }
            if (g == 0) {
                const int j = j0 + nt * 8 + 2 * t;
                if (j < blk_end) out[j] = j < n_full ? res[nt][0] : -CUDART_INF_F;
                if (j + 1 < blk_end) out[j + 1] = j + 1 < n_full ? res[nt][1] : -CUDART_INF_F;
            }
        }
    }
}

int score_blocks_tc(const oasis_dims_t *dims, const void *q_draft, int64_t q_batch_stride, int32_t n_draft,
                    const void *summaries, const int32_t *n_full_blocks, int32_t reduce_mode, float *scores,
                    int32_t *err_word, cudaStream_t st);          // score_tc.cu

}  // namespace oasis

extern "C" int oasis_score_blocks(const oasis_dims_t *dims, const void *q_draft,
                                  int64_t q_batch_stride, int32_t n_draft, const void *summaries,
                                  const int32_t *n_full_blocks, int32_t reduce_mode, float *scores,
                                  void *stream)
{
    using namespace oasis;
    if (int rc = check_dims(dims)) return rc;
    if (!q_draft || !summaries || !n_full_blocks || !scores)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_score_blocks: NULL pointer argument");
    if (!aligned16(q_draft) || !aligned16(summaries))
        return fail(OASIS_ERR_INVALID_ARG, "oasis_score_blocks: q_draft and summaries must be 16-byte aligned");
    if (n_draft < 1) return fail(OASIS_ERR_INVALID_ARG, "oasis_score_blocks: n_draft %d < 1", n_draft);
    if (reduce_mode != OASIS_REDUCE_MAX && reduce_mode != OASIS_REDUCE_SUM)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_score_blocks: reduce_mode %d", reduce_mode);
    const int G = dims->n_q_heads / dims->n_kv_heads;
    const int R = n_draft * G;
    if (R > 128) return fail(OASIS_ERR_UNSUPPORTED, "oasis_score_blocks: n_draft * group = %d rows > 128", R);
    if (q_batch_stride < (int64_t)n_draft * dims->n_q_heads * kHeadDim || q_batch_stride % 8 != 0)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_score_blocks: q_batch_stride %lld", (long long)q_batch_stride);
    if (dims->batch == 0) return OASIS_OK;
    if ((long long)dims->batch * dims->n_kv_heads * dims->max_blocks > 0x7fffffffLL)
        return fail(OASIS_ERR_UNSUPPORTED, "oasis_score_blocks: more than 2^31 summary rows");
    {
        static const bool legacy = getenv("OASIS_SCORE_MMA_SYNC") != nullptr;   // development switch
        if (!legacy)
            return score_blocks_tc(dims, q_draft, q_batch_stride, n_draft, summaries, n_full_blocks, reduce_mode,
                                   scores, error_word(), (cudaStream_t)stream);
    }

    ScoreParams p;
    p.q = (const uint8_t *)q_draft;
    p.q_batch_stride = q_batch_stride;
    p.summaries = (const uint8_t *)summaries;
    p.n_full = n_full_blocks;
    p.scores = scores;
    p.Hq = dims->n_q_heads; p.Hkv = dims->n_kv_heads; p.G = G; p.Td = n_draft; p.R = R;
    p.max_blocks = dims->max_blocks;
    p.reduce_sum = reduce_mode == OASIS_REDUCE_SUM;
    // Chunk of blocks per CTA: a multiple of one CTA iteration, small enough to give every
    // SM several CTAs, large enough to amortise the query set-up.
    const long long rows = (long long)dims->batch * dims->n_kv_heads;
    const long long want_ctas = 8LL * sm_count();
    long long per_row = (want_ctas + rows - 1) / rows;
    long long bpc = (dims->max_blocks + per_row - 1) / per_row;
    bpc = (bpc + kScoreCtaBlocksPerIter - 1) / kScoreCtaBlocksPerIter * kScoreCtaBlocksPerIter;
    if (bpc < 2 * kScoreCtaBlocksPerIter) bpc = 2 * kScoreCtaBlocksPerIter;
    p.blocks_per_cta = (int)bpc;
    p.chunks_per_row = (int)((dims->max_blocks + bpc - 1) / bpc);
    const long long grid = rows * p.chunks_per_row;
    if (grid > 0x7fffffffLL) return fail(OASIS_ERR_UNSUPPORTED, "oasis_score_blocks: grid too large");

    const int n_mt = (R + 15) / 16;
    const size_t smem = (size_t)n_mt * 16 * kQRowBytes;
    cudaStream_t st = (cudaStream_t)stream;
#define OASIS_SCORE_LAUNCH(NMT)                                                                   \
    do {                                                                                          \
        if (smem > 48 * 1024)                                                                     \
            cudaFuncSetAttribute(score_blocks_kernel<NMT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
        score_blocks_kernel<NMT><<<(unsigned)grid, kScoreWarps * 32, smem, st>>>(p);              \
    } while (0)
    switch (n_mt) {
        case 1: OASIS_SCORE_LAUNCH(1); break;
        case 2: OASIS_SCORE_LAUNCH(2); break;
        case 3: OASIS_SCORE_LAUNCH(3); break;
        case 4: OASIS_SCORE_LAUNCH(4); break;
        case 5: OASIS_SCORE_LAUNCH(5); break;
        case 6: OASIS_SCORE_LAUNCH(6); break;
        case 7: OASIS_SCORE_LAUNCH(7); break;
        default: OASIS_SCORE_LAUNCH(8); break;
    }
#undef OASIS_SCORE_LAUNCH
    return check_launch("oasis_score_blocks");
}
