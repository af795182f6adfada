// Step 1: entry point of the block scoring with the draft queries (Sec. 4.2.1): argument checks,
// then the tcgen05 / TMA kernel of score_tc.cu.
//
// U(q, j) = sum_x max(q_x * min_jx, q_x * max_jx) equals  q^- . min_j + q^+ . max_j  with
// q^- = min(q, 0), q^+ = max(q, 0), because min_j <= max_j coordinate-wise.  A summary is stored
// as [min row | max row] = 256 consecutive bf16, so the scores of the R = Td * G query rows that
// share a KV head against a run of blocks are a small dense contraction against ( q^- | q^+ ),
// followed by a max (or sum) over the R rows.  Every product of two bf16 values is exact in fp32,
// so only the order of the fp32 additions differs from a scalar evaluation.
#include "common.cuh"

namespace oasis {

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
    return score_blocks_tc(dims, q_draft, q_batch_stride, n_draft, summaries, n_full_blocks, reduce_mode, scores,
                           error_word(), (cudaStream_t)stream);
}
