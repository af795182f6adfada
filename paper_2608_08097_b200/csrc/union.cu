// Head-union block set for partial transfer (Sec. 4.4.1): per request, the union over the KV
// heads of the selected blocks, at block granularity, as an ascending id list.
//
// One CTA per request: a bitmap over the logical block ids in shared memory (atomicOr per
// selected id), then an ordered compaction -- every thread owns consecutive 32-bit words,
// a block-wide exclusive scan of their population counts gives the output position, and the
// set bits are written in ascending order.  Integer work on a few KiB per request.
#include "common.cuh"

namespace oasis {

constexpr int kUnionThreads = 256;

__global__ void __launch_bounds__(kUnionThreads)
union_blocks_kernel(const int32_t *__restrict__ sel, int Hkv, int max_blocks, int sel_cols, int k,
                    int max_union, int n_words, int32_t *__restrict__ union_idx, int32_t *__restrict__ n_union)
{
    extern __shared__ uint32_t bits[];                       // [n_words]
    __shared__ uint32_t warp_sum[kUnionThreads / 32];
    __shared__ uint32_t total;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x;

    for (int i = tid; i < n_words; i += kUnionThreads) bits[i] = 0;
    __syncthreads();
    for (int i = tid; i < Hkv * k; i += kUnionThreads) {
        const int h = i / k, r = i % k;
        const int j = sel[((long long)b * Hkv + h) * sel_cols + r];
        if (j >= 0 && j < max_blocks) atomicOr(&bits[j >> 5], 1u << (j & 31));
    }
    __syncthreads();

    // thread t owns words [t * wpt, (t + 1) * wpt)
    const int wpt = (n_words + kUnionThreads - 1) / kUnionThreads;
    const int w0 = tid * wpt, w1 = min(w0 + wpt, n_words);
    uint32_t mine = 0;
    for (int w = w0; w < w1; ++w) mine += __popc(bits[w]);
    uint32_t incl = mine;
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
        const uint32_t o = __shfl_up_sync(0xffffffffu, incl, m);
        if (lane >= m) incl += o;
    }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const uint32_t c = lane < kUnionThreads / 32 ? warp_sum[lane] : 0u;
        uint32_t s = c;
#pragma unroll
        for (int m = 1; m < 32; m <<= 1) {
            const uint32_t o = __shfl_up_sync(0xffffffffu, s, m);
            if (lane >= m) s += o;
        }
        if (lane < kUnionThreads / 32) warp_sum[lane] = s - c;      // exclusive prefix per warp
        if (lane == 31) total = s;
    }
    __syncthreads();
    uint32_t pos = warp_sum[warp] + incl - mine;
    int32_t *out = union_idx + (long long)b * max_union;
    for (int w = w0; w < w1; ++w) {
        uint32_t word = bits[w];
        while (word) {
            const int bit = __ffs(word) - 1;
            word &= word - 1;
            if (pos < (uint32_t)max_union) out[pos] = w * 32 + bit;
            ++pos;
        }
    }
    const uint32_t n = total;
    for (int i = (int)n + tid; i < max_union; i += kUnionThreads) out[i] = -1;
    if (tid == 0) n_union[b] = (int32_t)n;
}

}  // namespace oasis

extern "C" int oasis_union_blocks(const oasis_dims_t *dims, const int32_t *sel, int32_t sel_cols, int32_t k,
                                  int32_t max_union, int32_t *union_idx, int32_t *n_union, void *stream)
{
    using namespace oasis;
    if (int rc = check_dims(dims)) return rc;
    if (!sel || !union_idx || !n_union)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_union_blocks: NULL pointer argument");
    if (k < 1 || k > sel_cols) return fail(OASIS_ERR_INVALID_ARG, "oasis_union_blocks: k %d (sel_cols %d)", k, sel_cols);
    if (max_union < 1) return fail(OASIS_ERR_INVALID_ARG, "oasis_union_blocks: max_union %d < 1", max_union);
    if (dims->max_blocks > (1 << 20))
        return fail(OASIS_ERR_UNSUPPORTED, "oasis_union_blocks: max_blocks %d > %d", dims->max_blocks, 1 << 20);
    if (dims->batch == 0) return OASIS_OK;
    const int n_words = (dims->max_blocks + 31) / 32;
    const size_t smem = (size_t)n_words * 4;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(union_blocks_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return fail(OASIS_ERR_CUDA, "oasis_union_blocks: shared memory %zu B: %s", smem, cudaGetErrorString(e));
    }
    prefer_max_shared_carveout(union_blocks_kernel);
    union_blocks_kernel<<<dims->batch, kUnionThreads, smem, (cudaStream_t)stream>>>(
        sel, dims->n_kv_heads, dims->max_blocks, sel_cols, k, max_union, n_words, union_idx, n_union);
    return check_launch("oasis_union_blocks");
}
