// Step 0: per-block min/max key summaries (Sec. 4.2.1, Fig. "Look-ahead attention").
//
// One warp per (request, new block, KV head): it streams the 4 KiB K part of the entry
// with 16-byte loads (two 256-byte key rows per warp-wide load), keeps a running bf16x2
// min/max per lane, folds the two half-warps together and writes the 256-byte min row
// and max row.  bf16 min/max are exact, so the result does not depend on the order.
// Algorithmic traffic: 4096 B read + 512 B written per (block, head).
#include "common.cuh"

namespace oasis {

constexpr int kSummWarps = 4;

// bf16x2 min / max on raw 32-bit patterns (exact: the result is one of the inputs)
__device__ __forceinline__ uint32_t min2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("min.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t max2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

__device__ __forceinline__ void
summarise_item(const uint8_t *__restrict__ kv_pool, const int32_t *__restrict__ block_table,
               const int32_t *__restrict__ first_block, const int32_t *__restrict__ n_blocks,
               uint8_t *__restrict__ summaries, int Hkv, int max_blocks, int max_new, long long n_items, const Bounds &bd)
{
    const int lane = threadIdx.x & 31;
    const long long item = (long long)blockIdx.x * kSummWarps + (threadIdx.x >> 5);
    if (item >= n_items) return;
    const int h = (int)(item % Hkv);
    const int jj = (int)((item / Hkv) % max_new);
    const int b = (int)(item / ((long long)Hkv * max_new));
    if (jj >= n_blocks[b]) return;
    const int j = first_block[b] + jj;
    if (j < 0 || j >= max_blocks) {
        in_range(j, max_blocks, bd, kErrBlockCount);       // (checked build: reported; always skipped)
        return;
    }
    const long long phys = block_table[(long long)b * max_blocks + j];
    if (!in_range(phys * Hkv + h, bd.n_entries, bd, kErrHostEntry)) return;
    const uint8_t *src = kv_pool + (phys * Hkv + h) * (long long)kEntryBytes;

    // lane -> 16-byte chunk (lane & 15) of token (lane >> 4) + 2*i
    uint4 v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = ld_stream_v4(src + i * 512 + lane * 16);
    uint32_t lo[4] = {v[0].x, v[0].y, v[0].z, v[0].w};
    uint32_t hi[4] = {v[0].x, v[0].y, v[0].z, v[0].w};
#pragma unroll
    for (int i = 1; i < 8; ++i) {
        const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            lo[p] = min2(lo[p], w[p]);
            hi[p] = max2(hi[p], w[p]);
        }
    }
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        lo[p] = min2(lo[p], __shfl_xor_sync(0xffffffffu, lo[p], 16));
        hi[p] = max2(hi[p], __shfl_xor_sync(0xffffffffu, hi[p], 16));
    }
    uint8_t *dst = summaries + (((long long)b * Hkv + h) * max_blocks + j) * (long long)kSummaryBytes;
    // lanes 0..15 write the min row, lanes 16..31 the max row
    const bool low_half = lane < 16;
    uint4 o;
    o.x = low_half ? lo[0] : hi[0];
    o.y = low_half ? lo[1] : hi[1];
    o.z = low_half ? lo[2] : hi[2];
    o.w = low_half ? lo[3] : hi[3];
    *reinterpret_cast<uint4 *>(dst + lane * 16) = o;
}

__global__ void __launch_bounds__(kSummWarps * 32)
build_summaries_kernel(const uint8_t *__restrict__ kv_pool, const int32_t *__restrict__ block_table,
                       const int32_t *__restrict__ first_block, const int32_t *__restrict__ n_blocks,
                       uint8_t *__restrict__ summaries, int B, int Hkv, int max_blocks,
                       int max_new, long long n_items, const Bounds bd)
{
    summarise_item(kv_pool, block_table, first_block, n_blocks, summaries, Hkv, max_blocks, max_new, n_items, bd);
}

// The same for several layers in one launch (blockIdx.y = layer): a decode step appends to every layer's cache
// at once, and one launch instead of one per layer keeps 31 small launches out of the step.
struct SummLayers {
    const uint8_t *kv_pool[OASIS_MAX_LAYERS];
    const int32_t *block_table[OASIS_MAX_LAYERS];
    uint8_t *summaries[OASIS_MAX_LAYERS];
};

__global__ void __launch_bounds__(kSummWarps * 32)
build_summaries_layers_kernel(const __grid_constant__ SummLayers ly, const int32_t *__restrict__ first_block,
                              const int32_t *__restrict__ n_blocks, int Hkv, int max_blocks, int max_new, long long n_items,
                              const Bounds bd)
{
    const int l = blockIdx.y;
    summarise_item(ly.kv_pool[l], ly.block_table[l], first_block, n_blocks, ly.summaries[l], Hkv, max_blocks, max_new,
                   n_items, bd);
}

}  // namespace oasis

extern "C" int oasis_build_summaries(const oasis_dims_t *dims, const void *kv_pool,
                                     const int32_t *block_table, const int32_t *first_block,
                                     const int32_t *n_blocks, int32_t max_new_blocks,
                                     void *summaries, void *stream)
{
    using namespace oasis;
    if (int rc = check_dims(dims)) return rc;
    if (!kv_pool || !block_table || !first_block || !n_blocks || !summaries)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_build_summaries: NULL pointer argument");
    if (!aligned16(kv_pool) || !aligned16(summaries))
        return fail(OASIS_ERR_INVALID_ARG, "oasis_build_summaries: kv_pool and summaries must be 16-byte aligned");
    if (max_new_blocks < 0 || max_new_blocks > dims->max_blocks)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_build_summaries: max_new_blocks %d outside [0, %d]",
                    max_new_blocks, dims->max_blocks);
    const long long n_items = (long long)dims->batch * dims->n_kv_heads * max_new_blocks;
    if (n_items == 0) return OASIS_OK;
    const long long grid = (n_items + kSummWarps - 1) / kSummWarps;
    if (grid > 0x7fffffffLL) return fail(OASIS_ERR_UNSUPPORTED, "oasis_build_summaries: too many blocks");
    prefer_max_shared_carveout(build_summaries_kernel);
    build_summaries_kernel<<<(unsigned)grid, kSummWarps * 32, 0, (cudaStream_t)stream>>>(
        (const uint8_t *)kv_pool, block_table, first_block, n_blocks, (uint8_t *)summaries,
        dims->batch, dims->n_kv_heads, dims->max_blocks, max_new_blocks, n_items, bounds());
    return check_launch("oasis_build_summaries");
}

extern "C" int oasis_build_summaries_layers(const oasis_dims_t *dims, int32_t n_layers, const void *const *kv_pools,
                                            const int32_t *const *block_tables, const int32_t *first_block,
                                            const int32_t *n_blocks, int32_t max_new_blocks, void *const *summaries,
                                            void *stream)
{
    using namespace oasis;
    const char *who = "oasis_build_summaries_layers";
    if (int rc = check_dims(dims)) return rc;
    if (n_layers < 0 || n_layers > OASIS_MAX_LAYERS)
        return fail(OASIS_ERR_INVALID_ARG, "%s: n_layers %d outside [0, %d]", who, n_layers, OASIS_MAX_LAYERS);
    if (!kv_pools || !block_tables || !summaries || !first_block || !n_blocks)
        return fail(OASIS_ERR_INVALID_ARG, "%s: NULL pointer argument", who);
    if (max_new_blocks < 0 || max_new_blocks > dims->max_blocks)
        return fail(OASIS_ERR_INVALID_ARG, "%s: max_new_blocks %d outside [0, %d]", who, max_new_blocks, dims->max_blocks);
    SummLayers ly = {};
    for (int l = 0; l < n_layers; ++l) {
        if (!kv_pools[l] || !block_tables[l] || !summaries[l])
            return fail(OASIS_ERR_INVALID_ARG, "%s: NULL pointer for layer %d", who, l);
        if (!aligned16(kv_pools[l]) || !aligned16(summaries[l]))
            return fail(OASIS_ERR_INVALID_ARG, "%s: kv_pools and summaries must be 16-byte aligned (layer %d)", who, l);
        ly.kv_pool[l] = (const uint8_t *)kv_pools[l];
        ly.block_table[l] = block_tables[l];
        ly.summaries[l] = (uint8_t *)summaries[l];
    }
    const long long n_items = (long long)dims->batch * dims->n_kv_heads * max_new_blocks;
    if (n_items == 0 || n_layers == 0) return OASIS_OK;
    const long long grid = (n_items + kSummWarps - 1) / kSummWarps;
    if (grid > 0x7fffffffLL) return fail(OASIS_ERR_UNSUPPORTED, "%s: too many blocks", who);
    prefer_max_shared_carveout(build_summaries_layers_kernel);
    build_summaries_layers_kernel<<<dim3((unsigned)grid, (unsigned)n_layers), kSummWarps * 32, 0, (cudaStream_t)stream>>>(
        ly, first_block, n_blocks, dims->n_kv_heads, dims->max_blocks, max_new_blocks, n_items, bounds());
    return check_launch(who);
}
