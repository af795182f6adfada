// Step 3: gather of selected (block, head) entries from the host-resident full KV cache
// into HBM slots (Sec. 5.1: a gather kernel reads the selected entries from the pinned CPU
// cache through unified addressing and writes them straight into the resident GPU pages).
//
// One warp per 8 KiB entry: sixteen 16-byte loads per lane are issued back to back (the
// whole entry is in flight before the first store), each warp-wide load covering 512
// contiguous bytes, then sixteen stores.  The source may equally be device memory.  Requests
// with a negative source index are skipped, so list lengths never have to be read back by
// the host.  Algorithmic traffic: 8 KiB over the host link and 8 KiB written per request.
#include "common.cuh"

namespace oasis {

constexpr int kStageWarps = 8;

__global__ void __launch_bounds__(kStageWarps * 32)
stage_blocks_kernel(const uint8_t *__restrict__ host_kv, const long long *__restrict__ idx,
                    const int32_t *__restrict__ slots, int n, uint8_t *__restrict__ pool)
{
    const int lane = threadIdx.x & 31;
    const int warps_total = gridDim.x * kStageWarps;
    for (int i = blockIdx.x * kStageWarps + (threadIdx.x >> 5); i < n; i += warps_total) {
        const long long src_entry = idx[i];
        if (src_entry < 0) continue;
        const uint8_t *src = host_kv + src_entry * (long long)kEntryBytes + lane * 16;
        uint8_t *dst = pool + (long long)slots[i] * kEntryBytes + lane * 16;
        uint4 v[16];
#pragma unroll
        for (int c = 0; c < 16; ++c) v[c] = ld_stream_v4(src + c * 512);
        asm volatile("" ::: "memory");          // keeps the stores behind all sixteen loads
#pragma unroll
        for (int c = 0; c < 16; ++c) *reinterpret_cast<uint4 *>(dst + c * 512) = v[c];
    }
}

}  // namespace oasis

extern "C" int oasis_stage_blocks(const void *host_kv, const int64_t *idx, const int32_t *slots,
                                  int32_t n, void *hbm_pool, void *stream)
{
    using namespace oasis;
    if (n < 0) return fail(OASIS_ERR_INVALID_ARG, "oasis_stage_blocks: n %d < 0", n);
    if (n == 0) return OASIS_OK;
    if (!host_kv || !idx || !slots || !hbm_pool)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_stage_blocks: NULL pointer argument");
    if (!aligned16(host_kv) || !aligned16(hbm_pool))
        return fail(OASIS_ERR_INVALID_ARG, "oasis_stage_blocks: host_kv and hbm_pool must be 16-byte aligned");
    const int max_ctas = 16 * sm_count();
    int grid = (n + kStageWarps - 1) / kStageWarps;
    if (grid > max_ctas) grid = max_ctas;
    prefer_max_shared_carveout(stage_blocks_kernel);
    stage_blocks_kernel<<<grid, kStageWarps * 32, 0, (cudaStream_t)stream>>>(
        (const uint8_t *)host_kv, (const long long *)idx, slots, n, (uint8_t *)hbm_pool);
    return check_launch("oasis_stage_blocks");
}
