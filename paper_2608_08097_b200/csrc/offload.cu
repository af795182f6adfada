// Dense -> sparse hand-over (Sec. 4.3): when a request crosses the sparsification threshold its
// dense KV blocks, kept by the GPU pool as separate key and value blocks in Head-Token-Dimension
// order, are copied to the CPU pool as 8 KiB [K | V] entries, and the summaries of the copied
// blocks are taken from the keys while they pass through the registers (step 0 fused into the
// copy, so the keys are read once).
//
// One warp per (request, block, KV head): eight 16-byte loads per lane bring the 4 KiB key block,
// eight more the value block; both go out as sixteen 16-byte stores to the entry in mapped pinned
// host memory (or device memory), each warp-wide store covering 512 contiguous bytes.  The key
// chunks also feed the bf16x2 min / max of step 0 (half-warp fold, 256-byte min row and max row).
// Algorithmic traffic: 8 KiB read from HBM + 8 KiB over the host link + 512 B of summaries per
// (block, head).
#include "common.cuh"

namespace oasis {

constexpr int kOffloadWarps = 4;

__device__ __forceinline__ uint32_t off_min2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("min.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t off_max2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

__global__ void __launch_bounds__(kOffloadWarps * 32)
offload_blocks_kernel(const uint8_t *__restrict__ dense_k, const uint8_t *__restrict__ dense_v,
                      const int32_t *__restrict__ gpu_table, const int32_t *__restrict__ block_table,
                      const int32_t *__restrict__ first_block, const int32_t *__restrict__ n_blocks,
                      uint8_t *__restrict__ host_kv, uint8_t *__restrict__ summaries, int Hkv, int max_blocks,
                      int max_new, long long n_items, const Bounds bd)
{
    const int lane = threadIdx.x & 31;
    const long long item = (long long)blockIdx.x * kOffloadWarps + (threadIdx.x >> 5);
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
    const long long src_blk = gpu_table[(long long)b * max_blocks + j];
    const long long dst_blk = block_table[(long long)b * max_blocks + j];
    if (!in_range(dst_blk * Hkv + h, bd.n_entries, bd, kErrHostEntry)) return;
    constexpr int kPart = kEntryBytes / 2;                          // 4 KiB of keys, 4 KiB of values
    const uint8_t *ksrc = dense_k + (src_blk * Hkv + h) * (long long)kPart + lane * 16;
    const uint8_t *vsrc = dense_v + (src_blk * Hkv + h) * (long long)kPart + lane * 16;
    uint8_t *dst = host_kv + (dst_blk * Hkv + h) * (long long)kEntryBytes + lane * 16;

    // lane -> 16-byte chunk (lane & 15) of token (lane >> 4) + 2 * i
    uint4 k[8], v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) k[i] = ld_stream_v4(ksrc + i * 512);
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = ld_stream_v4(vsrc + i * 512);
#pragma unroll
    for (int i = 0; i < 8; ++i) *reinterpret_cast<uint4 *>(dst + i * 512) = k[i];
#pragma unroll
    for (int i = 0; i < 8; ++i) *reinterpret_cast<uint4 *>(dst + kPart + i * 512) = v[i];
    if (!summaries) return;

    uint32_t lo[4] = {k[0].x, k[0].y, k[0].z, k[0].w};
    uint32_t hi[4] = {k[0].x, k[0].y, k[0].z, k[0].w};
#pragma unroll
    for (int i = 1; i < 8; ++i) {
        const uint32_t w[4] = {k[i].x, k[i].y, k[i].z, k[i].w};
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            lo[p] = off_min2(lo[p], w[p]);
            hi[p] = off_max2(hi[p], w[p]);
        }
    }
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        lo[p] = off_min2(lo[p], __shfl_xor_sync(0xffffffffu, lo[p], 16));
        hi[p] = off_max2(hi[p], __shfl_xor_sync(0xffffffffu, hi[p], 16));
    }
    uint8_t *sdst = summaries + (((long long)b * Hkv + h) * max_blocks + j) * (long long)kSummaryBytes;
    const bool low_half = lane < 16;                                 // lanes 0..15: min row, lanes 16..31: max row
    uint4 o;
    o.x = low_half ? lo[0] : hi[0];
    o.y = low_half ? lo[1] : hi[1];
    o.z = low_half ? lo[2] : hi[2];
    o.w = low_half ? lo[3] : hi[3];
    *reinterpret_cast<uint4 *>(sdst + lane * 16) = o;
}

}  // namespace oasis

extern "C" int oasis_offload_blocks(const oasis_dims_t *dims, const void *dense_k, const void *dense_v,
                                    const int32_t *gpu_table, const int32_t *block_table,
                                    const int32_t *first_block, const int32_t *n_blocks, int32_t max_new_blocks,
                                    void *host_kv, void *summaries, void *stream)
{
    using namespace oasis;
    if (int rc = check_dims(dims)) return rc;
    if (!dense_k || !dense_v || !gpu_table || !block_table || !first_block || !n_blocks || !host_kv)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_offload_blocks: NULL pointer argument");
    if (!aligned16(dense_k) || !aligned16(dense_v) || !aligned16(host_kv) || !aligned16(summaries))
        return fail(OASIS_ERR_INVALID_ARG, "oasis_offload_blocks: dense_k, dense_v, host_kv and summaries must be 16-byte aligned");
    if (max_new_blocks < 0 || max_new_blocks > dims->max_blocks)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_offload_blocks: max_new_blocks %d outside [0, %d]", max_new_blocks,
                    dims->max_blocks);
    const long long n_items = (long long)dims->batch * dims->n_kv_heads * max_new_blocks;
    if (n_items == 0) return OASIS_OK;
    const long long grid = (n_items + kOffloadWarps - 1) / kOffloadWarps;
    if (grid > 0x7fffffffLL) return fail(OASIS_ERR_UNSUPPORTED, "oasis_offload_blocks: too many blocks");
    offload_blocks_kernel<<<(unsigned)grid, kOffloadWarps * 32, 0, (cudaStream_t)stream>>>(
        (const uint8_t *)dense_k, (const uint8_t *)dense_v, gpu_table, block_table, first_block, n_blocks,
        (uint8_t *)host_kv, (uint8_t *)summaries, dims->n_kv_heads, dims->max_blocks, max_new_blocks, n_items, bounds());
    return check_launch("oasis_offload_blocks");
}
