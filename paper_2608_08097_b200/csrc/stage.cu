// Step 3: gather of selected (block, head) entries from the host-resident full KV cache
// into HBM slots (Sec. 5.1: a gather kernel reads the selected entries from the pinned CPU
// cache through unified addressing and writes them straight into the resident GPU pages).
//
// One warp per 8 KiB entry: sixteen 16-byte loads per lane are issued back to back (the
// whole entry is in flight before the first store), each warp-wide load covering 512
// contiguous bytes, then sixteen stores.  The source may equally be device memory.  Requests
// with a negative source index are skipped, so list lengths never have to be read back by
// the host.  A launch keeps at most kStageDefaultCtas thread blocks busy (grid-stride over the list).
// oasis_stage_blocks_bulk moves the entries with the copy unit instead (see its kernel).
// Algorithmic traffic: 8 KiB over the host link and 8 KiB written per request.
#include "common.cuh"
#include "tc_common.cuh"

namespace oasis {

constexpr int kStageWarps = 4;
// Thread blocks of a gather launch unless the caller says otherwise: 128 x 4 warps x 8 KiB = 4 MiB of reads in
// flight.  Measured on B200 with the pool in pinned host memory: beyond about 4 MiB in flight (one launch, or
// several concurrent ones together) the host link delivers less, not more -- 0.89 of the copy-engine rate at 64
// thread blocks, 0.80 at 96, 0.66 with every request of a 3,000-entry list in flight at once.
constexpr int kStageDefaultCtas = 128;
constexpr int kStageBulkBufs = 1;                           // 8 KiB buffers per CTA of the copy-unit gather

__global__ void __launch_bounds__(kStageWarps * 32)
stage_blocks_kernel(const uint8_t *__restrict__ host_kv, const long long *__restrict__ idx,
                    const int32_t *__restrict__ slots, int n, uint8_t *__restrict__ pool, const Bounds bd)
{
    const int lane = threadIdx.x & 31;
    const int warps_total = gridDim.x * kStageWarps;
    for (int i = blockIdx.x * kStageWarps + (threadIdx.x >> 5); i < n; i += warps_total) {
        const long long src_entry = idx[i];
        if (src_entry < 0) continue;
        if (!in_range(src_entry, bd.n_entries, bd, kErrHostEntry) || !in_range(slots[i], bd.n_slots, bd, kErrSlot)) continue;
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

// The same for several layers in one launch (blockIdx.y = layer): each layer has its own source pool, request
// lists and working-set pool.  Larger launches keep the host link busier than a train of small ones.
struct StageLayers {
    const uint8_t *host_kv[OASIS_MAX_STAGE_LAYERS];
    const long long *idx[OASIS_MAX_STAGE_LAYERS];
    const int32_t *slots[OASIS_MAX_STAGE_LAYERS];
    uint8_t *pool[OASIS_MAX_STAGE_LAYERS];
};

__global__ void __launch_bounds__(kStageWarps * 32)
stage_blocks_layers_kernel(const __grid_constant__ StageLayers ly, int n, const Bounds bd)
{
    const int l = blockIdx.y;
    const uint8_t *host_kv = ly.host_kv[l];
    const long long *idx = ly.idx[l];
    const int32_t *slots = ly.slots[l];
    uint8_t *pool = ly.pool[l];
    const int lane = threadIdx.x & 31;
    const int warps_total = gridDim.x * kStageWarps;
    for (int i = blockIdx.x * kStageWarps + (threadIdx.x >> 5); i < n; i += warps_total) {
        const long long src_entry = idx[i];
        if (src_entry < 0) continue;
        if (!in_range(src_entry, bd.n_entries, bd, kErrHostEntry) || !in_range(slots[i], bd.n_slots, bd, kErrSlot)) continue;
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

// The several-layers gather through the copy unit: one thread per CTA moves its share of the list as 8 KiB bulk
// copies, CPU pool -> shared memory -> working-set pool, one buffer per CTA; no warp spends an instruction on the
// bytes, and the CTA (32 threads, 8 KiB of shared memory) fits on an SM beside the fused attention + scoring CTA.
// Alone it moves what the warp-per-entry kernel moves (49-51 GB/s from pinned memory), and so it does inside a decode
// step that the host link bounds while the queries are resident (3.99 ms either way at fetch ratio 0.05, 128 entry
// streams and eight layers per launch); end to end, with the query uploads on the same link, it is the faster one (4.45-4.47
// against 4.55-4.60 ms).  Where compute bounds the step the two are equal (1.66-1.67 ms at fetch ratio 0.02, two layers
// per launch) and the warp kernel disturbs the query uploads of the end-to-end step less (2.07 against 2.41 ms).  Two
// buffers per CTA no longer fit beside the fused CTA and are slower.
__global__ void __launch_bounds__(32)
stage_blocks_bulk_kernel(const __grid_constant__ StageLayers ly, int n, int nbuf, int32_t *err, const Bounds bd)
{
    extern __shared__ __align__(128) uint8_t bulk_smem[];
    __shared__ uint64_t bars[4];
    if (threadIdx.x != 0) return;
    const int l = blockIdx.y;
    const uint8_t *host_kv = ly.host_kv[l];
    const long long *idx = ly.idx[l];
    const int32_t *slots = ly.slots[l];
    uint8_t *pool = ly.pool[l];
    const uint32_t sm = smem_u32(bulk_smem), bar0 = smem_u32(bars);
    for (int b = 0; b < nbuf; ++b) mbar_init(bar0 + 8u * b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    auto load = [&](int i, int buf) -> bool {           // false: nothing to copy for list position i
        const long long src_entry = idx[i];
        if (src_entry < 0) return false;
        if (!in_range(src_entry, bd.n_entries, bd, kErrHostEntry) || !in_range(slots[i], bd.n_slots, bd, kErrSlot)) return false;
        mbar_arrive_expect_tx(bar0 + 8u * buf, (uint32_t)kEntryBytes);
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(sm + (uint32_t)buf * kEntryBytes), "l"(host_kv + src_entry * (long long)kEntryBytes), "r"((uint32_t)kEntryBytes),
                       "r"(bar0 + 8u * buf) : "memory");
        return true;
    };
    // this CTA's list positions: blockIdx.x, + gridDim.x, ...; position k of them uses buffer k % nbuf
    bool have[4] = {false, false, false, false};
    uint32_t phase[4] = {0, 0, 0, 0};
    int i_load = blockIdx.x;
    for (int b = 0; b < nbuf && i_load < n; ++b, i_load += gridDim.x) have[b] = load(i_load, b);
    int buf = 0;
    for (int i = blockIdx.x; i < n; i += gridDim.x) {
        if (have[buf]) {
            if (!mbar_wait(bar0 + 8u * buf, phase[buf], err, 71)) break;
            phase[buf] ^= 1u;
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                         ::"l"(pool + (long long)slots[i] * kEntryBytes), "r"(sm + (uint32_t)buf * kEntryBytes), "r"((uint32_t)kEntryBytes) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        have[buf] = false;
        if (i_load < n) {
            // the buffer is read by the store just issued: wait until that read is over, then refill it
            asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            have[buf] = load(i_load, buf);
            i_load += gridDim.x;
        }
        buf = buf + 1 == nbuf ? 0 : buf + 1;
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

}  // namespace oasis

extern "C" int oasis_stage_blocks_layers(int32_t n_layers, const void *const *host_kvs, const int64_t *const *idx,
                                         const int32_t *const *slots, int32_t n, void *const *hbm_pools,
                                         int32_t max_ctas_arg, void *stream)
{
    using namespace oasis;
    const char *who = "oasis_stage_blocks_layers";
    if (n < 0) return fail(OASIS_ERR_INVALID_ARG, "%s: n %d < 0", who, n);
    if (n_layers < 0 || n_layers > OASIS_MAX_STAGE_LAYERS)
        return fail(OASIS_ERR_INVALID_ARG, "%s: n_layers %d outside [0, %d]", who, n_layers, OASIS_MAX_STAGE_LAYERS);
    if (n == 0 || n_layers == 0) return OASIS_OK;
    if (!host_kvs || !idx || !slots || !hbm_pools) return fail(OASIS_ERR_INVALID_ARG, "%s: NULL pointer argument", who);
    StageLayers ly = {};
    for (int l = 0; l < n_layers; ++l) {
        if (!host_kvs[l] || !idx[l] || !slots[l] || !hbm_pools[l])
            return fail(OASIS_ERR_INVALID_ARG, "%s: NULL pointer for layer %d", who, l);
        if (!aligned16(host_kvs[l]) || !aligned16(hbm_pools[l]))
            return fail(OASIS_ERR_INVALID_ARG, "%s: host_kv and hbm_pool must be 16-byte aligned (layer %d)", who, l);
        ly.host_kv[l] = (const uint8_t *)host_kvs[l];
        ly.idx[l] = (const long long *)idx[l];
        ly.slots[l] = slots[l];
        ly.pool[l] = (uint8_t *)hbm_pools[l];
    }
    if (max_ctas_arg < 0) return fail(OASIS_ERR_INVALID_ARG, "%s: max_ctas %d < 0", who, max_ctas_arg);
    int max_ctas = (max_ctas_arg > 0 ? max_ctas_arg : kStageDefaultCtas) / n_layers;
    if (max_ctas < 1) max_ctas = 1;
    int grid = (n + kStageWarps - 1) / kStageWarps;
    if (grid > max_ctas) grid = max_ctas;
    prefer_max_shared_carveout(stage_blocks_layers_kernel);
    stage_blocks_layers_kernel<<<dim3((unsigned)grid, (unsigned)n_layers), kStageWarps * 32, 0, (cudaStream_t)stream>>>(ly, n, bounds());
    return check_launch(who);
}

extern "C" int oasis_stage_blocks_bulk(int32_t n_layers, const void *const *host_kvs, const int64_t *const *idx,
                                       const int32_t *const *slots, int32_t n, void *const *hbm_pools,
                                       int32_t max_streams, void *stream)
{
    using namespace oasis;
    const char *who = "oasis_stage_blocks_bulk";
    if (n < 0) return fail(OASIS_ERR_INVALID_ARG, "%s: n %d < 0", who, n);
    if (n_layers < 0 || n_layers > OASIS_MAX_STAGE_LAYERS)
        return fail(OASIS_ERR_INVALID_ARG, "%s: n_layers %d outside [0, %d]", who, n_layers, OASIS_MAX_STAGE_LAYERS);
    if (n == 0 || n_layers == 0) return OASIS_OK;
    if (!host_kvs || !idx || !slots || !hbm_pools) return fail(OASIS_ERR_INVALID_ARG, "%s: NULL pointer argument", who);
    StageLayers ly = {};
    for (int l = 0; l < n_layers; ++l) {
        if (!host_kvs[l] || !idx[l] || !slots[l] || !hbm_pools[l])
            return fail(OASIS_ERR_INVALID_ARG, "%s: NULL pointer for layer %d", who, l);
        if (!aligned16(host_kvs[l]) || !aligned16(hbm_pools[l]))
            return fail(OASIS_ERR_INVALID_ARG, "%s: host_kv and hbm_pool must be 16-byte aligned (layer %d)", who, l);
        ly.host_kv[l] = (const uint8_t *)host_kvs[l];
        ly.idx[l] = (const long long *)idx[l];
        ly.slots[l] = slots[l];
        ly.pool[l] = (uint8_t *)hbm_pools[l];
    }
    if (max_streams < 0) return fail(OASIS_ERR_INVALID_ARG, "%s: max_streams %d < 0", who, max_streams);
    int per_layer = (max_streams > 0 ? max_streams : kStageDefaultCtas) / n_layers;
    if (per_layer < 1) per_layer = 1;
    const int grid = n < per_layer ? n : per_layer;
    prefer_max_shared_carveout(stage_blocks_bulk_kernel);
    stage_blocks_bulk_kernel<<<dim3((unsigned)grid, (unsigned)n_layers), 32, (size_t)kStageBulkBufs * kEntryBytes, (cudaStream_t)stream>>>(
        ly, n, kStageBulkBufs, error_word(), bounds());
    return check_launch(who);
}

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
    const int max_ctas = kStageDefaultCtas;
    int grid = (n + kStageWarps - 1) / kStageWarps;
    if (grid > max_ctas) grid = max_ctas;
    prefer_max_shared_carveout(stage_blocks_kernel);
    stage_blocks_kernel<<<grid, kStageWarps * 32, 0, (cudaStream_t)stream>>>(
        (const uint8_t *)host_kv, (const long long *)idx, slots, n, (uint8_t *)hbm_pool, bounds());
    return check_launch("oasis_stage_blocks");
}
