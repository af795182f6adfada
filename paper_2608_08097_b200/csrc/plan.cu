// KV selection stage: delta selection with capped eviction (Sec. 4.2.3, cap from Sec. 5.5.1).
//
// One CTA per (request, KV head) row.  Two bitmaps over the logical block ids (predicted,
// resident) make the set intersections O(1) per element; the eviction targets are ordered
// with a bitonic sort of (empty first, last-selected step, column) keys; the candidates keep
// their rank order through a ballot/prefix-sum compaction; the first min(cap, candidates,
// targets) pairs are applied to the resident table and emitted as gather requests.
// Integer work on a few hundred elements per row: latency bound, no roofline to speak of.  The loops are kept
// rolled: the kernel shares SMs with the attention / scoring kernel, whose instruction fetches a large
// co-resident kernel slows down.
#include "common.cuh"

namespace oasis {

struct PlanParams {
    const int32_t *sel;
    const int32_t *block_table;
    int32_t *resident;
    int32_t *stamp;
    long long *plan_idx;
    int32_t *plan_slots;
    int32_t *n_admitted;
    int Hkv, max_blocks, sel_cols, k, n_res, res_stride, n_local, slot_stride, cap, step, sort_len, bitmap_words;
    Bounds bd;
};

constexpr int kPlanThreads = 256;

__global__ void __launch_bounds__(kPlanThreads)
plan_delta_kernel(const PlanParams p)
{
    extern __shared__ __align__(16) uint8_t smem_raw[];
    unsigned long long *tkey = reinterpret_cast<unsigned long long *>(smem_raw);   // [sort_len]
    int32_t *cand = reinterpret_cast<int32_t *>(tkey + p.sort_len);                // [k]
    uint32_t *pred_bits = reinterpret_cast<uint32_t *>(cand + p.k);                // [bitmap_words]
    uint32_t *res_bits = pred_bits + p.bitmap_words;                               // [bitmap_words]
    __shared__ uint32_t warp_cnt[kPlanThreads / 32], warp_pre[kPlanThreads / 32];
    __shared__ uint32_t sh_tile_total, sh_n_target;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int nwarps = kPlanThreads / 32;
    const int row = blockIdx.x;
    const int b = row / p.Hkv, h = row % p.Hkv;
    const int32_t *pred = p.sel + (long long)row * p.sel_cols;
    int32_t *res = p.resident + (long long)row * p.res_stride;
    int32_t *stp = p.stamp + (long long)row * p.res_stride;
    const int plan_cols = p.cap + p.n_local;

#pragma unroll 1
    for (int i = tid; i < 2 * p.bitmap_words; i += kPlanThreads) pred_bits[i] = 0;
    if (tid == 0) sh_n_target = 0;
    __syncthreads();
#pragma unroll 1
    for (int r = tid; r < p.k; r += kPlanThreads) {
        const int j = pred[r];
        if (j >= 0 && j < p.max_blocks) atomicOr(&pred_bits[j >> 5], 1u << (j & 31));
        else if (kBoundsCheck && j >= p.max_blocks) in_range(j, p.max_blocks, p.bd, kErrBlockId);
    }
#pragma unroll 1
    for (int c = tid; c < p.n_res; c += kPlanThreads) {
        const int j = res[c];
        if (j >= 0 && j < p.max_blocks) atomicOr(&res_bits[j >> 5], 1u << (j & 31));
    }
    __syncthreads();

    // ---- hits keep their column; everything else is an eviction target ------------------------------
#pragma unroll 1
    for (int c = tid; c < p.sort_len; c += kPlanThreads) {
        unsigned long long key = ~0ull;                       // non-targets sort to the end
        if (c < p.n_res) {
            const int j = res[c];
            const bool hit = j >= 0 && j < p.max_blocks && ((pred_bits[j >> 5] >> (j & 31)) & 1u);
            if (hit) {
                stp[c] = p.step;
            } else {
                const unsigned long long age = j < 0 ? 0ull : (unsigned long long)((uint32_t)stp[c] ^ 0x80000000u) + 1ull;
                key = (age << 12) | (unsigned long long)c;      // n_res <= 2048 < 2^12
                atomicAdd(&sh_n_target, 1u);
            }
        }
        tkey[c] = key;
    }
    __syncthreads();
#pragma unroll 1
    for (int size = 2; size <= p.sort_len; size <<= 1) {
#pragma unroll 1
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
#pragma unroll 1
            for (int i = tid; i < (p.sort_len >> 1); i += kPlanThreads) {
                const int pos = 2 * i - (i & (stride - 1));
                const unsigned long long x = tkey[pos], y = tkey[pos + stride];
                const bool ascending = (pos & size) == 0;
                if ((x > y) == ascending) {
                    tkey[pos] = y;
                    tkey[pos + stride] = x;
                }
            }
            __syncthreads();
        }
    }

    // ---- candidates: predicted blocks that are not resident, in rank order -----------------------------
    uint32_t n_cand = 0;
    const int k_pad = (p.k + kPlanThreads - 1) / kPlanThreads * kPlanThreads;
#pragma unroll 1
    for (int base = 0; base < k_pad; base += kPlanThreads) {
        const int r = base + tid;
        const int j = r < p.k ? pred[r] : -1;
        const bool is_cand = j >= 0 && j < p.max_blocks && !((res_bits[j >> 5] >> (j & 31)) & 1u);
        const unsigned ballot = __ballot_sync(0xffffffffu, is_cand);
        if (lane == 0) warp_cnt[warp] = __popc(ballot);
        __syncthreads();
        if (warp == 0) {
            const uint32_t c = lane < nwarps ? warp_cnt[lane] : 0u;
            uint32_t incl = c;
#pragma unroll
            for (int m = 1; m < 32; m <<= 1) {
                const uint32_t o = __shfl_up_sync(0xffffffffu, incl, m);
                if (lane >= m) incl += o;
            }
            if (lane < nwarps) warp_pre[lane] = incl - c;
            if (lane == 31) sh_tile_total = incl;
        }
        __syncthreads();
        if (is_cand) cand[n_cand + warp_pre[warp] + __popc(ballot & ((1u << lane) - 1u))] = j;
        n_cand += sh_tile_total;
        __syncthreads();
    }

    // ---- pair candidates with targets, bounded by the cap ------------------------------------------------
    const int n_pair = min(p.cap, min((int)n_cand, (int)sh_n_target));
#pragma unroll 1
    for (int i = tid; i < p.cap; i += kPlanThreads) {
        long long idx = -1;
        int slot = 0;
        if (i < n_pair) {
            const int c = (int)(tkey[i] & 0xfffull);
            const int j = cand[i];
            res[c] = j;
            stp[c] = p.step;
            idx = (long long)p.block_table[(long long)b * p.max_blocks + j] * p.Hkv + h;
            slot = row * p.slot_stride + c;
            if (!in_range(idx, p.bd.n_entries, p.bd, kErrHostEntry) || !in_range(slot, p.bd.n_slots, p.bd, kErrSlot)) idx = -1;
        }
        p.plan_idx[(long long)row * plan_cols + i] = idx;
        p.plan_slots[(long long)row * plan_cols + i] = slot;
    }
    // the always-kept local blocks (Sec. 4.3: selected blocks plus a local window)
#pragma unroll 1
    for (int i = tid; i < p.n_local; i += kPlanThreads) {
        const int j = pred[p.k + i];
        res[p.n_res + i] = j;
        p.plan_slots[(long long)row * plan_cols + p.cap + i] = row * p.slot_stride + p.n_res + i;
        long long lidx = (j < 0 || j >= p.max_blocks) ? -1ll : (long long)p.block_table[(long long)b * p.max_blocks + j] * p.Hkv + h;
        if (kBoundsCheck && j >= p.max_blocks) in_range(j, p.max_blocks, p.bd, kErrBlockId);
        if (lidx >= 0 && (!in_range(lidx, p.bd.n_entries, p.bd, kErrHostEntry) ||
                          !in_range((long long)row * p.slot_stride + p.n_res + i, p.bd.n_slots, p.bd, kErrSlot)))
            lidx = -1;
        p.plan_idx[(long long)row * plan_cols + p.cap + i] = lidx;
    }
    if (tid == 0 && p.n_admitted) p.n_admitted[row] = n_pair;
}

}  // namespace oasis

extern "C" int oasis_plan_delta(const oasis_dims_t *dims, const int32_t *sel, int32_t sel_cols, int32_t k,
                                const int32_t *block_table, int32_t *resident, int32_t *stamp,
                                int32_t n_res, int32_t res_stride, int32_t n_local, int32_t slot_stride,
                                int32_t cap, int32_t step,
                                int64_t *plan_idx, int32_t *plan_slots, int32_t *n_admitted, void *stream)
{
    using namespace oasis;
    if (int rc = check_dims(dims)) return rc;
    if (!sel || !block_table || !resident || !stamp)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_plan_delta: NULL pointer argument");
    if (k < 1 || k > OASIS_MAX_K || k > sel_cols)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_plan_delta: k %d (sel_cols %d, max %d)", k, sel_cols, OASIS_MAX_K);
    if (n_res < 1 || n_res > OASIS_MAX_K)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_plan_delta: n_res %d outside [1, %d]", n_res, OASIS_MAX_K);
    if (cap < 0 || cap > k) return fail(OASIS_ERR_INVALID_ARG, "oasis_plan_delta: cap %d outside [0, k]", cap);
    if (n_local < 0 || n_local > 2 || k + n_local > sel_cols)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_plan_delta: n_local %d (k %d, sel_cols %d)", n_local, k, sel_cols);
    if (res_stride < n_res + n_local)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_plan_delta: res_stride %d < n_res + n_local = %d", res_stride, n_res + n_local);
    if (cap + n_local > 0 && (!plan_idx || !plan_slots))
        return fail(OASIS_ERR_INVALID_ARG, "oasis_plan_delta: plan_idx / plan_slots are NULL");
    if (slot_stride < n_res + n_local)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_plan_delta: slot_stride %d < n_res + n_local = %d", slot_stride, n_res + n_local);
    if ((long long)dims->batch * dims->n_kv_heads * slot_stride > 0x7fffffffLL)
        return fail(OASIS_ERR_UNSUPPORTED, "oasis_plan_delta: more than 2^31 slots");
    if (dims->max_blocks > (1 << 19))
        return fail(OASIS_ERR_UNSUPPORTED, "oasis_plan_delta: max_blocks %d > %d", dims->max_blocks, 1 << 19);
    if (dims->batch == 0) return OASIS_OK;

    PlanParams p;
    p.sel = sel; p.block_table = block_table; p.resident = resident; p.stamp = stamp;
    p.plan_idx = (long long *)plan_idx; p.plan_slots = plan_slots; p.n_admitted = n_admitted;
    p.Hkv = dims->n_kv_heads; p.max_blocks = dims->max_blocks; p.sel_cols = sel_cols; p.k = k;
    p.n_res = n_res; p.res_stride = res_stride; p.n_local = n_local; p.slot_stride = slot_stride; p.cap = cap; p.step = step;
    p.bd = bounds();
    int sort_len = 2;
    while (sort_len < n_res) sort_len <<= 1;
    p.sort_len = sort_len;
    p.bitmap_words = (dims->max_blocks + 31) / 32;
    const size_t smem = (size_t)sort_len * 8 + (size_t)k * 4 + (size_t)p.bitmap_words * 8;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(plan_delta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return fail(OASIS_ERR_CUDA, "oasis_plan_delta: shared memory %zu B: %s", smem, cudaGetErrorString(e));
    }
    prefer_max_shared_carveout(plan_delta_kernel);
    plan_delta_kernel<<<dims->batch * dims->n_kv_heads, kPlanThreads, smem, (cudaStream_t)stream>>>(p);
    return check_launch("oasis_plan_delta");
}
