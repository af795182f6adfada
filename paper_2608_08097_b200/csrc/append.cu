// Local window and KV append (Sec. 4.3: the selected blocks and a local window stay in GPU memory;
// Sec. 5.2: the active local block is kept on top of the K selected ones).
//
// The tokens of a decode step are produced on the GPU, so their keys and values go straight into the local
// window of the working set and never cross the host link in that direction; the tokens the step commits
// are also written through to the CPU full-KV pool (zero-copy stores into mapped pinned memory), so that a
// block that fills up is complete there.  Local block j lives in column local_col + (j & 1) of its
// (request, KV head) row: a block keeps its column -- and slot -- while it is local.
//
// One warp per (request, token, KV head): lanes 0-15 carry the 256-byte key row, lanes 16-31 the value row,
// 16 bytes each.  The warp of token 0 also sets the row's two local columns.  Traffic per step and layer:
// B * T * Hkv * 512 B read and written in HBM, B * n_commit * Hkv * 512 B over the host link.
#include "common.cuh"

namespace oasis {

constexpr int kAppendWarps = 8;

// Per-layer pointers travel as a kernel argument (blockIdx.y = layer): 6 x 8 x 64 bytes.
struct AppendLayers {
    const uint8_t *new_kv[OASIS_MAX_APPEND_LAYERS];
    const int32_t *block_table[OASIS_MAX_APPEND_LAYERS];
    const int32_t *slot_tbl[OASIS_MAX_APPEND_LAYERS];
    int32_t *blk_tbl[OASIS_MAX_APPEND_LAYERS];
    uint8_t *pool[OASIS_MAX_APPEND_LAYERS];
    uint8_t *host_kv[OASIS_MAX_APPEND_LAYERS];
};

struct AppendParams {
    const int32_t *seq_len;
    int B, T, Hkv, max_blocks, n_cols, local_col, n_commit;
};

__device__ __forceinline__ void set_local_columns(int32_t *cols, int lo, int hi)
{
    cols[lo & 1] = lo;
    cols[(lo & 1) ^ 1] = hi > lo ? hi : -1;
}

__global__ void __launch_bounds__(kAppendWarps * 32)
append_kv_kernel(const __grid_constant__ AppendLayers ly_all, const AppendParams p, const Bounds bd)
{
    const int l = blockIdx.y;
    struct {
        const uint8_t *new_kv; const int32_t *block_table; const int32_t *slot_tbl; int32_t *blk_tbl; uint8_t *pool; uint8_t *host_kv;
    } ly = {ly_all.new_kv[l], ly_all.block_table[l], ly_all.slot_tbl[l], ly_all.blk_tbl[l], ly_all.pool[l], ly_all.host_kv[l]};
    const int lane = threadIdx.x & 31;
    const int total = p.B * p.T * p.Hkv;
    for (int w = blockIdx.x * kAppendWarps + (threadIdx.x >> 5); w < total; w += gridDim.x * kAppendWarps) {
        const int h = w % p.Hkv;
        const int t = (w / p.Hkv) % p.T;
        const int b = w / (p.Hkv * p.T);
        const int L = p.seq_len[b];
        const int pos = L + t;
        const int j = pos / kBlock, i = pos % kBlock;
        const long long row = (long long)b * p.Hkv + h;
        if (t == 0 && lane == 0)
            set_local_columns(ly.blk_tbl + row * p.n_cols + p.local_col, L / kBlock, (L + p.T - 1) / kBlock);
        const int part = lane >> 4;                                  // 0: key row, 1: value row
        const int off = (lane & 15) * 16;
        const uint4 v = *reinterpret_cast<const uint4 *>(ly.new_kv + (long long)w * 2 * kRowBytes + part * kRowBytes + off);
        const long long slot = ly.slot_tbl[row * p.n_cols + p.local_col + (j & 1)];
        const long long in_entry = (long long)part * kPartBytes + (long long)i * kRowBytes + off;
        if (in_range(slot, bd.n_slots, bd, kErrSlot))
            *reinterpret_cast<uint4 *>(ly.pool + slot * kEntryBytes + in_entry) = v;
        if (ly.host_kv && t < p.n_commit && in_range(j, p.max_blocks, bd, kErrBlockId)) {
            const long long phys = ly.block_table[(long long)b * p.max_blocks + j];
            if (in_range(phys * p.Hkv + h, bd.n_entries, bd, kErrHostEntry))
                *reinterpret_cast<uint4 *>(ly.host_kv + (phys * p.Hkv + h) * kEntryBytes + in_entry) = v;
        }
    }
}

__global__ void __launch_bounds__(128)
local_window_kernel(const int32_t *__restrict__ seq_len, const int32_t *__restrict__ block_table,
                    int32_t *__restrict__ blk_tbl, long long *__restrict__ stage_idx, int32_t *__restrict__ stage_slots,
                    int B, int T, int Hkv, int max_blocks, int n_cols, int local_col, int slot_stride, const Bounds bd)
{
    const int row = blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= B * Hkv) return;
    const int b = row / Hkv, h = row % Hkv;
    const int L = seq_len[b];
    int32_t *cols = blk_tbl + (long long)row * n_cols + local_col;
    const int lo = L / kBlock, hi = (L + T - 1) / kBlock;
    set_local_columns(cols, lo, hi);
    if (stage_idx) {
        const int c[2] = {(lo & 1) ? (hi > lo ? hi : -1) : lo, (lo & 1) ? lo : (hi > lo ? hi : -1)};
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            stage_slots[row * 2 + r] = row * slot_stride + local_col + r;
            stage_idx[row * 2 + r] = (c[r] < 0 || !in_range(c[r], max_blocks, bd, kErrBlockId))
                                         ? -1ll : (long long)block_table[(long long)b * max_blocks + c[r]] * Hkv + h;
        }
    }
}

static int check_append(const oasis_dims_t *dims, int T, int n_commit, int n_cols, int local_col, const char *who)
{
    if (int rc = check_dims(dims)) return rc;
    if (T < 1 || T > kBlock)
        return fail(OASIS_ERR_INVALID_ARG, "%s: n_q_tokens %d outside [1, %d]", who, T, kBlock);
    if (n_commit < 0 || n_commit > T)
        return fail(OASIS_ERR_INVALID_ARG, "%s: n_commit %d outside [0, n_q_tokens]", who, n_commit);
    if (local_col < 0 || local_col + 2 > n_cols)
        return fail(OASIS_ERR_INVALID_ARG, "%s: local columns %d, %d outside the %d columns", who, local_col, local_col + 1, n_cols);
    if ((long long)dims->batch * T * dims->n_kv_heads > 0x7fffffffLL)
        return fail(OASIS_ERR_UNSUPPORTED, "%s: too many (request, token, head) rows", who);
    return OASIS_OK;
}

static int launch_append(const oasis_dims_t *dims, int n_layers, const void *const *new_kv, int T, int n_commit,
                         const int32_t *seq_len, const int32_t *const *block_tables, const int32_t *const *slot_tbls,
                         int32_t *const *blk_tbls, int n_cols, int local_col, void *const *pools, void *const *host_kvs,
                         cudaStream_t st, const char *who)
{
    if (int rc = check_append(dims, T, n_commit, n_cols, local_col, who)) return rc;
    if (n_layers < 0 || n_layers > OASIS_MAX_APPEND_LAYERS)
        return fail(OASIS_ERR_INVALID_ARG, "%s: n_layers %d outside [0, %d]", who, n_layers, OASIS_MAX_APPEND_LAYERS);
    if (!new_kv || !seq_len || !block_tables || !slot_tbls || !blk_tbls || !pools)
        return fail(OASIS_ERR_INVALID_ARG, "%s: NULL pointer argument", who);
    AppendLayers ly = {};
    for (int l = 0; l < n_layers; ++l) {
        void *host = host_kvs ? host_kvs[l] : nullptr;
        if (!new_kv[l] || !block_tables[l] || !slot_tbls[l] || !blk_tbls[l] || !pools[l])
            return fail(OASIS_ERR_INVALID_ARG, "%s: NULL pointer for layer %d", who, l);
        if (n_commit > 0 && !host)
            return fail(OASIS_ERR_INVALID_ARG, "%s: n_commit %d but no host_kv (layer %d)", who, n_commit, l);
        if (!aligned16(new_kv[l]) || !aligned16(pools[l]) || !aligned16(host))
            return fail(OASIS_ERR_INVALID_ARG, "%s: new_kv, hbm_pool and host_kv must be 16-byte aligned (layer %d)", who, l);
        ly.new_kv[l] = (const uint8_t *)new_kv[l];
        ly.block_table[l] = block_tables[l];
        ly.slot_tbl[l] = slot_tbls[l];
        ly.blk_tbl[l] = blk_tbls[l];
        ly.pool[l] = (uint8_t *)pools[l];
        ly.host_kv[l] = n_commit > 0 ? (uint8_t *)host : nullptr;
    }
    const long long total = (long long)dims->batch * T * dims->n_kv_heads;
    if (total == 0 || n_layers == 0) return OASIS_OK;
    AppendParams p;
    p.seq_len = seq_len;
    p.B = dims->batch; p.T = T; p.Hkv = dims->n_kv_heads; p.max_blocks = dims->max_blocks;
    p.n_cols = n_cols; p.local_col = local_col; p.n_commit = n_commit;
    long long grid = (total + kAppendWarps - 1) / kAppendWarps;
    if (grid > 4096) grid = 4096;
    prefer_max_shared_carveout(append_kv_kernel);
    append_kv_kernel<<<dim3((unsigned)grid, (unsigned)n_layers), kAppendWarps * 32, 0, st>>>(ly, p, bounds());
    return check_launch(who);
}

}  // namespace oasis

extern "C" int oasis_append_kv(const oasis_dims_t *dims, const void *new_kv, int32_t n_q_tokens, int32_t n_commit,
                               const int32_t *seq_len, const int32_t *block_table, const int32_t *slot_tbl,
                               int32_t *blk_tbl, int32_t n_cols, int32_t local_col, void *hbm_pool, void *host_kv,
                               void *stream)
{
    return oasis::launch_append(dims, 1, &new_kv, n_q_tokens, n_commit, seq_len, &block_table, &slot_tbl, &blk_tbl, n_cols,
                                local_col, &hbm_pool, &host_kv, (cudaStream_t)stream, "oasis_append_kv");
}

extern "C" int oasis_append_kv_layers(const oasis_dims_t *dims, int32_t n_layers, const void *const *new_kv,
                                      int32_t n_q_tokens, int32_t n_commit, const int32_t *seq_len,
                                      const int32_t *const *block_tables, const int32_t *const *slot_tbls,
                                      int32_t *const *blk_tbls, int32_t n_cols, int32_t local_col,
                                      void *const *hbm_pools, void *const *host_kvs, void *stream)
{
    return oasis::launch_append(dims, n_layers, new_kv, n_q_tokens, n_commit, seq_len, block_tables, slot_tbls, blk_tbls,
                                n_cols, local_col, hbm_pools, host_kvs, (cudaStream_t)stream, "oasis_append_kv_layers");
}

extern "C" int oasis_local_window(const oasis_dims_t *dims, const int32_t *seq_len, int32_t n_q_tokens,
                                  const int32_t *block_table, int32_t *blk_tbl, int32_t n_cols, int32_t local_col,
                                  int32_t slot_stride, int64_t *stage_idx, int32_t *stage_slots, void *stream)
{
    using namespace oasis;
    const char *who = "oasis_local_window";
    if (int rc = check_append(dims, n_q_tokens, 0, n_cols, local_col, who)) return rc;
    if (!seq_len || !blk_tbl) return fail(OASIS_ERR_INVALID_ARG, "%s: NULL pointer argument", who);
    if ((stage_idx == nullptr) != (stage_slots == nullptr))
        return fail(OASIS_ERR_INVALID_ARG, "%s: stage_idx and stage_slots must both be given or both be NULL", who);
    if (stage_idx && (!block_table || slot_stride < local_col + 2))
        return fail(OASIS_ERR_INVALID_ARG, "%s: block_table missing or slot_stride %d < local_col + 2", who, slot_stride);
    const int rows = dims->batch * dims->n_kv_heads;
    if (rows == 0) return OASIS_OK;
    if ((long long)rows * slot_stride > 0x7fffffffLL) return fail(OASIS_ERR_UNSUPPORTED, "%s: more than 2^31 slots", who);
    prefer_max_shared_carveout(local_window_kernel);
    local_window_kernel<<<(rows + 127) / 128, 128, 0, (cudaStream_t)stream>>>(
        seq_len, block_table, blk_tbl, (long long *)stage_idx, stage_slots, dims->batch, n_q_tokens, dims->n_kv_heads,
        dims->max_blocks, n_cols, local_col, slot_stride, bounds());
    return check_launch(who);
}
