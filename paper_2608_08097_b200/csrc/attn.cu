// Step 4: entry points of the sparse paged decode attention (Sec. 4.2.1, 4.3): launch plan
// (how far the column list of a (request, KV head) row is split so that one CTA per SM is
// resident), the kernel that merges the splits' partial outputs, and the variant whose scratch
// is a fixed device array.  The attention kernel itself is in attn_tc.cu.
#include <math_constants.h>

#include "common.cuh"

namespace oasis {

constexpr int kAttnStages = 7;       // 32 KiB shared-memory stages of the attention kernel's K/V ring
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct AttnParams {
    const uint8_t *q;
    const uint8_t *pool;
    const int32_t *slot_tbl;
    const int32_t *blk_tbl;
    const int32_t *seq_len;
    uint8_t *out;
    float *lse;
    float *part_o;      // [items][rows_per_group][128] fp32 (split runs only)
    float *part_lse;    // [items][rows_per_group]      log2 domain
    float scale_log2;
    int T, Hq, Hkv, G, n_cols, R;           // R = T * G query rows per KV head
    int n_splits, cols_per_split, n_groups, rows_per_group;
};

// Merges the splits of one (request, KV head, row): out = sum_s w_s o_s / sum_s w_s with
// w_s = 2^(lse_s - max lse).  One warp per row, four output dims per thread (16-byte loads of the partials, the loads
// of four splits in flight at a time); CTAs of 256 threads take the `total` rows in turn, eight at a time.  Launched
// behind the fused layer kernel with programmatic stream serialization it lets the launch after it start early and
// itself waits for the partials (both instructions do nothing in an ordinary launch).
__global__ void __launch_bounds__(256)
attn_combine_kernel(const AttnParams p, long long total)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int lane = threadIdx.x & 31;
#pragma unroll 1
    for (long long wi = 8ll * blockIdx.x + (threadIdx.x >> 5); wi < total; wi += 8ll * gridDim.x) {
        const int row = (int)(wi % p.R);
        const int bh = (int)(wi / p.R);
        const int b = bh / p.Hkv, h = bh % p.Hkv;
        const int grp = row / p.rows_per_group, r = row % p.rows_per_group;
        // partial row of split s: prow0 + s * pstride
        const long long prow0 = ((long long)bh * p.n_splits * p.n_groups + grp) * p.rows_per_group + r;
        const long long pstride = (long long)p.n_groups * p.rows_per_group;
        float mx = -CUDART_INF_F;
        for (int s = lane; s < p.n_splits; s += 32) mx = fmaxf(mx, p.part_lse[prow0 + s * pstride]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float den = 0.f;
        if (mx > -CUDART_INF_F) {
#pragma unroll 1
            for (int s0 = 0; s0 < p.n_splits; s0 += 4) {
                float w[4];
                float4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const bool in = s0 + u < p.n_splits;
                    const long long prow = prow0 + (in ? s0 + u : s0) * pstride;
                    w[u] = in ? p.part_lse[prow] : -CUDART_INF_F;
                    v[u] = reinterpret_cast<const float4 *>(p.part_o + prow * kHeadDim)[lane];
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float ws = fast_exp2(w[u] - mx);           // 0 for the splits past the last one
                    acc.x += ws * v[u].x; acc.y += ws * v[u].y; acc.z += ws * v[u].z; acc.w += ws * v[u].w;
                    den += ws;
                }
            }
        }
        const bool any = den > 0.f;                                  // some split saw a key
        if (!any) { acc = make_float4(0.f, 0.f, 0.f, 0.f); den = 1.f; }
        const int tq = row / p.G, a = h * p.G + row % p.G;
        const long long orow = ((long long)b * p.T + tq) * p.Hq + a;
        reinterpret_cast<uint2 *>(p.out + orow * kHeadDim * 2)[lane] =
            make_uint2(pack_bf16x2(acc.x / den, acc.y / den), pack_bf16x2(acc.z / den, acc.w / den));
        if (p.lse && lane == 0) p.lse[orow] = any ? (mx + log2f(den)) * kLn2 : -CUDART_INF_F;
    }
}

// Launch geometry shared by the entry point and the workspace query.
struct AttnPlan {
    int n_groups, rows_per_group, n_splits, cols_per_split;
    long long items;
    size_t workspace;
};

int launch_attn_tc(const oasis_dims_t *dims, const void *q, int n_q_tokens, const void *hbm_pool,
                   const int32_t *slot_tbl, const int32_t *blk_tbl, int n_cols, const int32_t *seq_len, float scale,
                   void *out, float *lse, float *part_o, float *part_lse, int n_splits, int cols_per_split,
                   int stages, int32_t *err_word, cudaStream_t st, const char *who);      // attn_tc.cu

static AttnPlan attn_plan(const oasis_dims_t *dims, int T, int n_cols)
{
    AttnPlan pl;
    const int G = dims->n_q_heads / dims->n_kv_heads;
    const int R = T * G;
    pl.n_groups = 1;                     // all rows of a KV head share one CTA (they are the MMA's M rows)
    pl.rows_per_group = R;
    const long long base = (long long)dims->batch * dims->n_kv_heads * pl.n_groups;
    // All CTAs should be resident at once (one per SM): a bandwidth-bound kernel then has no
    // tail.  Split the column list only as far as that allows, at least 8 columns per split.
    const long long slots = sm_count();
    long long s = base > 0 ? slots / base : 1;
    const long long max_s = (n_cols + 7) / 8;
    if (s > max_s) s = max_s;
    if (s < 1) s = 1;
    pl.cols_per_split = (int)((n_cols + s - 1) / s);
    pl.n_splits = (n_cols + pl.cols_per_split - 1) / pl.cols_per_split;
    if (pl.n_splits < 1) pl.n_splits = 1;
    pl.items = base * pl.n_splits;
    pl.workspace = pl.n_splits > 1
                       ? (size_t)pl.items * pl.rows_per_group * (kHeadDim + 1) * sizeof(float)
                       : 0;
    return pl;
}

// Enqueues the attention kernel (and the split combine) for a plan.
static int launch_attn(const oasis_dims_t *dims, const AttnPlan &pl, const AttnParams &p, const void *q,
                       const void *pool, float scale, long long combine_ctas, cudaStream_t st, const char *who)
{
    if (int rc = launch_attn_tc(dims, q, p.T, pool, p.slot_tbl, p.blk_tbl, p.n_cols, p.seq_len, scale, p.out, p.lse,
                                p.part_o, p.part_lse, pl.n_splits, pl.cols_per_split, kAttnStages, error_word(), st, who))
        return rc;
    if (pl.n_splits > 1) {
        // programmatic stream serialization: the merge's thread blocks become resident while the attention still runs
        // and wait there for its partials, which hides their launch
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)((combine_ctas + 7) / 8));
        cfg.blockDim = dim3(256);
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e = cudaLaunchKernelEx(&cfg, attn_combine_kernel, p, combine_ctas);
        if (e != cudaSuccess) return fail(OASIS_ERR_CUDA, "%s: combine launch: %s", who, cudaGetErrorString(e));
        return check_launch(who);
    }
    return OASIS_OK;
}

// How the attention splits the column lists for these shapes (the fused layer launch splits the same way, so
// that its results equal the separate call's bit for bit) and the scratch bytes the partials need.
void attn_split_plan(const oasis_dims_t *dims, int T, int n_cols, int *n_splits, int *cols_per_split, size_t *workspace)
{
    const AttnPlan pl = attn_plan(dims, T, n_cols);
    *n_splits = pl.n_splits;
    *cols_per_split = pl.cols_per_split;
    *workspace = pl.workspace;
}

// The combine launch behind the fused layer kernel: a few CTAs per SM that are all resident at once, started
// early by programmatic stream serialization (the kernel itself waits for the partials).
int launch_attn_combine_after(const oasis_dims_t *dims, int T, void *out, float *lse, float *part_o, float *part_lse,
                              int n_splits, cudaStream_t st, const char *who)
{
    AttnParams p = {};
    p.out = (uint8_t *)out; p.lse = lse; p.part_o = part_o; p.part_lse = part_lse;
    p.T = T; p.Hq = dims->n_q_heads; p.Hkv = dims->n_kv_heads; p.G = dims->n_q_heads / dims->n_kv_heads;
    p.R = T * p.G; p.n_splits = n_splits; p.n_groups = 1; p.rows_per_group = p.R;
    const long long total = (long long)dims->batch * dims->n_kv_heads * p.R;
    long long grid = (long long)sm_count() * 2;          // all resident beside the fused kernel's thread blocks
    if (grid > (total + 7) / 8) grid = (total + 7) / 8;
    prefer_max_shared_carveout(attn_combine_kernel);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, attn_combine_kernel, p, total);
    if (e != cudaSuccess) return fail(OASIS_ERR_CUDA, "%s: combine launch: %s", who, cudaGetErrorString(e));
    return check_launch(who);
}

}  // namespace oasis

extern "C" size_t oasis_attn_workspace_bytes(const oasis_dims_t *dims, int32_t n_q_tokens, int32_t n_cols)
{
    using namespace oasis;
    if (check_dims(dims) != OASIS_OK || n_q_tokens < 1 || n_cols < 1) return 0;
    return attn_plan(dims, n_q_tokens, n_cols).workspace;
}

extern "C" int oasis_sparse_attn(const oasis_dims_t *dims, const void *q, int32_t n_q_tokens,
                                 const void *hbm_pool, const int32_t *slot_tbl, const int32_t *blk_tbl,
                                 int32_t n_cols, const int32_t *seq_len, float scale, void *out,
                                 float *lse, void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace oasis;
    if (int rc = check_dims(dims)) return rc;
    if (!q || !hbm_pool || !slot_tbl || !blk_tbl || !seq_len || !out)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_sparse_attn: NULL pointer argument");
    if (!aligned16(q) || !aligned16(hbm_pool) || !aligned16(out))
        return fail(OASIS_ERR_INVALID_ARG, "oasis_sparse_attn: q, hbm_pool and out must be 16-byte aligned");
    if (n_q_tokens < 1 || n_cols < 1)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_sparse_attn: n_q_tokens %d, n_cols %d", n_q_tokens, n_cols);
    const int G = dims->n_q_heads / dims->n_kv_heads;
    if (n_q_tokens * G > 128)
        return fail(OASIS_ERR_UNSUPPORTED, "oasis_sparse_attn: n_q_tokens * group = %d rows > 128", n_q_tokens * G);
    if (dims->batch == 0) return OASIS_OK;
    const AttnPlan pl = attn_plan(dims, n_q_tokens, n_cols);
    if (pl.workspace > 0) {
        if (!workspace || workspace_bytes < pl.workspace)
            return fail(OASIS_ERR_WORKSPACE, "oasis_sparse_attn: workspace of %zu bytes required, %zu given",
                        pl.workspace, workspace ? workspace_bytes : (size_t)0);
        if (!aligned16(workspace))
            return fail(OASIS_ERR_INVALID_ARG, "oasis_sparse_attn: workspace must be 16-byte aligned");
    }
    if (pl.items > 0x7fffffffLL) return fail(OASIS_ERR_UNSUPPORTED, "oasis_sparse_attn: grid too large");

    AttnParams p;
    p.q = (const uint8_t *)q; p.pool = (const uint8_t *)hbm_pool;
    p.slot_tbl = slot_tbl; p.blk_tbl = blk_tbl; p.seq_len = seq_len;
    p.out = (uint8_t *)out; p.lse = lse;
    p.part_o = (float *)workspace;
    p.part_lse = p.part_o ? p.part_o + (size_t)pl.items * pl.rows_per_group * kHeadDim : nullptr;
    p.scale_log2 = scale * kLog2e;
    p.T = n_q_tokens; p.Hq = dims->n_q_heads; p.Hkv = dims->n_kv_heads; p.G = G;
    p.n_cols = n_cols; p.R = n_q_tokens * G;
    p.n_splits = pl.n_splits; p.cols_per_split = pl.cols_per_split;
    p.n_groups = pl.n_groups; p.rows_per_group = pl.rows_per_group;

    return launch_attn(dims, pl, p, q, hbm_pool, scale, (long long)dims->batch * dims->n_kv_heads * p.R,
                       (cudaStream_t)stream, "oasis_sparse_attn");
}

// ---------------------------------------------------------------------------------------------
// Sparse attention with built-in scratch memory.
//
// oasis_sparse_attn needs a caller-supplied workspace whenever it splits the column list.  Some
// callers have no way to supply one: an inference engine that hands every free byte of the
// device to its KV-cache pool at start-up has nothing left to carve scratch from later, and a
// decode loop cannot afford cudaMalloc, which may fail at that point and synchronises the device
// when it succeeds.  For them the split-KV partials live in the fixed array below, which is part
// of the library image: every GPU that loads the library holds these bytes until the process
// exits.
//
// In host code `g_attn_scratch` is only a stand-in for the device array -- its host address is
// not a device address -- so the device address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and that pointer is what the kernels get.
#include <mutex>

namespace oasis {

constexpr size_t kStaticScratchBytes = 4u << 20;      // 4 MiB
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_attn_scratch[kStaticScratchBytes];

static std::mutex g_scratch_mutex;
static void *g_scratch_ptr[kMaxDevices] = {};          // device address of g_attn_scratch, per device

// Device address of the scratch array on the current device; looked up on first use.
static int static_scratch(void **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(OASIS_ERR_CUDA, "oasis_sparse_attn_static_scratch: cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices)
        return fail(OASIS_ERR_UNSUPPORTED, "oasis_sparse_attn_static_scratch: device ordinal %d >= %d", dev, kMaxDevices);
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_attn_scratch);
        if (e != cudaSuccess || !p) {
            cudaGetLastError();
            return fail(OASIS_ERR_CUDA, "oasis_sparse_attn_static_scratch: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        }
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return OASIS_OK;
}

}  // namespace oasis

extern "C" size_t oasis_static_scratch_bytes(void) { return oasis::kStaticScratchBytes; }

extern "C" int oasis_sparse_attn_static_scratch(const oasis_dims_t *dims, const void *q, int32_t n_q_tokens,
                                                const void *hbm_pool, const int32_t *slot_tbl,
                                                const int32_t *blk_tbl, int32_t n_cols, const int32_t *seq_len,
                                                float scale, void *out, float *lse, void *stream)
{
    using namespace oasis;
    if (int rc = check_dims(dims)) return rc;
    if (!q || !hbm_pool || !slot_tbl || !blk_tbl || !seq_len || !out)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_sparse_attn_static_scratch: NULL pointer argument");
    if (!aligned16(q) || !aligned16(hbm_pool) || !aligned16(out))
        return fail(OASIS_ERR_INVALID_ARG, "oasis_sparse_attn_static_scratch: q, hbm_pool and out must be 16-byte aligned");
    if (n_q_tokens < 1 || n_cols < 1)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_sparse_attn_static_scratch: n_q_tokens %d, n_cols %d", n_q_tokens, n_cols);
    const int G = dims->n_q_heads / dims->n_kv_heads;
    if (n_q_tokens * G > 128)
        return fail(OASIS_ERR_UNSUPPORTED, "oasis_sparse_attn_static_scratch: n_q_tokens * group = %d rows > 128", n_q_tokens * G);
    if (dims->batch == 0) return OASIS_OK;
    const AttnPlan pl = attn_plan(dims, n_q_tokens, n_cols);
    if (pl.workspace > kStaticScratchBytes)
        return fail(OASIS_ERR_WORKSPACE,
                    "oasis_sparse_attn_static_scratch: these shapes need %zu bytes of scratch, the built-in array holds %zu; "
                    "use oasis_sparse_attn with a caller-owned workspace",
                    pl.workspace, kStaticScratchBytes);
    if (pl.items > 0x7fffffffLL) return fail(OASIS_ERR_UNSUPPORTED, "oasis_sparse_attn_static_scratch: grid too large");
    void *scratch = nullptr;
    if (int rc = static_scratch(&scratch)) return rc;

    AttnParams p;
    p.q = (const uint8_t *)q; p.pool = (const uint8_t *)hbm_pool;
    p.slot_tbl = slot_tbl; p.blk_tbl = blk_tbl; p.seq_len = seq_len;
    p.out = (uint8_t *)out; p.lse = lse;
    p.part_o = (float *)scratch;
    p.part_lse = p.part_o + (size_t)pl.items * pl.rows_per_group * kHeadDim;
    p.scale_log2 = scale * kLog2e;
    p.T = n_q_tokens; p.Hq = dims->n_q_heads; p.Hkv = dims->n_kv_heads; p.G = G;
    p.n_cols = n_cols; p.R = n_q_tokens * G;
    p.n_splits = pl.n_splits; p.cols_per_split = pl.cols_per_split;
    p.n_groups = pl.n_groups; p.rows_per_group = pl.rows_per_group;

    return launch_attn(dims, pl, p, q, hbm_pool, scale, (long long)dims->batch * dims->n_kv_heads * p.R,
                       (cudaStream_t)stream, "oasis_sparse_attn_static_scratch");
}
