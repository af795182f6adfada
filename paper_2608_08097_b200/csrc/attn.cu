// Step 4: sparse paged decode attention over the staged working set (Sec. 4.2.1, 4.3).
//
// Work item = (request, KV head, split of the column list, group of query rows).  All
// query rows that share the KV head -- the G = Hq/Hkv heads of every verify-step token --
// are packed into the M dimension of the tensor-core tiles, so each K/V block is read from
// HBM once per item however many rows use it.
//
// A CTA has four warps.  Warp w owns the columns c0 + w, c0 + w + 4, ... of its item: it
// fetches each 8 KiB entry with sixteen 16-byte cp.async per lane into a private 3-deep
// shared-memory ring (XOR-swizzled 16-byte chunks, so ldmatrix is conflict-free), computes
// S = Q K^T for the 16 keys with mma.sync.m16n8k16 (bf16 in, fp32 out), applies the causal
// limit of local blocks, updates a running max / sum in fp32 (online softmax, quad shuffles
// for the row reductions), rounds P to bf16 and accumulates O += P V on the tensor cores.
// The ring is warp-private, so the main loop has no CTA-wide barrier.  At the end the four
// warps' (m, l, O) are merged through shared memory; if the column list was split, the
// item's normalised partial output and its log-sum-exp go to the workspace and a second
// small kernel merges the splits.
// Algorithmic traffic: 8 KiB per (request, KV head, column) plus Q and O.
#include <math_constants.h>

#include "common.cuh"

namespace oasis {

constexpr int kAttnWarps = 4;
constexpr int kAttnStages = 3;
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

__device__ __forceinline__ uint32_t swz(int row, int chunk)   // byte offset inside a [rows][256 B] tile
{
    return (uint32_t)(row * kRowBytes + ((chunk ^ (row & 7)) << 4));
}

template <int N_MT>
__global__ void __launch_bounds__(kAttnWarps * 32, 2)
sparse_attn_kernel(const AttnParams p)
{
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int QROWS = N_MT * 16;
    uint8_t *q_sm = smem;                                  // [QROWS][256 B], swizzled
    uint8_t *kv_sm = smem + QROWS * kRowBytes;             // [warps][stages][8 KiB]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t4 = lane & 3;

    // item -> (bh, split, row group); groups of one (bh, split) are adjacent in the grid
    int item = blockIdx.x;
    const int grp = item % p.n_groups; item /= p.n_groups;
    const int split = item % p.n_splits;
    const int bh = item / p.n_splits;
    const int b = bh / p.Hkv, h = bh % p.Hkv;
    const int row0 = grp * p.rows_per_group;
    const int nrows = min(p.rows_per_group, p.R - row0);
    const int c0 = split * p.cols_per_split;
    const int c1 = min(c0 + p.cols_per_split, p.n_cols);
    const int L = p.seq_len[b];

    // ---- Q rows of this group -> shared memory (zero rows past nrows) -------------------------
    for (int i = tid; i < QROWS * 16; i += blockDim.x) {
        const int r = i >> 4, ch = i & 15;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (r < nrows) {
            const int row = row0 + r;
            const int tq = row / p.G, a = h * p.G + row % p.G;
            v = *reinterpret_cast<const uint4 *>(p.q + ((((long long)b * p.T + tq) * p.Hq + a) * kHeadDim) * 2 + ch * 16);
        }
        *reinterpret_cast<uint4 *>(q_sm + swz(r, ch)) = v;
    }
    __syncthreads();

    // causal limit (last visible position) of the two rows this lane owns in every m-tile
    int limit[N_MT][2];
#pragma unroll
    for (int mt = 0; mt < N_MT; ++mt) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int r = mt * 16 + g + 8 * e;
            limit[mt][e] = (r < nrows) ? L + (row0 + r) / p.G : -1;
        }
    }

    float o[N_MT][16][4];
    float m_run[N_MT][2], l_run[N_MT][2];
#pragma unroll
    for (int mt = 0; mt < N_MT; ++mt) {
        m_run[mt][0] = m_run[mt][1] = -CUDART_INF_F;
        l_run[mt][0] = l_run[mt][1] = 0.f;
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) o[mt][nt][0] = o[mt][nt][1] = o[mt][nt][2] = o[mt][nt][3] = 0.f;
    }

    // Q fragments stay in registers when there is a single m-tile
    uint32_t qf[N_MT == 1 ? 8 : 1][4];
    if constexpr (N_MT == 1) {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const int m = lane >> 3, r = lane & 7;
            ldmatrix_x4(qf[ks], smem_u32(q_sm + swz((m & 1) * 8 + r, ks * 2 + (m >> 1))));
        }
    }

    // ---- this warp's columns ---------------------------------------------------------------------
    const int my_first = c0 + warp;
    const int n_mine = (c1 > my_first) ? (c1 - my_first + kAttnWarps - 1) / kAttnWarps : 0;
    const int32_t *slot_row = p.slot_tbl + (long long)bh * p.n_cols;
    const int32_t *blk_row = p.blk_tbl + (long long)bh * p.n_cols;
    uint8_t *ring = kv_sm + warp * (kAttnStages * kEntryBytes);
    const uint32_t ring_u32 = smem_u32(ring);

    // lane i of a 32-column window holds the table entries of this warp's column i
    int win_slot = -1, win_blk = -1;
    auto load_window = [&](int first_i) {
        const int c = my_first + (first_i + lane) * kAttnWarps;
        win_blk = (first_i + lane < n_mine) ? blk_row[c] : -1;
        win_slot = (win_blk >= 0) ? slot_row[c] : -1;
    };
    auto issue = [&](int i, int slot) {             // fetch this warp's i-th column into ring stage i % stages
        if (slot >= 0) {
            const uint8_t *src = p.pool + (long long)slot * kEntryBytes;
            const uint32_t dst = ring_u32 + (i % kAttnStages) * kEntryBytes;
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const int gch = lane + 32 * c;                 // 16-byte chunk of the entry
                const int part = gch >> 8, r = (gch >> 4) & 15, ch = gch & 15;
                cp_async16(dst + part * kPartBytes + swz(r, ch), src + gch * 16);
            }
        }
        cp_async_commit();
    };

    load_window(0);
#pragma unroll
    for (int s = 0; s < kAttnStages - 1; ++s) {
        const int slot = __shfl_sync(0xffffffffu, win_slot, s);     // s < 32 always
        issue(s, s < n_mine ? slot : -1);
    }

    for (int i = 0; i < n_mine; ++i) {
        if ((i & 31) == 0 && i > 0) load_window(i);
        // prefetch column i + stages - 1 (its ring stage was released at the end of iteration i - 1)
        {
            const int nx = i + kAttnStages - 1;
            int slot = -1;
            if (nx < n_mine) {
                // the window covers columns [32 * (i / 32), +32); nx may fall into the next one
                const int base = (i >> 5) << 5;
                if (nx < base + 32) slot = __shfl_sync(0xffffffffu, win_slot, nx - base);
                else {
                    const int c = my_first + nx * kAttnWarps;
                    const int bk = blk_row[c];
                    slot = bk >= 0 ? slot_row[c] : -1;
                }
            }
            issue(nx, slot);
        }
        const int blk = __shfl_sync(0xffffffffu, win_blk, i & 31);
        cp_async_wait<kAttnStages - 1>();
        __syncwarp();
        if (blk >= 0) {
            const uint32_t k_u32 = ring_u32 + (i % kAttnStages) * kEntryBytes;
            const uint32_t v_u32 = k_u32 + kPartBytes;

            // ---- S = Q K^T for 16 keys -------------------------------------------------------------
            float s[N_MT][2][4];
#pragma unroll
            for (int mt = 0; mt < N_MT; ++mt)
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) s[mt][nt][0] = s[mt][nt][1] = s[mt][nt][2] = s[mt][nt][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                uint32_t kf[4];
                {
                    const int m = lane >> 3, r = lane & 7;
                    ldmatrix_x4(kf, k_u32 + swz((m >> 1) * 8 + r, ks * 2 + (m & 1)));
                }
#pragma unroll
                for (int mt = 0; mt < N_MT; ++mt) {
                    uint32_t a[4];
                    if constexpr (N_MT == 1) {
#pragma unroll
                        for (int e = 0; e < 4; ++e) a[e] = qf[ks][e];
                    } else {
                        const int m = lane >> 3, r = lane & 7;
                        ldmatrix_x4(a, smem_u32(q_sm + swz(mt * 16 + (m & 1) * 8 + r, ks * 2 + (m >> 1))));
                    }
                    mma_bf16_16816(s[mt][0], a, kf[0], kf[1]);
                    mma_bf16_16816(s[mt][1], a, kf[2], kf[3]);
                }
            }

            // ---- online softmax -----------------------------------------------------------------------
            const int pos0 = blk * kBlock;                       // position of key 0 of the block
            uint32_t pf[N_MT][4];
#pragma unroll
            for (int mt = 0; mt < N_MT; ++mt) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {                    // e = 0: row g, e = 1: row g + 8
                    float x[4];                                  // keys 2*t4, 2*t4+1, 8+2*t4, 8+2*t4+1
                    x[0] = s[mt][0][2 * e]; x[1] = s[mt][0][2 * e + 1];
                    x[2] = s[mt][1][2 * e]; x[3] = s[mt][1][2 * e + 1];
                    const int lim = limit[mt][e] - pos0;         // keys with index <= lim are visible
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int key = (c >> 1) * 8 + 2 * t4 + (c & 1);
                        x[c] = key <= lim ? x[c] * p.scale_log2 : -CUDART_INF_F;
                    }
                    float mx = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                    const float m_new = fmaxf(m_run[mt][e], mx);
                    const float m_use = m_new == -CUDART_INF_F ? 0.f : m_new;
                    const float alpha = fast_exp2(m_run[mt][e] - m_use);
                    m_run[mt][e] = m_new;
                    // round P to bf16 first and sum the rounded values, so that the normaliser
                    // matches what the tensor cores multiply with V
                    const __nv_bfloat162 p01 = __floats2bfloat162_rn(fast_exp2(x[0] - m_use), fast_exp2(x[1] - m_use));
                    const __nv_bfloat162 p23 = __floats2bfloat162_rn(fast_exp2(x[2] - m_use), fast_exp2(x[3] - m_use));
                    const float2 f01 = __bfloat1622float2(p01), f23 = __bfloat1622float2(p23);
                    l_run[mt][e] = l_run[mt][e] * alpha + (f01.x + f01.y) + (f23.x + f23.y);
                    pf[mt][e] = *reinterpret_cast<const uint32_t *>(&p01);         // a0 / a1: keys 0..7
                    pf[mt][2 + e] = *reinterpret_cast<const uint32_t *>(&p23);     // a2 / a3: keys 8..15
#pragma unroll
                    for (int nt = 0; nt < 16; ++nt) {
                        o[mt][nt][2 * e] *= alpha;
                        o[mt][nt][2 * e + 1] *= alpha;
                    }
                }
            }

            // ---- O += P V --------------------------------------------------------------------------------
#pragma unroll
            for (int np = 0; np < 8; ++np) {
                uint32_t vf[4];
                {
                    const int m = lane >> 3, r = lane & 7;
                    ldmatrix_x4_trans(vf, v_u32 + swz((m & 1) * 8 + r, np * 2 + (m >> 1)));
                }
#pragma unroll
                for (int mt = 0; mt < N_MT; ++mt) {
                    mma_bf16_16816(o[mt][2 * np], pf[mt], vf[0], vf[1]);
                    mma_bf16_16816(o[mt][2 * np + 1], pf[mt], vf[2], vf[3]);
                }
            }
        }
        __syncwarp();        // every lane is done with this ring stage before it is refilled
    }
    cp_async_wait<0>();

    // ---- merge the four warps through shared memory ----------------------------------------------------
#pragma unroll
    for (int mt = 0; mt < N_MT; ++mt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            float l = l_run[mt][e];
            l += __shfl_xor_sync(0xffffffffu, l, 1);
            l += __shfl_xor_sync(0xffffffffu, l, 2);
            l_run[mt][e] = l;
        }
    __syncthreads();                                        // all rings idle: reuse them
    float *mo = reinterpret_cast<float *>(kv_sm);           // [warps][QROWS][128]
    float *mm = mo + kAttnWarps * QROWS * kHeadDim;         // [warps][QROWS]
    float *ml = mm + kAttnWarps * QROWS;                    // [warps][QROWS]
#pragma unroll
    for (int mt = 0; mt < N_MT; ++mt) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int r = mt * 16 + g + 8 * e;
            float *dst = mo + ((warp * QROWS + r) * kHeadDim);
#pragma unroll
            for (int nt = 0; nt < 16; ++nt)
                *reinterpret_cast<float2 *>(dst + nt * 8 + 2 * t4) = make_float2(o[mt][nt][2 * e], o[mt][nt][2 * e + 1]);
            if (t4 == 0) {
                mm[warp * QROWS + r] = m_run[mt][e];
                ml[warp * QROWS + r] = l_run[mt][e];
            }
        }
    }
    __syncthreads();

    const int d = tid;                                       // 128 threads <-> 128 output dims
    for (int r = 0; r < nrows; ++r) {
        float mw[kAttnWarps], mx = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < kAttnWarps; ++w) {
            mw[w] = mm[w * QROWS + r];
            mx = fmaxf(mx, mw[w]);
        }
        float acc = 0.f, den = 0.f;
        if (mx > -CUDART_INF_F) {
#pragma unroll
            for (int w = 0; w < kAttnWarps; ++w) {
                const float f = fast_exp2(mw[w] - mx);       // 0 for a warp that saw no key
                acc += f * mo[(w * QROWS + r) * kHeadDim + d];
                den += f * ml[w * QROWS + r];
            }
        }
        const float val = den > 0.f ? acc / den : 0.f;
        const float lse2 = den > 0.f ? mx + log2f(den) : -CUDART_INF_F;
        const int row = row0 + r;
        if (p.n_splits == 1) {
            const int tq = row / p.G, a = h * p.G + row % p.G;
            const long long orow = ((long long)b * p.T + tq) * p.Hq + a;
            reinterpret_cast<__nv_bfloat16 *>(p.out)[orow * kHeadDim + d] = __float2bfloat16_rn(val);
            if (p.lse && d == 0) p.lse[orow] = lse2 * kLn2;
        } else {
            const long long prow = (long long)blockIdx.x * p.rows_per_group + r;
            p.part_o[prow * kHeadDim + d] = val;
            if (d == 0) p.part_lse[prow] = lse2;
        }
    }
}

// Merges the splits of one (request, KV head, row): out = sum_s w_s o_s / sum_s w_s with
// w_s = 2^(lse_s - max lse).  One CTA of 128 threads per row.
__global__ void __launch_bounds__(128)
attn_combine_kernel(const AttnParams p)
{
    const int row = blockIdx.x % p.R;
    const int bh = blockIdx.x / p.R;
    const int b = bh / p.Hkv, h = bh % p.Hkv;
    const int grp = row / p.rows_per_group, r = row % p.rows_per_group;
    const int d = threadIdx.x;
    float mx = -CUDART_INF_F;
    for (int s = 0; s < p.n_splits; ++s) {
        const long long item = ((long long)bh * p.n_splits + s) * p.n_groups + grp;
        mx = fmaxf(mx, p.part_lse[item * p.rows_per_group + r]);
    }
    float acc = 0.f, den = 0.f;
    if (mx > -CUDART_INF_F) {
        for (int s = 0; s < p.n_splits; ++s) {
            const long long prow = (((long long)bh * p.n_splits + s) * p.n_groups + grp) * p.rows_per_group + r;
            const float w = fast_exp2(p.part_lse[prow] - mx);
            acc += w * p.part_o[prow * kHeadDim + d];
            den += w;
        }
    }
    const int tq = row / p.G, a = h * p.G + row % p.G;
    const long long orow = ((long long)b * p.T + tq) * p.Hq + a;
    reinterpret_cast<__nv_bfloat16 *>(p.out)[orow * kHeadDim + d] = __float2bfloat16_rn(den > 0.f ? acc / den : 0.f);
    if (p.lse && d == 0) p.lse[orow] = den > 0.f ? (mx + log2f(den)) * kLn2 : -CUDART_INF_F;
}

// Launch geometry shared by the entry point and the workspace query.
struct AttnPlan {
    int n_mt, n_groups, rows_per_group, n_splits, cols_per_split;
    long long items;
    size_t workspace;
};

static AttnPlan attn_plan(const oasis_dims_t *dims, int T, int n_cols)
{
    AttnPlan pl;
    const int G = dims->n_q_heads / dims->n_kv_heads;
    const int R = T * G;
    pl.n_groups = (R + 31) / 32;
    pl.rows_per_group = (R + pl.n_groups - 1) / pl.n_groups;
    pl.n_mt = pl.rows_per_group <= 16 ? 1 : 2;
    const long long base = (long long)dims->batch * dims->n_kv_heads * pl.n_groups;
    // All CTAs should be resident at once (two per SM): a bandwidth-bound kernel then has no
    // tail.  Split the column list only as far as that allows, at least 8 columns per split.
    const long long slots = 2LL * sm_count();
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

    cudaStream_t st = (cudaStream_t)stream;
    const size_t smem = (size_t)pl.n_mt * 16 * kRowBytes + (size_t)kAttnWarps * kAttnStages * kEntryBytes;
    cudaError_t e;
    if (pl.n_mt == 1) {
        e = cudaFuncSetAttribute(sparse_attn_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) sparse_attn_kernel<1><<<(unsigned)pl.items, kAttnWarps * 32, smem, st>>>(p);
    } else {
        e = cudaFuncSetAttribute(sparse_attn_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) sparse_attn_kernel<2><<<(unsigned)pl.items, kAttnWarps * 32, smem, st>>>(p);
    }
    if (e != cudaSuccess) return fail(OASIS_ERR_CUDA, "oasis_sparse_attn: %s", cudaGetErrorString(e));
    if (int rc = check_launch("oasis_sparse_attn")) return rc;
    if (pl.n_splits > 1) {
        attn_combine_kernel<<<(unsigned)((long long)dims->batch * dims->n_kv_heads * p.R), 128, 0, st>>>(p);
        return check_launch("oasis_sparse_attn (combine)");
    }
    return OASIS_OK;
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

    cudaStream_t st = (cudaStream_t)stream;
    const size_t smem = (size_t)pl.n_mt * 16 * kRowBytes + (size_t)kAttnWarps * kAttnStages * kEntryBytes;
    cudaError_t e;
    if (pl.n_mt == 1) {
        e = cudaFuncSetAttribute(sparse_attn_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) sparse_attn_kernel<1><<<(unsigned)pl.items, kAttnWarps * 32, smem, st>>>(p);
    } else {
        e = cudaFuncSetAttribute(sparse_attn_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) sparse_attn_kernel<2><<<(unsigned)pl.items, kAttnWarps * 32, smem, st>>>(p);
    }
    if (e != cudaSuccess) return fail(OASIS_ERR_CUDA, "oasis_sparse_attn_static_scratch: %s", cudaGetErrorString(e));
    if (int rc = check_launch("oasis_sparse_attn_static_scratch")) return rc;
    if (pl.n_splits > 1) {
        attn_combine_kernel<<<(unsigned)((long long)dims->batch * dims->n_kv_heads * p.R), 128, 0, st>>>(p);
        return check_launch("oasis_sparse_attn_static_scratch (combine)");
    }
    return OASIS_OK;
}
