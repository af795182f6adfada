// Step 4: sparse paged decode attention over the staged working set (Sec. 4.2.1, 4.3).
//
// Work item = (request, KV head, split of the column list, group of query rows).  All
// query rows that share the KV head -- the G = Hq/Hkv heads of every verify-step token --
// are packed into the M dimension of the tensor-core tiles, so each K/V block is read from
// HBM once per item however many rows use it.
//
// A CTA has four column slots; slot s owns the columns c0 + s, c0 + s + 4, ... of its item.
// A slot is served by one warp per 16-row m-tile (one or two warps): together they fetch each
// 8 KiB entry with 16-byte cp.async into the slot's private 3-deep shared-memory ring
// (XOR-swizzled 16-byte chunks, so ldmatrix is conflict-free) and meet on the slot's named
// barrier; each warp then computes S = Q K^T for its 16 rows x 16 keys with mma.sync.m16n8k16
// (bf16 in, fp32 out), applies the causal limit (local blocks only), keeps a running max / sum
// in fp32 (online softmax, quad shuffles; the running max is only raised when a row's new max
// exceeds it by 2^8, so the accumulator is rarely rescaled), rounds P to bf16 and accumulates
// O += P V on the tensor cores.  There is no CTA-wide barrier in the main loop.  At the end
// the slots' (m, l, O) are merged through shared memory; if the column list was split, the
// item's normalised partial output and its log-sum-exp go to the workspace and a second
// small kernel merges the splits.
// Algorithmic traffic: 8 KiB per (request, KV head, column) plus Q and O.
#include <math_constants.h>

#include <cstdlib>

#include "common.cuh"

namespace oasis {

constexpr int kAttnSlots = 4;       // column slots per CTA (each served by one warp per m-tile)
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

__device__ __forceinline__ void slot_barrier(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

template <int N_MT>
__global__ void __launch_bounds__(kAttnSlots * N_MT * 32, 2)
sparse_attn_kernel(const AttnParams p)
{
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int QROWS = N_MT * 16;
    constexpr int SLOT_THREADS = N_MT * 32;
    constexpr int NTHREADS = kAttnSlots * SLOT_THREADS;
    uint8_t *q_sm = smem;                                  // [QROWS][256 B], swizzled
    uint8_t *kv_sm = smem + QROWS * kRowBytes;             // [slots][stages][8 KiB]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t4 = lane & 3;
    const int mt = warp % N_MT, slot = warp / N_MT;
    const int slot_lane = mt * 32 + lane;                  // 0 .. SLOT_THREADS-1

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
    for (int i = tid; i < QROWS * 16; i += NTHREADS) {
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

    // causal limit (last visible position) of the two rows this lane owns: rows g and g + 8 of m-tile mt
    int limit[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int r = mt * 16 + g + 8 * e;
        limit[e] = (r < nrows) ? L + (row0 + r) / p.G : -1;
    }

    float o[16][4];
    float m_run[2] = {-CUDART_INF_F, -CUDART_INF_F}, l_run[2] = {0.f, 0.f};
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;

    // Q fragments of this warp's m-tile stay in registers when the CTA is small enough to afford them
    constexpr bool kQInRegs = (N_MT == 1);
    uint32_t qf[kQInRegs ? 8 : 1][4];
    const int lm = lane >> 3, lr = lane & 7;               // ldmatrix: matrix index, row within it
    const uint32_t q_u32 = smem_u32(q_sm);
    if constexpr (kQInRegs) {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
            ldmatrix_x4(qf[ks], q_u32 + swz(mt * 16 + (lm & 1) * 8 + lr, ks * 2 + (lm >> 1)));
    }

    // ---- this slot's columns ---------------------------------------------------------------------
    const int my_first = c0 + slot;
    const int n_mine = (c1 > my_first) ? (c1 - my_first + kAttnSlots - 1) / kAttnSlots : 0;
    const int32_t *slot_row = p.slot_tbl + (long long)bh * p.n_cols;
    const int32_t *blk_row = p.blk_tbl + (long long)bh * p.n_cols;
    const uint32_t ring_u32 = smem_u32(kv_sm + slot * (kAttnStages * kEntryBytes));

    // lane i of a 32-column window holds the table entries of this slot's column i
    int win_slot = -1, win_blk = -1;
    auto load_window = [&](int first_i) {
        const int c = my_first + (first_i + lane) * kAttnSlots;
        win_blk = (first_i + lane < n_mine) ? blk_row[c] : -1;
        win_slot = (win_blk >= 0) ? slot_row[c] : -1;
    };
    auto issue = [&](int i, int entry) {           // fetch this slot's i-th column into ring stage i % stages
        if (entry >= 0) {
            const uint8_t *src = p.pool + (long long)entry * kEntryBytes;
            const uint32_t dst = ring_u32 + (i % kAttnStages) * kEntryBytes;
#pragma unroll
            for (int c = 0; c < 16 / N_MT; ++c) {
                const int gch = slot_lane + SLOT_THREADS * c;          // 16-byte chunk of the entry
                const int part = gch >> 8, r = (gch >> 4) & 15, ch = gch & 15;
                cp_async16(dst + part * kPartBytes + swz(r, ch), src + gch * 16);
            }
        }
        cp_async_commit();
    };
    auto slot_sync = [&]() {
        if constexpr (N_MT == 1) __syncwarp();
        else slot_barrier(1 + slot, SLOT_THREADS);
    };

    load_window(0);
#pragma unroll
    for (int s = 0; s < kAttnStages - 1; ++s) {
        const int entry = __shfl_sync(0xffffffffu, win_slot, s);     // s < 32 always
        issue(s, s < n_mine ? entry : -1);
    }

    for (int i = 0; i < n_mine; ++i) {
        if ((i & 31) == 0 && i > 0) load_window(i);
        // prefetch column i + stages - 1 (its ring stage was released at the end of iteration i - 1)
        {
            const int nx = i + kAttnStages - 1;
            int entry = -1;
            if (nx < n_mine) {
                const int base = (i >> 5) << 5;                      // the window covers [base, base + 32)
                if (nx < base + 32) entry = __shfl_sync(0xffffffffu, win_slot, nx - base);
                else {
                    const int c = my_first + nx * kAttnSlots;
                    const int bk = blk_row[c];
                    entry = bk >= 0 ? slot_row[c] : -1;
                }
            }
            issue(nx, entry);
        }
        const int blk = __shfl_sync(0xffffffffu, win_blk, i & 31);
        cp_async_wait<kAttnStages - 1>();
        slot_sync();                                   // every thread's share of the entry has landed
        if (blk >= 0) {
            const uint32_t k_u32 = ring_u32 + (i % kAttnStages) * kEntryBytes;
            const uint32_t v_u32 = k_u32 + kPartBytes;

            // ---- S = Q K^T: 16 rows x 16 keys -------------------------------------------------------
            float s[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                uint32_t kf[4], a[4];
                ldmatrix_x4(kf, k_u32 + swz((lm >> 1) * 8 + lr, ks * 2 + (lm & 1)));
                if constexpr (kQInRegs) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) a[e] = qf[ks][e];
                } else {
                    ldmatrix_x4(a, q_u32 + swz(mt * 16 + (lm & 1) * 8 + lr, ks * 2 + (lm >> 1)));
                }
                mma_bf16_16816(s[0], a, kf[0], kf[1]);
                mma_bf16_16816(s[1], a, kf[2], kf[3]);
            }

            // ---- online softmax with a lazily raised running max -----------------------------------------
            const int pos0 = blk * kBlock;                       // position of key 0 of the block
            const bool masked = pos0 + kBlock - 1 > L;           // only local blocks reach past the history
            float x[2][4], mxs[2];
            bool raise = false;
#pragma unroll
            for (int e = 0; e < 2; ++e) {                        // e = 0: row g, e = 1: row g + 8
                x[e][0] = s[0][2 * e]; x[e][1] = s[0][2 * e + 1];        // keys 2*t4, 2*t4+1
                x[e][2] = s[1][2 * e]; x[e][3] = s[1][2 * e + 1];        // keys 8+2*t4, 8+2*t4+1
                if (masked) {
                    const int lim = limit[e] - pos0;             // keys with index <= lim are visible
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int key = (c >> 1) * 8 + 2 * t4 + (c & 1);
                        if (key > lim) x[e][c] = -CUDART_INF_F;
                    }
                }
                float mx = fmaxf(fmaxf(x[e][0], x[e][1]), fmaxf(x[e][2], x[e][3]));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                mxs[e] = mx * p.scale_log2;                      // scale > 0: max commutes with scaling
                raise |= mxs[e] > m_run[e] + 8.0f;               // also true for the first visible key
            }
            if (__any_sync(0xffffffffu, raise)) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const float m_new = mxs[e] > m_run[e] + 8.0f ? mxs[e] : m_run[e];
                    const float alpha = m_new == -CUDART_INF_F ? 1.f : fast_exp2(m_run[e] - m_new);
                    m_run[e] = m_new;
                    l_run[e] *= alpha;
#pragma unroll
                    for (int nt = 0; nt < 16; ++nt) {
                        o[nt][2 * e] *= alpha;
                        o[nt][2 * e + 1] *= alpha;
                    }
                }
            }
            uint32_t pf[4];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const float neg_m = m_run[e] == -CUDART_INF_F ? 0.f : -m_run[e];
                float pr[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) pr[c] = fast_exp2(fmaf(x[e][c], p.scale_log2, neg_m));
                l_run[e] += (pr[0] + pr[1]) + (pr[2] + pr[3]);
                pf[e] = pack_bf16x2(pr[0], pr[1]);               // a0 / a1: keys 0..7
                pf[2 + e] = pack_bf16x2(pr[2], pr[3]);           // a2 / a3: keys 8..15
            }

            // ---- O += P V --------------------------------------------------------------------------------
#pragma unroll
            for (int np = 0; np < 8; ++np) {
                uint32_t vf[4];
                ldmatrix_x4_trans(vf, v_u32 + swz((lm & 1) * 8 + lr, np * 2 + (lm >> 1)));
                mma_bf16_16816(o[2 * np], pf, vf[0], vf[1]);
                mma_bf16_16816(o[2 * np + 1], pf, vf[2], vf[3]);
            }
        }
        slot_sync();         // every thread of the slot is done with this ring stage before it is refilled
    }
    cp_async_wait<0>();

    // ---- merge the four slots through shared memory ----------------------------------------------------
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        float l = l_run[e];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        l_run[e] = l;
    }
    __syncthreads();                                        // all rings idle: reuse them
    float *mo = reinterpret_cast<float *>(kv_sm);           // [slots][QROWS][128]
    float *mm = mo + kAttnSlots * QROWS * kHeadDim;         // [slots][QROWS]
    float *ml = mm + kAttnSlots * QROWS;                    // [slots][QROWS]
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int r = mt * 16 + g + 8 * e;
        float *dst = mo + ((slot * QROWS + r) * kHeadDim);
#pragma unroll
        for (int nt = 0; nt < 16; ++nt)
            *reinterpret_cast<float2 *>(dst + nt * 8 + 2 * t4) = make_float2(o[nt][2 * e], o[nt][2 * e + 1]);
        if (t4 == 0) {
            mm[slot * QROWS + r] = m_run[e];
            ml[slot * QROWS + r] = l_run[e];
        }
    }
    __syncthreads();

    const int d = tid & (kHeadDim - 1);                      // 128 threads <-> 128 output dims
    for (int r = tid >> 7; r < nrows; r += NTHREADS / kHeadDim) {
        float mw[kAttnSlots], mx = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < kAttnSlots; ++w) {
            mw[w] = mm[w * QROWS + r];
            mx = fmaxf(mx, mw[w]);
        }
        float acc = 0.f, den = 0.f;
        if (mx > -CUDART_INF_F) {
#pragma unroll
            for (int w = 0; w < kAttnSlots; ++w) {
                const float f = fast_exp2(mw[w] - mx);       // 0 for a slot that saw no key
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

// The tcgen05 kernel (attn_tc.cu) is the product path; the mma.sync kernel above stays as a
// development cross-check behind an environment switch.
static bool use_tc()
{
    static const bool legacy = getenv("OASIS_ATTN_MMA_SYNC") != nullptr;
    return !legacy;
}

int launch_attn_tc(const oasis_dims_t *dims, const void *q, int n_q_tokens, const void *hbm_pool,
                   const int32_t *slot_tbl, const int32_t *blk_tbl, int n_cols, const int32_t *seq_len, float scale,
                   void *out, float *lse, float *part_o, float *part_lse, int n_splits, int cols_per_split,
                   int stages, int32_t *err_word, cudaStream_t st, const char *who);      // attn_tc.cu

static AttnPlan attn_plan(const oasis_dims_t *dims, int T, int n_cols)
{
    AttnPlan pl;
    const int G = dims->n_q_heads / dims->n_kv_heads;
    const int R = T * G;
    if (use_tc()) {                      // all rows of a KV head in one CTA (M = 128)
        pl.n_groups = 1;
        pl.rows_per_group = R;
    } else {
        pl.n_groups = (R + 31) / 32;
        pl.rows_per_group = (R + pl.n_groups - 1) / pl.n_groups;
    }
    pl.n_mt = pl.rows_per_group <= 16 ? 1 : 2;
    const long long base = (long long)dims->batch * dims->n_kv_heads * pl.n_groups;
    // All CTAs should be resident at once (two per SM): a bandwidth-bound kernel then has no
    // tail.  Split the column list only as far as that allows, at least 8 columns per split.
    const long long slots = (use_tc() ? 1LL : 2LL) * sm_count();   // resident CTAs: the tcgen05 kernel runs one per SM
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
    if (use_tc()) {
        if (int rc = launch_attn_tc(dims, q, p.T, pool, p.slot_tbl, p.blk_tbl, p.n_cols, p.seq_len, scale, p.out, p.lse,
                                    p.part_o, p.part_lse, pl.n_splits, pl.cols_per_split, 7, error_word(), st, who))
            return rc;
        if (pl.n_splits > 1) {
            attn_combine_kernel<<<(unsigned)combine_ctas, 128, 0, st>>>(p);
            return check_launch(who);
        }
        return OASIS_OK;
    }
    const size_t smem = (size_t)pl.n_mt * 16 * kRowBytes + (size_t)kAttnSlots * kAttnStages * kEntryBytes;
    cudaError_t e;
    if (pl.n_mt == 1) {
        e = cudaFuncSetAttribute(sparse_attn_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) sparse_attn_kernel<1><<<(unsigned)pl.items, kAttnSlots * 32, smem, st>>>(p);
    } else {
        e = cudaFuncSetAttribute(sparse_attn_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess) sparse_attn_kernel<2><<<(unsigned)pl.items, kAttnSlots * 64, smem, st>>>(p);
    }
    if (e != cudaSuccess) return fail(OASIS_ERR_CUDA, "%s: %s", who, cudaGetErrorString(e));
    if (int rc = check_launch(who)) return rc;
    if (pl.n_splits > 1) {
        attn_combine_kernel<<<(unsigned)combine_ctas, 128, 0, st>>>(p);
        return check_launch(who);
    }
    return OASIS_OK;
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
