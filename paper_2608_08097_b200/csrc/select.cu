// Step 2: per-(request, KV head) top-k over the block scores, plus the always-kept local
// blocks (Sec. 5.2: K selected blocks and the active local block per KV head).
//
// One CTA per (request, KV head) row, the whole row resident in shared memory:
//   1. scores -> order-preserving 32-bit keys (-0 folded into +0), row min / max;
//   2. radix select of the K-th largest key, 8 bits per pass, restricted to the bits in
//      which the row's keys actually differ (warp-aggregated shared-memory histograms);
//   3. index-ordered compaction: every key above the threshold, and the lowest-index keys
//      equal to it until K are taken (ballot + prefix sums), so ties go to the lowest id;
//   4. sort of the K winners by (score descending, id ascending): rank sort for up to 256, else bitonic;
//   5. sel row, local block ids, and the optional gather lists.
// The work is integer and shared-memory bound; it moves 4 B per block in and (k+2) * 16 B out.
#include "common.cuh"

namespace oasis {

struct SelectParams {
    const float *scores;
    const int32_t *n_full;
    const int32_t *seq_len;
    const int32_t *block_table;
    int32_t *sel;
    long long *stage_idx;
    int32_t *stage_slots;
    int Hkv, max_blocks, k, n_q_tokens, sort_len;   // sort_len: power of two >= k
    Bounds bd;
};

__device__ __forceinline__ uint32_t score_key(float f)
{
    const uint32_t u = __float_as_uint(f + 0.0f);           // -0 -> +0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

__global__ void __launch_bounds__(1024)
select_topk_kernel(const SelectParams p)
{
    extern __shared__ __align__(16) uint8_t smem_raw[];
    unsigned long long *cand = reinterpret_cast<unsigned long long *>(smem_raw);      // [sort_len]
    uint32_t *keys = reinterpret_cast<uint32_t *>(cand + p.sort_len);                 // [max_blocks]
    __shared__ uint32_t hist[256];
    __shared__ uint32_t warp_a[32], warp_b[32];
    __shared__ uint32_t sh_digit, sh_rank, sh_min, sh_max, sh_count;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthreads = blockDim.x, nwarps = nthreads >> 5;
    const int row = blockIdx.x;
    const int b = row / p.Hkv, h = row % p.Hkv;
    const int n_full_raw = p.n_full[b];
    const int n = max(0, min(n_full_raw, p.max_blocks));
    if (kBoundsCheck && threadIdx.x == 0 && n != n_full_raw) in_range(n_full_raw, p.max_blocks + 1, p.bd, kErrBlockCount);
    const int k_eff = min(p.k, n);
    const int n_pad = (n + 31) & ~31;
    const float *srow = p.scores + (long long)row * p.max_blocks;

    // ---- 1. keys, min, max ---------------------------------------------------------------
    uint32_t lo = 0xffffffffu, hi = 0u;
#pragma unroll 1
    for (int j = tid; j < n; j += nthreads) {
        const uint32_t key = score_key(srow[j]);
        keys[j] = key;
        lo = min(lo, key);
        hi = max(hi, key);
    }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) {
        lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, m));
        hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, m));
    }
    if (lane == 0) { warp_a[warp] = lo; warp_b[warp] = hi; }
    if (tid == 0) sh_count = 0;
    __syncthreads();
    if (warp == 0) {
        lo = lane < nwarps ? warp_a[lane] : 0xffffffffu;
        hi = lane < nwarps ? warp_b[lane] : 0u;
#pragma unroll
        for (int m = 16; m > 0; m >>= 1) {
            lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, m));
            hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, m));
        }
        if (lane == 0) { sh_min = lo; sh_max = hi; }
    }
    __syncthreads();
    const uint32_t kmin = sh_min;
    const uint32_t span = (n > 0) ? sh_max - kmin : 0u;
    const int npass = span ? (32 - __clz(span) + 7) / 8 : 0;

    // ---- 2. radix select of the k_eff-th largest (relative) key -----------------------------
    uint32_t prefix = 0;
    uint32_t rank = (uint32_t)k_eff;              // wanted: rank-th largest among keys matching prefix
    if (k_eff > 0) {
#pragma unroll 1
        for (int pass = npass - 1; pass >= 0; --pass) {
            const int shift = pass * 8;
            const uint32_t hi_mask = (shift + 8 >= 32) ? 0u : (0xffffffffu << (shift + 8));
            for (int i = tid; i < 256; i += nthreads) hist[i] = 0;
            __syncthreads();
#pragma unroll 1
            for (int j = tid; j < n_pad; j += nthreads) {
                const bool valid = j < n;
                const uint32_t kr = valid ? keys[j] - kmin : 0u;
                const bool match = valid && ((kr & hi_mask) == prefix);
                const uint32_t digit = (kr >> shift) & 0xffu;
                const unsigned active = __ballot_sync(0xffffffffu, match);
                if (match) {
                    const unsigned peers = __match_any_sync(active, digit);
                    if (lane == __ffs(peers) - 1) atomicAdd(&hist[digit], (uint32_t)__popc(peers));
                }
            }
            __syncthreads();
            if (warp == 0) {
                uint32_t c = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) c += hist[255 - (8 * lane + i)];
                uint32_t incl = c;
#pragma unroll
                for (int m = 1; m < 32; m <<= 1) {
                    const uint32_t o = __shfl_up_sync(0xffffffffu, incl, m);
                    if (lane >= m) incl += o;
                }
                const unsigned reach = __ballot_sync(0xffffffffu, incl >= rank);
                const int owner = __ffs(reach) - 1;      // exists: at least `rank` keys match
                if (lane == owner) {
                    uint32_t running = incl - c;
                    for (int i = 0; i < 8; ++i) {
                        const int d = 255 - (8 * lane + i);
                        const uint32_t cnt = hist[d];
                        if (running + cnt >= rank) {
                            sh_digit = (uint32_t)d;
                            sh_rank = rank - running;
                            break;
                        }
                        running += cnt;
                    }
                }
            }
            __syncthreads();
            prefix |= sh_digit << shift;
            rank = sh_rank;
            __syncthreads();                      // sh_digit / hist are rewritten in the next pass
        }
    }
    const uint32_t thresh = prefix;               // relative key of the k_eff-th largest
    const uint32_t take_equal = rank;             // how many keys equal to it are taken

    // ---- 3. index-ordered compaction ------------------------------------------------------------
    uint32_t equal_before = 0;                    // equal keys in earlier tiles
    if (k_eff > 0) {
#pragma unroll 1
        for (int base = 0; base < n_pad; base += nthreads) {
            const int j = base + tid;
            const bool valid = j < n;
            const uint32_t kr = valid ? keys[j] - kmin : 0u;
            const bool is_gt = valid && kr > thresh;
            const bool is_eq = valid && kr == thresh;
            const unsigned eq_ballot = __ballot_sync(0xffffffffu, is_eq);
            if (lane == 0) warp_a[warp] = __popc(eq_ballot);
            __syncthreads();
            if (warp == 0) {
                const uint32_t c = lane < nwarps ? warp_a[lane] : 0u;
                uint32_t incl = c;
#pragma unroll
                for (int m = 1; m < 32; m <<= 1) {
                    const uint32_t o = __shfl_up_sync(0xffffffffu, incl, m);
                    if (lane >= m) incl += o;
                }
                warp_b[lane] = incl - c;                                  // exclusive prefix per warp
                if (lane == 31) sh_rank = incl;                          // tile total
            }
            __syncthreads();
            const uint32_t eq_rank = equal_before + warp_b[warp] + __popc(eq_ballot & ((1u << lane) - 1u));
            const bool take = is_gt || (is_eq && eq_rank < take_equal);
            const unsigned take_ballot = __ballot_sync(0xffffffffu, take);
            uint32_t slot_base = 0;
            if (lane == 0 && take_ballot) slot_base = atomicAdd(&sh_count, (uint32_t)__popc(take_ballot));
            slot_base = __shfl_sync(0xffffffffu, slot_base, 0);
            if (take) {
                const uint32_t pos = slot_base + __popc(take_ballot & ((1u << lane) - 1u));
                cand[pos] = ((unsigned long long)kr << 32) | (uint32_t)(0xffffffffu - (uint32_t)j);
            }
            equal_before += sh_rank;
            __syncthreads();                       // warp_a / warp_b / sh_rank reused by the next tile
        }
    }
#pragma unroll 1
    for (int i = k_eff + tid; i < p.sort_len; i += nthreads) cand[i] = 0ull;   // sorts to the end
    __syncthreads();

    // ---- 4. sort, descending ----------------------------------------------------------------------
    // Plain loops over shared memory keep the code small: a large kernel that shares SMs with the attention /
    // scoring kernel costs that kernel instruction-cache misses even where little of it executes (a fully
    // unrolled register-resident sorting network made this kernel 75 KB and the decode step 8 % slower).
    if (k_eff > 1 && p.sort_len <= 256 && p.max_blocks >= 2 * p.sort_len) {
        // few winners: every thread ranks one of them against all others (the 64-bit keys are distinct) and
        // drops it at its rank; the key array, no longer needed, is the second buffer
        unsigned long long *sorted = reinterpret_cast<unsigned long long *>(keys);
        __syncthreads();
#pragma unroll 1
        for (int i = tid; i < p.sort_len; i += nthreads) {
            const unsigned long long mine = cand[i];
            int rank_i = 0;
#pragma unroll 4
            for (int o = 0; o < p.sort_len; ++o) rank_i += cand[o] > mine;
            if (mine != 0ull) sorted[rank_i] = mine;          // padding zeros stay behind the k_eff winners
        }
        __syncthreads();
#pragma unroll 1
        for (int i = tid; i < k_eff; i += nthreads) cand[i] = sorted[i];
        __syncthreads();
    } else if (k_eff > 1) {
        const int len = p.sort_len;
#pragma unroll 1
        for (int size = 2; size <= len; size <<= 1) {
#pragma unroll 1
            for (int stride = size >> 1; stride > 0; stride >>= 1) {
#pragma unroll 1
                for (int i = tid; i < (len >> 1); i += nthreads) {
                    const int pos = 2 * i - (i & (stride - 1));
                    const unsigned long long x = cand[pos], y = cand[pos + stride];
                    const bool descending = (pos & size) == 0;
                    if ((x < y) == descending) {
                        cand[pos] = y;
                        cand[pos + stride] = x;
                    }
                }
                __syncthreads();
            }
        }
    }

    // ---- 5. outputs --------------------------------------------------------------------------------
    const int cols = p.k + 2;
    const int end_block = (p.seq_len[b] + p.n_q_tokens + kBlock - 1) / kBlock;   // exclusive
#pragma unroll 1
    for (int c = tid; c < cols; c += nthreads) {
        int v = -1;
        if (c < k_eff) {
            v = (int)(0xffffffffu - (uint32_t)(cand[c] & 0xffffffffull));
        } else if (c >= p.k) {
            const int lb = n_full_raw + (c - p.k);
            if (lb >= 0 && lb < end_block) v = lb;
        }
        const long long o = (long long)row * cols + c;
        p.sel[o] = v;
        if (p.stage_idx) {
            p.stage_slots[o] = (int32_t)o;
            long long src = (v < 0 || v >= p.max_blocks)
                                ? -1ll
                                : (long long)p.block_table[(long long)b * p.max_blocks + v] * p.Hkv + h;
            if (src >= 0 && (!in_range(src, p.bd.n_entries, p.bd, kErrHostEntry) || !in_range(o, p.bd.n_slots, p.bd, kErrSlot)))
                src = -1ll;
            if (kBoundsCheck && v >= p.max_blocks) in_range(v, p.max_blocks, p.bd, kErrBlockId);
            p.stage_idx[o] = src;
        }
    }
}

}  // namespace oasis

extern "C" int oasis_select_topk(const oasis_dims_t *dims, const float *scores,
                                 const int32_t *n_full_blocks, const int32_t *seq_len,
                                 int32_t n_q_tokens, int32_t k, const int32_t *block_table,
                                 int32_t *sel, int64_t *stage_idx, int32_t *stage_slots, void *stream)
{
    using namespace oasis;
    if (int rc = check_dims(dims)) return rc;
    if (!scores || !n_full_blocks || !seq_len || !sel)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_select_topk: NULL pointer argument");
    if ((stage_idx == nullptr) != (stage_slots == nullptr))
        return fail(OASIS_ERR_INVALID_ARG, "oasis_select_topk: stage_idx and stage_slots must both be given or both be NULL");
    if (stage_idx && !block_table)
        return fail(OASIS_ERR_INVALID_ARG, "oasis_select_topk: block_table is required for the gather lists");
    if (k < 1 || k > OASIS_MAX_K) return fail(OASIS_ERR_INVALID_ARG, "oasis_select_topk: k %d outside [1, %d]", k, OASIS_MAX_K);
    if (n_q_tokens < 1) return fail(OASIS_ERR_INVALID_ARG, "oasis_select_topk: n_q_tokens %d < 1", n_q_tokens);
    if (dims->max_blocks > 49152)
        return fail(OASIS_ERR_UNSUPPORTED, "oasis_select_topk: max_blocks %d > 49152", dims->max_blocks);
    if ((long long)dims->batch * dims->n_kv_heads * (k + 2) > 0x7fffffffLL)
        return fail(OASIS_ERR_UNSUPPORTED, "oasis_select_topk: more than 2^31 slots");
    if (dims->batch == 0) return OASIS_OK;

    SelectParams p;
    p.scores = scores; p.n_full = n_full_blocks; p.seq_len = seq_len; p.block_table = block_table;
    p.bd = bounds();
    p.sel = sel; p.stage_idx = (long long *)stage_idx; p.stage_slots = stage_slots;
    p.Hkv = dims->n_kv_heads; p.max_blocks = dims->max_blocks; p.k = k; p.n_q_tokens = n_q_tokens;
    int sort_len = 2;
    while (sort_len < k) sort_len <<= 1;
    p.sort_len = sort_len;
    int threads = 128;
    // about 4 keys per thread: the kernel runs beside the fused attention + scoring kernel, and the shorter it is there
    // the less it costs that kernel (compute-only step of the reasoning-style workload: 1.71 ms with 256 threads per
    // row, 1.60 with 512, 1.58-1.62 with 1,024; with 128 and fewer the top-k itself becomes the step's bottleneck)
    while (threads < 1024 && threads * 4 < dims->max_blocks) threads <<= 1;
    const size_t smem = (size_t)sort_len * 8 + (size_t)dims->max_blocks * 4;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(select_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return fail(OASIS_ERR_CUDA, "oasis_select_topk: shared memory %zu B: %s", smem, cudaGetErrorString(e));
    }
    prefer_max_shared_carveout(select_topk_kernel);
    select_topk_kernel<<<dims->batch * dims->n_kv_heads, threads, smem, (cudaStream_t)stream>>>(p);
    return check_launch("oasis_select_topk");
}
