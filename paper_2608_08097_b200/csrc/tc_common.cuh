// PTX wrappers shared by the tcgen05 / TMA kernels (sm_100a): mbarriers with bounded waits,
// 2-D tensor copies, tcgen05 MMA / commit / fences / tensor-memory loads, shared-memory matrix
// descriptors, and the host-side tensor-map encoder lookup.
#pragma once
#include <cuda.h>
#include <math_constants.h>

#include "common.cuh"

namespace oasis {

constexpr uint32_t kSpinLimit = 1u << 22;

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait: false (and an error code in *err) if the phase did not complete within `limit` probes.
__device__ __forceinline__ bool mbar_wait_limit(uint32_t bar, uint32_t parity, int32_t *err, int code, uint32_t limit)
{
    {
        // one non-blocking probe first: try_wait on a phase that has already completed costs well over a hundred cycles
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
    }
#pragma unroll 1                 // the compiler otherwise unrolls the spin loop at every call site (half the kernel's code)
    for (uint32_t i = 0; i < limit; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done) return true;
    }
    if (err) atomicCAS(err, 0, code);
    return false;
}
// The wait every kernel uses: the compile-time limit of about four million probes (tens of milliseconds).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int32_t *err, int code)
{
    return mbar_wait_limit(bar, parity, err, code, kSpinLimit);
}
// The same wait made by all 32 lanes of a converged warp (the MMA-issuing warps); the lanes agree on the outcome, so the
// warp stays converged whatever happens.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, int32_t *err, int code)
{
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, err, code));
}
// One blocking probe (try_wait) made by the lanes with `active` set, as a predicated instruction of a converged warp:
// there is no branch, so the warp waits as one.
__device__ __forceinline__ bool mbar_try_lanes(uint32_t bar, uint32_t parity, bool active)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %3, 0;\n\t"
        "setp.eq.u32 p, %3, 0x7fffffff;\n\t"       // false
        "@q mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity), "r"((uint32_t)active)
        : "memory");
    return done != 0;
}
// Two waits of a converged warp in one: lane 0 probes barrier A, lane 1 barrier B, in one predicated instruction that
// all lanes execute, and a ballot tells when both phases have completed -- one round trip instead of two (a wait by
// all 32 lanes costs 300-400 cycles even when the phase has long completed, because the lanes take turns at the
// barrier).  Used by the scoring kernel's MMA warp (25.6 against 26.0 us at 16 query rows, 167.8 against 172.5 us at
// 128 K context); in the attention kernels, whose issuing warps share their schedulers with busy softmax warps, the
// plain waits were the faster ones.
__device__ __forceinline__ bool mbar_wait_warp2(uint32_t bar_a, uint32_t parity_a, uint32_t bar_b, uint32_t parity_b, int32_t *err, int code)
{
    const int lane = threadIdx.x & 31;
    const uint32_t bar = lane == 0 ? bar_a : bar_b, parity = lane == 0 ? parity_a : parity_b;
#pragma unroll 1
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        const bool done = mbar_try_lanes(bar, parity, lane < 2);
        if ((__ballot_sync(0xffffffffu, done) & 3u) == 3u) {
            __syncwarp();                        // what the probing lanes have observed is ordered before the others go on
            return true;
        }
    }
    if (lane == 0 && err) atomicCAS(err, 0, code);
    return false;
}
// One non-blocking probe of a phase.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done != 0;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// tcgen05.mma and tcgen05.commit are issued by ONE lane, but from a converged warp: all 32 lanes call these wrappers
// with the same arguments and elect.sync picks the issuing lane (always the same one for the full mask, so a commit
// tracks the MMAs before it).  Issued from inside an `if (lane == 0)` branch instead, every MMA costs about 60 cycles
// whatever its shape (measured: 8 MMAs of 128 x 64 x 16 in 497 cycles), because in divergent code the descriptors
// cannot stay in uniform registers; from a converged warp the same eight take 257 cycles, the tensor core's own time.
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile(
        "{\n\t.reg .pred q;\n\t"
        "elect.sync _|q, 0xffffffff;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "elect.sync _|q, 0xffffffff;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tc_ld16_nowait(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr));
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand stored as rows of 128 bytes with the
// 128-byte swizzle (8-row groups 1024 bytes apart).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);          // start address
    d |= (uint64_t)1 << 16;                           // leading-dimension byte offset (unused here)
    d |= (uint64_t)(1024 >> 4) << 32;                 // stride between 8-row groups
    d |= (uint64_t)1 << 46;                           // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                           // 128-byte swizzle
    return d;
}

// ---- host side -----------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
        else
            cudaGetLastError();
    }
    return fn;
}

// ---- shared by the attention kernels (attn_tc.cu, layer_tc.cu) ----------------------------------------
constexpr int kAtTileCols = 4;                              // blocks per tile
constexpr int kAtTileKeys = kAtTileCols * kBlock;           // 64
constexpr int kAtStageBytes = kAtTileCols * kEntryBytes;    // 32 KiB: one 8 KiB image per block
// Shared-memory image of one block (one 5-D tensor copy): [row group 0..1][dim half 0..1][K, V][8 rows][128 B].
constexpr int kImgGroup = 4096, kImgHalf = 2048, kImgPart = 1024;
constexpr int kAtSBufs = 4;                                 // S / P buffers in tensor memory (Q K^T runs 3 tiles ahead)
constexpr int kAtQBytes = 0;                                // Q lives in tensor memory
constexpr int kAtMaxStages = 7;
constexpr int kAtTmemCols = 512;                            // S buffers [0,256), O [256,384), Q [384,448)
// The softmax weights P go to the P V product as bf16, like V: the two operands of one tcgen05.mma kind::f16 must
// have the same format (fp16 weights against bf16 values raise an illegal-instruction fault on B200).
constexpr uint32_t kIdescPvFormats = (1u << 7) | (1u << 10);
__device__ __forceinline__ uint32_t pack_p(float lo, float hi) { return pack_bf16x2(lo, hi); }
constexpr float kAtLog2e = 1.4426950408889634f;
constexpr float kAtLn2 = 0.6931471805599453f;


__device__ __forceinline__ void tc_mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "elect.sync _|q, 0xffffffff;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
}
__device__ __forceinline__ void tc_st8(uint32_t taddr, const uint32_t (&v)[8])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// K-major operand with 128-byte rows and the 128-byte swizzle is described by smem_desc_sw128().
// MN-major operand (V: rows = keys, 64 dims = 128 bytes per row and half): 8-key groups 1024 bytes
// apart, the second 64-dim half `half_stride` bytes further.
__device__ __forceinline__ uint64_t smem_desc_sw128_mn(uint32_t addr, uint32_t half_stride, uint32_t group_stride)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)((half_stride >> 4) & 0x3fffu) << 16;   // leading-dimension byte offset
    d |= (uint64_t)((group_stride >> 4) & 0x3fffu) << 32;  // stride between 8-key groups
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// K-major operand, 128-byte swizzle, 8-row groups `group_stride` bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128_k(uint32_t addr, uint32_t group_stride)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)((group_stride >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, int c3, int c4,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar)
        : "memory");
}

// Named barrier 1 over the softmax warps (THREADS = 128 per set), returning the AND of their predicates.
template <int THREADS = 128>
__device__ __forceinline__ bool softmax_warps_all(bool pred)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, %2, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"((uint32_t)pred), "n"(THREADS) : "memory");
    return r != 0;
}

// ---- pieces shared by the scoring kernel, the attention kernel and the fused layer kernel ----------------------
// Instruction descriptors (kind::f16): fp32 accumulator (bit 4), operand formats (bits 7-9, 10-12: 1 = bf16),
// B transposed for the key-major V operand (bit 16), N >> 3 (bits 17-22), M >> 4 (bits 24-28).
__device__ __forceinline__ uint32_t idesc_qk(int mma_m)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kAtTileKeys >> 3) << 17) | ((uint32_t)(mma_m >> 4) << 24);
}
__device__ __forceinline__ uint32_t idesc_pv(int mma_m)
{
    return (1u << 4) | kIdescPvFormats | (1u << 16) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(mma_m >> 4) << 24);
}
__device__ __forceinline__ uint32_t idesc_score(int n_cols, int tile_blocks)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_cols >> 3) << 17) | ((uint32_t)(tile_blocks >> 4) << 24);
}

// S = Q K^T of one 64-key tile: Q (128 dims = 8 k-steps) from tensor memory, K from the stage's block images.
__device__ __forceinline__ void issue_qk_tile(uint32_t d_tmem, uint32_t tmem_q, uint64_t k_desc, uint32_t idesc)
{
#pragma unroll
    for (int kc = 0; kc < 2; ++kc)
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4)
            tc_mma_bf16_ts(d_tmem, tmem_q + (kc * 4 + k4) * 8, k_desc + (uint64_t)((kc * kImgHalf + k4 * 32) >> 4), idesc,
                           (kc | k4) ? 1u : 0u);
}
// Two softmax warp sets (the 128-row kernels with a single copy of the query rows, 65 to 128 rows).  A softmax warp
// with full 64-key rows needs 950-1,000 cycles per tile (64 ex2 at 8 cycles per warp instruction, about 240 other
// instructions at 2 or more), of which a lone warp per scheduler loses the latencies between dependent instructions
// and around its waits.  So the rows get two threads each, in two warps of the same scheduler, that take alternate
// tiles of the row; each set keeps a running maximum and sum and an O accumulator of its own (P V of the row's even
// tiles goes to the first, of its odd tiles to the second), merged when the row is written.  Tensor memory then holds
// three S buffers, the two O accumulators and Q.
__host__ __device__ constexpr int at_softmax_sets(int mma_m, int copies) { return (mma_m == 128 && copies == 1) ? 2 : 1; }
__host__ __device__ constexpr int at_s_bufs(int sets) { return sets == 2 ? 3 : kAtSBufs; }
// Ring stage and completion parity of the tile `n` tiles further on (run-time stage count: no division per tile).
__device__ __forceinline__ void ring_advance(int &s, uint32_t &ph, int n, int stages)
{
#pragma unroll
    for (int k = 0; k < n; ++k) {
        ph ^= (s + 1 == stages);
        s = (s + 1 == stages) ? 0 : s + 1;
    }
}
// O (+)= P V of one tile: 16 keys (one block image) per MMA, P from tensor memory.
__device__ __forceinline__ void issue_pv_tile(uint32_t tmem_o, uint32_t p_tmem, uint64_t v_desc, uint32_t idesc, bool first_of_row)
{
#pragma unroll
    for (int ks = 0; ks < kAtTileCols; ++ks)
        tc_mma_bf16_ts(tmem_o, p_tmem + ks * 8, v_desc + (uint64_t)((ks * kEntryBytes) >> 4), idesc,
                       (!first_of_row || ks) ? 1u : 0u);
}
// D[128 blocks x N] = [min | max][128 x 256] . (q^- | q^+)[256 x N] of one scoring tile: 16 MMAs of K = 16.
__device__ __forceinline__ void issue_score_tile(uint32_t d_tmem, uint32_t a_tile, uint32_t b_tile, int n_cols, uint32_t sub_tile_bytes,
                                                 uint32_t idesc)
{
#pragma unroll
    for (int kc = 0; kc < 4; ++kc) {
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4) {
            const uint64_t ad = smem_desc_sw128(a_tile + kc * sub_tile_bytes + k4 * 32);
            const uint64_t bd = smem_desc_sw128(b_tile + kc * n_cols * 128 + k4 * 32);
            tc_mma_bf16(d_tmem, ad, bd, idesc, (kc | k4) ? 1u : 0u);
        }
    }
}
// The four 2-D tensor copies (128 rows x 128 bytes each) that bring one scoring tile of 128 summaries.
__device__ __forceinline__ void load_score_tile(uint32_t dst, const CUtensorMap *map, int y, uint32_t sub_tile_bytes, uint32_t bar)
{
#pragma unroll
    for (int kc = 0; kc < 4; ++kc) tma_load_2d(dst + kc * sub_tile_bytes, map, kc * 64, y, bar);
}
// One block's score: the reduction (max or sum) over the N query columns of this thread's accumulator row.
__device__ __forceinline__ float reduce_score_row(uint32_t taddr, int n_cols, bool reduce_sum)
{
    float res = reduce_sum ? 0.f : -CUDART_INF_F;
#pragma unroll 1
    for (int c = 0; c < n_cols; c += 16) {
        uint32_t v[16];
        tc_ld16(taddr + c, v);
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            const float f = __uint_as_float(v[e]);
            res = reduce_sum ? res + f : fmaxf(res, f);
        }
    }
    return res;
}
// The scoring operand (q^- | q^+) of one (request, KV head): rows n = query rows (R = draft tokens x group; rows R..N-1
// repeat them, or are zero in sum mode), K-major with the 128-byte swizzle: element k of row n lives in sub-tile
// k / 64; k in [0, 128) holds min(q, 0) (it meets the min rows), k in [128, 256) max(q, 0).  `nthr` threads (index
// `me`) share the work; loads are issued eight at a time so their latencies overlap.
__device__ __forceinline__ void build_qpm_operand(uint8_t *dstb, const uint8_t *q, long long q_batch_stride, int b, int h, int R, int G,
                                                  int Hq, int n_cols, bool reduce_sum, int me, int nthr)
{
    const int tasks = n_cols * 16;                           // 16-byte chunks of the query rows
#pragma unroll 1
    for (int i0 = me; i0 < tasks; i0 += nthr * 8) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = i0 + nthr * u;
            v[u] = make_uint4(0, 0, 0, 0);
            const int n = i >> 4, c = i & 15;
            if (i < tasks && (n < R || !reduce_sum)) {
                const int r = n % R;
                const int tq = r / G, a = h * G + r % G;
                v[u] = *reinterpret_cast<const uint4 *>(q + ((long long)b * q_batch_stride + ((long long)tq * Hq + a) * kHeadDim) * 2 + c * 16);
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = i0 + nthr * u;
            if (i >= tasks) continue;
            const int n = i >> 4, c = i & 15;
            const __nv_bfloat162 zero2 = __floats2bfloat162_rn(0.f, 0.f);
            uint4 neg, pos;
            const __nv_bfloat162 *f = reinterpret_cast<const __nv_bfloat162 *>(&v[u]);
            __nv_bfloat162 *n2 = reinterpret_cast<__nv_bfloat162 *>(&neg);
            __nv_bfloat162 *p2 = reinterpret_cast<__nv_bfloat162 *>(&pos);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                n2[e] = __hmin2(f[e], zero2);
                p2[e] = __hmax2(f[e], zero2);
            }
            const int sub = c >> 3, ch = (c & 7) ^ (n & 7);
            uint8_t *row = dstb + n * 128 + ch * 16;
            *reinterpret_cast<uint4 *>(row + (size_t)sub * n_cols * 128) = neg;          // k in [0, 128): min rows
            *reinterpret_cast<uint4 *>(row + (size_t)(2 + sub) * n_cols * 128) = pos;    // k in [128, 256): max rows
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// ---- table windows of the attention producers ------------------------------------------------------------------
// The producer warp reads a row's block ids and slot ids 32 columns (eight tiles) at a time, one window ahead, by
// asynchronous copies into two small shared-memory buffers: lane j requests column j of the window, and the copies
// of a window are only waited for when its first tile comes up, eight tiles later.  (Loads into registers did not
// stay ahead: written as a rotation of current / next window registers, the warp stalled for a whole memory
// latency, 2,300-3,100 cycles, at every window switch, whatever form the load took.)
constexpr int kWinCols = 32;                                // columns per window
constexpr int kWinBytes = 2 * kWinCols * 4;                 // block ids [32], slot ids [32]
// Lane `lane` requests column `c` of the row (beyond the last column `c1 - 1`: -1) into the window buffer at `win_u32`.
__device__ __forceinline__ void window_request(uint32_t win_u32, int lane, const int32_t *blk_row, const int32_t *slot_row, int c, int c1)
{
    const uint32_t dst = win_u32 + (uint32_t)lane * 4u;
    if (c < c1) {
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(blk_row + c) : "memory");
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst + kWinCols * 4), "l"(slot_row + c) : "memory");
    } else {
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(dst), "r"(-1) : "memory");
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(dst + kWinCols * 4), "r"(-1) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}
// All requested windows have landed and are visible to the whole warp; earlier reads of the buffers are over.
__device__ __forceinline__ void window_wait()
{
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncwarp();
}
// Block id and slot id of this lane's column of tile `i` (lanes 0..3; -1 for the other lanes).
__device__ __forceinline__ void window_read(const int32_t *win, int i, int lane, int &blk, int &slot)
{
    const int32_t *w = win + ((i >> 3) & 1) * (2 * kWinCols) + (i & 7) * kAtTileCols;
    blk = -1;
    slot = -1;
    if (lane < kAtTileCols) {
        blk = w[lane];
        slot = w[kWinCols + lane];
    }
}
// Producer side of one attention tile (the producer warp; lanes 0..3 hold one block each): records the block ids for
// the softmax warps, zeroes the V part of a missing block's image (a missing block contributes P = 0, which must not
// meet stale NaN bit patterns in V), announces the bytes and issues one 5-D tensor copy per present block (the whole
// 8 KiB entry, gathered by slot id).
__device__ __forceinline__ void stage_attn_tile(int lane, int blk, int slot, int32_t *tile_blk_s, uint8_t *stage_ptr, uint32_t stage_u32,
                                                const CUtensorMap *map, uint32_t bar)
{
    const unsigned valid = __ballot_sync(0xffffffffu, lane < kAtTileCols && blk >= 0);
    if (lane < kAtTileCols) tile_blk_s[lane] = blk;
    if ((valid & 0xfu) != 0xfu) {
        // the whole warp zeroes the V part of each missing block: lane -> (row group, dim half) unit lane / 8, 128 bytes of it
#pragma unroll
        for (int c = 0; c < kAtTileCols; ++c) {
            if ((valid >> c) & 1u) continue;
            uint8_t *dst = stage_ptr + c * kEntryBytes + (lane >> 4) * kImgGroup + ((lane >> 3) & 1) * kImgHalf + kImgPart + (lane & 7) * 128;
#pragma unroll
            for (int j = 0; j < 8; ++j) *reinterpret_cast<uint4 *>(dst + j * 16) = make_uint4(0, 0, 0, 0);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    if (lane == 0) mbar_arrive_expect_tx(bar, (uint32_t)__popc(valid) * kEntryBytes);
    __syncwarp();
    if (lane < kAtTileCols && blk >= 0) tma_load_5d(stage_u32 + lane * kEntryBytes, map, 0, 0, 2 * slot, 0, 0, bar);
}
// One query row (128 dims, 16 x 16 bytes in v) to this thread's tensor-memory lane as the A operand of Q K^T.
__device__ __forceinline__ void q_row_to_tmem(uint32_t q_lane, const uint4 (&v)[16])
{
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const uint32_t w[16] = {v[4 * c].x, v[4 * c].y, v[4 * c].z, v[4 * c].w, v[4 * c + 1].x, v[4 * c + 1].y,
                                v[4 * c + 1].z, v[4 * c + 1].w, v[4 * c + 2].x, v[4 * c + 2].y, v[4 * c + 2].z,
                                v[4 * c + 2].w, v[4 * c + 3].x, v[4 * c + 3].y, v[4 * c + 3].z, v[4 * c + 3].w};
        tc_st16(q_lane + c * 16, w);
    }
    tc_wait_st();
}

// ---- packed fp32 arithmetic (two lanes per instruction) and the three-input maximum of sm_100 ------------------
__device__ __forceinline__ uint64_t f32x2(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f32x2_split(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b)
{
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// ---- one 64-key tile of the online softmax, shared by the attention kernel and the fused layer kernel --------
// The calling thread owns one MMA row (one tensor-memory lane).  It reads its row of S = Q K^T for the blocks of
// its copy, masks positions past `limit` (only tiles that hold a block of the local window need it), raises the
// reference maximum lazily -- only when a logit exceeds it by 2^8; the O row in tensor memory is then rescaled,
// after `wait_prev()` has made sure that the previous tile's P V has completed -- and writes P = 2^(s - m_ref),
// rounded to bf16, back over S; the columns of the other copies' blocks get P = 0.  Running maximum and sum stay
// in the thread's registers; there is no cross-thread reduction.
//   s_tmem      tensor-memory address of the tile's S buffer at this thread's lane
//   o_tmem      tensor-memory address of the O rows at this thread's lane
//   tile_blk    the four block ids of the tile (shared memory), -1 = missing
//   copy        which copy of the query rows this thread belongs to (0 when COPIES == 1)
//   have_o      O already holds earlier tiles of this row (else there is nothing to rescale)
// Returns false if wait_prev() gave up.
template <int COPIES, class WaitPrev>
__device__ __forceinline__ bool softmax_tile(const uint32_t s_tmem, const uint32_t o_tmem, const int32_t *tile_blk, const int copy_in,
                                             const int limit, const bool has_row, const float scale_log2, float &m_ref, float &l_sum,
                                             const bool have_o, WaitPrev &&wait_prev)
{
    constexpr int BPC = kAtTileCols / COPIES;               // blocks of a tile each copy handles
    constexpr int KPC = BPC * kBlock;                       // keys of a tile each copy handles
    const int copy = COPIES == 1 ? 0 : copy_in;
    bool alive = true;
    int nvis[BPC];                                          // visible keys of each of this copy's blocks
    bool masked = false;
#pragma unroll
    for (int c = 0; c < BPC; ++c) {
        const int blk = tile_blk[copy * BPC + c];
        int n = blk < 0 ? 0 : limit - blk * kBlock + 1;
        n = max(0, min(n, kBlock));
        nvis[c] = n;
        masked |= has_row && n < kBlock;                    // lanes without an MMA row are zeroed below instead
    }
    masked = __any_sync(0xffffffffu, masked);
    float x[KPC];
    {
        uint32_t v[BPC][16];
#pragma unroll
        for (int c = 0; c < BPC; ++c) tc_ld16_nowait(s_tmem + (copy * BPC + c) * 16, v[c]);
        tc_wait_ld();
#pragma unroll
        for (int c = 0; c < BPC; ++c)
#pragma unroll
            for (int e = 0; e < 16; ++e) x[c * 16 + e] = __uint_as_float(v[c][e]);
    }
    if (masked) {
#pragma unroll
        for (int c = 0; c < BPC; ++c)
#pragma unroll
            for (int e = 0; e < 16; ++e)
                if (e >= nvis[c]) x[c * 16 + e] = -CUDART_INF_F;
    }
    float mx4[4] = {x[0], x[1], x[2], x[3]};
#pragma unroll
    for (int e = 4; e < KPC; e += 8) {                      // three-input maxima: two elements per instruction
        mx4[0] = max3(mx4[0], x[e], x[e + 4]);
        mx4[1] = max3(mx4[1], x[e + 1], x[e + 5]);
        mx4[2] = max3(mx4[2], x[e + 2], x[e + 6]);
        mx4[3] = max3(mx4[3], x[e + 3], x[e + 7]);
    }
    // a lane without an MMA row read whatever its tensor-memory lane held: it must not raise the reference
    const float mx = has_row ? fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) : -CUDART_INF_F;
    const float mxs = mx * scale_log2;
    const bool raise = mxs > m_ref + 8.0f;
    if (__any_sync(0xffffffffu, raise)) {
        // the O rows must be complete up to the previous tile before they are rescaled
        if (have_o) alive = wait_prev();
        tc_fence_after();
        const float m_new = raise ? mxs : m_ref;
        const float alpha = m_new == -CUDART_INF_F ? 1.f : fast_exp2(m_ref - m_new);
        m_ref = m_new;
        l_sum *= alpha;
        if (have_o) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                uint32_t v[16];
                tc_ld16(o_tmem + c * 16, v);
#pragma unroll
                for (int e = 0; e < 16; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * alpha);
                tc_st16(o_tmem + c * 16, v);
            }
            tc_wait_st();
        }
    }
    const float neg_m = m_ref == -CUDART_INF_F ? 0.f : -m_ref;
    const uint64_t scale2 = f32x2(scale_log2, scale_log2), neg_m2 = f32x2(neg_m, neg_m);
    uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};            // eight partial sums, two per packed accumulator
    // P of the whole tile is 32 packed columns; this copy owns columns [copy*KPC/2, +KPC/2), the rest is 0
    uint32_t pk[KPC / 2];
#pragma unroll
    for (int e = 0; e < KPC / 2; ++e) {
        float t0, t1;
        f32x2_split(fma_f32x2(f32x2(x[2 * e], x[2 * e + 1]), scale2, neg_m2), t0, t1);
        const float p0 = fast_exp2(t0), p1 = fast_exp2(t1);
        sum2[e & 3] = add_f32x2(sum2[e & 3], f32x2(p0, p1));
        pk[e] = pack_p(p0, p1);
    }
    {
        float lo, hi;
        f32x2_split(add_f32x2(add_f32x2(sum2[0], sum2[1]), add_f32x2(sum2[2], sum2[3])), lo, hi);
        l_sum += lo + hi;
    }
    if (!has_row) {
#pragma unroll
        for (int e = 0; e < KPC / 2; ++e) pk[e] = 0u;       // and it stores P = 0
    }
#pragma unroll
    for (int g8 = 0; g8 < 4; ++g8) {                        // four groups of 8 packed columns = four blocks
        uint32_t w8[8];
        if (COPIES == 1) {
#pragma unroll
            for (int e = 0; e < 8; ++e) w8[e] = pk[g8 * 8 + e];
        } else {
            const int own = g8 - copy * BPC;                // index among this copy's blocks, if in [0, BPC)
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                uint32_t val = 0u;
#pragma unroll
                for (int c = 0; c < BPC; ++c)
                    if (own == c) val = pk[c * 8 + e];
                w8[e] = val;
            }
        }
        tc_st8(s_tmem + g8 * 8, w8);
    }
    tc_wait_st();
    return alive;
}

}  // namespace oasis
