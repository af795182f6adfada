// Shared device/host helpers of the OasisKV hot-path kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <mutex>

#include "../../include/oasis.h"

namespace oasis {

constexpr int kHeadDim = 128;
constexpr int kBlock = 16;                      // tokens per KV block
constexpr int kRowBytes = kHeadDim * 2;         // one bf16 key/value/summary row
constexpr int kPartBytes = kBlock * kRowBytes;  // K part (or V part) of an entry: 4 KiB
constexpr int kEntryBytes = 2 * kPartBytes;     // 8 KiB
constexpr int kSummaryBytes = 2 * kRowBytes;    // min row + max row: 512 B

// Records the message returned by oasis_last_error() and passes `code` through.
int fail(int code, const char *fmt, ...);
int check_dims(const oasis_dims_t *dims);
int check_launch(const char *what);   // cudaGetLastError() -> status
int sm_count();                       // multiprocessors of the current device (148 if unknown)
int32_t *error_word();                // device word registered with oasis_set_error_word (or NULL)

// ---- bounds-check build (-DOASIS_BOUNDS_CHECK) ---------------------------------------------------------
// In that build every index a kernel reads from a device array -- an entry of the full-KV pool, a slot of the
// working-set pool, a logical block id, a per-request block count -- is range-checked before it is used; a
// violation records a code in the registered error word (first one wins) and the access is skipped.  Nothing
// traps.  In the regular build the checks compile to nothing.
#ifdef OASIS_BOUNDS_CHECK
constexpr bool kBoundsCheck = true;
#else
constexpr bool kBoundsCheck = false;
#endif
constexpr int kErrHostEntry = 201;   // index into the full-KV pool outside [0, n_host_entries)
constexpr int kErrSlot = 202;        // slot outside [0, n_slots)
constexpr int kErrBlockId = 203;     // logical block id outside [0, max_blocks)
constexpr int kErrBlockCount = 204;  // per-request block count / range beyond max_blocks

struct Bounds {
    long long n_entries;   // entries ((block, head) pairs) of the full-KV pool
    long long n_slots;     // entries of the working-set pool
    int32_t *err;          // the registered error word (may be NULL)
};
Bounds bounds();           // what oasis_set_extents declared (huge when nothing was declared) + the error word

__device__ __forceinline__ bool in_range(long long v, long long n, const Bounds &bd, int code)
{
    if constexpr (!kBoundsCheck) return true;
    if (v >= 0 && v < n) return true;
    if (bd.err) atomicCAS(bd.err, 0, code);
    return false;
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- device helpers -----------------------------------------------------------------

__device__ __forceinline__ uint4 ld_stream_v4(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi)
{
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// The small kernels of the other streams (top-k, plan, gather, summaries) ask for the largest shared-memory
// carve-out although they need little: an SM they have configured otherwise could not take a thread block of the
// attention / scoring kernels (which need nearly all of it) until they have left.  The attention / scoring kernels ask
// for it too: an instantiation with four ring stages needs 173 KiB, the driver then configured the SM for the next
// size up, and a top-k thread block (20 KiB at 4,096 blocks per row) no longer fitted beside it and a gather thread
// block -- every gather waited for the following layer's launch (budget x draft sweep, 8 draft tokens: 0.75 -> 0.52 ms).
inline void prefer_max_shared_carveout_of(const void *kernel)
{
    // once per kernel (per instantiation: instantiations of one template share their pointer TYPE, so the flag cannot be
    // a static of a function template over that type); a process drives one GPU, so once per process is once per device
    static std::mutex lock;
    static const void *seen[256];
    static int n_seen = 0;
    std::lock_guard<std::mutex> guard(lock);
    for (int i = 0; i < n_seen; ++i)
        if (seen[i] == kernel) return;
    cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
    if (n_seen < 256) seen[n_seen++] = kernel;
}

template <typename K>
inline void prefer_max_shared_carveout(K kernel)
{
    prefer_max_shared_carveout_of(reinterpret_cast<const void *>(kernel));
}

}  // namespace oasis
