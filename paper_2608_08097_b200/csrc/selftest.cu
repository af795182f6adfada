// Self-test of the bounded waits.  Every wait inside the tcgen05 / TMA kernels is a bounded spin on a
// shared-memory barrier; when the bound runs out the kernel records a code in the registered error word,
// releases the tensor memory it holds and returns.  That path never runs in a healthy launch, so this file
// offers a launch that takes it on purpose and harmlessly: one thread block initialises a barrier that
// nobody will ever arrive at, allocates a little tensor memory, waits with a caller-chosen small bound,
// sees the wait give up, frees the tensor memory and reports.  Nothing is left in flight and the context
// stays usable.
#include "common.cuh"
#include "tc_common.cuh"

namespace oasis {

constexpr int kSelftestCode = 99;

__global__ void __launch_bounds__(64)
wait_timeout_selftest_kernel(uint32_t probes, int32_t *err, int32_t *result)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&tmem_slot)), "r"(32u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    bool completed = true;
    if (threadIdx.x == 0) completed = mbar_wait_limit(smem_u32(&bar), 0, err, kSelftestCode, probes);
    // wind-down, as in the real kernels: everybody meets, the allocating warp frees the tensor memory
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_slot), "r"(32u) : "memory");
    if (threadIdx.x == 0 && result) {
        result[0] = completed ? 0 : 1;          // 1 = the wait gave up, as it should
        result[1] = kSelftestCode;
    }
}

}  // namespace oasis

extern "C" int oasis_selftest_wait_timeout(uint32_t probes, int32_t *result, void *stream)
{
    using namespace oasis;
    if (probes == 0 || probes > (1u << 20))
        return fail(OASIS_ERR_INVALID_ARG, "oasis_selftest_wait_timeout: probes %u outside [1, 2^20]", probes);
    wait_timeout_selftest_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(probes, error_word(), result);
    return check_launch("oasis_selftest_wait_timeout");
}
