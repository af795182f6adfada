// Host-side plumbing shared by every entry point: last-error string, argument checks.
#include <cstdarg>
#include <cstdio>

#include "common.cuh"

namespace oasis {

static thread_local char g_last_error[512] = "";

int fail(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_last_error, sizeof g_last_error, fmt, ap);
    va_end(ap);
    return code;
}

int check_dims(const oasis_dims_t *d)
{
    if (!d) return fail(OASIS_ERR_INVALID_ARG, "dims is NULL");
    if (d->head_dim != kHeadDim)
        return fail(OASIS_ERR_UNSUPPORTED, "head_dim %d: only 128 is supported", d->head_dim);
    if (d->block_size != kBlock)
        return fail(OASIS_ERR_UNSUPPORTED, "block_size %d: only 16 is supported", d->block_size);
    if (d->batch < 0 || d->n_q_heads <= 0 || d->n_kv_heads <= 0 || d->max_blocks <= 0)
        return fail(OASIS_ERR_INVALID_ARG, "dims: batch %d, heads %d/%d, max_blocks %d", d->batch,
                    d->n_q_heads, d->n_kv_heads, d->max_blocks);
    if (d->n_q_heads % d->n_kv_heads != 0)
        return fail(OASIS_ERR_INVALID_ARG, "n_q_heads %d is not a multiple of n_kv_heads %d",
                    d->n_q_heads, d->n_kv_heads);
    if ((int64_t)d->batch * d->n_kv_heads > 0x7fffffffLL / 4)
        return fail(OASIS_ERR_UNSUPPORTED, "batch * n_kv_heads too large");
    return OASIS_OK;
}

int check_launch(const char *what)
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess)
        return fail(OASIS_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
    return OASIS_OK;
}

int sm_count()
{
    static thread_local int cached_dev = -1, cached = 148;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return 148;
    }
    if (dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
            cached = n;
        else
            cudaGetLastError();
        cached_dev = dev;
    }
    return cached;
}

static int32_t *g_error_word = nullptr;
int32_t *error_word() { return g_error_word; }

static long long g_n_entries = 1ll << 62, g_n_slots = 1ll << 31;
Bounds bounds() { return Bounds{g_n_entries, g_n_slots, g_error_word}; }

}  // namespace oasis

extern "C" int oasis_set_error_word(int32_t *device_word)
{
    oasis::g_error_word = device_word;
    return OASIS_OK;
}

extern "C" int oasis_set_extents(int64_t n_host_entries, int64_t n_slots)
{
    using namespace oasis;
    if (n_host_entries < 0 || n_slots < 0 || n_slots > (1ll << 31))
        return fail(OASIS_ERR_INVALID_ARG, "oasis_set_extents: n_host_entries %lld, n_slots %lld", (long long)n_host_entries,
                    (long long)n_slots);
    g_n_entries = n_host_entries > 0 ? n_host_entries : 1ll << 62;
    g_n_slots = n_slots > 0 ? n_slots : 1ll << 31;
    return OASIS_OK;
}

extern "C" int oasis_bounds_checked(void) { return oasis::kBoundsCheck ? 1 : 0; }

extern "C" const char *oasis_last_error(void) { return oasis::g_last_error; }
extern "C" const char *oasis_version(void) { return "0.1"; }
