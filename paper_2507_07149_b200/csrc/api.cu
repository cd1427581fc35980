// Host-side validation, size arithmetic and status plumbing of the C ABI.
#include <math.h>
#include <string.h>

#include "common.cuh"
#include "launch_cache.hpp"

namespace daf {

cudaError_t persistent_ctas(const void *kernel, int threads, int dyn_smem, int *ctas)
{
    static LaunchCache cache;
    int device = 0;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return e;
    const int err = cache.get(kernel, device, dyn_smem, ctas, [&](int *value) -> int {
        int sms = 0, per_sm = 0, optin = 0;
        cudaError_t q = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
        // the limit on dynamic shared memory is a property of the kernel on this device: raised to all the
        // device offers, so that later requests of any size find it high enough
        if (q == cudaSuccess && dyn_smem > 48 * 1024) {
            cudaFuncAttributes fa;
            q = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
            if (q == cudaSuccess) q = cudaFuncGetAttributes(&fa, kernel);
            if (q == cudaSuccess)   // static and dynamic shared memory share the device's limit
                q = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, optin - (int)fa.sharedSizeBytes);
        }
        if (q == cudaSuccess) q = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, (size_t)dyn_smem);
        if (q != cudaSuccess) return (int)q;
        *value = sms * (per_sm > 0 ? per_sm : 1);
        return 0;
    });
    return (cudaError_t)err;
}

static bool is_pow2(uint32_t v) { return v && !(v & (v - 1)); }

// Importance per stored bit of raising a group from width lo to width hi: with a uniform
// quantizer (Eq. 1 of the paper) the rounding-error variance of a group of range R is
// proportional to R^2 / (2^b - 1)^2; the sort key of a raise is R times the square root of
// the variance removed per added bit (Sec. 3.4.1: importance per memory footprint).
static float raise_factor(uint32_t lo, uint32_t hi)
{
    const double a = exp2((double)lo) - 1.0, b = exp2((double)hi) - 1.0;
    return (float)sqrt((1.0 / (a * a) - 1.0 / (b * b)) / (double)(hi - lo));
}

daf_status make_plan(const daf_params *p, Plan *pl)
{
    if (!p || p->struct_size != sizeof(daf_params) || (p->flags & 0xE0u) != 0) return DAF_ERR_INVALID_ARG;
    if (p->dtype > DAF_BF16 || p->rounding > DAF_ROUND_NEAREST) return DAF_ERR_INVALID_ARG;
    if ((p->flags & DAF_FLAG_STREAM_ALWAYS) && (p->flags & DAF_FLAG_STREAM_NEVER)) return DAF_ERR_INVALID_ARG;
    if ((p->flags & DAF_FLAG_ONE_PASS) && (p->flags & DAF_FLAG_TWO_PASS)) return DAF_ERR_INVALID_ARG;
    const uint32_t We = p->window_elems ? p->window_elems : 16384u;
    const uint32_t G = p->group_size;
    if (!is_pow2(G) || G < 32u) return DAF_ERR_INVALID_ARG;
    if (!is_pow2(We) || G > We) return DAF_ERR_INVALID_ARG;
    if (We != 4096u && We != 8192u && We != 16384u) return DAF_ERR_UNSUPPORTED;
    if (p->width_mask == 0 || (p->width_mask & ~0x116u)) return DAF_ERR_INVALID_ARG;
    if (p->elem_index_base & 7u) return DAF_ERR_INVALID_ARG;
    if (p->numel == 0 || p->numel % G) return DAF_ERR_SHAPE;
    if (!(p->bit_budget >= 0.0f) || p->bit_budget > 64.0f) return DAF_ERR_BUDGET;

    memset(pl, 0, sizeof(*pl));
    pl->G = G;
    pl->We = We;
    pl->chunks = We / (kThreads * kLaneElems);
    pl->W = We / G;
    for (uint32_t t = G; t > 1; t >>= 1) pl->log2G++;
    for (uint32_t b = 1; b <= 8; b <<= 1)
        if (p->width_mask & (1u << b)) pl->S[pl->m++] = b;
    for (uint32_t k = 0; k + 1 < pl->m; k++) {
        pl->cost[k] = pl->S[k + 1] - pl->S[k];
        pl->v[k] = raise_factor(pl->S[k], pl->S[k + 1]);
    }
    pl->beta_q8 = (uint32_t)floorf(p->bit_budget * 256.0f);
    if (pl->beta_q8 < 256u * pl->S[0]) return DAF_ERR_BUDGET;
    // a budget above the largest width buys nothing: every group reaches that width either way, and the packed
    // capacity and the kernels' buffers are sized from the budget
    if (pl->beta_q8 > 256u * pl->S[pl->m - 1]) pl->beta_q8 = 256u * pl->S[pl->m - 1];

    pl->n_groups = p->numel / G;
    pl->n_windows = (pl->n_groups + pl->W - 1) / pl->W;
    const uint64_t full = pl->n_groups / pl->W, last = pl->n_groups % pl->W;
    pl->capacity = full * ((((uint64_t)pl->beta_q8 * pl->W) >> 8) * G / 8) + (((uint64_t)pl->beta_q8 * last) >> 8) * G / 8;
    pl->workspace = sizeof(WorkspaceHeader) + 16ull * pl->n_windows;
    return DAF_OK;
}

}  // namespace daf

using namespace daf;

extern "C" daf_status daf_sizes(const daf_params *params, uint64_t *n_groups, uint64_t *n_windows,
                                uint64_t *packed_capacity_bytes, uint64_t *workspace_bytes)
{
    Plan pl;
    daf_status st = make_plan(params, &pl);
    if (st != DAF_OK) return st;
    if (n_groups) *n_groups = pl.n_groups;
    if (n_windows) *n_windows = pl.n_windows;
    if (packed_capacity_bytes) *packed_capacity_bytes = pl.capacity;
    if (workspace_bytes) *workspace_bytes = pl.workspace;
    return DAF_OK;
}

// The window-aligned slice of a tensor that rank `rank` of `world` takes: whole windows, as even as possible, in order.
extern "C" daf_status daf_shard(const daf_params *whole, uint32_t rank, uint32_t world, daf_params *shard, uint64_t *first_elem)
{
    Plan pl;
    const daf_status st = make_plan(whole, &pl);
    if (st != DAF_OK) return st;
    if (!shard || world == 0 || rank >= world) return DAF_ERR_INVALID_ARG;
    const uint64_t per = pl.n_windows / world, extra = pl.n_windows % world;
    const uint64_t w_lo = (uint64_t)rank * per + (rank < extra ? rank : extra), w_hi = w_lo + per + (rank < extra ? 1u : 0u);
    uint64_t lo = w_lo * pl.We, hi = w_hi * pl.We;
    if (lo > whole->numel) lo = whole->numel;
    if (hi > whole->numel) hi = whole->numel;
    *shard = *whole;
    shard->numel = hi - lo;                                       // 0: more ranks than windows, nothing for this one
    shard->elem_index_base = whole->elem_index_base + lo;
    if (first_elem) *first_elem = lo;
    return DAF_OK;
}

extern "C" daf_status daf_poll_status(const void *d_workspace, daf_stream stream)
{
    if (!d_workspace) return DAF_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    unsigned int status = 0;
    if (cudaMemcpyAsync(&status, d_workspace, sizeof(status), cudaMemcpyDeviceToHost, s) != cudaSuccess) return DAF_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return DAF_ERR_CUDA;
    return status <= DAF_ERR_UNSUPPORTED ? (daf_status)status : DAF_ERR_CUDA;
}

extern "C" const char *daf_status_string(daf_status status)
{
    switch (status) {
    case DAF_OK: return "ok";
    case DAF_ERR_INVALID_ARG: return "invalid argument";
    case DAF_ERR_SHAPE: return "numel is zero or not a multiple of the group size";
    case DAF_ERR_BUDGET: return "bit budget below the smallest allowed width";
    case DAF_ERR_CAPACITY: return "packed buffer or workspace too small";
    case DAF_ERR_CUDA: return "CUDA runtime error";
    case DAF_ERR_TIMEOUT: return "bounded device-side wait ran out";
    case DAF_ERR_UNSUPPORTED: return "not supported by this build";
    }
    return "unknown status";
}

extern "C" uint32_t daf_version(void) { return 0x000100u; }
