// Device-wide exclusive prefix sum of the group byte lengths G*b/8 (the "layout
// concatenation" of Sec. 3.3 of the paper needs every group's position in the packed buffer).
// Single pass: each CTA scans a tile of 8192 groups and obtains the sum of all earlier tiles
// through the same bounded decoupled look-back the compress kernel uses.
#include "common.cuh"

namespace daf {

constexpr int kScanItems = 16;                                    // groups per thread
constexpr int kScanTile = kThreads * kScanItems;                  // groups per CTA

struct ScanArgs {
    const uint8_t *bits;
    uint64_t *offsets;
    uint64_t n_groups;
    uint32_t n_tiles, bytes_per_bit;                              // bytes_per_bit = G / 8
    uint32_t poll_limit;                                          // polls after which the bounded look-back wait gives up
    WorkspaceHeader *hdr;
    uint64_t *flags;
};

__global__ void __launch_bounds__(kThreads) group_offsets_kernel(const __grid_constant__ ScanArgs a)
{
    __shared__ uint32_t s_wtot[kWarps];
    __shared__ uint32_t s_ticket;
    __shared__ uint64_t s_excl;
    __shared__ int s_failed;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(a.bits) & 15u) == 0;

    for (;;) {
        if (tid == 0) s_ticket = atomicAdd(&a.hdr->ticket, 1u);
        __syncthreads();
        const uint32_t tile = s_ticket;
        if (tile >= a.n_tiles) return;
        const uint64_t base = (uint64_t)tile * kScanTile + (uint64_t)tid * kScanItems;

        uint32_t b[kScanItems];
        if (vec_ok && base + kScanItems <= a.n_groups) {
            const uint4 v = *reinterpret_cast<const uint4 *>(a.bits + base);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int i = 0; i < kScanItems; i++) b[i] = (w[i >> 2] >> (8 * (i & 3))) & 0xFFu;
        } else {
#pragma unroll
            for (int i = 0; i < kScanItems; i++) b[i] = base + i < a.n_groups ? a.bits[base + i] : 0u;
        }
        uint32_t sum = 0;
#pragma unroll
        for (int i = 0; i < kScanItems; i++) sum += b[i];
        sum *= a.bytes_per_bit;

        uint32_t incl = sum;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += y;
        }
        if (lane == 31) s_wtot[warp] = incl;
        __syncthreads();
        uint32_t before = 0, total = 0;
#pragma unroll
        for (int i = 0; i < kWarps; i++) {
            const uint32_t t = s_wtot[i];
            if (i < warp) before += t;
            total += t;
        }
        if (warp == 0) {
            // decoupled look-back over the tile descriptors (state in the top two bits)
            uint64_t excl = 0;
            int bad = 0;                                          // 1: a tile before this one failed; 2: this tile's wait ran out
            if (tile == 0) {
                if (lane == 0) st_relaxed_u64(a.flags, (kFlagPrefix << kFlagShift) | total);
            } else {
                if (lane == 0) st_relaxed_u64(a.flags + tile, (kFlagAggregate << kFlagShift) | total);
                int64_t idx = (int64_t)tile - 1 - lane;
                for (;;) {
                    uint64_t f = 0;
                    unsigned polls = 0, stop_mask, upto;
                    for (;;) {
                        f = idx >= 0 ? ld_relaxed_u64(a.flags + idx) : (kFlagPrefix << kFlagShift);
                        const uint32_t st = (uint32_t)(f >> kFlagShift);
                        stop_mask = __ballot_sync(0xFFFFFFFFu, st == kFlagPrefix || st == kFlagPoison);
                        const unsigned empty_mask = __ballot_sync(0xFFFFFFFFu, st == kFlagEmpty);
                        upto = stop_mask ? ((2u << (__ffs(stop_mask) - 1)) - 1u) : 0xFFFFFFFFu;
                        if ((empty_mask & upto) == 0u) break;
                        if (++polls > a.poll_limit) { bad = 2; break; }
                        __nanosleep(64);
                    }
                    if (bad) break;
                    if (__ballot_sync(0xFFFFFFFFu, (uint32_t)(f >> kFlagShift) == kFlagPoison) & upto) { bad = 1; break; }
                    uint64_t v = ((upto >> lane) & 1u) ? (f & kFlagValueMask) : 0ull;
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
                    excl += v;
                    if (stop_mask) break;
                    idx -= 32;
                }
                if (lane == 0) {
                    // the tile whose wait ran out reports it BEFORE it poisons its descriptor; tiles that only meet the
                    // poison stop without a report of their own
                    if (bad == 2 && atomicCAS(&a.hdr->status, 0u, (unsigned)DAF_ERR_TIMEOUT) == 0u) a.hdr->fail_window = tile;
                    __threadfence();
                    st_relaxed_u64(a.flags + tile,
                                   bad ? (kFlagPoison << kFlagShift) : ((kFlagPrefix << kFlagShift) | (excl + total)));
                }
            }
            if (lane == 0) {
                s_excl = excl;
                s_failed = bad;
            }
        }
        __syncthreads();
        if (!s_failed) {
            uint64_t run = s_excl + before + incl - sum;
#pragma unroll
            for (int i = 0; i < kScanItems; i++) {
                if (base + i < a.n_groups) a.offsets[base + i] = run;
                run += (uint64_t)b[i] * a.bytes_per_bit;
                if (base + i + 1 == a.n_groups) a.offsets[a.n_groups] = run;
            }
        }
    }
}

}  // namespace daf

using namespace daf;

extern "C" uint64_t daf_group_offsets_workspace(uint64_t n_groups)
{
    const uint64_t tiles = (n_groups + kScanTile - 1) / kScanTile;
    return sizeof(WorkspaceHeader) + 8ull * (tiles ? tiles : 1);
}

static daf_status group_offsets_impl(const uint8_t *d_bits, uint64_t n_groups, uint32_t group_size, uint64_t *d_offsets,
                                     void *d_ws, uint64_t ws_bytes, uint32_t flags, daf_stream stream)
{
    if (!d_bits || !d_offsets || !d_ws || (reinterpret_cast<uintptr_t>(d_offsets) & 7u) || (reinterpret_cast<uintptr_t>(d_ws) & 15u))
        return DAF_ERR_INVALID_ARG;
    // (the upper bound also keeps a tile's 32-bit byte count in range)
    if (group_size < 32u || group_size > 16384u || (group_size & (group_size - 1u))) return DAF_ERR_INVALID_ARG;
    if (flags & 0xFBu) return DAF_ERR_INVALID_ARG;                // only DAF_FLAG_KEEP_WORKSPACE and DAF_FLAG_POLL_LIMIT mean something here
    if (n_groups == 0) return DAF_ERR_SHAPE;
    const uint64_t tiles = (n_groups + kScanTile - 1) / kScanTile;
    if (tiles > 0x7FFFFFFFull) return DAF_ERR_UNSUPPORTED;
    const uint64_t need = daf_group_offsets_workspace(n_groups);
    if (ws_bytes < need) return DAF_ERR_CAPACITY;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (!(flags & DAF_FLAG_KEEP_WORKSPACE) && cudaMemsetAsync(d_ws, 0, need, s) != cudaSuccess) return DAF_ERR_CUDA;
    int max_ctas = 0;
    if (persistent_ctas(reinterpret_cast<const void *>(&group_offsets_kernel), kThreads, 0, &max_ctas) != cudaSuccess) return DAF_ERR_CUDA;
    ScanArgs a;
    a.bits = d_bits;
    a.offsets = d_offsets;
    a.n_groups = n_groups;
    a.n_tiles = (uint32_t)tiles;
    a.bytes_per_bit = group_size / 8u;
    a.poll_limit = (flags >> 8) ? (flags >> 8) : kMaxPolls;
    a.hdr = reinterpret_cast<WorkspaceHeader *>(d_ws);
    a.flags = reinterpret_cast<uint64_t *>(reinterpret_cast<char *>(d_ws) + sizeof(WorkspaceHeader));
    const uint32_t grid = a.n_tiles < (uint32_t)max_ctas ? a.n_tiles : (uint32_t)max_ctas;
    group_offsets_kernel<<<grid, kThreads, 0, s>>>(a);
    return cudaGetLastError() == cudaSuccess ? DAF_OK : DAF_ERR_CUDA;
}

extern "C" daf_status daf_group_offsets(const uint8_t *d_bits, uint64_t n_groups, uint32_t group_size,
                                        uint64_t *d_offsets, void *d_ws, uint64_t ws_bytes, daf_stream stream)
{
    return group_offsets_impl(d_bits, n_groups, group_size, d_offsets, d_ws, ws_bytes, 0u, stream);
}

extern "C" daf_status daf_group_offsets_diag(const uint8_t *d_bits, uint64_t n_groups, uint32_t group_size,
                                             uint64_t *d_offsets, void *d_ws, uint64_t ws_bytes, uint32_t flags,
                                             daf_stream stream)
{
    return group_offsets_impl(d_bits, n_groups, group_size, d_offsets, d_ws, ws_bytes, flags, stream);
}
