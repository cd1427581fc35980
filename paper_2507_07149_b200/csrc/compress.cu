// Fused compress kernel: one persistent CTA processes one window (window_elems elements) at a
// time and reads the input from HBM exactly once.
//
//   load window into registers (8 consecutive elements per lane and chunk, 256-bit loads)
//   -> per-group min / max (lane-local 3-input min/max, warp redux or segmented shuffles)
//   -> per-window greedy bit-width choice (Sec. 3.4.1 of the paper: importance per bit)
//   -> intra-window exclusive scan of the group byte lengths, device-wide window offset by a
//      bounded decoupled look-back over 64-bit descriptors
//   -> Eq. 1 quantization with stochastic rounding (Philox4x32-10, 16 bits per element, float
//      -> uint through the power-of-two offset of Eq. 5) and lane-local LSB-first packing
//   -> stores of the packed bytes and of bits / min / scale.
//
// Windows are handed out by an atomic ticket, so every window with a smaller index than the
// one a CTA holds is already owned by a running (or finished) CTA and the look-back always
// makes progress; it is bounded all the same.
#include "common.cuh"

namespace daf {

struct TensorDesc {
    const void *in;
    uint8_t *packed;
    uint64_t capacity;
    uint8_t *bits;
    float *mn;
    float *scale;
    uint64_t *woff;
    uint64_t numel;
    uint64_t elem_base;
    uint64_t seed;
    uint32_t first_window;   // index of this tensor's window 0 among all windows of the launch
    uint32_t n_windows;
};

template <int NT> struct CompressArgs {
    WorkspaceHeader *hdr;
    uint64_t *flags;
    uint32_t total_windows, n_tensors;
    uint32_t G, log2G, beta_q8, m, nearest;
    uint32_t S[kMaxLevels], cost[kMaxLevels];
    float v[kMaxLevels];
    PhiloxKeys keys;          // round keys of tensor 0 (single-tensor launches)
    TensorDesc t[NT];
};

struct GroupRec {             // what the quantize pass needs per group (one 16-byte shared load)
    float mn, inv;
    uint32_t b, off;
};

// ------------------------------------------------------------------------------------------
// Eight codes of width B from eight values; o[] holds eight 16-bit random lanes (two per word).
// s = fma(x - mn, inv, 256) lies in [256, 512) where one ulp is 2^-15, so its mantissa field
// is the fixed-point quotient; adding a 15-bit random offset and dropping 15 bits rounds
// stochastically (offset 2^14 = round half up).
// ------------------------------------------------------------------------------------------
template <int B>
__device__ __forceinline__ void quantize8(const float (&x)[8], float mn, float inv, const uint32_t (&o)[4],
                                          uint32_t &w0, uint32_t &w1)
{
    constexpr uint32_t L = (1u << B) - 1u;
    w0 = 0u;
    w1 = 0u;
#pragma unroll
    for (int i = 0; i < 8; i++) {
        float d = __fsub_rn(x[i], mn);
        float s = __fmaf_rn(d, inv, 256.0f);
        uint32_t r15 = (i & 1) ? (o[i >> 1] >> 17) : ((o[i >> 1] >> 1) & 0x7FFFu);
        uint32_t t = __float_as_uint(s) - 0x43800000u + r15;
        uint32_t q = min(t >> 15, L);
        if (B == 8) {
            if (i < 4) w0 |= q << (8 * i);
            else w1 |= q << (8 * (i - 4));
        } else {
            w0 |= q << (B * i);
        }
    }
}

// ------------------------------------------------------------------------------------------
// Decoupled look-back over the window descriptors, executed by one full warp.  Returns the
// exclusive prefix (bytes before this window); *failed is set when a predecessor is poisoned
// or the bounded wait runs out.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t lookback(uint64_t *flags, uint32_t gw, uint32_t first, uint64_t total,
                                             int lane, int *failed, int *timed_out)
{
    uint64_t excl = 0;
    int bad = 0, tmo = 0;
    if (gw == first) {
        if (lane == 0) st_relaxed_u64(flags + gw, (kFlagPrefix << kFlagShift) | total);
        *failed = 0;
        *timed_out = 0;
        return 0;
    }
    if (lane == 0) st_relaxed_u64(flags + gw, (kFlagAggregate << kFlagShift) | total);
    int64_t idx = (int64_t)gw - 1 - lane;
    for (;;) {
        uint64_t f = 0;
        unsigned polls = 0;
        unsigned ready_mask, stop_mask;
        for (;;) {
            f = (idx >= (int64_t)first) ? ld_relaxed_u64(flags + idx) : (kFlagPrefix << kFlagShift);
            uint32_t st = (uint32_t)(f >> kFlagShift);
            stop_mask = __ballot_sync(0xFFFFFFFFu, st == kFlagPrefix || st == kFlagPoison);
            unsigned empty_mask = __ballot_sync(0xFFFFFFFFu, st == kFlagEmpty);
            // only descriptors up to and including the first prefix / poison matter
            unsigned upto = stop_mask ? ((2u << (__ffs(stop_mask) - 1)) - 1u) : 0xFFFFFFFFu;
            ready_mask = upto;
            if ((empty_mask & upto) == 0u) break;
            if (++polls > kMaxPolls) { tmo = 1; break; }
            __nanosleep(64);
        }
        if (tmo) { bad = 1; break; }
        uint32_t st = (uint32_t)(f >> kFlagShift);
        if (__ballot_sync(0xFFFFFFFFu, st == kFlagPoison) & ready_mask) { bad = 1; break; }
        uint64_t v = ((ready_mask >> lane) & 1u) ? (f & kFlagValueMask) : 0ull;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
        excl += v;
        if (stop_mask) break;
        idx -= 32;
    }
    if (lane == 0)
        st_relaxed_u64(flags + gw, bad ? (kFlagPoison << kFlagShift) : ((kFlagPrefix << kFlagShift) | (excl + total)));
    *failed = bad;
    *timed_out = tmo;
    return excl;
}

template <typename T, int CHUNKS, bool BATCH>
__global__ void __launch_bounds__(kThreads, 2)
compress_kernel(const __grid_constant__ CompressArgs<BATCH ? DAF_BATCH_MAX : 1> a)
{
    constexpr uint32_t WE = kThreads * kLaneElems * CHUNKS;

    __shared__ float s_umn[kMaxGroups], s_umx[kMaxGroups];      // per unit (min(G,256) elements)
    __shared__ float s_R[kMaxGroups], s_mn[kMaxGroups];
    __shared__ uint32_t s_key[kMaxLevels - 1][kMaxGroups];
    __shared__ uint32_t s_cum[kMaxLevels - 1][kMaxGroups];
    __shared__ __align__(16) GroupRec s_grp[kMaxGroups];
    __shared__ uint32_t s_wmin[kWarps], s_wmax[kWarps], s_wtot[kWarps];
    __shared__ uint32_t s_ticket;
    __shared__ uint64_t s_woff;
    __shared__ int s_skip;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t G = a.G, log2G = a.log2G, m = a.m;
    const uint32_t U = G < 256u ? G : 256u;                      // unit: elements reduced inside one warp pass
    const uint32_t log2U = G < 256u ? log2G : 8u;
    const uint32_t lpu = U >> 3;                                  // lanes per unit

    for (;;) {
        if (tid == 0) s_ticket = atomicAdd(&a.hdr->ticket, 1u);
        __syncthreads();
        const uint32_t gw = s_ticket;
        if (gw >= a.total_windows) return;

        uint32_t ti = 0;
        if (BATCH) {                                              // last tensor whose first window is <= gw
            uint32_t lo = 0, hi = a.n_tensors - 1;
            while (lo < hi) {
                uint32_t mid = (lo + hi + 1) >> 1;
                if (a.t[mid].first_window <= gw) lo = mid; else hi = mid - 1;
            }
            ti = lo;
        }
        const TensorDesc &td = a.t[ti];
        const uint32_t w = gw - td.first_window;
        const uint64_t wbase = (uint64_t)w * WE;
        const uint64_t left = td.numel - wbase;
        const uint32_t n_elems = left < WE ? (uint32_t)left : WE;
        const uint32_t n = n_elems >> log2G;                      // groups in this window
        const uint64_t g0 = wbase >> log2G;                       // first group of the window in the tensor

        // ---------------------------------------------------------------- load + unit min/max
        float x[CHUNKS][8];
        uint32_t e[CHUNKS];
#pragma unroll
        for (int c = 0; c < CHUNKS; c++) {
            e[c] = (uint32_t)((warp * CHUNKS + c) * 256 + lane * 8);
            if (e[c] < n_elems) {
                Elem<T>::load8(reinterpret_cast<const char *>(td.in) + (wbase + e[c]) * Elem<T>::kBytes, x[c]);
            } else {
#pragma unroll
                for (int i = 0; i < 8; i++) x[c][i] = 0.0f;
            }
        }
#pragma unroll
        for (int c = 0; c < CHUNKS; c++) {
            float lo = fmin3(fmin3(x[c][0], x[c][1], x[c][2]), fmin3(x[c][3], x[c][4], x[c][5]), fmin2(x[c][6], x[c][7]));
            float hi = fmax3(fmax3(x[c][0], x[c][1], x[c][2]), fmax3(x[c][3], x[c][4], x[c][5]), fmax2(x[c][6], x[c][7]));
            for (uint32_t off = 1; off < lpu; off <<= 1) {
                lo = fmin2(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, off));
                hi = fmax2(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, off));
            }
            if ((lane & (lpu - 1u)) == 0u && e[c] < n_elems) {
                s_umn[e[c] >> log2U] = lo;
                s_umx[e[c] >> log2U] = hi;
            }
        }
        __syncthreads();

        // ---------------------------------------------------------------- group range and keys
        const uint64_t T = ((uint64_t)a.beta_q8 * n) >> 8;        // bit units of the window
        const uint32_t rem = (uint32_t)(T - (uint64_t)a.S[0] * n);
        // largest level every group can be raised to within the budget
        uint32_t ell = 0;
        while (ell + 1 < m && (a.S[ell + 1] - a.S[0]) * n <= rem) ell++;
        const uint32_t rem_after = rem - (a.S[ell] - a.S[0]) * n;

        float mn = 0.0f, R = 0.0f;
        uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
        if ((uint32_t)tid < n) {
            float mx;
            if (G > 256u) {
                const uint32_t r = G >> 8;
                mn = s_umn[tid * r];
                mx = s_umx[tid * r];
                for (uint32_t j = 1; j < r; j++) {
                    mn = fmin2(mn, s_umn[tid * r + j]);
                    mx = fmax2(mx, s_umx[tid * r + j]);
                }
            } else {
                mn = s_umn[tid];
                mx = s_umx[tid];
            }
            R = __fsub_rn(mx, mn);
            if (R < 0x1p-118f) R = 0.0f;                          // degenerate group: constant
            s_mn[tid] = mn;
            s_R[tid] = R;
            for (uint32_t k = 0; k + 1 < m; k++) {
                uint32_t key = __float_as_uint(__fmul_rn(R, a.v[k]));
                s_key[k][tid] = key;
                s_cum[k][tid] = 0u;
                if (k + 1 == ell) kmin = key;
                if (k == ell) kmax = key;
            }
        }
        kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
        kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
        if (lane == 0) {
            s_wmin[warp] = kmin;
            s_wmax[warp] = kmax;
        }
        __syncthreads();
        kmin = 0xFFFFFFFFu;
        kmax = 0u;
#pragma unroll
        for (int i = 0; i < kWarps; i++) {
            kmin = min(kmin, s_wmin[i]);
            kmax = max(kmax, s_wmax[i]);
        }

        // ---------------------------------------------------------------- bit choice
        // Uniform outcome: every raise below level ell sorts ahead of every raise from level
        // ell upward, they all fit, and the best raise of level ell does not.
        uint32_t level = ell;
        const bool uniform = (ell + 1 == m) || (rem_after < a.cost[ell] && (ell == 0 || kmin >= kmax));
        if (!uniform) {
            // General case.  For each candidate (group g, raise k) add up the cost of all
            // candidates that sort at or ahead of it (key descending, level ascending, group
            // ascending); the candidate is accepted iff that total fits in the budget.
            const uint32_t nl = m - 1;
            const uint32_t items = n * nl * nl;
            for (uint32_t it = tid; it < items; it += kThreads) {
                const uint32_t g = it % n, kk = it / n;
                const uint32_t k = kk / nl, k2 = kk % nl;
                const uint32_t key = s_key[k][g];
                uint32_t cnt = 0;
                if (k2 < k) {
                    for (uint32_t h = 0; h < n; h++) cnt += (s_key[k2][h] >= key);
                } else if (k2 > k) {
                    for (uint32_t h = 0; h < n; h++) cnt += (s_key[k2][h] > key);
                } else {
                    for (uint32_t h = 0; h < n; h++) {
                        const uint32_t kh = s_key[k][h];
                        cnt += (kh > key) || (kh == key && h <= g);
                    }
                }
                atomicAdd(&s_cum[k][g], cnt * a.cost[k2]);
            }
            __syncthreads();
            level = 0;
            if ((uint32_t)tid < n)
                for (uint32_t k = 0; k + 1 < m; k++) level += (s_cum[k][tid] <= rem);
        }

        // ---------------------------------------------------------------- group parameters, sizes, scan
        uint32_t size = 0, b = 0;
        float inv = 0.0f;
        if ((uint32_t)tid < n) {
            b = a.S[level];
            const float Lf = (float)((1u << b) - 1u);
            const float scale = R > 0.0f ? __fdiv_rn(R, Lf) : 0.0f;
            inv = R > 0.0f ? __fdiv_rn(Lf, R) : 0.0f;
            td.bits[g0 + tid] = (uint8_t)b;
            td.mn[g0 + tid] = mn;
            td.scale[g0 + tid] = scale;
            size = (G >> 3) * b;
        }
        uint32_t incl = size;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += y;
        }
        if (lane == 31) s_wtot[warp] = incl;
        __syncthreads();
        uint32_t wbase_bytes = 0, total = 0;
#pragma unroll
        for (int i = 0; i < kWarps; i++) {
            const uint32_t t = s_wtot[i];
            if (i < warp) wbase_bytes += t;
            total += t;
        }
        if ((uint32_t)tid < n) {
            GroupRec rec;
            rec.mn = mn;
            rec.inv = inv;
            rec.b = b;
            rec.off = wbase_bytes + incl - size;
            s_grp[tid] = rec;
        }
        __syncthreads();

        // ---------------------------------------------------------------- window offset (warp 0)
        if (warp == 0) {
            int failed = 0, timed_out = 0;
            const uint64_t excl = lookback(a.flags, gw, td.first_window, total, lane, &failed, &timed_out);
            if (lane == 0) {
                int skip = failed;
                if (!failed) {
                    td.woff[w] = excl;
                    if (w + 1 == td.n_windows) td.woff[w + 1] = excl + total;
                    if (excl + total > td.capacity) skip = 1;
                }
                if (skip) {
                    const unsigned code = timed_out ? DAF_ERR_TIMEOUT : DAF_ERR_CAPACITY;
                    if (atomicCAS(&a.hdr->status, 0u, code) == 0u) a.hdr->fail_window = gw;
                }
                s_woff = excl;
                s_skip = skip;
            }
        }

        // ---------------------------------------------------------------- quantize + pack (registers)
        uint32_t pk0[CHUNKS], pk1[CHUNKS], pb[CHUNKS], poff[CHUNKS];
#pragma unroll
        for (int c = 0; c < CHUNKS; c++) {
            pk0[c] = pk1[c] = pb[c] = poff[c] = 0u;
            if (e[c] < n_elems) {
                const GroupRec rec = s_grp[e[c] >> log2G];
                uint32_t o[4];
                if (a.nearest) {
                    o[0] = o[1] = o[2] = o[3] = 0x80008000u;       // every 15-bit lane = 2^14
                } else {
                    const uint64_t blk = (td.elem_base + wbase + e[c]) >> 3;
                    if (BATCH) {
                        PhiloxSeedKeys sk{(uint32_t)td.seed, (uint32_t)(td.seed >> 32)};
                        philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), sk, o);
                    } else {
                        philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), a.keys, o);
                    }
                }
                switch (rec.b) {
                case 1: quantize8<1>(x[c], rec.mn, rec.inv, o, pk0[c], pk1[c]); break;
                case 2: quantize8<2>(x[c], rec.mn, rec.inv, o, pk0[c], pk1[c]); break;
                case 4: quantize8<4>(x[c], rec.mn, rec.inv, o, pk0[c], pk1[c]); break;
                default: quantize8<8>(x[c], rec.mn, rec.inv, o, pk0[c], pk1[c]); break;
                }
                pb[c] = rec.b;
                poff[c] = rec.off + ((e[c] & (G - 1u)) >> 3) * rec.b;
            }
        }
        __syncthreads();

        // ---------------------------------------------------------------- store
        if (!s_skip) {
            uint8_t *dst = td.packed + s_woff;
#pragma unroll
            for (int c = 0; c < CHUNKS; c++) {
                if (e[c] < n_elems) {
                    uint8_t *p = dst + poff[c];
                    switch (pb[c]) {
                    case 1: *p = (uint8_t)pk0[c]; break;
                    case 2: *reinterpret_cast<uint16_t *>(p) = (uint16_t)pk0[c]; break;
                    case 4: *reinterpret_cast<uint32_t *>(p) = pk0[c]; break;
                    default:
                        if (G >= 64u) {
                            *reinterpret_cast<uint2 *>(p) = make_uint2(pk0[c], pk1[c]);
                        } else {                                   // G = 32: groups are only 4-byte aligned
                            reinterpret_cast<uint32_t *>(p)[0] = pk0[c];
                            reinterpret_cast<uint32_t *>(p)[1] = pk1[c];
                        }
                        break;
                    }
                }
            }
        }
        // the next iteration's first barrier orders these reads of shared memory before any rewrite
    }
}

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
template <typename T, int CHUNKS, bool BATCH>
static cudaError_t launch(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    static int max_ctas = 0;                                      // resident CTAs on the current device
    if (max_ctas == 0) {
        int dev = 0, sms = 0, per_sm = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess)
            e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, compress_kernel<T, CHUNKS, BATCH>, kThreads, 0);
        if (e != cudaSuccess) return e;
        max_ctas = sms * (per_sm > 0 ? per_sm : 1);
    }
    const uint32_t grid = args.total_windows < (uint32_t)max_ctas ? args.total_windows : (uint32_t)max_ctas;
    compress_kernel<T, CHUNKS, BATCH><<<grid, kThreads, 0, stream>>>(args);
    return cudaGetLastError();
}

template <bool BATCH>
static cudaError_t dispatch(uint32_t dtype, uint32_t chunks, const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args,
                            cudaStream_t stream)
{
#define DAF_CASE(T)                                                     \
    switch (chunks) {                                                   \
    case 1: return launch<T, 1, BATCH>(args, stream);                   \
    case 2: return launch<T, 2, BATCH>(args, stream);                   \
    default: return launch<T, 4, BATCH>(args, stream);                  \
    }
    if (dtype == DAF_F32) { DAF_CASE(float) }
    if (dtype == DAF_F16) { DAF_CASE(__half) }
    DAF_CASE(__nv_bfloat16)
#undef DAF_CASE
}

template <int NT> static void fill_common(CompressArgs<NT> &a, const Plan &pl, const daf_params *p, void *ws)
{
    a.hdr = reinterpret_cast<WorkspaceHeader *>(ws);
    a.flags = reinterpret_cast<uint64_t *>(reinterpret_cast<char *>(ws) + sizeof(WorkspaceHeader));
    a.G = pl.G;
    a.log2G = pl.log2G;
    a.beta_q8 = pl.beta_q8;
    a.m = pl.m;
    a.nearest = p->rounding == DAF_ROUND_NEAREST;
    for (int k = 0; k < kMaxLevels; k++) {
        a.S[k] = pl.S[k];
        a.cost[k] = pl.cost[k];
        a.v[k] = pl.v[k];
    }
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace daf

using namespace daf;

extern "C" daf_status daf_compress(const daf_params *params, const void *d_in, void *d_packed,
                                   uint64_t packed_capacity, uint8_t *d_bits, float *d_min, float *d_scale,
                                   uint64_t *d_window_offsets, void *d_workspace, uint64_t workspace_bytes,
                                   daf_stream stream)
{
    Plan pl;
    daf_status st = make_plan(params, &pl);
    if (st != DAF_OK) return st;
    if (!d_in || !d_packed || !d_bits || !d_min || !d_scale || !d_window_offsets || !d_workspace) return DAF_ERR_INVALID_ARG;
    if (!aligned16(d_in) || !aligned16(d_packed) || !aligned16(d_workspace) || (reinterpret_cast<uintptr_t>(d_min) & 3u) ||
        (reinterpret_cast<uintptr_t>(d_scale) & 3u) || (reinterpret_cast<uintptr_t>(d_window_offsets) & 7u))
        return DAF_ERR_INVALID_ARG;
    if (workspace_bytes < pl.workspace) return DAF_ERR_CAPACITY;
    if (pl.n_windows > 0xFFFFFFF0ull) return DAF_ERR_UNSUPPORTED;

    CompressArgs<1> a;
    fill_common(a, pl, params, d_workspace);
    a.total_windows = (uint32_t)pl.n_windows;
    a.n_tensors = 1;
    a.keys = philox_keys(params->seed);
    a.t[0] = TensorDesc{d_in, reinterpret_cast<uint8_t *>(d_packed), packed_capacity, d_bits, d_min, d_scale,
                        d_window_offsets, params->numel, params->elem_index_base, params->seed, 0u,
                        (uint32_t)pl.n_windows};
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(d_workspace, 0, pl.workspace, s) != cudaSuccess) return DAF_ERR_CUDA;
    return dispatch<false>(params->dtype, pl.chunks, a, s) == cudaSuccess ? DAF_OK : DAF_ERR_CUDA;
}

extern "C" uint64_t daf_batch_workspace(uint32_t n, const daf_params *params)
{
    uint64_t windows = 0;
    for (uint32_t i = 0; i < n; i++) {
        Plan pl;
        if (make_plan(&params[i], &pl) != DAF_OK) return 0;
        windows += pl.n_windows;
    }
    return sizeof(WorkspaceHeader) + 8ull * windows;
}

extern "C" daf_status daf_compress_batch(uint32_t n, const daf_params *params, const void *const *d_in,
                                         void *const *d_packed, const uint64_t *packed_capacity,
                                         uint8_t *const *d_bits, float *const *d_min, float *const *d_scale,
                                         uint64_t *const *d_window_offsets, void *d_workspace,
                                         uint64_t workspace_bytes, daf_stream stream)
{
    if (n == 0 || n > DAF_BATCH_MAX || !params || !d_in || !d_packed || !packed_capacity || !d_bits || !d_min || !d_scale ||
        !d_window_offsets || !d_workspace || !aligned16(d_workspace))
        return DAF_ERR_INVALID_ARG;
    Plan pl0;
    daf_status st = make_plan(&params[0], &pl0);
    if (st != DAF_OK) return st;
    CompressArgs<DAF_BATCH_MAX> a;
    fill_common(a, pl0, &params[0], d_workspace);
    a.n_tensors = n;
    a.keys = philox_keys(params[0].seed);
    uint64_t windows = 0;
    for (uint32_t i = 0; i < n; i++) {
        const daf_params *p = &params[i];
        Plan pl;
        st = make_plan(p, &pl);
        if (st != DAF_OK) return st;
        if (p->dtype != params[0].dtype || pl.G != pl0.G || pl.We != pl0.We || p->width_mask != params[0].width_mask ||
            pl.beta_q8 != pl0.beta_q8 || p->rounding != params[0].rounding)
            return DAF_ERR_INVALID_ARG;
        if (!d_in[i] || !d_packed[i] || !d_bits[i] || !d_min[i] || !d_scale[i] || !d_window_offsets[i] || !aligned16(d_in[i]) ||
            !aligned16(d_packed[i]) || (reinterpret_cast<uintptr_t>(d_min[i]) & 3u) ||
            (reinterpret_cast<uintptr_t>(d_scale[i]) & 3u) || (reinterpret_cast<uintptr_t>(d_window_offsets[i]) & 7u))
            return DAF_ERR_INVALID_ARG;
        if (windows + pl.n_windows > 0xFFFFFFF0ull) return DAF_ERR_UNSUPPORTED;
        a.t[i] = TensorDesc{d_in[i], reinterpret_cast<uint8_t *>(d_packed[i]), packed_capacity[i], d_bits[i], d_min[i],
                            d_scale[i], d_window_offsets[i], p->numel, p->elem_index_base, p->seed, (uint32_t)windows,
                            (uint32_t)pl.n_windows};
        windows += pl.n_windows;
    }
    a.total_windows = (uint32_t)windows;
    const uint64_t need = sizeof(WorkspaceHeader) + 8ull * windows;
    if (workspace_bytes < need) return DAF_ERR_CAPACITY;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(d_workspace, 0, need, s) != cudaSuccess) return DAF_ERR_CUDA;
    return dispatch<true>(params[0].dtype, pl0.chunks, a, s) == cudaSuccess ? DAF_OK : DAF_ERR_CUDA;
}
