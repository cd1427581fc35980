// Streaming compress kernel for calls whose windows end with TWO neighbouring widths: a budget that lies between two
// allowed widths (3 bits with widths {1,2,4,8}: every group reaches 2 bits and half of them 4) on data whose ranges
// within a window are close enough that the raises of the levels do not interleave (Sec. 3.4.1 of the paper).
//
// Then the greedy has a closed form.  With ell the last level every group reaches and `left` the budget that remains,
// exactly k = min(n, left / cost) groups are raised once more, and they are the k groups with the largest ranges (ties:
// the lower index).  So the window's packed size does not depend on the data -- n groups of width S[ell], k of them
// widened to S[ell + 1] -- and neither does its offset in the packed buffer: no look-back, as in the one-width kernel.
// What is left to find out is WHICH groups are raised, and that is a rank: a group is raised iff fewer than k groups
// of its window sort ahead of it.
//
// Structure: that of the one-width streaming kernel (compress_stream.cuh) -- CTA c takes windows c, c + gridDim.x, ...,
// warp w takes strip w of each, the strip lives in registers -- plus two meetings of the CTA's sixteen warps per window:
//
//   load strip, per-group min / max, ranges to shared memory            | meeting 1
//   read all ranges (two per lane), test that the levels separate,
//   rank of the warp's own groups by ballots, raised-bits to shared     | meeting 2
//   read the raised-bits, byte offset of each own group by popcounts,
//   1/scale by IEEE division, quantize with the group's width, store
//
// The assumption can fail (ranges that do not separate, a ragged last window whose own budget arithmetic ends at another
// level, a range that needs the clamped quantizer): the CTA that sees it raises hdr->retry, everybody stops at their
// next window, and the fallback, enqueued behind, redoes the call.  Decisions to stop are taken from one word in
// shared memory that one thread fills before meeting 1, so that all warps of a CTA leave together.
//
// Groups of 256, 512 or 1024 elements (LG = 8, 9, 10: whole chunks inside a warp's strip), default window, stochastic
// rounding.
#pragma once
#include "compress_stream.cuh"

namespace daf {

template <typename T, int LG, bool BATCH>
__global__ void __launch_bounds__(kThreads, 2)
two_width_kernel(const __grid_constant__ CompressArgs<BATCH ? DAF_BATCH_MAX : 1> a)
{
    using namespace stream;
    constexpr int CHUNKS = 4;
    constexpr uint32_t STRIP = 256u * CHUNKS, WE = kWarps * STRIP;
    constexpr uint32_t EB = Elem<T>::kBytes;
    constexpr uint32_t G = 1u << LG;
    constexpr int GPW = (int)(STRIP >> LG);                       // groups per strip: 4, 2, 1
    constexpr int CPG = CHUNKS / GPW;                             // chunks per group: 1, 2, 4
    constexpr uint32_t kNoGroup = 0xFFFFFFFFu;                    // range slot of a group the window does not have
    static_assert(DAF_BATCH_MAX == 64, "two entries of s_first per lane");

    __shared__ uint32_t s_R[64];                                  // the window's ranges (bit patterns; all are >= +0)
    __shared__ uint32_t s_raised[kWarps];                         // per warp: which of its groups are raised
    __shared__ uint32_t s_stop;                                   // hdr->retry as one thread saw it before meeting 1
    __shared__ uint32_t s_first[BATCH ? DAF_BATCH_MAX : 1];
    __shared__ __align__(16) uint32_t s_rkeys[BATCH ? kWarps : 1][20];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (BATCH)
        for (uint32_t i = tid; i < DAF_BATCH_MAX; i += kThreads) s_first[i] = i < a.n_tensors ? a.t[i].first_window : 0xFFFFFFFFu;
    if (tid < 64) s_R[tid] = kNoGroup;                            // (slots past the window's group count stay that way)
    if (tid == 0) s_stop = ld_relaxed_u32(&a.hdr->retry);
    __syncthreads();
    if (s_stop != 0u) return;                                     // given up before this CTA started

    const uint32_t strip0 = (uint32_t)warp * STRIP, e0 = strip0 + (uint32_t)lane * 8u;
    const uint32_t s0 = (uint32_t)warp * GPW;                     // the strip's first group within its window
    const uint32_t ell = a.full_ell, m = a.m;
    uint32_t cur_keys = 0xFFFFFFFFu;

    // One window.  WHOLE: it has all its elements (no predicates anywhere).  Returns false when the CTA is to leave.
    auto window = [&](auto whole_tag, const TensorDesc &td, uint32_t gw, uint32_t w, uint32_t n_elems) -> bool {
        constexpr bool WHOLE = decltype(whole_tag)::value;
        float x[CHUNKS][8];
        {
            const char *const src = reinterpret_cast<const char *>(td.in) + ((uint64_t)w * WE + e0) * EB;
#pragma unroll
            for (int c = 0; c < CHUNKS; c++) {
                if (WHOLE) {
                    Elem<T>::load8(src + 256u * EB * c, x[c]);
                } else {
#pragma unroll
                    for (int i = 0; i < 8; i++) x[c][i] = 0.0f;
                    if (e0 + 256u * c < n_elems) Elem<T>::load8(src + 256u * EB * c, x[c]);
                }
            }
        }
        if (WHOLE && gw + gridDim.x + 1u < a.total_windows && (uint32_t)lane * 128u < STRIP * EB) {
            const char *const next = reinterpret_cast<const char *>(td.in) + ((uint64_t)(w + gridDim.x) * WE + strip0) * EB;
            if (!BATCH || w + gridDim.x + 1u < td.n_windows) asm volatile("prefetch.global.L2 [%0];" ::"l"(next + (uint32_t)lane * 128u));
        }
        if (tid == 0) s_stop = ld_relaxed_u32(&a.hdr->retry);
        const uint32_t n = WHOLE ? WE >> LG : n_elems >> LG;

        // ---- minimum and range of the strip's groups (the same values in every lane), ranges filed for the CTA
        float g_mn[GPW], g_R[GPW];
#pragma unroll
        for (int j = 0; j < GPW; j++) {
            float lo, hi;
            extremes8(x[j * CPG], lo, hi);
#pragma unroll
            for (int c = 1; c < CPG; c++) {
                float l2, h2;
                extremes8(x[j * CPG + c], l2, h2);
                lo = fmin2(lo, l2);
                hi = fmax2(hi, h2);
            }
            lo = warp_min(lo);
            hi = warp_max(hi);
            const float R0 = __fsub_rn(hi, lo);
            g_mn[j] = lo;
            g_R[j] = R0 >= 0x1p-118f ? R0 : 0.0f;                 // below: degenerate group, treated as constant
            if (lane == j) s_R[s0 + j] = (WHOLE || s0 + j < n) ? __float_as_uint(g_R[j]) : kNoGroup;
        }
        __syncthreads();                                          // ---- meeting 1: every range of the window is filed
        if (s_stop != 0u) return false;                           // (the same word for all warps: they leave together)

        // ---- the window's verdict, worked out by every warp for itself
        const uint32_t Ra = s_R[lane], Rb = s_R[lane + 32];
        const bool va = Ra != kNoGroup, vb = Rb != kNoGroup;
        uint32_t k = a.tw_k;
        bool give_up = false;
        if (!WHOLE) {                                             // ragged last window: its own budget arithmetic
            const uint32_t rem = (uint32_t)((((uint64_t)a.beta_q8 * n) >> 8) - (uint64_t)a.S[0] * n);
            uint32_t l2 = 0;
            while (l2 + 1u < m && (a.S[l2 + 1u] - a.S[0]) * n <= rem) l2++;
            give_up = l2 != ell;
            const uint32_t kk = give_up ? 0u : (rem - (a.S[ell] - a.S[0]) * n) / a.cost[ell];
            k = kk < n ? kk : n;
        }
        {
            const uint32_t Rmin = __reduce_min_sync(0xFFFFFFFFu, min(va ? Ra : 0xFFFFFFFFu, vb ? Rb : 0xFFFFFFFFu));
            const uint32_t Rmax = __reduce_max_sync(0xFFFFFFFFu, max(va ? Ra : 0u, vb ? Rb : 0u));
            const float fmin_ = __uint_as_float(Rmin), fmax_ = __uint_as_float(Rmax);
            // every raise below level ell must sort ahead of every raise of level ell, every raise above it behind (ties go
            // to the lower level); and 1/scale must be a normal number (the quantizer here has no clamp)
            const uint32_t k_lo = __float_as_uint(__fmul_rn(fmin_, a.tw_v_my)), k_hi = __float_as_uint(__fmul_rn(fmax_, a.tw_v_my));
            if (a.tw_test_lo != 0u && __float_as_uint(__fmul_rn(fmin_, a.tw_v_lo)) < k_hi) give_up = true;
            if (a.tw_test_hi != 0u && __float_as_uint(__fmul_rn(fmax_, a.tw_v_hi)) > k_lo) give_up = true;
            if (fmax_ > 0x1p125f) give_up = true;
        }
        // rank of each own group among the window's groups by (key descending, index ascending): raised iff rank < k
        const uint32_t ka = __float_as_uint(__fmul_rn(__uint_as_float(va ? Ra : 0u), a.tw_v_my));
        const uint32_t kb = __float_as_uint(__fmul_rn(__uint_as_float(vb ? Rb : 0u), a.tw_v_my));
        uint32_t raised = 0u;
#pragma unroll
        for (int j = 0; j < GPW; j++) {
            const uint32_t gi = s0 + j;
            const uint32_t K = __float_as_uint(__fmul_rn(g_R[j], a.tw_v_my));
            const bool ahead_a = va && (ka > K || (ka == K && (uint32_t)lane < gi));
            const bool ahead_b = vb && (kb > K || (kb == K && (uint32_t)lane + 32u < gi));
            const uint32_t rank = __popc(__ballot_sync(0xFFFFFFFFu, ahead_a)) + __popc(__ballot_sync(0xFFFFFFFFu, ahead_b));
            if ((WHOLE || gi < n) && rank < k) raised |= 1u << j;
        }
        if (lane == 0) {
            s_raised[warp] = raised;
            if (give_up) atomicExch(&a.hdr->retry, 1u);
        }
        __syncthreads();                                          // ---- meeting 2: who is raised

        // ---- byte offset of the strip inside the window: tw_size_lo per group ahead + tw_size_up per raised group ahead
        const uint32_t r = (uint32_t)lane < (uint32_t)kWarps ? s_raised[lane] : 0u;
        const uint32_t ahead = __reduce_add_sync(0xFFFFFFFFu, lane < warp ? (uint32_t)__popc(r) : 0u);
        const uint64_t wbase = (uint64_t)w * a.tw_wbytes;         // every window before this one is whole
        unsigned char *const out = td.packed + wbase + (size_t)s0 * a.tw_size_lo + (size_t)ahead * a.tw_size_up;
        const uint64_t blk0 = (td.elem_base >> 3) + (uint64_t)w * (WE >> 3) + (e0 >> 3);
#pragma unroll
        for (int c = 0; c < CHUNKS; c++) {
            const int j = c / CPG;                                // the chunk's group among the strip's
            const bool up = (raised >> j) & 1u;
            const uint32_t b = up ? a.tw_bhi : a.tw_blo;
            const uint32_t off = (uint32_t)j * a.tw_size_lo + (uint32_t)__popc(raised & ((1u << j) - 1u)) * a.tw_size_up;
            const uint32_t idx = 32u * (uint32_t)(c % CPG) + (uint32_t)lane;   // the lane's eight codes within the group
            const float R = g_R[j];
            const float inv = R > 0.0f ? __fdiv_rn(up ? a.tw_lf_hi : a.tw_lf_lo, R > 0.0f ? R : 1.0f) : 0.0f;
            // (a window whose arithmetic did not come out as assumed is not stored: its sizes are not the planned ones)
            const bool ok = (WHOLE || e0 + 256u * c < n_elems) && !give_up;
            unsigned char *const p = out + off + idx * b;
            uint32_t o[4], t[8], w0, w1;
            const uint64_t blk = blk0 + 32u * c;
            if (BATCH) {
                const PhiloxSharedKeys sk{reinterpret_cast<const uint4 *>(s_rkeys[warp])};
                philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), sk, o);
            } else {
                philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), a.keys, o);
            }
            noisy_sums8(x[c], g_mn[j], inv, o, t);
            switch (b) {                                          // (the same branch for the whole warp)
            case 1:
                close_codes8<1, false>(t, w0, w1);
                if (ok) store_packed<1>(p, w0, w1);
                break;
            case 2:
                close_codes8<2, false>(t, w0, w1);
                if (ok) store_packed<2>(p, w0, w1);
                break;
            case 4:
                close_codes8<4, false>(t, w0, w1);
                if (ok) store_packed<4>(p, w0, w1);
                break;
            default:
                close_codes8<8, false>(t, w0, w1);
                if (ok) store_packed<8>(p, w0, w1);
                break;
            }
        }
        // ---- metadata of the strip's groups (lane j: group j), the window's offset (and the total behind the last window)
        {
            float R_l = g_R[0], mn_l = g_mn[0];
#pragma unroll
            for (int j = 1; j < GPW; j++)
                if (lane == j) {
                    R_l = g_R[j];
                    mn_l = g_mn[j];
                }
            if (lane < GPW && (WHOLE || s0 + (uint32_t)lane < n)) {
                const bool up = (raised >> lane) & 1u;
                const uint64_t g = (uint64_t)w * (WE >> LG) + s0 + (uint32_t)lane;
                td.bits[g] = (uint8_t)(up ? a.tw_bhi : a.tw_blo);
                td.mn[g] = mn_l;
                td.scale[g] = R_l > 0.0f ? __fdiv_rn(R_l, up ? a.tw_lf_hi : a.tw_lf_lo) : 0.0f;
            }
        }
        if (tid == 0) {
            td.woff[w] = wbase;
            if (w + 1u == td.n_windows) td.woff[w + 1u] = wbase + (uint64_t)n * a.tw_size_lo + (uint64_t)k * a.tw_size_up;
        }
        return true;
    };

    for (uint32_t gw = blockIdx.x; gw < a.total_windows; gw += gridDim.x) {
        uint32_t ti = 0u;
        if (BATCH) {
            const uint32_t n0 = __popc(__ballot_sync(0xFFFFFFFFu, s_first[lane] <= gw));
            const uint32_t n1 = __popc(__ballot_sync(0xFFFFFFFFu, s_first[lane + 32] <= gw));
            ti = n0 + n1 - 1u;
            if (ti != cur_keys) {                                 // round keys of this tensor's seed
                __syncwarp();
                if (lane < 10) philox_store_round_keys(s_rkeys[warp], a.t[ti].seed, lane);
                __syncwarp();
                cur_keys = ti;
            }
        }
        const TensorDesc &td = a.t[ti];
        const uint32_t w = BATCH ? gw - td.first_window : gw;
        uint32_t n_elems = WE;
        if (w + 1u == td.n_windows) n_elems = (uint32_t)(td.numel - (uint64_t)w * WE);
        const bool go = n_elems == WE ? window(std::true_type{}, td, gw, w, n_elems) : window(std::false_type{}, td, gw, w, n_elems);
        if (!go) break;
    }
}

template <typename T, int LG, bool BATCH>
static cudaError_t launch_two_width(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    int ctas = 0;
    const cudaError_t e = persistent_ctas(reinterpret_cast<const void *>(&two_width_kernel<T, LG, BATCH>), kThreads, 0, &ctas);
    if (e != cudaSuccess) return e;
    const uint32_t want = (uint32_t)ctas * 8u;                    // several waves, as for the one-width kernel
    two_width_kernel<T, LG, BATCH><<<args.total_windows < want ? args.total_windows : want, kThreads, 0, stream>>>(args);
    return cudaGetLastError();
}

// Launch for element type T and groups of 256, 512 or 1024 elements; the two widths are S[full_ell] and S[full_ell + 1].
template <typename T, bool BATCH>
cudaError_t dispatch_two_width_t(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    switch (args.log2G) {
    case 8: return launch_two_width<T, 8, BATCH>(args, stream);
    case 9: return launch_two_width<T, 9, BATCH>(args, stream);
    default: return launch_two_width<T, 10, BATCH>(args, stream);
    }
}

#define DAF_INSTANTIATE_TWO_WIDTH(T)                                                                                \
    template cudaError_t dispatch_two_width_t<T, false>(const CompressArgs<1> &, cudaStream_t);                     \
    template cudaError_t dispatch_two_width_t<T, true>(const CompressArgs<DAF_BATCH_MAX> &, cudaStream_t);

}  // namespace daf
