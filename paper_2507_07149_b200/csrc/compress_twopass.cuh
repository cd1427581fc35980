// Two-pass compress for windows of mixed widths: three kernels that never wait for one another.
//
//   widths_kernel   one WARP per window: reads the window once, keeps every group's min / max in registers (group g in
//                   lane g mod 32), runs the greedy of Sec. 3.4.1 on them (the one-warp threshold search of
//                   accept_prefix) and writes the groups' metadata and the window's packed size.  Many windows are
//                   settled at once on every multiprocessor, so the long dependent chain of one decision is covered
//                   by the other warps' loads; no shared memory, no barrier.
//   offsets_kernel  one CTA per tensor: exclusive scan of the window sizes -> window offsets, the capacity check.
//   pack_kernel     the one-width streaming kernel's structure (compress_stream.cuh: CTA per window, warp per strip,
//                   strip in registers, codes stored straight to their final place) with the width of every group read
//                   back from the metadata: Eq. 1 with stochastic rounding and LSB-first packing, per-group widths.
//
// The input is read twice.  For 16-bit elements that is cheap next to the arithmetic (Philox and Eq. 1 cost the same
// per element whatever its size), and what is saved is the general kernel's waiting: there the sixteen warps of a CTA
// hold a window in registers while one or a few of them decide its widths.  Groups of 128 to 1024 elements, default
// window, no fused producer.
#pragma once
#include "compress_stream.cuh"

namespace daf {

namespace twopass {

constexpr int kWidthsThreads = 256;                               // widths_kernel: eight independent warps
constexpr uint32_t kWE = 16384;                                   // elements per window

// Tensor of window gw in a batched launch: the last one whose first window is <= gw (s_first: first windows, padded
// with 0xFFFFFFFF to 64 entries).
__device__ __forceinline__ uint32_t tensor_of_window(const uint32_t *s_first, uint32_t gw, int lane)
{
    const uint32_t n0 = __popc(__ballot_sync(0xFFFFFFFFu, s_first[lane] <= gw));
    const uint32_t n1 = __popc(__ballot_sync(0xFFFFFFFFu, s_first[lane + 32] <= gw));
    return n0 + n1 - 1u;
}

}  // namespace twopass

// ------------------------------------------------------------------------------------------
// Pass 1: widths.  LG = log2 of the group size (7 .. 10).
// ------------------------------------------------------------------------------------------
template <typename T, int LG, bool BATCH>
__global__ void __launch_bounds__(twopass::kWidthsThreads, 3)
widths_kernel(const __grid_constant__ CompressArgs<BATCH ? DAF_BATCH_MAX : 1> a)
{
    using namespace stream;
    using namespace twopass;
    static_assert(DAF_BATCH_MAX == 64, "tensor_of_window reads two entries per lane");
    constexpr uint32_t EB = Elem<T>::kBytes;
    constexpr uint32_t G = 1u << LG, NMAX = kWE >> LG;            // groups per whole window: 128, 64, 32, 16
    constexpr int NQ = NMAX > 32u ? (int)(NMAX / 32u) : 1;        // groups a lane looks after (group lane + 32 q)
    constexpr uint32_t CPQ = 64u / NQ;                            // 256-element chunks that hold the groups of one q
    constexpr int NK = 3 * NQ;                                    // candidate raises per lane
    constexpr int U = EB == 2u ? 8 : 4;                           // chunks whose loads are in flight together

    __shared__ uint32_t s_first[BATCH ? DAF_BATCH_MAX : 1];
    if (a.gated != 0u && ld_relaxed_u32(&a.hdr->retry) == 0u) return;   // nothing to redo
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (BATCH) {
        for (uint32_t i = tid; i < DAF_BATCH_MAX; i += kWidthsThreads) s_first[i] = i < a.n_tensors ? a.t[i].first_window : 0xFFFFFFFFu;
        __syncthreads();
    }
    const uint32_t nl = a.m - 1u;
    const uint32_t warps = gridDim.x * (kWidthsThreads / 32);

    for (uint32_t gw = blockIdx.x * (kWidthsThreads / 32) + (uint32_t)warp; gw < a.total_windows; gw += warps) {
        const TensorDesc &td = a.t[BATCH ? tensor_of_window(s_first, gw, lane) : 0u];
        const uint32_t w = BATCH ? gw - td.first_window : gw;
        uint32_t n_elems = kWE;                                   // a ragged last window has fewer (whole groups)
        if (w + 1u == td.n_windows) n_elems = (uint32_t)(td.numel - (uint64_t)w * kWE);
        const uint32_t n = n_elems >> LG;
        const char *const src = reinterpret_cast<const char *>(td.in) + ((uint64_t)w * kWE + (uint32_t)lane * 8u) * EB;

        // ---- min / max of every group; group g ends up in lane g mod 32, slot g / 32
        float p_mn[NQ], p_mx[NQ];
#pragma unroll
        for (int q = 0; q < NQ; q++) {
            p_mn[q] = p_mx[q] = 0.0f;
            // the extremes of four chunks -> group extremes -> the lanes that keep them
            auto reduce_quad = [&](uint32_t c0, const float (&x)[4][8]) {
                float lo[4], hi[4];
#pragma unroll
                for (int u = 0; u < 4; u++) extremes8(x[u], lo[u], hi[u]);
                if (LG == 7) {
                    // two groups per chunk: a warp-wide reduction for each half, the other half's lanes holding the identity
                    const bool upper = lane >= 16;
                    const float inf = __uint_as_float(0x7F800000u), ninf = __uint_as_float(0xFF800000u);
#pragma unroll
                    for (int u = 0; u < 4; u++) {
                        const float lo_a = warp_min(upper ? inf : lo[u]), lo_b = warp_min(upper ? lo[u] : inf);
                        const float hi_a = warp_max(upper ? ninf : hi[u]), hi_b = warp_max(upper ? hi[u] : ninf);
                        const uint32_t t = (uint32_t)lane - ((2u * (c0 + u)) & 31u);   // 0 / 1: this lane keeps the first / second group
                        if (t < 2u) {
                            p_mn[q] = t ? lo_b : lo_a;
                            p_mx[q] = t ? hi_b : hi_a;
                        }
                    }
                } else if (LG == 8) {
#pragma unroll
                    for (int u = 0; u < 4; u++) {
                        const float l = warp_min(lo[u]), h = warp_max(hi[u]);
                        if ((uint32_t)lane == ((c0 + u) & 31u)) {
                            p_mn[q] = l;
                            p_mx[q] = h;
                        }
                    }
                } else if (LG == 9) {
#pragma unroll
                    for (int u = 0; u < 4; u += 2) {
                        const float l = warp_min(fmin2(lo[u], lo[u + 1])), h = warp_max(fmax2(hi[u], hi[u + 1]));
                        if ((uint32_t)lane == (c0 + u) >> 1) {
                            p_mn[q] = l;
                            p_mx[q] = h;
                        }
                    }
                } else {
                    const float l = warp_min(fmin2(fmin2(lo[0], lo[1]), fmin2(lo[2], lo[3])));
                    const float h = warp_max(fmax2(fmax2(hi[0], hi[1]), fmax2(hi[2], hi[3])));
                    if ((uint32_t)lane == c0 >> 2) {
                        p_mn[q] = l;
                        p_mx[q] = h;
                    }
                }
            };
            for (uint32_t c0 = (uint32_t)q * CPQ; c0 < (uint32_t)(q + 1) * CPQ; c0 += U) {
                if (c0 * 256u >= n_elems) break;
                if constexpr (EB == 2u) {
                    // 16-bit elements: eight chunks' loads in flight (16 bytes per lane each), widened four at a time
                    uint4 raw[U];
#pragma unroll
                    for (int u = 0; u < U; u++) {
                        raw[u] = make_uint4(0u, 0u, 0u, 0u);
                        if (c0 * 256u + 256u * U <= n_elems || (c0 + u) * 256u + (uint32_t)lane * 8u < n_elems)
                            asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                                         : "=r"(raw[u].x), "=r"(raw[u].y), "=r"(raw[u].z), "=r"(raw[u].w)
                                         : "l"(src + (size_t)(c0 + u) * 256u * EB));
                    }
#pragma unroll
                    for (int h = 0; h < U; h += 4) {
                        if ((c0 + h) * 256u >= n_elems) break;
                        float x[4][8];
#pragma unroll
                        for (int u = 0; u < 4; u++) Elem<T>::widen8(raw[h + u], x[u]);
                        reduce_quad(c0 + h, x);
                    }
                } else {
                    float x[4][8];
                    if (c0 * 256u + 1024u <= n_elems) {
#pragma unroll
                        for (int u = 0; u < 4; u++) Elem<T>::load8(src + (size_t)(c0 + u) * 256u * EB, x[u]);
                    } else {
#pragma unroll
                        for (int u = 0; u < 4; u++) {
#pragma unroll
                            for (int i = 0; i < 8; i++) x[u][i] = 0.0f;
                            if ((c0 + u) * 256u + (uint32_t)lane * 8u < n_elems) Elem<T>::load8(src + (size_t)(c0 + u) * 256u * EB, x[u]);
                        }
                    }
                    reduce_quad(c0, x);
                }
            }
        }

        // ---- the window's budget; then the greedy, by the cheapest route that settles it
        uint32_t ell = a.full_ell, rem = a.full_rem, rem_after = a.full_rem_after;
        if (n != NMAX) {                                          // ragged last window: its own arithmetic
            rem = (uint32_t)((((uint64_t)a.beta_q8 * n) >> 8) - (uint64_t)a.S[0] * n);
            ell = 0u;
            while (ell + 1u < a.m && (a.S[ell + 1u] - a.S[0]) * n <= rem) ell++;
            rem_after = rem - (a.S[ell] - a.S[0]) * n;
        }
        const bool all_max = ell + 1u == a.m;                     // every group reaches the largest width
        const bool need_sep = !all_max && rem_after < a.cost[ell];   // not even one raise of level ell fits
        float R[NQ];
        bool on[NQ];
#pragma unroll
        for (int q = 0; q < NQ; q++) {
            const float R0 = __fsub_rn(p_mx[q], p_mn[q]);
            R[q] = R0 >= 0x1p-118f ? R0 : 0.0f;                   // below: degenerate group, treated as constant
            on[q] = (uint32_t)lane + 32u * q < n;
        }
        // extremes of the keys of the raises below level ell, of level ell, and above it
        uint32_t up_min = 0xFFFFFFFFu, my_min = 0xFFFFFFFFu, my_max = 0u, dn_max = 0u;
#pragma unroll
        for (int k = 0; k < 3; k++) {
            if ((uint32_t)k >= nl) continue;
#pragma unroll
            for (int q = 0; q < NQ; q++) {
                if (!on[q]) continue;
                const uint32_t kk = __float_as_uint(__fmul_rn(R[q], a.v[k]));
                if ((uint32_t)k < ell) up_min = min(up_min, kk);
                else if ((uint32_t)k > ell) dn_max = max(dn_max, kk);
                else {
                    my_min = min(my_min, kk);
                    my_max = max(my_max, kk);
                }
            }
        }
        up_min = __reduce_min_sync(0xFFFFFFFFu, up_min);
        my_max = __reduce_max_sync(0xFFFFFFFFu, my_max);
        uint32_t lvl[NQ];
        if (all_max || (need_sep && up_min >= my_max)) {
            // one width: every raise below level ell sorts ahead of every raise of level ell (ties go to the lower
            // level), they all fit, and the next does not
#pragma unroll
            for (int q = 0; q < NQ; q++) lvl[q] = ell;
        } else {
            my_min = __reduce_min_sync(0xFFFFFFFFu, my_min);
            dn_max = __reduce_max_sync(0xFFFFFFFFu, dn_max);
            if (up_min >= my_max && dn_max <= my_min) {
                // the levels do not interleave: all raises below level ell are taken (they fit by the definition of
                // ell), none above it, and the search runs over the raises of level ell alone
                uint32_t key[NQ], cw[NQ], slot_cost[NQ];
                bool take[NQ];
#pragma unroll
                for (int q = 0; q < NQ; q++) {
                    key[q] = on[q] ? __float_as_uint(__fmul_rn(R[q], a.v[ell])) : 0u;
                    cw[q] = on[q] ? a.cost[ell] | 0x10000u : 0u;
                    slot_cost[q] = a.cost[ell];
                }
                accept_prefix<NQ, true>(key, cw, slot_cost, rem_after, my_max, my_min, lane, take);
#pragma unroll
                for (int q = 0; q < NQ; q++) lvl[q] = ell + (uint32_t)take[q];
            } else {
                // candidate raise k of group lane + 32 q sits in slot k NQ + q, so that equal keys are taken level by
                // level and, within a level, group by group (the order accept_prefix defines)
                uint32_t key[NK], cw[NK], slot_cost[NK];
                bool take[NK];
#pragma unroll
                for (int k = 0; k < 3; k++)
#pragma unroll
                    for (int q = 0; q < NQ; q++) {
                        const bool c = (uint32_t)k < nl && on[q];
                        key[k * NQ + q] = c ? __float_as_uint(__fmul_rn(R[q], a.v[k])) : 0u;
                        cw[k * NQ + q] = c ? a.cost[k] | 0x10000u : 0u;
                        slot_cost[k * NQ + q] = a.cost[k];
                    }
                accept_prefix<NK, false>(key, cw, slot_cost, rem, 0u, 0u, lane, take);
#pragma unroll
                for (int q = 0; q < NQ; q++) lvl[q] = (uint32_t)take[q] + take[NQ + q] + take[2 * NQ + q];
            }
        }

        // ---- metadata of the groups, packed size of the window
        const uint64_t g0 = (uint64_t)w * NMAX;
        uint32_t total = 0u;
#pragma unroll
        for (int q = 0; q < NQ; q++) {
            const uint32_t g = (uint32_t)lane + 32u * q;
            if (g < n) {
                const uint32_t b = a.S[lvl[q]];
                const float Lf = (float)((1u << b) - 1u);
                td.bits[g0 + g] = (uint8_t)b;
                td.mn[g0 + g] = p_mn[q];
                td.scale[g0 + g] = R[q] > 0.0f ? __fdiv_rn(R[q], Lf) : 0.0f;
                total += (G >> 3) * b;
            }
        }
        total = __reduce_add_sync(0xFFFFFFFFu, total);
        if (lane == 0) a.flags2[gw] = total;
    }
}

// ------------------------------------------------------------------------------------------
// Between the passes: window offsets of tensor blockIdx.x = exclusive scan of its windows' sizes (left in the
// descriptor array by widths_kernel), the total behind the last window, and the capacity check: the first window
// that does not fit is reported; pack_kernel stores no window that ends beyond the capacity.
// ------------------------------------------------------------------------------------------
template <int NT>
__global__ void __launch_bounds__(1024) offsets_kernel(const __grid_constant__ CompressArgs<NT> a)
{
    __shared__ uint64_t s_warp[32];
    __shared__ uint32_t s_bad;
    if (a.gated != 0u && stream::ld_relaxed_u32(&a.hdr->retry) == 0u) return;
    const TensorDesc &td = a.t[blockIdx.x];
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint64_t *const size = a.flags2 + td.first_window;
    const uint32_t nw = td.n_windows, per = (nw + 1023u) / 1024u;
    const uint32_t lo = min(tid * per, nw), hi = min(lo + per, nw);   // this thread's windows
    if (tid == 0) s_bad = 0xFFFFFFFFu;
    uint64_t sum = 0;
    for (uint32_t w = lo; w < hi; w++) sum += size[w];
    uint64_t incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint64_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= (uint32_t)o) incl += y;
    }
    if (lane == 31u) s_warp[warp] = incl;
    __syncthreads();
    uint64_t before = 0, all = 0;
    for (uint32_t k = 0; k < 32u; k++) {
        const uint64_t t = s_warp[k];
        if (k < warp) before += t;
        all += t;
    }
    uint64_t at = before + incl - sum;
    uint32_t bad = 0xFFFFFFFFu;
    for (uint32_t w = lo; w < hi; w++) {
        td.woff[w] = at;
        at += size[w];
        if (at > td.capacity && bad == 0xFFFFFFFFu) bad = w;
    }
    if (bad != 0xFFFFFFFFu) atomicMin(&s_bad, bad);
    __syncthreads();
    if (tid == 0) {
        td.woff[nw] = all;
        if (s_bad != 0xFFFFFFFFu && atomicCAS(&a.hdr->status, 0u, (unsigned)DAF_ERR_CAPACITY) == 0u)
            a.hdr->fail_window = td.first_window + s_bad;
    }
}

// ------------------------------------------------------------------------------------------
// Pass 2: quantize and pack with the widths pass 1 chose.  CTA c takes windows c, c + gridDim.x, ...; warp w takes
// strip w (1024 elements) of each.  A strip's groups recompute their own min / max (the strip is in registers anyway;
// the same operations on the same values as in pass 1), read their widths from the metadata and their place from the
// window's offset plus the sizes of the window's groups ahead of them.
// ------------------------------------------------------------------------------------------
template <typename T, int LG, bool BATCH>
__global__ void __launch_bounds__(kThreads, 2)
pack_kernel(const __grid_constant__ CompressArgs<BATCH ? DAF_BATCH_MAX : 1> a)
{
    using namespace stream;
    using namespace twopass;
    constexpr int CHUNKS = 4;
    constexpr uint32_t STRIP = 256u * CHUNKS;
    constexpr uint32_t EB = Elem<T>::kBytes;
    constexpr uint32_t G = 1u << LG, NMAX = kWE >> LG;
    constexpr int NQ = NMAX > 32u ? (int)(NMAX / 32u) : 1;
    constexpr uint32_t GPW = STRIP >> LG;                         // groups per strip: 8, 4, 2, 1

    __shared__ uint32_t s_first[BATCH ? DAF_BATCH_MAX : 1];
    __shared__ __align__(16) uint32_t s_rkeys[BATCH ? kWarps : 1][20];   // Philox round keys of the warp's current tensor

    if (a.gated != 0u && ld_relaxed_u32(&a.hdr->retry) == 0u) return;    // nothing to redo
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (BATCH) {
        for (uint32_t i = tid; i < DAF_BATCH_MAX; i += kThreads) s_first[i] = i < a.n_tensors ? a.t[i].first_window : 0xFFFFFFFFu;
        __syncthreads();
    }
    const uint32_t strip0 = (uint32_t)warp * STRIP, e0 = strip0 + (uint32_t)lane * 8u;
    const uint32_t s0 = (uint32_t)warp * GPW;                     // the strip's first group within its window
    const bool nearest = a.nearest != 0u;
    uint32_t cur_keys = 0xFFFFFFFFu;

    auto strip = [&](auto whole_tag, const TensorDesc &td, uint32_t gw, uint32_t w, uint32_t n_elems) {
        constexpr bool WHOLE = decltype(whole_tag)::value;
        float x[CHUNKS][8];
        {
            const char *const src = reinterpret_cast<const char *>(td.in) + ((uint64_t)w * kWE + e0) * EB;
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
        // the strip this warp takes next is asked into L2 (one 128-byte line per lane; whole windows only)
        if (WHOLE && gw + gridDim.x + 1u < a.total_windows && (uint32_t)lane * 128u < STRIP * EB) {
            const char *const next = reinterpret_cast<const char *>(td.in) + ((uint64_t)(w + gridDim.x) * kWE + strip0) * EB;
            if (!BATCH || w + gridDim.x + 1u < td.n_windows) asm volatile("prefetch.global.L2 [%0];" ::"l"(next + (uint32_t)lane * 128u));
        }
        // ---- where the strip's codes go: the window's offset, then the groups of the window ahead of the strip
        const uint32_t n = WHOLE ? NMAX : n_elems >> LG;
        const uint64_t wo = td.woff[w];
        const bool room = td.woff[w + 1u] <= td.capacity;         // a window that ends beyond the capacity is not stored
        // widths of the window's groups, four to a lane (group 4 lane + i in byte i of the lane's word)
        const uint8_t *const bits_w = td.bits + (uint64_t)w * NMAX;
        uint32_t bw = 0u;
        if (WHOLE && (reinterpret_cast<uintptr_t>(td.bits) & 3u) == 0u) {
            if ((uint32_t)lane * 4u < NMAX) bw = *reinterpret_cast<const uint32_t *>(bits_w + 4u * lane);
        } else {
#pragma unroll
            for (uint32_t i = 0; i < 4u; i++)
                if (4u * lane + i < n) bw |= (uint32_t)bits_w[4u * lane + i] << (8u * i);
        }
        // widths of the groups ahead of the strip: the words below the strip's first, and the low bytes of that one
        const uint32_t wi = s0 >> 2, part = 8u * (s0 & 3u);
        const uint32_t mine = (uint32_t)lane < wi ? bw : (uint32_t)lane == wi ? bw & ((1u << part) - 1u) : 0u;
        const uint32_t ahead = __reduce_add_sync(0xFFFFFFFFu, (mine * 0x01010101u) >> 24);   // (a width is at most 8: the byte sum fits)
        // the strip's own widths, group j in byte j of (W0, W1)
        const uint32_t W0 = __shfl_sync(0xFFFFFFFFu, bw, (int)wi) >> part;
        const uint32_t W1 = GPW > 4u ? __shfl_sync(0xFFFFFFFFu, bw, (int)wi + 1) : 0u;
        uint32_t pre = 0u;                                        // widths of the strip's groups before the current one
        unsigned char *const out = td.packed + wo + (size_t)ahead * (G >> 3);
        const uint64_t blk0 = (td.elem_base >> 3) + (uint64_t)w * (kWE >> 3) + (e0 >> 3);

        float lo = 0.0f, hi = 0.0f;
        if (LG == 10) {
            extremes8(x[0], lo, hi);
#pragma unroll
            for (int c = 1; c < CHUNKS; c++) {
                float l2, h2;
                extremes8(x[c], l2, h2);
                lo = fmin2(lo, l2);
                hi = fmax2(hi, h2);
            }
            lo = warp_min(lo);
            hi = warp_max(hi);
        }
#pragma unroll
        for (int c = 0; c < CHUNKS; c++) {
            // ---- the chunk's group (LG = 7: the lane's one of two): extremes, width, place
            if (LG == 7) {
                extremes8(x[c], lo, hi);
                const bool upper = lane >= 16;
                const float inf = __uint_as_float(0x7F800000u), ninf = __uint_as_float(0xFF800000u);
                const float lo_a = warp_min(upper ? inf : lo), lo_b = warp_min(upper ? lo : inf);
                const float hi_a = warp_max(upper ? ninf : hi), hi_b = warp_max(upper ? hi : ninf);
                lo = upper ? lo_b : lo_a;
                hi = upper ? hi_b : hi_a;
            } else if (LG == 8) {
                extremes8(x[c], lo, hi);
                lo = warp_min(lo);
                hi = warp_max(hi);
            } else if (LG == 9) {
                if ((c & 1) == 0) {
                    float l2, h2;
                    extremes8(x[c], lo, hi);
                    extremes8(x[(c + 1) % CHUNKS], l2, h2);
                    lo = warp_min(fmin2(lo, l2));
                    hi = warp_max(fmax2(hi, h2));
                }
            }
            uint32_t b, off, idx;
            if (LG == 7) {
                const uint32_t Wx = c < 2 ? W0 : W1;
                const uint32_t bA = (Wx >> (8 * ((2 * c) & 3))) & 0xFFu, bB = (Wx >> (8 * ((2 * c + 1) & 3))) & 0xFFu;
                const bool upper = lane >= 16;
                b = upper ? bB : bA;
                off = (pre + (upper ? bA : 0u)) * (G >> 3);
                idx = (uint32_t)lane & 15u;
                pre += bA + bB;
            } else if (LG == 8) {
                b = (W0 >> (8 * c)) & 0xFFu;
                off = pre * (G >> 3);
                idx = (uint32_t)lane;
                pre += b;
            } else if (LG == 9) {
                b = (W0 >> (8 * (c >> 1))) & 0xFFu;
                off = pre * (G >> 3);
                idx = 32u * (c & 1) + (uint32_t)lane;
                if (c & 1) pre += b;
            } else {
                b = W0 & 0xFFu;
                off = 0u;
                idx = 32u * c + (uint32_t)lane;
            }
            const float R0 = __fsub_rn(hi, lo);
            const bool pos = R0 >= 0x1p-118f;                     // below: degenerate group, treated as constant
            const float Lf = (float)((1u << b) - 1u);
            const float inv = pos ? __fdiv_rn(Lf, pos ? R0 : 1.0f) : 0.0f;
            unsigned char *const p = out + off + idx * b;
            const bool ok = (WHOLE || e0 + 256u * c < n_elems) && room;

            uint32_t o[4], w0, w1;
            if (nearest) {
                o[0] = o[1] = o[2] = o[3] = 0x80008000u;          // every 16-bit lane = 2 * 2^14
            } else {
                const uint64_t blk = blk0 + 32u * c;
                if (BATCH) {
                    const PhiloxSharedKeys sk{reinterpret_cast<const uint4 *>(s_rkeys[warp])};
                    philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), sk, o);
                } else {
                    philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), a.keys, o);
                }
            }
            if (__any_sync(0xFFFFFFFFu, R0 > 0x1p125f)) {
                // 1/scale may not be a normal number: the codes may need the clamp
                quantize8_any(x[c], lo, inv, o, b, w0, w1);
                if (ok) {
                    if (b == 1u) store_packed<1>(p, w0, w1);
                    else if (b == 2u) store_packed<2>(p, w0, w1);
                    else if (b == 4u) store_packed<4>(p, w0, w1);
                    else store_packed<8>(p, w0, w1);
                }
            } else {
                uint32_t t[8];
                noisy_sums8(x[c], lo, inv, o, t);                 // (the arithmetic all widths share stays outside the split)
                switch (b) {
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
        }
    };

    for (uint32_t gw = blockIdx.x; gw < a.total_windows; gw += gridDim.x) {
        uint32_t ti = 0u;
        if (BATCH) {
            ti = tensor_of_window(s_first, gw, lane);
            if (ti != cur_keys) {                                 // round keys of this tensor's seed
                __syncwarp();
                if (lane < 10) philox_store_round_keys(s_rkeys[warp], a.t[ti].seed, lane);
                __syncwarp();
                cur_keys = ti;
            }
        }
        const TensorDesc &td = a.t[ti];
        const uint32_t w = BATCH ? gw - td.first_window : gw;
        uint32_t n_elems = kWE;
        if (w + 1u == td.n_windows) n_elems = (uint32_t)(td.numel - (uint64_t)w * kWE);
        if (n_elems == kWE) strip(std::true_type{}, td, gw, w, n_elems);
        else strip(std::false_type{}, td, gw, w, n_elems);
    }
}

// ------------------------------------------------------------------------------------------
// Launch
// ------------------------------------------------------------------------------------------
template <typename T, int LG, bool BATCH>
static cudaError_t launch_twopass(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    constexpr int NT = BATCH ? DAF_BATCH_MAX : 1;
    int ctas = 0;
    cudaError_t e = persistent_ctas(reinterpret_cast<const void *>(&widths_kernel<T, LG, BATCH>), twopass::kWidthsThreads, 0, &ctas);
    if (e != cudaSuccess) return e;
    constexpr uint32_t wpc = twopass::kWidthsThreads / 32;
    // four waves of CTAs (eight for the pack kernel): the block scheduler evens out the finishing times, which differ
    // with the windows' decisions (one wave: 279 against 246 us and 625 against 597 us on the ViT set at full size)
    uint32_t want = (args.total_windows + wpc - 1u) / wpc, most = (uint32_t)ctas * 4u;
    widths_kernel<T, LG, BATCH><<<want < most ? want : most, twopass::kWidthsThreads, 0, stream>>>(args);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    offsets_kernel<NT><<<args.n_tensors, 1024, 0, stream>>>(args);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    e = persistent_ctas(reinterpret_cast<const void *>(&pack_kernel<T, LG, BATCH>), kThreads, 0, &ctas);
    if (e != cudaSuccess) return e;
    want = (uint32_t)ctas * 8u;
    pack_kernel<T, LG, BATCH><<<args.total_windows < want ? args.total_windows : want, kThreads, 0, stream>>>(args);
    return cudaGetLastError();
}

// Launch for element type T and groups of 128, 256, 512 or 1024 elements (default window).
template <typename T, bool BATCH>
cudaError_t dispatch_twopass_t(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    switch (args.log2G) {
    case 7: return launch_twopass<T, 7, BATCH>(args, stream);
    case 8: return launch_twopass<T, 8, BATCH>(args, stream);
    case 9: return launch_twopass<T, 9, BATCH>(args, stream);
    default: return launch_twopass<T, 10, BATCH>(args, stream);
    }
}

#define DAF_INSTANTIATE_TWOPASS(T)                                                                                  \
    template cudaError_t dispatch_twopass_t<T, false>(const CompressArgs<1> &, cudaStream_t);                       \
    template cudaError_t dispatch_twopass_t<T, true>(const CompressArgs<DAF_BATCH_MAX> &, cudaStream_t);

}  // namespace daf
