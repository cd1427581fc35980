// Streaming compress kernel for calls whose windows all end with one width (the common case:
// a budget that one allowed width meets exactly, ranges within a window close enough that no
// raise of a higher level sorts ahead of one of a lower level, Sec. 3.4.1 of the paper).
//
// With one width B = S[ell] for every group, the packed position of every code follows from its
// index, and a warp can take 8 * 32 * CHUNKS consecutive elements (a "strip") from global memory
// to packed bytes on its own, with no shared memory and no meeting with other warps:
//
//   strip -> registers (32 bytes per lane and load, all loads of the strip in flight)
//   -> per-group min / max (3-input min/max, warp redux or segmented shuffles)
//   -> range, 1/scale and scale by IEEE division, metadata stores
//   -> Eq. 1 with stochastic rounding (Philox4x32-10, the float -> uint step by the power-of-two
//      offset of Eq. 5), lane-local LSB-first packing, coalesced stores.
//
// A CTA takes windows blockIdx.x, blockIdx.x + gridDim.x, ...; its warp w takes strip w of each.
// That every window really is of one width is an assumption while the strips are processed.
// Each warp adds the extremes of the importance keys of its groups to the window's word in the
// workspace (two atomic max); verify_stream_kernel, enqueued behind, compares them window by
// window, checks the budget arithmetic of ragged last windows and writes the window offsets.  If
// a test fails anywhere (or a group needs the clamped quantizer), hdr->retry is raised and the
// general kernel, enqueued behind both, redoes the call; the streaming kernel itself stops as
// soon as it sees the flag, and raises it itself when the keys of one strip alone do not
// separate.  Groups larger than a strip are the one case where warps meet: those that
// share a group exchange their extremes through shared memory at a named barrier of their own.
//
// The kernel is a template over the element type, the strip length, the width B, the relation
// of group size and strip (GC: 0 = groups below 128 elements, 3 = groups of 128, 1 = groups of whole chunks inside
// a strip, 2 = groups of one or more strips), batched calls and the fused ReLU; this header is
// included by one translation unit per element type.
#pragma once
#include <type_traits>

#include "compress_shared.cuh"

namespace daf {

namespace stream {

__device__ __forceinline__ uint32_t ld_relaxed_u32(const unsigned int *p)
{
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void named_bar_sync(uint32_t id, uint32_t threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
// Lane-local extremes of eight values.
__device__ __forceinline__ void extremes8(const float (&x)[8], float &lo, float &hi)
{
    lo = fmin3(fmin3(x[0], x[1], x[2]), fmin3(x[3], x[4], x[5]), fmin2(x[6], x[7]));
    hi = fmax3(fmax3(x[0], x[1], x[2]), fmax3(x[3], x[4], x[5]), fmax2(x[6], x[7]));
}
__device__ __forceinline__ float warp_min(float v)
{
    asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(v) : "f"(v));
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(v) : "f"(v));
    return v;
}
template <int B> __device__ __forceinline__ void store_packed(unsigned char *p, uint32_t w0, uint32_t w1)
{
    if (B == 1) *p = (unsigned char)w0;
    else if (B == 2) *reinterpret_cast<uint16_t *>(p) = (uint16_t)w0;
    else if (B == 4) *reinterpret_cast<uint32_t *>(p) = w0;
    else *reinterpret_cast<uint2 *>(p) = make_uint2(w0, w1);
}

// What a group's elements need before they can be quantized: the minimum and 1/scale = L / R (IEEE division).  R comes
// back as the range the oracle uses (zero for a degenerate group).
template <int B> __device__ __forceinline__ float inverse_scale(float lo, float hi, float &R)
{
    constexpr float Lf = (float)((1u << B) - 1u);
    const float R0 = __fsub_rn(hi, lo);
    const bool pos = R0 >= 0x1p-118f;                             // below: degenerate group, treated as constant
    R = pos ? R0 : 0.0f;
    // (a constant group divides by one: the division stays on its fast path)
    return pos ? __fdiv_rn(Lf, pos ? R0 : 1.0f) : 0.0f;
}

}  // namespace stream

template <typename T, int CHUNKS, int B, int GC, bool BATCH, int ACT>
__global__ void __launch_bounds__(kThreads, 2)
stream_compress_kernel(const __grid_constant__ CompressArgs<BATCH ? DAF_BATCH_MAX : 1> a)
{
    using namespace stream;
    constexpr uint32_t STRIP = 256u * CHUNKS;                     // elements per warp and window
    constexpr uint32_t WE = kWarps * STRIP;
    constexpr uint32_t EB = Elem<T>::kBytes;
    constexpr uint32_t WBYTES = (WE >> 3) * B;                    // packed bytes of a whole window

    __shared__ float s_ext[2][kWarps][2];                         // strip extremes of groups that span warps
    __shared__ uint32_t s_stop[2][kWarps];                        // ... and each warp's wish to stop
    __shared__ uint32_t s_first[BATCH ? DAF_BATCH_MAX : 1];       // first window of every tensor
    __shared__ __align__(16) uint32_t s_rkeys[BATCH ? kWarps : 1][20];   // Philox round keys of the warp's current tensor

    __shared__ uint32_t s_late;                                   // the call was given up before this CTA started

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (BATCH)
        for (uint32_t i = tid; i < DAF_BATCH_MAX; i += kThreads) s_first[i] = i < a.n_tensors ? a.t[i].first_window : 0xFFFFFFFFu;
    // Whoever starts after somebody has asked for the fallback leaves at once: the grid is several times what the
    // device holds, so after a failure in the first wave the rest of the grid costs next to nothing.  Warps that
    // share a group (GC = 2) must take the same decision: there one thread reads the flag for the CTA.
    // Independent warps read the flag themselves: at once (groups of 128 elements and more; 8-bit codes), or with the
    // wait for it moved behind the first strip's loads (smaller groups) -- whichever the instantiation runs faster
    // with when nothing fails (differences of half a percent, measured on the 16 sweep points).
    constexpr bool kWaitAtStart = GC != 0 || B == 8;
    uint32_t retry_seen = 0u;
    if (GC == 2) {
        if (tid == 0) s_late = ld_relaxed_u32(&a.hdr->retry);
        __syncthreads();
        if (s_late != 0u) return;
    } else {
        if (BATCH) __syncthreads();
        retry_seen = ld_relaxed_u32(&a.hdr->retry);
        if (kWaitAtStart && retry_seen != 0u) return;
    }
    const uint32_t log2G = a.log2G;
    const uint32_t strip0 = (uint32_t)warp * STRIP;               // the strip's first element within its window
    const uint32_t e0 = strip0 + (uint32_t)lane * 8u;             // the lane's first element of chunk 0
    uint32_t cur_keys = 0xFFFFFFFFu;
    uint32_t stop = 0u;
    uint32_t it = 0;

    // One strip.  WHOLE: the window has all its elements (no predicates anywhere).
    auto strip = [&](auto whole_tag, const TensorDesc &td, uint32_t gw, uint32_t w, uint32_t n_elems) {
        constexpr bool WHOLE = decltype(whole_tag)::value;
        // ---- the strip's loads go out first
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
        // ---- the strip this warp takes next is asked into L2 now, a whole strip's work ahead of its loads (one 128-byte
        // line per lane; whole windows only: the line must exist)
#ifndef DAF_PF_DIST
#define DAF_PF_DIST 1u
#endif
        if (WHOLE && gw + DAF_PF_DIST * gridDim.x + 1u < a.total_windows && (uint32_t)lane * 128u < STRIP * EB) {
            const char *const next = reinterpret_cast<const char *>(td.in) + ((uint64_t)(w + DAF_PF_DIST * gridDim.x) * WE + strip0) * EB;
            if (!BATCH || w + DAF_PF_DIST * gridDim.x + 1u < td.n_windows)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(next + (uint32_t)lane * 128u));
        }
        // ---- meanwhile: has anybody asked to stop?
        stop |= retry_seen;
        retry_seen = ld_relaxed_u32(&a.hdr->retry);               // consumed one window later
        if (GC != 2 && !kWaitAtStart && stop != 0u) return;       // (nobody waits for this warp: the strip is dropped here)
        if (ACT != kActNone) {
            // fused producer: the activation is written out and (ReLU, ReLU6) replaces x as what is compressed; a lane
            // stores the chunk it loaded, so the output may be the input buffer
            char *const act = reinterpret_cast<char *>(td.act) + ((uint64_t)w * WE + e0) * EB;
#pragma unroll
            for (int c = 0; c < CHUNKS; c++) {
                float y[8];
                activate8<ACT>(x[c], y);
                if (WHOLE || e0 + 256u * c < n_elems) Elem<T>::store8(act + 256u * EB * c, y);
            }
        }

        const uint64_t blk0 = (td.elem_base >> 3) + (uint64_t)w * (WE >> 3) + (e0 >> 3);
        unsigned char *const out = td.packed + (uint64_t)w * WBYTES + (size_t)(e0 >> 3) * B;
        const uint64_t g0 = (uint64_t)w * (WE >> log2G) + (strip0 >> log2G);   // the strip's first group in the tensor
        uint8_t *const bits_p = td.bits + g0;
        float *const mn_p = td.mn + g0, *const scale_p = td.scale + g0;
        // Each group's (minimum, range) is parked in one lane while the chunks are quantized; afterwards one pass over the
        // lanes works out the scales and the importance keys and stores the metadata of the whole strip.
        float p_mn = 0.0f, p_R = 0.0f;
        uint32_t p_idx = 0xFFFFFFFFu;                             // the parked group's index within the strip (none yet)
        // Philox + Eq. 1 + pack + store of chunk c with the group's minimum and 1/scale
        auto quantize = [&](auto chunk_tag, float mn, float inv) {
            constexpr int c = decltype(chunk_tag)::value;
            uint32_t o[4], w0, w1;
            const uint64_t blk = blk0 + 32u * c;
            if (BATCH) {
                const PhiloxSharedKeys sk{reinterpret_cast<const uint4 *>(s_rkeys[warp])};
                philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), sk, o);
            } else {
                philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), a.keys, o);
            }
            quantize8<B, false>(x[c], mn, inv, o, w0, w1);
            if (WHOLE || e0 + 256u * c < n_elems) store_packed<B>(out + 32 * B * c, w0, w1);
        };
        auto for_chunks = [&](auto f) {                           // f(integral_constant<int, c>) for every chunk of the strip
            f(std::integral_constant<int, 0>{});
            if constexpr (CHUNKS > 1) f(std::integral_constant<int, 1>{});
            if constexpr (CHUNKS > 2) {
                f(std::integral_constant<int, 2>{});
                f(std::integral_constant<int, 3>{});
            }
        };

        if (GC == 0 || GC == 3) {
            // ---- several groups per chunk: a segmented shuffle leaves every lane with its own group's extremes; the lane
            // whose position in its group equals the chunk number parks the group
            const uint32_t lpg = 1u << (log2G - 3u);              // lanes per group (4, 8 or 16)
            for_chunks([&](auto ct) {
                constexpr int c = decltype(ct)::value;
                float lo, hi;
                extremes8(x[c], lo, hi);
                if (GC == 3) {
                    // two groups per chunk: a warp-wide reduction for each half, the other half's lanes holding the
                    // identity (four redux and four selects instead of eight shuffles and eight min / max)
                    const bool upper = lane >= 16;
                    const float inf = __uint_as_float(0x7F800000u), ninf = __uint_as_float(0xFF800000u);
                    const float lo_a = warp_min(upper ? inf : lo), lo_b = warp_min(upper ? lo : inf);
                    const float hi_a = warp_max(upper ? ninf : hi), hi_b = warp_max(upper ? hi : ninf);
                    lo = upper ? lo_b : lo_a;
                    hi = upper ? hi_b : hi_a;
                } else {
                    lo = fmin2(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, 1));
                    hi = fmax2(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, 1));
                    lo = fmin2(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, 2));
                    hi = fmax2(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, 2));
                    if (lpg > 4u) {
                        lo = fmin2(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, 4));
                        hi = fmax2(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, 4));
                    }
                }
                float R;
                const float inv = inverse_scale<B>(lo, hi, R);
                // (groups are whole: the lane's group exists iff its elements do)
                if ((WHOLE || e0 + 256u * c < n_elems) && ((uint32_t)lane & (lpg - 1u)) == (uint32_t)c) {
                    p_mn = lo;
                    p_R = R;
                    p_idx = (((uint32_t)c << 8) >> log2G) + ((uint32_t)lane >> (log2G - 3u));
                }
                quantize(ct, lo, inv);
            });
        } else if (GC == 1) {
            // ---- groups of one chunk, or of two (strips of four chunks, groups of 512 elements): lane j parks group j
            const bool pairs = CHUNKS == 4 && log2G == 9u;
            float l_prev = 0.0f, h_prev = 0.0f, mn_pair = 0.0f, inv_pair = 0.0f;
            for_chunks([&](auto ct) {
                constexpr int c = decltype(ct)::value;
                float lo, hi;
                if (!pairs || (c & 1) == 0) {
                    extremes8(x[c], lo, hi);
                    if (pairs && c + 1 < CHUNKS) {
                        extremes8(x[(c + 1) % CHUNKS], l_prev, h_prev);
                        lo = fmin2(lo, l_prev);
                        hi = fmax2(hi, h_prev);
                    }
                    lo = warp_min(lo);
                    hi = warp_max(hi);
                    float R;
                    const float inv = inverse_scale<B>(lo, hi, R);
                    const uint32_t j = pairs ? (uint32_t)c >> 1 : (uint32_t)c;
                    if ((WHOLE || strip0 + 256u * c < n_elems) && (uint32_t)lane == j) {
                        p_mn = lo;
                        p_R = R;
                        p_idx = j;
                    }
                        mn_pair = lo;
                    inv_pair = inv;
                }
                quantize(ct, mn_pair, inv_pair);
            });
        } else {
            // ---- the strip lies in one group, which k warps share
            const uint32_t k = (1u << log2G) / STRIP;
            float lo, hi;
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
            if (k > 1u) {
                // exchange the strips' extremes (and the wish to stop, so that the k warps leave together and nobody is
                // left at the barrier)
                const uint32_t buf = it & 1u, first = (uint32_t)warp & ~(k - 1u);
                if (lane == 0) {
                    s_ext[buf][warp][0] = lo;
                    s_ext[buf][warp][1] = hi;
                    s_stop[buf][warp] = stop;
                }
                named_bar_sync(1u + first / k, 32u * k);
                for (uint32_t j = 0; j < k; j++) {
                    lo = fmin2(lo, s_ext[buf][first + j][0]);
                    hi = fmax2(hi, s_ext[buf][first + j][1]);
                    stop |= s_stop[buf][first + j];
                }
            }
            float R;
            const float inv = inverse_scale<B>(lo, hi, R);
            // the group's first warp parks it (in lane 0) and stores its metadata
            if ((WHOLE || strip0 < n_elems) && lane == 0 && ((uint32_t)warp & (k - 1u)) == 0u) {
                p_mn = lo;
                p_R = R;
                p_idx = 0u;
            }
            for_chunks([&](auto ct) { quantize(ct, lo, inv); });
        }

        // ---- the strip's metadata and its part of the test that the window ends with one width
        {
            constexpr float Lf = (float)((1u << B) - 1u);
            const bool on = p_idx != 0xFFFFFFFFu, pos = p_R > 0.0f;
            const float scale = pos ? __fdiv_rn(p_R, Lf) : 0.0f;  // (lanes without a group divide zero)
            // importance keys of the last raise taken and of the first raise not taken (Sec. 3.4.1)
            uint32_t kmin = on ? __float_as_uint(__fmul_rn(p_R, a.stream_v_lo)) : 0xFFFFFFFFu;
            uint32_t kmax = on ? __float_as_uint(__fmul_rn(p_R, a.stream_v_hi)) : 0u;
            if (on) {
                bits_p[p_idx] = (uint8_t)B;
                mn_p[p_idx] = p_mn;
                scale_p[p_idx] = scale;
            }
            kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
            kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
            // 1/scale = L / R is not a normal number when R passes about 2^126: the codes may then need the clamp, which
            // this kernel does not have.  (Any range above 2^125 is sent to the general kernel: sooner than needed is fine.)
            bool give_up = __any_sync(0xFFFFFFFFu, p_R > 0x1p125f);
            if (lane == 0) {
                if (a.full_test != 0u) {
                    // every raise below level ell must sort ahead of every raise from level ell upward: the window's
                    // word gathers the smallest key of the former (complemented) and the largest of the latter, for the
                    // kernel that runs behind this one; keys of this strip alone that do not separate settle the matter
                    unsigned int *const word = reinterpret_cast<unsigned int *>(a.flags + gw);
                    atomicMax(word, ~kmin);
                    atomicMax(word + 1, kmax);
                    give_up |= kmin < kmax;
                }
                if (give_up) atomicExch(&a.hdr->retry, 1u);       // the general kernel redoes the call
            }
        }
    };

    for (uint32_t gw = blockIdx.x; gw < a.total_windows; gw += gridDim.x, it++) {
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
        uint32_t n_elems = WE;                                    // a ragged last window has fewer (whole groups)
        if (w + 1u == td.n_windows) n_elems = (uint32_t)(td.numel - (uint64_t)w * WE);
        if (n_elems == WE) strip(std::true_type{}, td, gw, w, n_elems);
        else strip(std::false_type{}, td, gw, w, n_elems);
        if (stop != 0u) break;                                    // (the same decision in all warps that share a group)
    }
}

template <typename T, int CHUNKS, int B, int GC, bool BATCH, int ACT>
static cudaError_t launch_stream(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    int ctas = 0;
    const cudaError_t e = persistent_ctas(reinterpret_cast<const void *>(&stream_compress_kernel<T, CHUNKS, B, GC, BATCH, ACT>),
                                          kThreads, 0, &ctas);
    if (e != cudaSuccess) return e;
    // eight times the CTAs the device holds at once: no CTA waits for another here, and with several waves the block
    // scheduler evens out the CTAs' finishing times (measured on 2^30 elements: 0.839 ms at 1x, 0.824 at 2x, 0.815 at 4x,
    // 0.814 at 8x, 0.818 at 16x, 0.831 at 32x, 0.926 with one CTA per window)
    const uint32_t want = (uint32_t)ctas * 8u;
    const uint32_t grid = args.total_windows < want ? args.total_windows : want;
    stream_compress_kernel<T, CHUNKS, B, GC, BATCH, ACT><<<grid, kThreads, 0, stream>>>(args);
    return cudaGetLastError();
}

template <typename T, int CHUNKS, bool BATCH, int ACT>
static cudaError_t launch_stream_c(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    const uint32_t strip = 256u * CHUNKS;
    const int gc = args.G < 128u ? 0 : args.G == 128u ? 3 : args.G < strip ? 1 : 2;
#define DAF_CASE(BB)                                                                                                 \
    case BB:                                                                                                         \
        if (gc == 0) return launch_stream<T, CHUNKS, BB, 0, BATCH, ACT>(args, stream);                              \
        if (gc == 3) return launch_stream<T, CHUNKS, BB, 3, BATCH, ACT>(args, stream);                              \
        if constexpr (CHUNKS > 1) { if (gc == 1) return launch_stream<T, CHUNKS, BB, 1, BATCH, ACT>(args, stream); } \
        return launch_stream<T, CHUNKS, BB, 2, BATCH, ACT>(args, stream);
    switch (args.S[args.full_ell]) {
        DAF_CASE(1)
        DAF_CASE(2)
        DAF_CASE(4)
    default:
        DAF_CASE(8)
    }
#undef DAF_CASE
}

// Launch for element type T: strip length from the window size, GC from the group size, B = the
// width every whole window ends with.
template <typename T, bool BATCH, int ACT>
cudaError_t dispatch_stream_t(uint32_t chunks, const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    if constexpr (ACT != kActNone) {                              // fused producer: single tensor, default window
        return launch_stream_c<T, 4, false, ACT>(args, stream);
    } else {
        if (chunks == 1) return launch_stream_c<T, 1, BATCH, kActNone>(args, stream);
        if (chunks == 2) return launch_stream_c<T, 2, BATCH, kActNone>(args, stream);
        return launch_stream_c<T, 4, BATCH, kActNone>(args, stream);
    }
}

#define DAF_INSTANTIATE_STREAM(T)                                                                                          \
    template cudaError_t dispatch_stream_t<T, false, kActNone>(uint32_t, const CompressArgs<1> &, cudaStream_t);              \
    template cudaError_t dispatch_stream_t<T, true, kActNone>(uint32_t, const CompressArgs<DAF_BATCH_MAX> &, cudaStream_t);   \
    template cudaError_t dispatch_stream_t<T, false, kActRelu>(uint32_t, const CompressArgs<1> &, cudaStream_t);              \
    template cudaError_t dispatch_stream_t<T, false, kActRelu6>(uint32_t, const CompressArgs<1> &, cudaStream_t);             \
    template cudaError_t dispatch_stream_t<T, false, kActGelu>(uint32_t, const CompressArgs<1> &, cudaStream_t);

}  // namespace daf
