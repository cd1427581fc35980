// Streaming compress kernel for calls whose windows all end with one width (the common case:
// a budget that one allowed width meets exactly, ranges within a window close enough that no
// raise of a higher level sorts ahead of one of a lower level, Sec. 3.4.1 of the paper).
//
// One persistent CTA of 32 warps per multiprocessor takes windows blockIdx.x, blockIdx.x +
// gridDim.x, ...; its warps have two roles and never meet at a CTA-wide barrier:
//
//   stats warps (NS of them) run ahead.  Per window each reads its share of the 256-element
//     chunks (32 bytes per lane and load, four loads in flight), reduces them to per-group
//     min / max (3-input min/max, warp redux or segmented shuffles) and leaves these in the
//     window's slot of a small ring in shared memory.  The warp that finishes a window last
//     does the per-group arithmetic for all its groups, one group per lane: range, importance
//     keys, 1/scale and scale by IEEE division, group records into the slot, metadata to global
//     memory, and the test that the window really ends with one width.  Then it completes the
//     slot's "full" barrier.  They also ask for the window two ahead to be brought into L2
//     (one bulk prefetch per warp), so that HBM latency is paid long before anybody waits.
//   quantize warps take the CTA's chunks round-robin.  A chunk's 8 elements per lane come from
//     L1 / L2 (the stats warps had them a moment ago), the group record from the slot; then
//     Eq. 1 with stochastic rounding (Philox4x32-10, the float -> uint step by the power-of-two
//     offset of Eq. 5), lane-local LSB-first packing, one coalesced store.  Every chunk done
//     counts on the slot's "empty" barrier, which frees the slot for the stats warps.
//
// With every window of one width B, the packed position of a code follows from its index, so
// nothing here depends on another CTA.  If a window fails the test (or a group needs the clamped
// quantizer, or a ragged last window has a budget that asks for another width), the kernel raises
// hdr->retry and stops; the general kernel, enqueued behind it, then redoes the call.
//
// The kernel is a template over the element type, the window size, the width B, batched calls
// and the fused ReLU; this header is included by one translation unit per element type.
#pragma once
#include "compress_shared.cuh"

namespace daf {

namespace stream {

constexpr int kWarpsPerCta = 32, kCtaThreads = 32 * kWarpsPerCta;
constexpr int kSlots = 4;                                         // windows between the stats warps and the slowest quantize warp
constexpr int kMaxUnits = 512;                                    // per window: 256-element chunks, or groups when they are smaller

struct Slot {
    uint64_t full;            // mbarrier: the window's records are complete (one arrival)
    uint64_t empty;           // mbarrier: every chunk of the window has been quantized (one arrival per chunk)
    const char *src;          // the window's first element
    unsigned char *out;       // the window's first packed byte
    char *act;                // fused ReLU: where the window's activation goes
    uint64_t blk;             // Philox block of the window's first element
    uint32_t n_elems;         // elements of the window (a ragged last window has fewer)
    uint32_t done;            // stats warps that have finished the window
    uint32_t pad[2];
    uint32_t rkeys[20];       // Philox round keys of the window's tensor (batched calls)
    float umn[kMaxUnits], umx[kMaxUnits];
    float2 rec[kMaxUnits];    // per group: min, 1/scale
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool bar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cta.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok)
                 : "r"(smem_u32(bar)), "r"(parity)
                 : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint32_t ld_volatile_shared(const uint32_t *p)
{
    return *reinterpret_cast<const volatile uint32_t *>(p);
}
__device__ __forceinline__ void st_volatile_shared(uint32_t *p, uint32_t v)
{
    *reinterpret_cast<volatile uint32_t *>(p) = v;
}
__device__ __forceinline__ uint32_t ld_relaxed_u32(const unsigned int *p)
{
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
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

}  // namespace stream

template <typename T, int WE, int B, int NS, bool BATCH, bool RELU>
__global__ void __launch_bounds__(stream::kCtaThreads, 1)
stream_compress_kernel(const __grid_constant__ CompressArgs<BATCH ? DAF_BATCH_MAX : 1> a)
{
    using namespace stream;
    constexpr uint32_t CPW = WE / 256u;                           // chunks per window
    constexpr uint32_t NQ = kWarpsPerCta - NS;                    // quantize warps
    constexpr uint32_t SHARE = CPW / NS;                          // chunks of a window per stats warp
    constexpr uint32_t EB = Elem<T>::kBytes;
    constexpr uint32_t WBYTES = (WE >> 3) * B;                    // packed bytes of a whole window
    static_assert(CPW % NS == 0 && SHARE >= 1, "the stats warps share a window's chunks evenly");
    constexpr int BATCHED = SHARE < 4 ? (int)SHARE : 4;           // loads a stats warp keeps in flight

    __shared__ __align__(16) Slot s_slot[kSlots];
    __shared__ uint32_t s_abort;                                  // this CTA stops: the call is redone (or a wait ran out)
    __shared__ uint32_t s_first[BATCH ? DAF_BATCH_MAX : 1];       // first window of every tensor

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid < kSlots) {
        bar_init(&s_slot[tid].full, 1u);
        bar_init(&s_slot[tid].empty, CPW);
        s_slot[tid].done = 0u;
    }
    if (tid == 0) {
        s_abort = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (BATCH) {
        for (uint32_t i = tid; i < DAF_BATCH_MAX; i += kCtaThreads) s_first[i] = i < a.n_tensors ? a.t[i].first_window : 0xFFFFFFFFu;
    }
    __syncthreads();

    const uint32_t log2G = a.log2G;
    auto tensor_index = [&](uint32_t gw) -> uint32_t {
        if (!BATCH) return 0u;
        const uint32_t n0 = __popc(__ballot_sync(0xFFFFFFFFu, s_first[lane] <= gw));
        const uint32_t n1 = __popc(__ballot_sync(0xFFFFFFFFu, s_first[lane + 32] <= gw));
        return n0 + n1 - 1u;
    };
    auto give_up = [&]() {                                        // the general kernel redoes the call
        atomicExch(&a.hdr->retry, 1u);
        st_volatile_shared(&s_abort, 1u);
    };
    // Bounded wait on one of the slots' barriers; false: stop (another warp gave up, or the wait ran out).
    auto wait = [&](uint64_t *bar, uint32_t parity, uint32_t gw, uint32_t site) -> bool {
        for (unsigned polls = 0;; polls++) {
            if (bar_try_wait(bar, parity)) return true;
            if (ld_volatile_shared(&s_abort) != 0u) return false;
            if (polls > a.poll_limit) {
                if (lane == 0 && atomicCAS(&a.hdr->status, 0u, (unsigned)DAF_ERR_TIMEOUT) == 0u) {
                    a.hdr->fail_window = gw;
                    a.hdr->fail_site = site;
                }
                st_volatile_shared(&s_abort, 1u);
                return false;
            }
        }
    };

    if (warp < NS) {
        // ============================================================ stats warps
        uint32_t retry_seen = 0u;
        for (uint32_t it = 0;; it++) {
            const uint32_t gw = blockIdx.x + it * gridDim.x;
            if (gw >= a.total_windows) break;
            if ((retry_seen | ld_volatile_shared(&s_abort)) != 0u) {
                st_volatile_shared(&s_abort, 1u);                 // the quantize warps stop waiting for this window
                break;
            }
            retry_seen = ld_relaxed_u32(&a.hdr->retry);           // consumed one window later
            Slot &sl = s_slot[it % kSlots];
            const uint32_t use = it / kSlots;
            const uint32_t ti = tensor_index(gw);
            const TensorDesc &td = a.t[ti];
            const uint32_t w = BATCH ? gw - td.first_window : gw;
            uint32_t n_elems = WE;
            if (w + 1u == td.n_windows) n_elems = (uint32_t)(td.numel - (uint64_t)w * WE);
            const char *const src = reinterpret_cast<const char *>(td.in) + (uint64_t)w * (WE * EB);

            // ---- the window two ahead is requested into L2 now (this warp's share of it)
            {
                const uint32_t gw_p = gw + 2u * gridDim.x;
                if (gw_p < a.total_windows) {
                    const TensorDesc &tp = a.t[tensor_index(gw_p)];
                    const uint64_t at = (uint64_t)(BATCH ? gw_p - tp.first_window : gw_p) * WE + (uint32_t)warp * (SHARE * 256u);
                    if (lane == 0 && at < tp.numel) {
                        const uint64_t left = (tp.numel - at) * EB;
                        const uint32_t bytes = left < SHARE * 256u * EB ? (uint32_t)left : SHARE * 256u * EB;
                        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(reinterpret_cast<const char *>(tp.in) + at * EB),
                                     "r"(bytes & ~15u));
                    }
                }
            }
            // ---- the slot must have been drained by the quantize warps
            if (use > 0u && !wait(&sl.empty, (use - 1u) & 1u, gw, 8u)) break;

            // ---- this warp's chunks: per-unit min / max into the slot
            const uint32_t c0 = (uint32_t)warp * SHARE;
#pragma unroll 1
            for (uint32_t cb = 0; cb < SHARE; cb += BATCHED) {
                float x[BATCHED][8];
#pragma unroll
                for (int j = 0; j < BATCHED; j++) {
                    const uint32_t e = (c0 + cb + j) * 256u + (uint32_t)lane * 8u;
                    if (e < n_elems) {
                        Elem<T>::load8_keep(src + (size_t)e * EB, x[j]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; i++) x[j][i] = 0.0f;
                    }
                }
#pragma unroll
                for (int j = 0; j < BATCHED; j++) {
                    if (RELU) {
#pragma unroll
                        for (int i = 0; i < 8; i++) x[j][i] = fmaxf(x[j][i], 0.0f);
                    }
                    float lo, hi;
                    extremes8(x[j], lo, hi);
                    const uint32_t c = c0 + cb + j;
                    if (log2G >= 8u) {
                        lo = warp_min(lo);
                        hi = warp_max(hi);
                        if (lane == 0) {
                            sl.umn[c] = lo;
                            sl.umx[c] = hi;
                        }
                    } else {
                        const uint32_t lpu = 1u << (log2G - 3u);  // lanes per group
                        for (uint32_t off = 1; off < lpu; off <<= 1) {
                            lo = fmin2(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, off));
                            hi = fmax2(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, off));
                        }
                        if (((uint32_t)lane & (lpu - 1u)) == 0u) {
                            const uint32_t u = (c << (8u - log2G)) + ((uint32_t)lane >> (log2G - 3u));
                            sl.umn[u] = lo;
                            sl.umx[u] = hi;
                        }
                    }
                }
            }
            // ---- the warp that finishes the window last settles its groups
            __syncwarp();
            uint32_t last = 0u;
            if (lane == 0) {
                __threadfence_block();
                last = atomicAdd(&sl.done, 1u) + 1u == (uint32_t)NS;
                __threadfence_block();
            }
            last = __shfl_sync(0xFFFFFFFFu, last, 0);
            if (last == 0u) continue;

            const uint32_t n = n_elems >> log2G;                  // groups of the window
            bool ok = true;
            if (n_elems != WE) {
                // ragged last window: its own budget arithmetic must ask for the same single width
                const uint32_t rem = (uint32_t)((((uint64_t)a.beta_q8 * n) >> 8) - (uint64_t)a.S[0] * n);
                uint32_t ell = 0;
                while (ell + 1 < a.m && (a.S[ell + 1] - a.S[0]) * n <= rem) ell++;
                const uint32_t rem_after = rem - (a.S[ell] - a.S[0]) * n;
                const bool all_max = ell + 1 == a.m;
                ok = ell == a.full_ell && (all_max || rem_after < a.cost[ell]);
            }
            const float Lf = (float)((1u << B) - 1u);
            const float v_lo = a.v[a.full_ell > 0u ? a.full_ell - 1u : 0u], v_hi = a.v[a.full_ell];
            const uint32_t cpg = log2G > 8u ? 1u << (log2G - 8u) : 1u;   // units per group
            const uint64_t g0 = (uint64_t)w * (WE >> log2G);      // first group of the window in the tensor
            uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
            bool slow = false;
            for (uint32_t g = lane; g < n; g += 32u) {
                float lo = sl.umn[g * cpg], hi = sl.umx[g * cpg];
                for (uint32_t j = 1; j < cpg; j++) {
                    lo = fmin2(lo, sl.umn[g * cpg + j]);
                    hi = fmax2(hi, sl.umx[g * cpg + j]);
                }
                float R = __fsub_rn(hi, lo);
                if (R < 0x1p-118f) R = 0.0f;                      // degenerate group: constant
                kmin = min(kmin, __float_as_uint(__fmul_rn(R, v_lo)));
                kmax = max(kmax, __float_as_uint(__fmul_rn(R, v_hi)));
                const float inv = R > 0.0f ? __fdiv_rn(Lf, R) : 0.0f;
                const float scale = R > 0.0f ? __fdiv_rn(R, Lf) : 0.0f;
                // 1/scale not a normal number: the codes may need the clamp, which this kernel does not have
                slow |= R > 0.0f && inv < 0x1p-126f;
                sl.rec[g] = make_float2(lo, inv);
                td.bits[g0 + g] = (uint8_t)B;
                td.mn[g0 + g] = lo;
                td.scale[g0 + g] = scale;
            }
            if (a.full_test != 0u) {
                // every raise below level ell must sort ahead of every raise from level ell upward
                kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
                kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
                ok = ok && kmin >= kmax;
            }
            ok = ok && !__any_sync(0xFFFFFFFFu, slow);
            if (lane < 10 && BATCH) philox_store_round_keys(sl.rkeys, td.seed, lane);
            if (lane == 0) {
                if (!ok) give_up();
                sl.src = src;
                sl.out = td.packed + (uint64_t)w * WBYTES;
                sl.act = RELU ? reinterpret_cast<char *>(td.act) + (uint64_t)w * (WE * EB) : nullptr;
                sl.blk = (td.elem_base >> 3) + (uint64_t)w * (WE >> 3);
                sl.n_elems = n_elems;
                sl.done = 0u;
                td.woff[w] = (uint64_t)w * WBYTES;
                if (w + 1u == td.n_windows) td.woff[w + 1u] = (uint64_t)w * WBYTES + (uint64_t)(n_elems >> 3) * B;
            }
            __syncwarp();
            if (lane == 0) bar_arrive(&sl.full);                  // (release: the slot's contents are visible to who sees the phase)
        }
        return;
    }

    // ================================================================ quantize warps
    uint32_t cur_it = 0xFFFFFFFFu;
    const char *src = nullptr;
    unsigned char *out = nullptr;
    char *act = nullptr;
    uint64_t blk0 = 0;
    uint32_t n_elems = 0;
    for (uint32_t nseq = (uint32_t)warp - NS;; nseq += NQ) {
        const uint32_t it = nseq / CPW, c = nseq % CPW;
        const uint32_t gw = blockIdx.x + it * gridDim.x;
        if (gw >= a.total_windows) break;
        Slot &sl = s_slot[it % kSlots];
        if (it != cur_it) {
            if (!wait(&sl.full, (it / kSlots) & 1u, gw, 9u)) break;
            cur_it = it;
            src = sl.src;
            out = sl.out;
            act = sl.act;
            blk0 = sl.blk;
            n_elems = sl.n_elems;
        }
        const uint32_t e = c * 256u + (uint32_t)lane * 8u;
        const bool on = e < n_elems;
        float x[8];
        if (on) {
            Elem<T>::load8(src + (size_t)e * EB, x);
        } else {
#pragma unroll
            for (int i = 0; i < 8; i++) x[i] = 0.0f;
        }
        const float2 rec = sl.rec[on ? e >> log2G : 0u];
        uint32_t o[4], w0, w1;
        const uint64_t blk = blk0 + (e >> 3);
        if (BATCH) {
            const PhiloxSharedKeys sk{reinterpret_cast<const uint4 *>(sl.rkeys)};
            philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), sk, o);
        } else {
            philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), a.keys, o);
        }
        if (RELU) {
            // fused producer: what is compressed (and written out) is max(x, +0); the lane stores what it loaded, so
            // the output may be the input buffer (the stats warps are done with this window)
#pragma unroll
            for (int i = 0; i < 8; i++) x[i] = fmaxf(x[i], 0.0f);
            if (on) Elem<T>::store8(act + (size_t)e * EB, x);
        }
        quantize8<B, false>(x, rec.x, rec.y, o, w0, w1);
        if (on) store_packed<B>(out + (size_t)(e >> 3) * B, w0, w1);
        __syncwarp();                                             // every lane has read its record
        if (lane == 0) bar_arrive(&sl.empty);
    }
}

template <typename T, int WE, int B, int NS, bool BATCH, bool RELU>
static cudaError_t launch_stream(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    int ctas = 0;
    const cudaError_t e = persistent_ctas(reinterpret_cast<const void *>(&stream_compress_kernel<T, WE, B, NS, BATCH, RELU>),
                                          stream::kCtaThreads, 0, &ctas);
    if (e != cudaSuccess) return e;
    const uint32_t grid = args.total_windows < (uint32_t)ctas ? args.total_windows : (uint32_t)ctas;
    stream_compress_kernel<T, WE, B, NS, BATCH, RELU><<<grid, stream::kCtaThreads, 0, stream>>>(args);
    return cudaGetLastError();
}

template <typename T, int WE, bool BATCH, bool RELU>
static cudaError_t launch_stream_w(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    // groups below 256 elements cost the stats warps segmented shuffles and more groups to settle: eight of them
    const bool many = args.G < 256u;
#define DAF_CASE(BB)                                                                              \
    case BB:                                                                                      \
        return many ? launch_stream<T, WE, BB, 8, BATCH, RELU>(args, stream)                      \
                    : launch_stream<T, WE, BB, 4, BATCH, RELU>(args, stream);
    switch (args.S[args.full_ell]) {
        DAF_CASE(1)
        DAF_CASE(2)
        DAF_CASE(4)
    default:
        DAF_CASE(8)
    }
#undef DAF_CASE
}

// Launch for element type T: window size from the plan's chunk count, B = the width every whole window ends with.
template <typename T, bool BATCH, bool RELU>
cudaError_t dispatch_stream_t(uint32_t chunks, const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    if constexpr (RELU) {                                         // fused producer: single tensor, default window
        return launch_stream_w<T, 16384, false, true>(args, stream);
    } else {
        if (chunks == 1) return launch_stream_w<T, 4096, BATCH, false>(args, stream);
        if (chunks == 2) return launch_stream_w<T, 8192, BATCH, false>(args, stream);
        return launch_stream_w<T, 16384, BATCH, false>(args, stream);
    }
}

#define DAF_INSTANTIATE_STREAM(T)                                                                                          \
    template cudaError_t dispatch_stream_t<T, false, false>(uint32_t, const CompressArgs<1> &, cudaStream_t);              \
    template cudaError_t dispatch_stream_t<T, true, false>(uint32_t, const CompressArgs<DAF_BATCH_MAX> &, cudaStream_t);   \
    template cudaError_t dispatch_stream_t<T, false, true>(uint32_t, const CompressArgs<1> &, cudaStream_t);

}  // namespace daf
