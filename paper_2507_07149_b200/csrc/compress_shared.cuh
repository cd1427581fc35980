// Argument structures and the lane-local quantize-and-pack routines shared by the compress kernels
// (the streaming kernel for windows of one width and the window-synchronous general kernel).
#pragma once
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
    void *act;               // fused producer (daf_relu_compress): where the activation itself goes
};

constexpr int kGeneralSelWords = 180;                         // shared words of the general kernel's bit choice with more than 64 groups

struct SmemLayout {          // byte offsets into the general kernel's dynamic shared memory
    uint32_t out0, out_stride, umn, umx, sel, grp, total;
};

template <int NT> struct CompressArgs {
    WorkspaceHeader *hdr;
    uint64_t *flags;          // per window: key extremes gathered by the streaming kernel
    uint64_t *flags2;         // per window: look-back descriptor of the general kernel
    uint32_t gated;           // the general kernel runs only if the streaming one (or its verifier) asked for it
    uint32_t poll_limit;      // polls after which a bounded wait gives up
    uint32_t total_windows, n_tensors;
    uint32_t G, log2G, beta_q8, m, nearest, bulk_store, n_max;
    uint32_t full_ell, full_rem, full_rem_after;   // budget arithmetic of a full window (n_max groups)
    uint32_t full_test;       // ... whose groups share a width only if the keys of the levels around full_ell separate
    float stream_v_lo, stream_v_hi;   // importance factors of the raise into level full_ell and of the raise out of it
    uint32_t S[kMaxLevels], cost[kMaxLevels];
    float v[kMaxLevels];
    SmemLayout lay;
    PhiloxKeys keys;          // round keys of tensor 0 (single-tensor launches)
    TensorDesc t[NT];
    // two-width streaming kernel: groups of a full window that are raised above level full_ell; the two widths, their
    // largest codes as floats, bytes of a group at the lower width and what the raise adds, bytes of a whole window
    uint32_t tw_k, tw_blo, tw_bhi, tw_size_lo, tw_size_up;
    float tw_lf_lo, tw_lf_hi;
    float tw_v_my, tw_v_lo, tw_v_hi;   // importance factors of the raise out of level full_ell, into it, and of the next one
    uint32_t tw_test_lo, tw_test_hi;   // ... the latter two exist
    uint64_t tw_wbytes;
};

// ------------------------------------------------------------------------------------------
// Bulk asynchronous copies (TMA, non-tensor form) and the mbarrier that signals a landed
// window.  All waits are bounded.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_addr(dst_smem)),
                 "l"(src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}
__device__ __forceinline__ void bulk_store(void *dst, const void *src_smem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_addr(src_smem)), "r"(bytes)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void bulk_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Orders this thread's earlier writes to shared memory before later reads by the async proxy.
__device__ __forceinline__ void fence_async_shared() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok)
                 : "r"(smem_addr(bar)), "r"(parity)
                 : "memory");
    return ok != 0;
}
// Returns false if the copy did not land within the poll budget (try_wait itself blocks for a
// hardware-defined interval, so the loop turns slowly).
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity, unsigned limit)
{
    for (unsigned polls = 0; polls < limit; polls++)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// Eight consecutive elements of a lane from the staged window (two 16-byte shared loads for
// 4-byte elements, one for 2-byte elements).
template <typename T> __device__ __forceinline__ void load8_staged(const unsigned char *chunk, int lane, float (&x)[8]);

template <> __device__ __forceinline__ void load8_staged<float>(const unsigned char *chunk, int lane, float (&x)[8])
{
    // a lane owns 32 bytes; which half it reads first depends on the lane, so that each
    // quarter-warp touches all 32 banks
    const int odd = (lane >> 2) & 1;
    const float4 a = *reinterpret_cast<const float4 *>(chunk + lane * 32 + 16 * odd);
    const float4 b = *reinterpret_cast<const float4 *>(chunk + lane * 32 + 16 * (odd ^ 1));
    x[0] = odd ? b.x : a.x; x[1] = odd ? b.y : a.y; x[2] = odd ? b.z : a.z; x[3] = odd ? b.w : a.w;
    x[4] = odd ? a.x : b.x; x[5] = odd ? a.y : b.y; x[6] = odd ? a.z : b.z; x[7] = odd ? a.w : b.w;
}
template <> __device__ __forceinline__ void load8_staged<__half>(const unsigned char *chunk, int lane, float (&x)[8])
{
    const uint4 v = *reinterpret_cast<const uint4 *>(chunk + lane * 16);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
        x[2 * i] = f.x;
        x[2 * i + 1] = f.y;
    }
}
template <> __device__ __forceinline__ void load8_staged<__nv_bfloat16>(const unsigned char *chunk, int lane, float (&x)[8])
{
    const uint4 v = *reinterpret_cast<const uint4 *>(chunk + lane * 16);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; i++) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

// ------------------------------------------------------------------------------------------
// Decoupled look-back over the window descriptors, executed by one full warp.  Each round
// inspects DEPTH * 32 predecessors with all loads in flight at once.  Returns 1 when the
// exclusive prefix was found (*excl), 0 when a needed descriptor is still empty and `block`
// is false, -1 on a poisoned predecessor, -2 when the bounded wait ran out.
// ------------------------------------------------------------------------------------------
constexpr int kLookDepth = 4;                                 // measured: 2 is 5 % slower with groups of 1024 elements, 8 is 13 % slower everywhere

template <int DEPTH>
__device__ __forceinline__ int lookback(const uint64_t *flags, uint32_t gw, uint32_t first, int lane, bool block,
                                        unsigned limit, uint64_t *excl_out)
{
    uint64_t excl = 0;
    int64_t idx = (int64_t)gw - 1 - lane;                         // lane's nearest predecessor of this round
    unsigned polls = 0;
    for (;;) {
        uint64_t f[DEPTH];
        bool done = false;                                        // a prefix (or poison) ends the walk in this round
        for (;;) {
#pragma unroll
            for (int j = 0; j < DEPTH; j++) {
                const int64_t i = idx - 32 * j;
                f[j] = (i >= (int64_t)first) ? ld_relaxed_u64(flags + i) : (kFlagPrefix << kFlagShift);
            }
            bool ready = true;                                    // walk the chunks from the nearest predecessor outward
            done = false;
#pragma unroll
            for (int j = 0; j < DEPTH; j++) {
                if (!done && ready) {
                    const uint32_t st = (uint32_t)(f[j] >> kFlagShift);
                    const unsigned stop_mask = __ballot_sync(0xFFFFFFFFu, st == kFlagPrefix || st == kFlagPoison);
                    const unsigned empty_mask = __ballot_sync(0xFFFFFFFFu, st == kFlagEmpty);
                    const unsigned upto = stop_mask ? ((2u << (__ffs(stop_mask) - 1)) - 1u) : 0xFFFFFFFFu;
                    if (empty_mask & upto) ready = false;
                    else if (stop_mask) done = true;
                }
            }
            if (ready) break;
            if (!block) return 0;
            if (++polls > limit) return -2;
            __nanosleep(64);
        }
        // accumulate up to and including the first prefix; a poisoned predecessor fails the window
        uint64_t v = 0;
        bool stop = false, bad = false;
#pragma unroll
        for (int j = 0; j < DEPTH; j++) {
            if (!stop) {
                const uint32_t st = (uint32_t)(f[j] >> kFlagShift);
                const unsigned stop_mask = __ballot_sync(0xFFFFFFFFu, st == kFlagPrefix || st == kFlagPoison);
                const unsigned upto = stop_mask ? ((2u << (__ffs(stop_mask) - 1)) - 1u) : 0xFFFFFFFFu;
                if (__ballot_sync(0xFFFFFFFFu, st == kFlagPoison) & upto) bad = true;
                if ((upto >> lane) & 1u) v += f[j] & kFlagValueMask;
                if (stop_mask) stop = true;
            }
        }
        if (bad) return -1;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
        excl += v;
        if (done) break;
        idx -= 32 * DEPTH;
    }
    *excl_out = excl;
    return 1;
}

// The streaming kernel for calls whose windows all end with one width (compress_stream.cuh; one
// translation unit per element type).
template <typename T, bool BATCH, int ACT>
cudaError_t dispatch_stream_t(uint32_t chunks, const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream);

// The streaming kernel for calls whose windows end with two neighbouring widths (compress_twowidth.cuh; one translation
// unit per element type).
template <typename T, bool BATCH>
cudaError_t dispatch_two_width_t(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream);

template <bool BATCH>
inline cudaError_t dispatch_two_width(uint32_t dtype, const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    if (dtype == DAF_F32) return dispatch_two_width_t<float, BATCH>(args, stream);
    if (dtype == DAF_F16) return dispatch_two_width_t<__half, BATCH>(args, stream);
    return dispatch_two_width_t<__nv_bfloat16, BATCH>(args, stream);
}

// The two-pass kernels for windows of mixed widths (compress_twopass.cuh; one translation unit per element type).
template <typename T, bool BATCH>
cudaError_t dispatch_twopass_t(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream);

template <bool BATCH>
inline cudaError_t dispatch_twopass(uint32_t dtype, const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    if (dtype == DAF_F32) return dispatch_twopass_t<float, BATCH>(args, stream);
    if (dtype == DAF_F16) return dispatch_twopass_t<__half, BATCH>(args, stream);
    return dispatch_twopass_t<__nv_bfloat16, BATCH>(args, stream);
}

// The general kernel: any mix of widths within a window (compress_general.cuh; one translation unit per element type).
template <typename T, bool BATCH, int ACT>
cudaError_t dispatch_general_t(uint32_t chunks, const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream);

template <bool BATCH, int ACT>
inline cudaError_t dispatch_general(uint32_t dtype, uint32_t chunks, const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args,
                                    cudaStream_t stream)
{
    if (dtype == DAF_F32) return dispatch_general_t<float, BATCH, ACT>(chunks, args, stream);
    if (dtype == DAF_F16) return dispatch_general_t<__half, BATCH, ACT>(chunks, args, stream);
    return dispatch_general_t<__nv_bfloat16, BATCH, ACT>(chunks, args, stream);
}

template <bool BATCH, int ACT>
inline cudaError_t dispatch_stream(uint32_t dtype, uint32_t chunks, const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args,
                                   cudaStream_t stream)
{
    if (dtype == DAF_F32) return dispatch_stream_t<float, BATCH, ACT>(chunks, args, stream);
    if (dtype == DAF_F16) return dispatch_stream_t<__half, BATCH, ACT>(chunks, args, stream);
    return dispatch_stream_t<__nv_bfloat16, BATCH, ACT>(chunks, args, stream);
}

struct GroupRec {             // what the quantize pass needs per group (one 16-byte shared load)
    float mn, inv;
    uint32_t b, off;
};

// ------------------------------------------------------------------------------------------
// Eight codes of width B from eight values; o[] holds eight 16-bit random lanes (two per word).
// s = fma(x - mn, inv, 256) lies in [256, 512) where one ulp is 2^-15, so its mantissa field
// is the fixed-point quotient; adding a 15-bit random offset r15 and dropping 15 bits rounds
// stochastically (r15 = 2^14: round half up).  With h = 2*r15 + (one more random bit),
// (fixed + r15) >> 15 == (2*bits(s) + h - 2*bits(256)) >> 16, which needs one add, one shift
// and one fused subtract-and-clamp per element.
// ------------------------------------------------------------------------------------------
// t[i] = 2 * bits(s_i) + h_i (mod 2^32): bits 16 .. 31 of t[i], less 0x8700, are code i before any clamp.
__device__ __forceinline__ void noisy_sums8(const float (&x)[8], float mn, float inv, const uint32_t (&o)[4], uint32_t (&t)[8])
{
#pragma unroll
    for (int i = 0; i < 8; i++) {
        const float d = __fsub_rn(x[i], mn);
        const float s = __fmaf_rn(d, inv, 256.0f);
        const uint32_t h = (i & 1) ? (o[i >> 1] >> 16) : (o[i >> 1] & 0xFFFFu);
        t[i] = __float_as_uint(s) * 2u + h;                       // mod 2^32; 2*bits(256) = 0x87000000
    }
}

// The eight codes of width B out of t[], packed LSB first into w0 (and w1 for B = 8).
template <int B, bool CLAMP>
__device__ __forceinline__ void close_codes8(const uint32_t (&t)[8], uint32_t &w0, uint32_t &w1)
{
    constexpr uint32_t L = (1u << B) - 1u;
    if (CLAMP) {
        w0 = 0u;
        w1 = 0u;
#pragma unroll
        for (int i = 0; i < 8; i++) {
            const int pos = (B * i) & 31;                         // bit position of code i in its word (unrolled: constant)
            const uint32_t field = min((t[i] >> 16) - 0x8700u, L) << pos;
            if (B == 8 && i >= 4) w1 |= field;
            else w0 |= field;
        }
    } else {
        // The code never exceeds L when 1/scale is a normal number, so byte 2 of t is the code
        // itself (bits 16+B .. 23 are zero).  Byte permutes gather the eight code bytes; widths
        // below 8 then close the gaps: 4-bit codes by interleaving two words of nibbles, 2- and
        // 1-bit codes by a multiplication that lines the four fields of a word up in its top byte.
        if (B == 4) {
            // bytes (c0, c2, c4, c6) and (c1, c3, c5, c7): the odd codes become the high nibbles
            const uint32_t ev = __byte_perm(__byte_perm(t[0], t[2], 0x0062), __byte_perm(t[4], t[6], 0x0062), 0x5410);
            const uint32_t od = __byte_perm(__byte_perm(t[1], t[3], 0x0062), __byte_perm(t[5], t[7], 0x0062), 0x5410);
            w0 = od * 16u + ev;
            w1 = 0u;
        } else {
            const uint32_t c0123 = __byte_perm(__byte_perm(t[0], t[1], 0x0062), __byte_perm(t[2], t[3], 0x0062), 0x5410);
            const uint32_t c4567 = __byte_perm(__byte_perm(t[4], t[5], 0x0062), __byte_perm(t[6], t[7], 0x0062), 0x5410);
            if (B == 8) {
                w0 = c0123;
                w1 = c4567;
            } else {
                constexpr uint32_t M = B == 2 ? 0x01041040u : 0x01020408u;   // field i of a word moves up by 24 - (8 - B) i bits
                w0 = (((c4567 * M) >> 24) << (4 * B)) | ((c0123 * M) >> 24);
                w1 = 0u;
            }
        }
    }
}

template <int B, bool CLAMP>
__device__ __forceinline__ void quantize8(const float (&x)[8], float mn, float inv, const uint32_t (&o)[4],
                                          uint32_t &w0, uint32_t &w1)
{
    uint32_t t[8];
    noisy_sums8(x, mn, inv, o, t);
    close_codes8<B, CLAMP>(t, w0, w1);
}

// The same for a width known only at run time (and possibly different in every lane): the
// codes are clamped to 2^b - 1, then joined pairwise with multiply-adds by 2^b, 2^2b, 2^4b.
__device__ __forceinline__ void quantize8_any(const float (&x)[8], float mn, float inv, const uint32_t (&o)[4],
                                              uint32_t b, uint32_t &w0, uint32_t &w1)
{
    const uint32_t m1 = 1u << b, L = m1 - 1u, m2 = m1 * m1;
    const uint32_t m4 = b == 8u ? 0u : m2 * m2;                   // eight 8-bit codes fill two words
    uint32_t q[8];
#pragma unroll
    for (int i = 0; i < 8; i++) {
        const float d = __fsub_rn(x[i], mn);
        const float s = __fmaf_rn(d, inv, 256.0f);
        const uint32_t h = (i & 1) ? (o[i >> 1] >> 16) : (o[i >> 1] & 0xFFFFu);
        const uint32_t t = __float_as_uint(s) * 2u + h;
        q[i] = min((t >> 16) - 0x8700u, L);
    }
    const uint32_t q01 = q[1] * m1 + q[0], q23 = q[3] * m1 + q[2], q45 = q[5] * m1 + q[4], q67 = q[7] * m1 + q[6];
    const uint32_t lo = q23 * m2 + q01, hi = q67 * m2 + q45;
    w0 = hi * m4 + lo;
    w1 = hi;
}

// ------------------------------------------------------------------------------------------
// The greedy of Sec. 3.4.1 on one warp.  Every lane holds NK candidate raises (key, cw = cost
// | 1 << 16, or cw = 0 for "no candidate"); slot s of lane l sorts, among equal keys, before
// slot s' > s of any lane and before slot s of lane l' > l.  Accepted is the longest prefix,
// in the order (key descending, then that order), whose summed cost is at most rem; take[s]
// says whether this lane's slot s is in it.  F(t), the cost of all raises with key >= t, falls
// as t grows, so the prefix is every raise with a key above Kp, the largest t with F(t) > rem,
// and then the raises with key Kp in order while they fit.  One warp reduction gives F(t) and
// N(t), the number of raises with key >= t; the interval that holds Kp starts from the keys'
// common leading bits (BOUNDS: the caller passes the largest and the smallest key) and is
// halved bit by bit; as soon as a single raise is left in it, its key is Kp.
// ------------------------------------------------------------------------------------------
template <int NK, bool BOUNDS>
__device__ __forceinline__ void accept_prefix(const uint32_t (&key)[NK], const uint32_t (&cw)[NK],
                                              const uint32_t (&slot_cost)[NK], uint32_t rem, uint32_t hi, uint32_t lo,
                                              int lane, bool (&take)[NK])
{
    if (!BOUNDS) {
        hi = 0u;
        lo = 0xFFFFFFFFu;
#pragma unroll
        for (int s = 0; s < NK; s++)
            if (cw[s] != 0u) {
                hi = max(hi, key[s]);
                lo = min(lo, key[s]);
            }
        hi = __reduce_max_sync(0xFFFFFFFFu, hi);
        lo = __reduce_min_sync(0xFFFFFFFFu, lo);
    }
    auto from = [&](uint32_t t) {                                 // F(t) | N(t) << 16
        uint32_t f = 0;
#pragma unroll
        for (int s = 0; s < NK; s++) f += key[s] >= t ? cw[s] : 0u;
        return __reduce_add_sync(0xFFFFFFFFu, f);
    };
    uint32_t Kp = 0u, at_lo = from(0u), at_hi;                    // F | N at the two ends of the interval
    if ((at_lo & 0xFFFFu) > rem) {
        const uint32_t diff = hi ^ lo;
        int bit = diff != 0u ? 31 - __clz(diff) : -1;             // the interval is [Kp, Kp + 2^(bit+1))
        Kp = diff != 0u ? hi & ~((2u << bit) - 1u) : hi;
        at_hi = 0u;
        while (bit >= 0 && (at_lo >> 16) - (at_hi >> 16) > 1u) {
            const uint32_t t = Kp | (1u << bit);
            const uint32_t e = from(t);
            if ((e & 0xFFFFu) > rem) {
                Kp = t;
                at_lo = e;
            } else {
                at_hi = e;
            }
            bit--;
        }
        if (bit >= 0) {                                           // one raise left in the interval: Kp is its key
            const uint32_t sh = (uint32_t)bit + 1u;
            uint32_t only = 0u;
#pragma unroll
            for (int s = 0; s < NK; s++)
                if (cw[s] != 0u && (sh >= 32u || (key[s] >> sh) == (Kp >> sh))) only = key[s];
            Kp = __reduce_max_sync(0xFFFFFFFFu, only);
        }
    } else {
        at_hi = from(1u);                                         // every raise fits (Kp = 0)
    }
    uint32_t left = rem - (at_hi & 0xFFFFu);                      // after every raise with a key above Kp
    bool open = true;                                             // no raise has been turned down yet
    const uint32_t below = (1u << lane) - 1u;
#pragma unroll
    for (int s = 0; s < NK; s++) {
        const bool on = cw[s] != 0u, tie = on && key[s] == Kp;
        const uint32_t ties = __ballot_sync(0xFFFFFFFFu, tie);
        uint32_t fit = 0u;
        if (ties != 0u && open) {
            const uint32_t cnt = (uint32_t)__popc(ties);
            fit = min(cnt, left / slot_cost[s]);
            left -= fit * slot_cost[s];
            open = fit == cnt;                                    // the walk stops at the first raise that does not fit
        }
        take[s] = on && (key[s] > Kp || (tie && (uint32_t)__popc(ties & below) < fit));
    }
}

}  // namespace daf
