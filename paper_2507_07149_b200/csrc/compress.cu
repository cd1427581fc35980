// Fused compress kernel: one persistent CTA processes one window (window_elems elements) at a
// time and reads the input from HBM exactly once.
//
//   - the next window is staged into shared memory by one bulk asynchronous copy (TMA,
//     completion on an mbarrier) while the current one is processed;
//   - staged window -> registers (8 consecutive elements per lane and chunk), per-group
//     min / max (3-input min/max, warp redux or segmented shuffles);
//   - per-window greedy bit-width choice (Sec. 3.4.1 of the paper: importance per bit);
//   - intra-window exclusive scan of the group byte lengths; the window's byte count is
//     published at once in a 64-bit descriptor;
//   - Eq. 1 quantization with stochastic rounding (Philox4x32-10, 16 bits per element, the
//     float -> uint step done with the power-of-two offset of Eq. 5) and lane-local LSB-first
//     packing into a shared-memory buffer;
//   - the window's device-wide byte offset comes from a bounded decoupled look-back over the
//     descriptors, resolved opportunistically after the quantize pass and otherwise one
//     window later, so that no CTA waits for its neighbours; the packed window then leaves
//     shared memory as one bulk asynchronous store.
//
// Windows are handed out by an atomic ticket, so every window with a smaller index than the
// one a CTA holds is owned by a running (or finished) CTA and the look-back always makes
// progress; every wait is bounded all the same.
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

struct SmemLayout {          // byte offsets into dynamic shared memory
    uint32_t out0, out_stride, umn, umx, key, cum, grp, srt, total;
};

template <int NT> struct CompressArgs {
    WorkspaceHeader *hdr;
    uint64_t *flags;
    uint32_t total_windows, n_tensors;
    uint32_t G, log2G, beta_q8, m, nearest, bulk_store, n_max, nbuf;
    uint32_t full_ell, full_rem, full_rem_after;   // budget arithmetic of a full window (n_max groups)
    uint32_t S[kMaxLevels], cost[kMaxLevels];
    float v[kMaxLevels];
    SmemLayout lay;
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
// is the fixed-point quotient; adding a 15-bit random offset r15 and dropping 15 bits rounds
// stochastically (r15 = 2^14: round half up).  With h = 2*r15 + (one more random bit),
// (fixed + r15) >> 15 == (2*bits(s) + h - 2*bits(256)) >> 16, which needs one add, one shift
// and one fused subtract-and-clamp per element.
// ------------------------------------------------------------------------------------------
template <int B, bool CLAMP>
__device__ __forceinline__ void quantize8(const float (&x)[8], float mn, float inv, const uint32_t (&o)[4],
                                          uint32_t &w0, uint32_t &w1)
{
    constexpr uint32_t L = (1u << B) - 1u;
    w0 = 0u;
    w1 = 0u;
#pragma unroll
    for (int i = 0; i < 8; i++) {
        const float d = __fsub_rn(x[i], mn);
        const float s = __fmaf_rn(d, inv, 256.0f);
        const uint32_t h = (i & 1) ? (o[i >> 1] >> 16) : (o[i >> 1] & 0xFFFFu);
        const uint32_t t = __float_as_uint(s) * 2u + h;           // mod 2^32; 2*bits(256) = 0x87000000
        const int pos = (B * i) & 31;                             // bit position of code i in its word (unrolled: constant)
        uint32_t field;
        if (CLAMP) {
            field = min((t >> 16) - 0x8700u, L) << pos;
        } else {
            // the code is the B-bit field of t at bit 16 (never above L when 1/scale is a normal
            // number): move it to its place and mask, without materialising it
            const uint32_t moved = pos < 16 ? (t >> (16 - pos)) : (pos == 16 ? t : (t << (pos - 16)));
            field = moved & (L << pos);
        }
        if (B == 8 && i >= 4) w1 |= field;
        else w0 |= field;
    }
}

// ------------------------------------------------------------------------------------------
// Decoupled look-back over the window descriptors, executed by one full warp.  Each round
// inspects DEPTH * 32 predecessors with all loads in flight at once.  Returns 1 when the
// exclusive prefix was found (*excl), 0 when a needed descriptor is still empty and `block`
// is false, -1 on a poisoned predecessor, -2 when the bounded wait ran out.
// ------------------------------------------------------------------------------------------
constexpr int kLookDepth = 16;

template <int DEPTH>
__device__ __forceinline__ int lookback(const uint64_t *flags, uint32_t gw, uint32_t first, int lane, bool block,
                                        uint64_t *excl_out)
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
            if (++polls > kMaxPolls) return -2;
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
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity)
{
    for (unsigned polls = 0; polls < kMaxPolls; polls++)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// Eight consecutive elements of a lane from the staged window (two 16-byte shared loads for
// 4-byte elements, one for 2-byte elements).  For 4-byte elements a lane owns 32 bytes; the
// two halves are read in an order that depends on the lane so that each quarter-warp touches
// all 32 banks.  ORDERED = false leaves the halves as read (enough for min / max).
template <typename T, bool ORDERED> __device__ __forceinline__ void load8_staged(const unsigned char *chunk, int lane, float (&x)[8]);

template <> __device__ __forceinline__ void load8_staged<float, false>(const unsigned char *chunk, int lane, float (&x)[8])
{
    const int odd = (lane >> 2) & 1;
    const unsigned char *p = chunk + lane * 32;
    const float4 a = *reinterpret_cast<const float4 *>(p + odd * 16);
    const float4 b = *reinterpret_cast<const float4 *>(p + (odd ^ 1) * 16);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
    x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
template <> __device__ __forceinline__ void load8_staged<float, true>(const unsigned char *chunk, int lane, float (&x)[8])
{
    const bool odd = (lane >> 2) & 1;
    float y[8];
    load8_staged<float, false>(chunk, lane, y);
#pragma unroll
    for (int i = 0; i < 4; i++) {
        x[i] = odd ? y[i + 4] : y[i];
        x[i + 4] = odd ? y[i] : y[i + 4];
    }
}
template <bool ORDERED> __device__ __forceinline__ void load8_staged_half(const unsigned char *chunk, int lane, float (&x)[8])
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
template <bool ORDERED> __device__ __forceinline__ void load8_staged_bf16(const unsigned char *chunk, int lane, float (&x)[8])
{
    const uint4 v = *reinterpret_cast<const uint4 *>(chunk + lane * 16);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; i++) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}
template <> __device__ __forceinline__ void load8_staged<__half, false>(const unsigned char *c, int l, float (&x)[8]) { load8_staged_half<false>(c, l, x); }
template <> __device__ __forceinline__ void load8_staged<__half, true>(const unsigned char *c, int l, float (&x)[8]) { load8_staged_half<true>(c, l, x); }
template <> __device__ __forceinline__ void load8_staged<__nv_bfloat16, false>(const unsigned char *c, int l, float (&x)[8]) { load8_staged_bf16<false>(c, l, x); }
template <> __device__ __forceinline__ void load8_staged<__nv_bfloat16, true>(const unsigned char *c, int l, float (&x)[8]) { load8_staged_bf16<true>(c, l, x); }

// Staged window -> registers, then min / max per unit of LPU lanes (a full warp uses the
// redux instruction).  Every lane of a unit ends up with the unit's min / max (lo[c], hi[c]);
// the unit's first lane also writes them to shared memory for the general bit choice.
// Chunks past a ragged window's end read stale bytes; their results are never used.
template <typename T, int CHUNKS, int LPU>
__device__ __forceinline__ void load_and_reduce(const unsigned char *stage, int warp, int lane, float (&x)[CHUNKS][8],
                                                float (&lo)[CHUNKS], float (&hi)[CHUNKS], float *s_umn, float *s_umx)
{
    constexpr int kChunkBytes = 256 * Elem<T>::kBytes;
#pragma unroll
    for (int c = 0; c < CHUNKS; c++) load8_staged<T, false>(stage + (warp * CHUNKS + c) * kChunkBytes, lane, x[c]);
#pragma unroll
    for (int c = 0; c < CHUNKS; c++) {
        float l = fmin3(fmin3(x[c][0], x[c][1], x[c][2]), fmin3(x[c][3], x[c][4], x[c][5]), fmin2(x[c][6], x[c][7]));
        float h = fmax3(fmax3(x[c][0], x[c][1], x[c][2]), fmax3(x[c][3], x[c][4], x[c][5]), fmax2(x[c][6], x[c][7]));
        if (LPU == 32) {
            asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(l) : "f"(l));
            asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(h) : "f"(h));
        } else {
#pragma unroll
            for (int off = 1; off < LPU; off <<= 1) {
                l = fmin2(l, __shfl_xor_sync(0xFFFFFFFFu, l, off));
                h = fmax2(h, __shfl_xor_sync(0xFFFFFFFFu, h, off));
            }
        }
        if ((lane & (LPU - 1)) == 0) {
            const int u = (warp * CHUNKS + c) * (32 / LPU) + lane / LPU;
            s_umn[u] = l;
            s_umx[u] = h;
        }
        lo[c] = l;
        hi[c] = h;
    }
}

template <int NT> __device__ __forceinline__ uint32_t find_tensor(const CompressArgs<NT> &a, uint32_t gw)
{
    uint32_t lo = 0, hi = a.n_tensors - 1;                        // last tensor whose first window is <= gw
    while (lo < hi) {
        const uint32_t mid = (lo + hi + 1) >> 1;
        if (a.t[mid].first_window <= gw) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// One persistent CTA per SM: 16 compute warps plus three service warps, synchronised only through
// shared-memory mbarriers (every wait on them is bounded) except inside the general bit choice.
//   s_full[s]  : the bulk copy into stage s has landed (or the control warp has marked the
//                window behind it as "no more work");
//   s_cons[s]  : all compute warps have moved stage s into registers and have finished packing
//                the previous window (16 arrivals);
//   s_exch     : all compute warps have contributed their part of a window's min / max test
//                (16 arrivals) -- arrival and wait are split so that the exchange of window
//                j+1 completes while window j is being quantized;
//   s_wid      : the group records of a window that needed the general bit choice are ready;
//   s_ready[b] : the window using packed-bytes buffer b is completely packed (16 arrivals);
//   s_free[b]  : the packed bytes of the window that used buffer b have left shared memory.
// Window j uses stage j & 1, packed-bytes buffer j % 3 and slot j & 3 (tickets: j & 7) of the
// small per-window arrays.  A loader warp owns tickets and bulk copies in; two storer warps
// alternate over the windows for look-back and bulk stores out.
constexpr uint32_t kBarOwners = 3;

__device__ __forceinline__ void bar_sync(uint32_t id, uint32_t threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// Philox4x32-10 for CHUNKS consecutive counter blocks at once (blk0 + 32 c): the rounds of the
// independent blocks are interleaved in program order so that their long dependency chains
// overlap.
template <typename KEYS, int CHUNKS>
__device__ __forceinline__ void philox_chunks(uint64_t blk0, const KEYS &keys, uint32_t (&o)[CHUNKS][4])
{
    uint32_t c0[CHUNKS], c1[CHUNKS], c2[CHUNKS], c3[CHUNKS];
#pragma unroll
    for (int c = 0; c < CHUNKS; c++) {
        const uint64_t blk = blk0 + 32u * c;
        c0[c] = (uint32_t)blk;
        c1[c] = (uint32_t)(blk >> 32);
        c2[c] = 0u;
        c3[c] = 0u;
    }
#pragma unroll
    for (int r = 0; r < 10; r++) {
#pragma unroll
        for (int c = 0; c < CHUNKS; c++) {
            const uint64_t p0 = (uint64_t)kPhiloxM0 * c0[c], p1 = (uint64_t)kPhiloxM1 * c2[c];
            c0[c] = (uint32_t)(p1 >> 32) ^ c1[c] ^ philox_key0(keys, r);
            c1[c] = (uint32_t)p1;
            c2[c] = (uint32_t)(p0 >> 32) ^ c3[c] ^ philox_key1(keys, r);
            c3[c] = (uint32_t)p0;
        }
    }
#pragma unroll
    for (int c = 0; c < CHUNKS; c++) {
        o[c][0] = c0[c];
        o[c][1] = c1[c];
        o[c][2] = c2[c];
        o[c][3] = c3[c];
    }
}

// Quantize + pack CHUNKS chunks that all have width B, with per-chunk (min, 1/scale) in
// registers: no per-chunk decisions, packed position computed from the element index alone.
template <typename KEYS, int CHUNKS, int B, bool CLAMP>
__device__ __forceinline__ void quantize_uniform(const float (&x)[CHUNKS][8], const float (&mn)[CHUNKS],
                                                 const float (&inv)[CHUNKS], uint32_t e0, uint64_t blk0, const KEYS &keys,
                                                 unsigned char *s_out)
{
    unsigned char *const out = s_out + (e0 >> 3) * B;
    uint32_t o[CHUNKS][4];
    philox_chunks<KEYS, CHUNKS>(blk0, keys, o);
#pragma unroll
    for (int c = 0; c < CHUNKS; c++) {
        uint32_t w0, w1;
        quantize8<B, CLAMP>(x[c], mn[c], inv[c], o[c], w0, w1);
        unsigned char *p = out + 32 * B * c;
        if (B == 1) *p = (unsigned char)w0;
        else if (B == 2) *reinterpret_cast<uint16_t *>(p) = (uint16_t)w0;
        else if (B == 4) *reinterpret_cast<uint32_t *>(p) = w0;
        else *reinterpret_cast<uint2 *>(p) = make_uint2(w0, w1);
    }
}

template <typename KEYS, int CHUNKS, bool CLAMP>
__device__ __forceinline__ void quantize_uniform_b(uint32_t b, const float (&x)[CHUNKS][8], const float (&mn)[CHUNKS],
                                                   const float (&inv)[CHUNKS], uint32_t e0, uint64_t blk0, const KEYS &keys,
                                                   unsigned char *s_out)
{
    switch (b) {
    case 1: quantize_uniform<KEYS, CHUNKS, 1, CLAMP>(x, mn, inv, e0, blk0, keys, s_out); break;
    case 2: quantize_uniform<KEYS, CHUNKS, 2, CLAMP>(x, mn, inv, e0, blk0, keys, s_out); break;
    case 4: quantize_uniform<KEYS, CHUNKS, 4, CLAMP>(x, mn, inv, e0, blk0, keys, s_out); break;
    default: quantize_uniform<KEYS, CHUNKS, 8, CLAMP>(x, mn, inv, e0, blk0, keys, s_out); break;
    }
}

// Budget arithmetic of a window of n groups.
struct Budget {
    uint32_t ell;          // largest level every group can be raised to
    uint32_t rem;          // bit units left after the smallest width
    bool all_max;          // every group reaches the largest width
    bool need_sep;         // the best raise of level ell does not fit: uniform iff the levels separate
};

// T: element type; CHUNKS: 256-element chunks per compute warp; NW: compute warps; NSTAGE: staged
// windows per CTA (2: one CTA per SM with a window of look-ahead; 1: two CTAs per SM that cover
// each other's copy latency); NSTO: storer warps.
template <typename T, int CHUNKS, int NW, int NSTAGE, int NSTO, bool BATCH>
__global__ void __launch_bounds__(NW * 32 + 32 + 32 * NSTO, NSTAGE == 1 ? 2 : 1)
compress_kernel(const __grid_constant__ CompressArgs<BATCH ? DAF_BATCH_MAX : 1> a)
{
    constexpr int kComputeWarps = NW;
    constexpr uint32_t WE = NW * 256u * CHUNKS;
    constexpr uint32_t kStageBytes = WE * Elem<T>::kBytes;

    extern __shared__ __align__(128) unsigned char smem[];       // [stage 0 | stage 1 | packed x3 | group arrays]
    __shared__ __align__(8) uint64_t s_full[NSTAGE], s_cons[NSTAGE], s_ready[3], s_free[3], s_exch, s_wid;   // mbarriers
    __shared__ uint32_t s_next[8];                               // ticket of window j
    __shared__ uint32_t s_kmin[4], s_kmax[4], s_flag[4];         // per-window exchange: key extremes, "a wait ran out"
    __shared__ uint32_t s_tot[4];                                // packed bytes of window j
    __shared__ uint32_t s_wtot[NW], s_coll;
    __shared__ uint32_t s_lost, s_end;                           // s_end: number of windows this CTA packed (set on leaving)

    float *const s_umn = reinterpret_cast<float *>(smem + a.lay.umn);    // [2][units]
    float *const s_umx = reinterpret_cast<float *>(smem + a.lay.umx);
    uint32_t *const s_key = reinterpret_cast<uint32_t *>(smem + a.lay.key);   // [level][n_max]
    uint32_t *const s_cum = reinterpret_cast<uint32_t *>(smem + a.lay.cum);
    GroupRec *const s_grp = reinterpret_cast<GroupRec *>(smem + a.lay.grp);   // [2][n_max]
    uint32_t *const s_srt = reinterpret_cast<uint32_t *>(smem + a.lay.srt);   // [2][n_max]: sorted group, its range

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t G = a.G, log2G = a.log2G;

    auto record_error = [&](unsigned code, uint32_t window, unsigned site) {
        if (atomicCAS(&a.hdr->status, 0u, code) == 0u) {
            a.hdr->fail_window = window;
            a.hdr->fail_site = site;
        }
    };
    auto tensor_of = [&](uint32_t gw) -> const TensorDesc & { return a.t[BATCH ? find_tensor(a, gw) : 0u]; };
    auto budget_of = [&](uint32_t n) {
        Budget b;
        uint32_t rem_after = a.full_rem_after;
        b.ell = a.full_ell;
        b.rem = a.full_rem;
        if (n != a.n_max) {                                       // ragged last window: work it out here
            const uint64_t Tbits = ((uint64_t)a.beta_q8 * n) >> 8;
            b.rem = (uint32_t)(Tbits - (uint64_t)a.S[0] * n);
            b.ell = 0;
            while (b.ell + 1 < a.m && (a.S[b.ell + 1] - a.S[0]) * n <= b.rem) b.ell++;
            rem_after = b.rem - (a.S[b.ell] - a.S[0]) * n;
        }
        b.all_max = (b.ell + 1 == a.m);
        b.need_sep = !b.all_max && rem_after < a.cost[b.ell];
        return b;
    };

    if (warp == kComputeWarps) {
        // ============================================================ loader warp
        // Publishes the ticket of window j and starts its bulk copy into stage j & 1, or completes
        // the stage's barrier empty-handed when there is no such window.  Round r: once the
        // compute warps have moved window r into registers, stage r & 1 takes window r+2.
        auto issue = [&](uint32_t j, uint32_t t) {
            s_next[j & 7u] = t;
            uint64_t *bar = &s_full[j % NSTAGE];
            if (t < a.total_windows) {
                const TensorDesc &nd = tensor_of(t);
                const uint64_t base = (uint64_t)(t - nd.first_window) * WE;
                const uint64_t left = nd.numel - base;
                const uint32_t bytes = (uint32_t)(left < WE ? left : WE) * Elem<T>::kBytes;
                mbar_expect_tx(bar, bytes);
                bulk_load(smem + (j % NSTAGE) * kStageBytes, reinterpret_cast<const char *>(nd.in) + base * Elem<T>::kBytes, bytes, bar);
            } else {
                mbar_arrive(bar);
            }
        };
        uint32_t next_w = 0;                                      // next window index to issue
        uint32_t tk = 0xFFFFFFFFu;                                // its ticket, reserved ahead of time
        bool more = true;                                         // no "no more work" window issued yet
        auto issue_next = [&]() {
            issue(next_w, tk);
            more = tk < a.total_windows;
            next_w++;
            if (more) tk = atomicAdd(&a.hdr->ticket, 1u);         // its latency is off the compute warps' path
        };
        if (lane == 0) {
            for (int k = 0; k < NSTAGE; k++) {
                mbar_init(&s_full[k], 1);
                mbar_init(&s_cons[k], kComputeWarps);
            }
            for (int k = 0; k < 3; k++) {
                mbar_init(&s_ready[k], kComputeWarps);
                mbar_init(&s_free[k], 1);
            }
            mbar_init(&s_exch, kComputeWarps);
            mbar_init(&s_wid, kComputeWarps);
            s_lost = 0u;
            s_end = 0xFFFFFFFFu;
            for (int k = 0; k < 4; k++) {
                s_kmin[k] = 0xFFFFFFFFu;
                s_kmax[k] = 0u;
                s_flag[k] = 0u;
            }
            tk = atomicAdd(&a.hdr->ticket, 1u);
            for (int k = 0; k < NSTAGE && more; k++) issue_next();
        }
        __syncthreads();
        if (lane != 0) return;
        // Round r: once the compute warps have moved window r into registers, its stage takes
        // window r + NSTAGE.  Windows 0 .. next_w-1 have been issued, the last of them possibly
        // as "no more work".
        for (uint32_t r = 0; more || r + 1u < next_w; r++) {
            if (!mbar_wait_bounded(&s_cons[r % NSTAGE], (r / NSTAGE) & 1u)) {
                s_lost = 1u;
                record_error(DAF_ERR_TIMEOUT, s_next[r & 7u], 2u + 16u * r);
            }
            if (s_lost != 0u) {
                // leaving: windows still held will never be published; copies in flight must land
                for (uint32_t q = r + 1u; q < next_w; q++) {
                    const uint32_t t = s_next[q & 7u];
                    if (t < a.total_windows) {
                        st_relaxed_u64(a.flags + t, kFlagPoison << kFlagShift);
                        mbar_wait_bounded(&s_full[q % NSTAGE], (q / NSTAGE) & 1u);
                    }
                }
                if (more && tk < a.total_windows) st_relaxed_u64(a.flags + tk, kFlagPoison << kFlagShift);
                if (more) {                                       // release anyone still waiting for the next window
                    tk = 0xFFFFFFFFu;
                    issue_next();
                }
                break;
            }
            if (more) issue_next();
        }
        return;
    }
    if (warp > kComputeWarps) {
        // ============================================================ storer warps (taking windows in turn)
        // For window p: once it is packed, find its byte offset by look-back, publish its inclusive
        // prefix, send its packed bytes to global memory with one bulk store, free the buffer.
        __syncthreads();
        for (uint32_t p = (uint32_t)(warp - kComputeWarps - 1);; p += NSTO) {
            // s_ready[p % 3] fires when window p is packed -- or when the compute warps have left
            // their loop without ever reaching a window p (s_end tells which)
            const bool ok = mbar_wait_bounded(&s_ready[p % 3u], (p / 3u) & 1u);
            if (ok && p >= s_end) break;
            const uint32_t p_gw = s_next[p & 7u];
            if (!ok || s_lost != 0u) {
                s_lost = 1u;
                if (lane == 0 && !ok) record_error(DAF_ERR_TIMEOUT, 0u, 8u + 16u * p);
                if (lane == 0 && ok) st_relaxed_u64(a.flags + p_gw, kFlagPoison << kFlagShift);
                break;
            }
            const TensorDesc &pd = tensor_of(p_gw);
            const uint32_t p_total = s_tot[p & 3u];
            const unsigned char *src = smem + a.lay.out0 + (p % 3u) * a.lay.out_stride;
            uint64_t excl = 0;
            int state = 1;
            if (p_gw != pd.first_window) {
                state = lookback<kLookDepth>(a.flags, p_gw, pd.first_window, lane, true, &excl);
                if (lane == 0)
                    st_relaxed_u64(a.flags + p_gw, state == 1 ? ((kFlagPrefix << kFlagShift) | (excl + p_total))
                                                                : (kFlagPoison << kFlagShift));
            }
            const uint32_t pw = p_gw - pd.first_window;
            bool skip = state != 1;
            if (!skip) {
                if (lane == 0) {
                    pd.woff[pw] = excl;
                    if (pw + 1 == pd.n_windows) pd.woff[pw + 1] = excl + p_total;
                }
                skip = excl + p_total > pd.capacity;
            }
            if (skip) {
                if (lane == 0)
                    record_error(state == -2 ? DAF_ERR_TIMEOUT : DAF_ERR_CAPACITY, p_gw, state == 1 ? 5u : (state == -2 ? 3u : 4u));
            } else if (a.bulk_store) {
                if (lane == 0 && p_total) {
                    bulk_store(pd.packed + excl, src, p_total);
                    bulk_store_wait_read();
                }
            } else {                                              // groups of 32 / 64: windows are only 4-byte aligned
                uint32_t *dst = reinterpret_cast<uint32_t *>(pd.packed + excl);
                const uint32_t *s32 = reinterpret_cast<const uint32_t *>(src);
                for (uint32_t k = lane; k < (p_total >> 2); k += 32) dst[k] = s32[k];
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_free[p % 3u]);          // the buffer may be rewritten from now on
        }
        if (lane == 0) bulk_store_wait_all();
        return;
    }

    // ================================================================ compute warps
    __syncthreads();                                              // barriers initialised by the control warp
    const uint32_t e0 = (uint32_t)(warp * CHUNKS * 256 + lane * 8);    // this lane's first element of chunk 0
    const uint32_t lpu = (G < 256u ? G : 256u) >> 3;              // lanes per unit
    const uint32_t units = WE >> (G < 256u ? log2G : 8u);         // units per window
    // Launch-wide facts about full windows (the ragged last window of a tensor always takes the
    // general path): can the quick uniform-width decision apply, and with which numbers?
    const Budget fb = budget_of(a.n_max);
    const bool fast_launch = G <= 256u * CHUNKS && !a.nearest && (fb.all_max || fb.need_sep);
    const bool test_sep = fast_launch && fb.need_sep && fb.ell > 0;
    const uint32_t fast_b = a.S[fb.ell];
    const float fast_L = (float)((1u << fast_b) - 1u);
    const float v_lo = a.v[fb.ell > 0 ? fb.ell - 1 : 0], v_hi = a.v[fb.ell];
    // lane k of a unit looks after chunk k's group in the uniform case
    const int uk = lane & (int)(lpu - 1u), usb = lane - uk;
    const uint32_t unit_elem = (uint32_t)((warp * CHUNKS + uk) * 256 + usb * 8);   // first element of that unit
    const bool meta_lane = uk < CHUNKS && (unit_elem & (G - 1u)) == 0u;            // the unit opens a group

    // the window being quantized (registers) and how
    float x[CHUNKS][8];
    float q_mn[CHUNKS], q_inv[CHUNKS];                            // uniform windows: per-chunk min and 1/scale
    uint32_t q_b = 0;                                             // uniform windows: the width; 0 = use the group records
    uint32_t q_gw = 0, q_elems = 0;
    uint32_t n_generic = 0;                                       // windows that took the general bit choice so far
    uint32_t n_packed = 0;                                        // windows 0 .. n_packed-1 are packed
    bool my_lost = false;

    uint32_t j = 0;
    for (;; j++) {
        // ---------------------------------------------------------------- window j has landed (or there is none)
        if (!mbar_wait_bounded(&s_full[j % NSTAGE], (j / NSTAGE) & 1u)) {
            my_lost = true;
            s_lost = 1u;
            if (lane == 0) record_error(DAF_ERR_TIMEOUT, 0u, 1u + 16u * j);
        }
        const uint32_t gw = my_lost ? 0xFFFFFFFFu : s_next[j & 7u];
        const bool valid = gw < a.total_windows;
        const unsigned char *stage = smem + (j % NSTAGE) * kStageBytes;

        // ---------------------------------------------------------------- min / max of window j, contribution to its exchange
        const TensorDesc &td = tensor_of(valid ? gw : 0u);
        const uint32_t w = gw - td.first_window;
        const bool full = (uint64_t)(w + 1u) * WE <= td.numel;
        const bool fast_ok = fast_launch && full;
        float lo[CHUNKS], hi[CHUNKS];
        if (valid) {
            float y[CHUNKS][8];                                   // transient: only the min / max are kept
            float *umn = s_umn + (j & 1u) * units, *umx = s_umx + (j & 1u) * units;
            if (lpu == 32u) load_and_reduce<T, CHUNKS, 32>(stage, warp, lane, y, lo, hi, umn, umx);
            else if (lpu == 16u) load_and_reduce<T, CHUNKS, 16>(stage, warp, lane, y, lo, hi, umn, umx);
            else if (lpu == 8u) load_and_reduce<T, CHUNKS, 8>(stage, warp, lane, y, lo, hi, umn, umx);
            else load_and_reduce<T, CHUNKS, 4>(stage, warp, lane, y, lo, hi, umn, umx);
            if (fast_ok) {
                // groups of 512 / 1024 span 2 / 4 chunks of this warp
                if (G == 512u) {
#pragma unroll
                    for (int c = 0; c + 1 < CHUNKS; c += 2) {
                        lo[c] = lo[c + 1] = fmin2(lo[c], lo[c + 1]);
                        hi[c] = hi[c + 1] = fmax2(hi[c], hi[c + 1]);
                    }
                } else if (G == 1024u && CHUNKS == 4) {
                    const float l = fmin2(fmin2(lo[0], lo[1]), fmin2(lo[2], lo[3]));
                    const float h = fmax2(fmax2(hi[0], hi[1]), fmax2(hi[2], hi[3]));
#pragma unroll
                    for (int c = 0; c < CHUNKS; c++) {
                        lo[c] = l;
                        hi[c] = h;
                    }
                }
                // Contribution to the window's exchange: the separation test of the uniform outcome
                // (min over groups of the key of the last raise taken, max over groups of the key of
                // the first raise not taken) and "some range is so large that 1/scale is not a normal
                // number" (bit 1 of the flag word: such windows take the careful general path).
                uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
                float rmax = 0.0f;
#pragma unroll
                for (int c = 0; c < CHUNKS; c++) {
                    float R = __fsub_rn(hi[c], lo[c]);
                    if (R < 0x1p-118f) R = 0.0f;                  // degenerate group: constant
                    rmax = fmax2(rmax, R);
                    if (test_sep) {
                        kmin = min(kmin, __float_as_uint(__fmul_rn(R, v_lo)));
                        kmax = max(kmax, __float_as_uint(__fmul_rn(R, v_hi)));
                    }
                }
                if (lpu != 32u) {
                    if (test_sep) {
                        kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
                        kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
                    }
                    rmax = __uint_as_float(__reduce_max_sync(0xFFFFFFFFu, __float_as_uint(rmax)));   // rmax >= 0
                }
                if (lane == 0) {
                    if (test_sep) {
                        atomicMin(&s_kmin[j & 3u], kmin);
                        atomicMax(&s_kmax[j & 3u], kmax);
                    }
                    if (!(rmax < 0x1p126f)) atomicOr(&s_flag[j & 3u], 2u);
                }
            }
            if (lane == 0 && s_lost != 0u) atomicOr(&s_flag[j & 3u], 1u);
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_exch);
        }

        // ---------------------------------------------------------------- quantize + pack window j-1 (registers -> shared)
        if (j > 0) {
            unsigned char *const s_out = smem + a.lay.out0 + ((j - 1u) % 3u) * a.lay.out_stride;
            if (j > 3u && !mbar_wait_bounded(&s_free[(j - 1u) % 3u], (((j - 1u) / 3u) - 1u) & 1u)) {
                s_lost = 1u;                                      // the buffer's previous window never left: give up
                if (lane == 0) record_error(DAF_ERR_TIMEOUT, q_gw, 9u + 16u * j);
                break;
            }
            const TensorDesc &qd = tensor_of(q_gw);
            const uint64_t blk0 = ((qd.elem_base >> 3) + (uint64_t)(q_gw - qd.first_window) * (WE / 8u)) + (e0 >> 3);
            if (q_b != 0u) {
                if (BATCH) {
                    const PhiloxSeedKeys sk{(uint32_t)qd.seed, (uint32_t)(qd.seed >> 32)};
                    quantize_uniform_b<PhiloxSeedKeys, CHUNKS, false>(q_b, x, q_mn, q_inv, e0, blk0, sk, s_out);
                } else {
                    quantize_uniform_b<PhiloxKeys, CHUNKS, false>(q_b, x, q_mn, q_inv, e0, blk0, a.keys, s_out);
                }
            } else {
                const GroupRec *grp = s_grp + ((j - 1u) & 1u) * a.n_max;
#pragma unroll
                for (int c = 0; c < CHUNKS; c++) {
                    const uint32_t e = e0 + 256u * c;
                    const GroupRec rec = grp[e >> log2G];
                    uint32_t o[4];
                    if (a.nearest) {
                        o[0] = o[1] = o[2] = o[3] = 0x80008000u;   // every 16-bit lane = 2 * 2^14
                    } else {
                        const uint64_t blk = blk0 + 32u * c;
                        if (BATCH) {
                            const PhiloxSeedKeys sk{(uint32_t)qd.seed, (uint32_t)(qd.seed >> 32)};
                            philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), sk, o);
                        } else {
                            philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), a.keys, o);
                        }
                    }
                    uint32_t w0, w1;
                    unsigned char *p = s_out + rec.off + ((e & (G - 1u)) >> 3) * rec.b;
                    if (e < q_elems) {
                        switch (rec.b) {
                        case 1: quantize8<1, true>(x[c], rec.mn, rec.inv, o, w0, w1); *p = (unsigned char)w0; break;
                        case 2: quantize8<2, true>(x[c], rec.mn, rec.inv, o, w0, w1); *reinterpret_cast<uint16_t *>(p) = (uint16_t)w0; break;
                        case 4: quantize8<4, true>(x[c], rec.mn, rec.inv, o, w0, w1); *reinterpret_cast<uint32_t *>(p) = w0; break;
                        default:
                            quantize8<8, true>(x[c], rec.mn, rec.inv, o, w0, w1);
                            if (G >= 64u) {
                                *reinterpret_cast<uint2 *>(p) = make_uint2(w0, w1);
                            } else {                               // G = 32: groups are only 4-byte aligned
                                reinterpret_cast<uint32_t *>(p)[0] = w0;
                                reinterpret_cast<uint32_t *>(p)[1] = w1;
                            }
                            break;
                        }
                    }
                }
            }
            if (a.bulk_store) fence_async_shared();               // packed bytes visible to the bulk store issued later
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_ready[(j - 1u) % 3u]);  // this warp's share of window j-1 is packed
            n_packed = j;
        }
        if (!valid) break;

        // ---------------------------------------------------------------- the exchange of window j is complete: widths
        if (!mbar_wait_bounded(&s_exch, j & 1u)) {
            s_lost = 1u;
            if (lane == 0) record_error(DAF_ERR_TIMEOUT, gw, 6u + 16u * j);
            break;
        }
        const uint32_t flag = s_flag[j & 3u];
        if (flag & 1u) break;                                     // some warp ran out of patience: all leave together
        if (tid == 0) {                                           // recycle the slots two windows ahead
            s_kmin[(j + 2u) & 3u] = 0xFFFFFFFFu;
            s_kmax[(j + 2u) & 3u] = 0u;
            s_flag[(j + 2u) & 3u] = 0u;
        }
        const bool uniform = fast_ok && flag == 0u && (!test_sep || s_kmin[j & 3u] >= s_kmax[j & 3u]);
        if (uniform) {
            // -------------------------------------------------------------- every group gets width S[ell]
            // lane k of a unit works out (scale, 1/scale) of chunk k's group, then the unit shares them
            float Rk = 0.0f, mnk = 0.0f;
#pragma unroll
            for (int c = 0; c < CHUNKS; c++)
                if (uk == c) {
                    Rk = __fsub_rn(hi[c], lo[c]);
                    mnk = lo[c];
                }
            if (Rk < 0x1p-118f) Rk = 0.0f;                        // degenerate group: constant
            const float scale_k = Rk > 0.0f ? __fdiv_rn(Rk, fast_L) : 0.0f;
            const float inv_k = Rk > 0.0f ? __fdiv_rn(fast_L, Rk) : 0.0f;
            if (meta_lane) {
                const uint64_t g = (((uint64_t)w * WE) >> log2G) + (unit_elem >> log2G);
                td.bits[g] = (uint8_t)fast_b;
                td.mn[g] = mnk;
                td.scale[g] = scale_k;
            }
#pragma unroll
            for (int c = 0; c < CHUNKS; c++) {
                q_inv[c] = __shfl_sync(0xFFFFFFFFu, inv_k, usb + c);
                q_mn[c] = lo[c];
            }
            q_b = fast_b;
            if (tid == 0) {
                const uint32_t total = a.n_max * (G >> 3) * fast_b;
                const bool first = (w == 0u);
                st_relaxed_u64(a.flags + gw, ((first ? kFlagPrefix : kFlagAggregate) << kFlagShift) | total);
                s_tot[j & 3u] = total;
            }
        } else {
            const uint64_t wbase = (uint64_t)w * WE;
            const uint64_t left = td.numel - wbase;
            const uint32_t n_elems = left < WE ? (uint32_t)left : WE;
            const uint32_t n = n_elems >> log2G;                  // groups in window j
            const Budget bud = budget_of(n);
            const uint64_t g0 = wbase >> log2G;                   // first group of the window in the tensor
            // -------------------------------------------------------------- general bit choice, group records
            // All compute warps take this branch together.  The greedy of Sec. 3.4.1 accepts the
            // longest prefix of the candidate raises, sorted by (key descending, level ascending,
            // group ascending), whose summed cost fits the window's budget.  Within one level the
            // keys fl(R v_k) are a non-decreasing function of the range R, so one ranking of the
            // groups by (R descending, group ascending) sorts every level at once; a candidate's
            // position in the merged order then follows from binary searches in the other levels'
            // sorted keys.  Only if two different ranges round to the same key (their order would then
            // be by group index, not by range) does the window fall back to ranking by counting.
            constexpr uint32_t kBarCompute = 2;                   // hardware barrier of the 16 compute warps
            constexpr uint32_t kComputeThreads = NW * 32u;
            const uint32_t owners = (n + 31u) >> 5;               // warps that own group records
            const uint32_t m = a.m, n_max = a.n_max, nl = a.m - 1u;
            const bool mine = (uint32_t)tid < n;
            uint32_t *const s_Rb = s_cum, *const s_rank = s_cum + n_max, *const s_lvl = s_cum + 2u * n_max;
            uint32_t *const s_sorted = s_srt, *const s_sR = s_srt + n_max;
            float mn = 0.0f, Rg = 0.0f;
            if (mine) {
                const float *umn = s_umn + (j & 1u) * units, *umx = s_umx + (j & 1u) * units;
                float mx;
                if (G > 256u) {
                    const uint32_t rr = G >> 8;
                    mn = umn[tid * rr];
                    mx = umx[tid * rr];
                    for (uint32_t k = 1; k < rr; k++) {
                        mn = fmin2(mn, umn[tid * rr + k]);
                        mx = fmax2(mx, umx[tid * rr + k]);
                    }
                } else {
                    mn = umn[tid];
                    mx = umx[tid];
                }
                Rg = __fsub_rn(mx, mn);
                if (Rg < 0x1p-118f) Rg = 0.0f;                    // degenerate group: constant
                s_Rb[tid] = __float_as_uint(Rg);
                s_rank[tid] = 0u;
                s_lvl[tid] = 0u;
            }
            if (tid == 0) s_coll = 0u;
            bar_sync(kBarCompute, kComputeThreads);

            // Does every group end at level ell after all?  (every warp works it out for itself)
            bool same = bud.all_max;
            if (!bud.all_max && bud.need_sep) {
                // every raise below level ell sorts ahead of every raise from level ell upward (ties go
                // to the lower level), they all fit, the next does not
                same = true;
                if (bud.ell > 0) {
                    const float vl = a.v[bud.ell - 1], vh = a.v[bud.ell];
                    uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
                    for (uint32_t g = lane; g < n; g += 32) {
                        const float R = __uint_as_float(s_Rb[g]);
                        kmin = min(kmin, __float_as_uint(__fmul_rn(R, vl)));
                        kmax = max(kmax, __float_as_uint(__fmul_rn(R, vh)));
                    }
                    kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
                    kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
                    same = kmin >= kmax;
                }
            }
            uint32_t level = bud.ell;
            if (!same) {
                // (1) rank of every group by (range descending, group ascending): the range list is cut
                //     into slices so that all threads count, a warp reads one range at a time (broadcast)
                const uint32_t slices = n >= kComputeThreads ? 1u : kComputeThreads / n;
                const uint32_t len = (n + slices - 1u) / slices;
                for (uint32_t it = tid; it < n * slices; it += kComputeThreads) {
                    const uint32_t g = it % n, sl = it / n;
                    const uint32_t Rb = s_Rb[g];
                    const uint32_t h1 = min(n, (sl + 1u) * len);
                    uint32_t cnt = 0;
                    for (uint32_t h = sl * len; h < h1; h++) {
                        const uint32_t Rh = s_Rb[h];
                        cnt += (Rh > Rb) || (Rh == Rb && h < g);
                    }
                    if (cnt) atomicAdd(&s_rank[g], cnt);
                }
                bar_sync(kBarCompute, kComputeThreads);
                if (mine) {
                    const uint32_t r = s_rank[tid];
                    s_sorted[r] = (uint32_t)tid;
                    s_sR[r] = __float_as_uint(Rg);
                }
                bar_sync(kBarCompute, kComputeThreads);
                // (2) keys of every level in sorted order
                for (uint32_t it = tid; it < n * nl; it += kComputeThreads) {
                    const uint32_t r = it % n, k = it / n;
                    s_key[k * n_max + r] = __float_as_uint(__fmul_rn(__uint_as_float(s_sR[r]), a.v[k]));
                }
                bar_sync(kBarCompute, kComputeThreads);
                // (3) two different ranges with the same key?
                for (uint32_t it = tid; it < (n - 1u) * nl; it += kComputeThreads) {
                    const uint32_t r = it % (n - 1u), k = it / (n - 1u);
                    if (s_key[k * n_max + r] == s_key[k * n_max + r + 1u] && s_sR[r] != s_sR[r + 1u]) s_coll = 1u;
                }
                bar_sync(kBarCompute, kComputeThreads);
                if (s_coll == 0u) {
                    // (4) position of every candidate in the merged order -> accepted or not
                    for (uint32_t it = tid; it < n * nl; it += kComputeThreads) {
                        const uint32_t r = it % n, k = it / n;
                        const uint32_t key = s_key[k * n_max + r];
                        uint32_t cum = (r + 1u) * a.cost[k];
                        for (uint32_t k2 = 0; k2 < nl; k2++) {
                            if (k2 == k) continue;
                            // number of level-k2 candidates sorting ahead: keys >= key (lower level: ties
                            // first) or keys > key (higher level); the row is non-increasing
                            const uint32_t *row = s_key + k2 * n_max;
                            uint32_t lo_i = 0, hi_i = n;
                            while (lo_i < hi_i) {
                                const uint32_t mid = (lo_i + hi_i) >> 1;
                                const bool ahead = k2 < k ? row[mid] >= key : row[mid] > key;
                                if (ahead) lo_i = mid + 1u; else hi_i = mid;
                            }
                            cum += lo_i * a.cost[k2];
                        }
                        if (cum <= bud.rem) atomicAdd(&s_lvl[s_sorted[r]], 1u);
                    }
                    bar_sync(kBarCompute, kComputeThreads);
                    if (mine) level = s_lvl[tid];
                } else if ((uint32_t)warp < owners) {
                    // Fallback.  For each candidate (group g, raise k) add up the cost of all candidates
                    // that sort at or ahead of it; the candidate is accepted iff that total fits.
                    if (mine) {
#pragma unroll
                        for (int k = 0; k < kMaxLevels - 1; k++) {
                            s_key[k * n_max + tid] = __float_as_uint(__fmul_rn(Rg, a.v[k]));
                            s_cum[k * n_max + tid] = 0u;
                        }
                    }
                    if (owners > 1) bar_sync(kBarOwners, owners * 32u);
                    else __syncwarp();
                    const uint32_t items = n * nl * nl;
                    for (uint32_t it = tid; it < items; it += owners * 32u) {
                        const uint32_t g = it % n, kk = it / n;
                        const uint32_t k = kk / nl, k2 = kk % nl;
                        const uint32_t kg = s_key[k * n_max + g];
                        const uint32_t *row = s_key + k2 * n_max;
                        uint32_t cnt = 0;
                        if (k2 < k) {
                            for (uint32_t h = 0; h < n; h++) cnt += (row[h] >= kg);
                        } else if (k2 > k) {
                            for (uint32_t h = 0; h < n; h++) cnt += (row[h] > kg);
                        } else {
                            for (uint32_t h = 0; h < n; h++) cnt += (row[h] > kg) || (row[h] == kg && h <= g);
                        }
                        atomicAdd(&s_cum[k * n_max + g], cnt * a.cost[k2]);
                    }
                    if (owners > 1) bar_sync(kBarOwners, owners * 32u);
                    else __syncwarp();
                    level = 0;
                    if (mine)
                        for (uint32_t k = 0; k + 1 < m; k++) level += (s_cum[k * n_max + tid] <= bud.rem);
                }
            }
            if ((uint32_t)warp < owners) {
                uint32_t size = 0, b = 0;
                float inv = 0.0f;
                if (mine) {
                    b = a.S[level];
                    const float Lf = (float)((1u << b) - 1u);
                    const float scale = Rg > 0.0f ? __fdiv_rn(Rg, Lf) : 0.0f;
                    inv = Rg > 0.0f ? __fdiv_rn(Lf, Rg) : 0.0f;
                    td.bits[g0 + tid] = (uint8_t)b;
                    td.mn[g0 + tid] = mn;
                    td.scale[g0 + tid] = scale;
                    size = (G >> 3) * b;
                }
                // byte offset of each group inside the window: exclusive scan of the sizes
                uint32_t incl = size;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                    if (lane >= off) incl += y;
                }
                uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 31), before = 0;
                if (owners > 1) {
                    if (lane == 0) s_wtot[warp] = total;
                    bar_sync(kBarOwners, owners * 32u);
                    total = 0;
                    for (uint32_t k = 0; k < owners; k++) {
                        const uint32_t t = s_wtot[k];
                        if (k < (uint32_t)warp) before += t;
                        total += t;
                    }
                    bar_sync(kBarOwners, owners * 32u);           // s_wtot may be rewritten by the next general window
                }
                if (mine) {
                    GroupRec rec;
                    rec.mn = mn;
                    rec.inv = inv;
                    rec.b = b;
                    rec.off = before + incl - size;
                    s_grp[(j & 1u) * n_max + tid] = rec;
                }
                if (tid == 0) {
                    const bool first = (gw == td.first_window);
                    st_relaxed_u64(a.flags + gw, ((first ? kFlagPrefix : kFlagAggregate) << kFlagShift) | total);
                    s_tot[j & 3u] = total;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_wid);
            if (!mbar_wait_bounded(&s_wid, n_generic & 1u)) {     // group records visible to all compute warps
                s_lost = 1u;
                if (lane == 0) record_error(DAF_ERR_TIMEOUT, gw, 7u + 16u * j);
                break;
            }
            n_generic++;
            q_b = 0u;
            q_elems = n_elems;
        }
        q_gw = gw;

        // ---------------------------------------------------------------- window j: stage -> registers, stage released
        {
            constexpr int kChunkBytes = 256 * Elem<T>::kBytes;
#pragma unroll
            for (int c = 0; c < CHUNKS; c++) load8_staged<T, true>(stage + (warp * CHUNKS + c) * kChunkBytes, lane, x[c]);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_cons[j % NSTAGE]);          // stage consumed
    }
    // Out of the loop with windows 0 .. n_packed-1 packed: wake the storer warps, which wait for the
    // windows from n_packed on.  The wake-up goes through the same barriers as a packed
    // window, so it honours the same rule: never before the buffer's previous window has left.
    if (tid == 0) s_end = n_packed;
    for (uint32_t q = n_packed; q < n_packed + NSTO; q++)
        if (q >= 3u) mbar_wait_bounded(&s_free[q % 3u], ((q / 3u) - 1u) & 1u);
    __syncwarp();
    if (lane == 0)
        for (uint32_t q = n_packed; q < n_packed + NSTO; q++) mbar_arrive(&s_ready[q % 3u]);
}

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
// Shared-memory carve-up for one launch configuration.
static SmemLayout make_layout(uint32_t we, uint32_t elem_bytes, uint32_t G, uint32_t window_cap_bytes, uint32_t nstage)
{
    auto up = [](uint32_t v) { return (v + 127u) & ~127u; };
    const uint32_t n_max = we / G, units = we / (G < 256u ? G : 256u);
    SmemLayout l;
    uint32_t at = nstage * up(we * elem_bytes);                   // the stages
    l.out0 = at;
    l.out_stride = up(window_cap_bytes < 16u ? 16u : window_cap_bytes);
    at += 3u * l.out_stride;                                      // three packed-bytes buffers
    l.umn = at; at += up(2u * 4u * units);
    l.umx = at; at += up(2u * 4u * units);
    l.key = at; at += up(4u * (kMaxLevels - 1) * n_max);
    l.cum = at; at += up(4u * (kMaxLevels - 1) * n_max);
    l.grp = at; at += up(2u * 16u * n_max);
    l.srt = at; at += up(2u * 4u * n_max);
    l.total = at;
    return l;
}

// Staged windows per CTA.  Two stages and one CTA per SM measured faster on B200 than one stage
// and two CTAs per SM (which leaves 56 registers per thread and spills).
constexpr uint32_t kStages = 2, kStorers = 2;

template <typename T, int CHUNKS, int NW, int NSTAGE, int NSTO, bool BATCH>
static cudaError_t launch(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    constexpr int kBlock = NW * 32 + 32 + 32 * NSTO;
    static int sms = 0, smem_set = 0, cached_smem = -1, cached_ctas = 0;   // per instantiation, current device
    const int smem = (int)args.lay.total;
    cudaError_t e = cudaSuccess;
    if (sms == 0) {
        int dev = 0;
        e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
    }
    if (smem > smem_set) {
        e = cudaFuncSetAttribute(compress_kernel<T, CHUNKS, NW, NSTAGE, NSTO, BATCH>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        smem_set = smem;
    }
    if (smem != cached_smem) {
        int per_sm = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, compress_kernel<T, CHUNKS, NW, NSTAGE, NSTO, BATCH>, kBlock, smem);
        if (e != cudaSuccess) return e;
        cached_smem = smem;
        cached_ctas = sms * (per_sm > 0 ? per_sm : 1);
    }
    const uint32_t grid = args.total_windows < (uint32_t)cached_ctas ? args.total_windows : (uint32_t)cached_ctas;
    compress_kernel<T, CHUNKS, NW, NSTAGE, NSTO, BATCH><<<grid, kBlock, smem, stream>>>(args);
    return cudaGetLastError();
}

// `chunks4k` = window_elems / 4096: the window is spread over 16 compute warps (a CTA holds at
// most 1024 threads, and the service warps take some of its 32 warp slots).
template <bool BATCH>
static cudaError_t dispatch(uint32_t dtype, uint32_t chunks4k, const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args,
                            cudaStream_t stream)
{
#define DAF_CASE(T)                                                                     \
    switch (chunks4k) {                                                                 \
    case 1: return launch<T, 1, 16, kStages, kStorers, BATCH>(args, stream);            \
    case 2: return launch<T, 2, 16, kStages, kStorers, BATCH>(args, stream);            \
    default: return launch<T, 4, 16, kStages, kStorers, BATCH>(args, stream);           \
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
    a.bulk_store = pl.G >= 128u;                                  // every group is then a multiple of 16 bytes
    a.n_max = pl.We / pl.G;
    const uint32_t elem_bytes = p->dtype == DAF_F32 ? 4u : 2u;
    {
        const uint32_t n = a.n_max;
        a.full_rem = (uint32_t)((((uint64_t)pl.beta_q8 * n) >> 8) - (uint64_t)pl.S[0] * n);
        a.full_ell = 0;
        while (a.full_ell + 1 < pl.m && (pl.S[a.full_ell + 1] - pl.S[0]) * n <= a.full_rem) a.full_ell++;
        a.full_rem_after = a.full_rem - (pl.S[a.full_ell] - pl.S[0]) * n;
    }
    a.nbuf = 3;
    a.lay = make_layout(pl.We, elem_bytes, pl.G, (uint32_t)((((uint64_t)pl.beta_q8 * pl.W) >> 8) * pl.G / 8), kStages);
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

// ------------------------------------------------------------------------------------------
// Compress with the kernel's scratch in a fixed device array instead of a caller's workspace,
// for callers that cannot allocate one (see include/daf.h).  In host code the array's name is
// only a handle: the address a kernel can use comes from cudaGetSymbolAddress, looked up once
// per device with that device current.
// ------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(WorkspaceHeader) + 8ull * DAF_STATIC_MAX_WINDOWS];

extern "C" daf_status daf_compress_static(const daf_params *params, const void *d_in, void *d_packed,
                                          uint64_t packed_capacity, uint8_t *d_bits, float *d_min, float *d_scale,
                                          uint64_t *d_window_offsets, uint32_t *d_status, daf_stream stream)
{
    Plan pl;
    daf_status st = make_plan(params, &pl);
    if (st != DAF_OK) return st;
    if (!d_in || !d_packed || !d_bits || !d_min || !d_scale || !d_window_offsets) return DAF_ERR_INVALID_ARG;
    if (!aligned16(d_in) || !aligned16(d_packed) || (reinterpret_cast<uintptr_t>(d_min) & 3u) ||
        (reinterpret_cast<uintptr_t>(d_scale) & 3u) || (reinterpret_cast<uintptr_t>(d_window_offsets) & 7u) ||
        (reinterpret_cast<uintptr_t>(d_status) & 3u))
        return DAF_ERR_INVALID_ARG;
    if (pl.n_windows > DAF_STATIC_MAX_WINDOWS) return DAF_ERR_CAPACITY;      // the fixed array has no room for more

    // device address of the array, once per device
    constexpr int kMaxDevices = 64;
    static void *scratch_of[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DAF_ERR_CUDA;
    if (!scratch_of[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return DAF_ERR_CUDA;
        scratch_of[dev] = ptr;
    }
    void *scratch = scratch_of[dev];

    CompressArgs<1> a;
    fill_common(a, pl, params, scratch);
    a.total_windows = (uint32_t)pl.n_windows;
    a.n_tensors = 1;
    a.keys = philox_keys(params->seed);
    a.t[0] = TensorDesc{d_in, reinterpret_cast<uint8_t *>(d_packed), packed_capacity, d_bits, d_min, d_scale,
                        d_window_offsets, params->numel, params->elem_index_base, params->seed, 0u,
                        (uint32_t)pl.n_windows};
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    // header (ticket, status) and this call's descriptors must start at zero: the array keeps the last call's contents
    if (cudaMemsetAsync(scratch, 0, pl.workspace, s) != cudaSuccess) return DAF_ERR_CUDA;
    if (dispatch<false>(params->dtype, pl.chunks, a, s) != cudaSuccess) return DAF_ERR_CUDA;
    if (d_status && cudaMemcpyAsync(d_status, scratch, sizeof(uint32_t), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return DAF_ERR_CUDA;
    return DAF_OK;
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
