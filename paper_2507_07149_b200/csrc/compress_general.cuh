// General compress kernel: any mix of widths within a window (Sec. 3.4.1 of the paper: the widths of a
// window's groups are chosen greedily by importance per bit under the window's budget).
//
// A persistent CTA (two per multiprocessor) takes one window at a time, handed out by an atomic ticket.
// Its 16 worker warps never wait for the choice of the window they have just measured, because every
// window passes through the CTA twice, one window apart:
//
//   pass A, window i   : a worker loads its strip (8 * 32 * CHUNKS elements) from HBM, reduces it to
//                        per-group min / max (3-input min/max, warp redux or segmented shuffles) and
//                        leaves these in the window's slot of a small ring in shared memory;
//   decider, window i  : one of two decider warps (they alternate) takes the slot: ranges, importance
//                        keys, the test for a window of one width, else the greedy choice (threshold
//                        search on the keys, ties in level / group order), byte offsets of the groups by
//                        an exclusive scan, the window's offset in the packed buffer by a bounded decoupled
//                        look-back over the other CTAs' windows, 1/scale and scale by IEEE division, group
//                        records into the slot, metadata and the window offset to global memory;
//   pass B, window i-1 : the worker loads the same strip of the previous window again (it is still in
//                        L2), and with the group records of that window: Eq. 1 with stochastic rounding
//                        (Philox4x32-10, the float -> uint step by the power-of-two offset of Eq. 5),
//                        lane-local LSB-first packing at the group's width, stores straight to the
//                        group's place in the packed buffer.
//
// So the input crosses HBM once and L2 twice, nothing of a window lives in registers or shared memory
// between the passes, and the decider has a whole window's time before anybody asks for its result.
// Every wait is bounded: on a timeout the status word is set, the window's descriptor is poisoned (so
// that the CTAs behind it stop too) and the CTA leaves.
//
// Windows are handed out by ticket, so every window with a smaller index than the one a CTA holds
// belongs to a CTA that is running (or done) and the look-back always makes progress.
#pragma once
#include <type_traits>

#include "compress_shared.cuh"

namespace daf {

namespace general {

constexpr int kWorkers = kWarps;                                  // 16 worker warps: one strip of the window each
constexpr int kDeciders = 2;
constexpr int kCtaThreads = 32 * (kWorkers + kDeciders);
constexpr int kLag = 3;                                           // pass B runs this many windows behind pass A
constexpr int kRing = kLag + 2;                                   // window slots

struct WinHead {                                                  // fixed part of a window's slot
    uint64_t stats_in;        // mbarrier: every worker's min / max of the window are in (one arrival per worker)
    uint64_t ready;           // mbarrier: the decider has settled the window (one arrival)
    unsigned char *out;       // where the window's packed bytes go
    uint32_t n_elems;         // elements of the window
    uint32_t store;           // 0: the window's packed bytes must not be stored (no room, or a window before it failed)
    uint32_t ti;              // tensor of the window (batched calls)
    uint32_t pad[3];
    uint32_t rkeys[20];       // Philox round keys of the window's tensor (batched calls)
};
static_assert(sizeof(WinHead) % 16 == 0, "arrays behind the head stay 16-byte aligned");

// Slot layout behind the head: rec[n_max] (16 bytes each), umn[units], umx[units], mn[n_max], R[n_max], key[3][n_max].
struct SlotLayout {
    uint32_t rec, umn, umx, mn, R, key, bytes;
};
__host__ __device__ inline SlotLayout slot_layout(uint32_t n_max, uint32_t units)
{
    SlotLayout l;
    uint32_t at = (uint32_t)sizeof(WinHead);
    l.rec = at; at += 16u * n_max;
    l.umn = at; at += 4u * units;
    l.umx = at; at += 4u * units;
    l.mn = at; at += 4u * n_max;
    l.R = at; at += 4u * n_max;
    l.key = at; at += 12u * n_max;
    l.bytes = (at + 15u) & ~15u;
    return l;
}

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
__device__ __forceinline__ uint32_t ld_volatile_shared(const uint32_t *p) { return *reinterpret_cast<const volatile uint32_t *>(p); }
__device__ __forceinline__ void st_volatile_shared(uint32_t *p, uint32_t v) { *reinterpret_cast<volatile uint32_t *>(p) = v; }

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

// Eight codes of the lane at width b (1, 2, 4 or 8) -> packed bytes at p.  CLAMP: the group's 1/scale is not a
// normal number, so a code may pass 2^b - 1 and must be clamped.  wide8: an 8-byte store is aligned.
template <bool CLAMP>
__device__ __forceinline__ void quantize_store(uint32_t b, const float (&x)[8], float mn, float inv, const uint32_t (&o)[4],
                                               unsigned char *p, bool wide8)
{
    uint32_t w0, w1;
    switch (b) {
    case 1:
        quantize8<1, CLAMP>(x, mn, inv, o, w0, w1);
        *p = (unsigned char)w0;
        break;
    case 2:
        quantize8<2, CLAMP>(x, mn, inv, o, w0, w1);
        *reinterpret_cast<uint16_t *>(p) = (uint16_t)w0;
        break;
    case 4:
        quantize8<4, CLAMP>(x, mn, inv, o, w0, w1);
        *reinterpret_cast<uint32_t *>(p) = w0;
        break;
    default:
        quantize8<8, CLAMP>(x, mn, inv, o, w0, w1);
        if (wide8) {
            *reinterpret_cast<uint2 *>(p) = make_uint2(w0, w1);
        } else {                                                  // groups of 32 elements are only 4-byte aligned
            reinterpret_cast<uint32_t *>(p)[0] = w0;
            reinterpret_cast<uint32_t *>(p)[1] = w1;
        }
        break;
    }
}

// ------------------------------------------------------------------------------------------
// The greedy of Sec. 3.4.1 on one warp, candidates in registers.  Every lane holds NK candidate raises (key, cw =
// cost | 1 << 16, or cw = 0 for "no candidate"); slot s of lane l sorts, among equal keys, before slot s' > s of
// any lane and before slot s of lane l' > l.  Accepted is the longest prefix, in the order (key descending, then
// that order), whose summed cost is at most rem; take[s] says whether this lane's slot s is in it.  F(t), the cost
// of all raises with key >= t, falls as t grows, so the prefix is every raise with a key above Kp, the largest t
// with F(t) > rem, and then the raises with key Kp in order while they fit.  One warp reduction gives F(t) and N(t),
// the number of raises with key >= t; the interval that holds Kp starts from the keys' common leading bits and is
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

}  // namespace general

// Development aid: time stamps of the first CTA's deciders into the (here unused) first descriptor array.
#ifdef DAF_STAMPS
#define DAF_GSTAMP(k) do { if (blockIdx.x == 0 && lane == 0 && it < 24u) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); a.flags[it * 8u + (k)] = t_; } } while (0)
#else
#define DAF_GSTAMP(k) do { } while (0)
#endif

template <typename T, int CHUNKS, bool BATCH, bool RELU>
__global__ void __launch_bounds__(general::kCtaThreads, 2)
general_compress_kernel(const __grid_constant__ CompressArgs<BATCH ? DAF_BATCH_MAX : 1> a)
{
    using namespace general;
    constexpr uint32_t STRIP = 256u * CHUNKS;                     // elements per worker and window
    constexpr uint32_t WE = kWorkers * STRIP;
    constexpr uint32_t EB = Elem<T>::kBytes;

    extern __shared__ __align__(16) unsigned char smem[];        // kRing window slots
    __shared__ uint32_t s_gw[kRing];                              // window of iteration i (slot i % kRing)
    __shared__ uint32_t s_tag[kRing];                             // i + 1 once that window is known
    __shared__ uint32_t s_claim;                                  // the last iteration whose window somebody has set out to draw
    __shared__ uint32_t s_abort;                                  // a wait ran out, or a window before ours failed: the CTA leaves

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (a.gated != 0u && *reinterpret_cast<volatile unsigned int *>(&a.hdr->retry) == 0u) return;   // nothing to redo

    const uint32_t G = a.G, log2G = a.log2G, n_max = a.n_max;
    const uint32_t units = G >= 256u ? WE / 256u : n_max;         // min / max are left per chunk, or per group when groups are smaller
    const SlotLayout lay = slot_layout(n_max, units);
    auto head = [&](uint32_t it) -> WinHead & { return *reinterpret_cast<WinHead *>(smem + (it % kRing) * lay.bytes); };
    auto slot_at = [&](uint32_t it, uint32_t off) -> unsigned char * { return smem + (it % kRing) * lay.bytes + off; };

    if (tid < kRing) {
        WinHead &h = *reinterpret_cast<WinHead *>(smem + tid * lay.bytes);
        bar_init(&h.stats_in, kWorkers);
        bar_init(&h.ready, 1u);
    }
    if (tid == 0) {
        s_abort = 0u;
        s_gw[0] = atomicAdd(&a.hdr->ticket2, 1u);
        s_tag[0] = 1u;
        for (int r = 1; r < kRing; r++) s_tag[r] = 0u;
        s_claim = 0u;
    }
    __syncthreads();

    auto tensor_index = [&](uint32_t gw) -> uint32_t {            // last tensor whose first window is <= gw
        if (!BATCH) return 0u;
        uint32_t lo = 0, hi = a.n_tensors - 1;
        while (lo < hi) {
            const uint32_t mid = (lo + hi + 1) >> 1;
            if (a.t[mid].first_window <= gw) lo = mid; else hi = mid - 1;
        }
        return lo;
    };
    auto record_error = [&](unsigned code, uint32_t window, uint32_t site) {
        if (atomicCAS(&a.hdr->status, 0u, code) == 0u) {
            a.hdr->fail_window = window;
            a.hdr->fail_site = site;
        }
    };
    // Bounded wait on a slot's barrier; false: the CTA is leaving (somebody gave up, or this wait ran out).
    auto wait = [&](uint64_t *bar, uint32_t parity, uint32_t gw, uint32_t site) -> bool {
        for (unsigned polls = 0;; polls++) {
            if (bar_try_wait(bar, parity)) return true;
            if (ld_volatile_shared(&s_abort) != 0u) return false;
            if (polls > a.poll_limit) {
                if (lane == 0) record_error(DAF_ERR_TIMEOUT, gw, site);
                st_volatile_shared(&s_abort, 1u);
                return false;
            }
            if (polls > 2u) __nanosleep(64);
        }
    };

    if (warp >= kWorkers) {
        // ============================================================ decider warps: warp d settles windows d, d + 2, ...
        const uint32_t nl = a.m - 1u;                             // raises per group
        uint32_t pend_it = 0xFFFFFFFFu, pend_gw = 0u, pend_total = 0u;   // the window whose place is still to be looked up
        // Looks up the pending window's place in the packed buffer (bounded decoupled look-back over the windows
        // before it), publishes its inclusive prefix, writes its offset and lets the workers have the slot.
        // block: wait (bounded) for the windows before it; else give up for now when one of them has not published yet.
        auto finish = [&](bool block) {
            if (pend_it == 0xFFFFFFFFu) return;
            WinHead &ph = head(pend_it);
            const TensorDesc &td = a.t[BATCH ? ph.ti : 0u];
            const uint32_t w = pend_gw - td.first_window;
            uint64_t excl = 0;
            int state = 1;
            if (w != 0u) {
                state = lookback<kLookDepth>(a.flags2, pend_gw, td.first_window, lane, block, a.poll_limit, &excl);
                if (state == 0) return;                           // not yet
                if (lane == 0)
                    st_relaxed_u64(a.flags2 + pend_gw, state == 1 ? ((kFlagPrefix << kFlagShift) | (excl + pend_total))
                                                                   : (kFlagPoison << kFlagShift));
            }
            bool store = state == 1;
            if (store) {
                if (lane == 0) {
                    td.woff[w] = excl;
                    if (w + 1u == td.n_windows) td.woff[w + 1u] = excl + pend_total;
                }
                if (excl + pend_total > td.capacity) {            // no room: nothing of the window is stored
                    store = false;
                    if (lane == 0) record_error(DAF_ERR_CAPACITY, pend_gw, 12u);
                }
            } else {
                if (state == -2 && lane == 0) record_error(DAF_ERR_TIMEOUT, pend_gw, 13u);   // (a poisoned predecessor has reported itself)
                st_volatile_shared(&s_abort, 1u);                 // the windows behind a failed one are lost: the CTA leaves
            }
            if (lane == 0) {
                ph.out = td.packed + excl;
                ph.store = store ? 1u : 0u;
            }
            __syncwarp();
            if (lane == 0) bar_arrive(&ph.ready);                 // (release: the slot is visible to who sees the phase)
            pend_it = 0xFFFFFFFFu;
        };
        for (uint32_t it = (uint32_t)warp - kWorkers;; it += kDeciders) {
            WinHead &h = head(it);
            // wait for the window's statistics; meanwhile keep trying to place the window this warp settled last
            bool go = true;
            for (unsigned polls = 0;; polls++) {
                if (bar_try_wait(&h.stats_in, (it / kRing) & 1u)) break;
                if (ld_volatile_shared(&s_abort) != 0u) { go = false; break; }
                if (polls > a.poll_limit) {
                    if (lane == 0) record_error(DAF_ERR_TIMEOUT, 0xFFFFFFFFu, 11u);
                    st_volatile_shared(&s_abort, 1u);
                    go = false;
                    break;
                }
                if (pend_it != 0xFFFFFFFFu) finish(false);
                else __nanosleep(200);
            }
            finish(true);                                         // (the workers ask for that window next)
            if (!go) break;
            const uint32_t gw = ld_volatile_shared(&s_gw[it % kRing]);
            if (gw >= a.total_windows) break;
            DAF_GSTAMP(0);
            const uint32_t ti = tensor_index(gw);
            const TensorDesc &td = a.t[ti];
            const uint32_t w = gw - td.first_window;
            uint32_t n_elems = WE;
            if (w + 1u == td.n_windows) n_elems = (uint32_t)(td.numel - (uint64_t)w * WE);
            const uint32_t n = n_elems >> log2G;                  // groups of the window
            const uint64_t g0 = (uint64_t)w * n_max;              // first group of the window in the tensor
            GroupRec *const rec = reinterpret_cast<GroupRec *>(slot_at(it, lay.rec));
            const float *const umn = reinterpret_cast<const float *>(slot_at(it, lay.umn));
            const float *const umx = reinterpret_cast<const float *>(slot_at(it, lay.umx));
            float *const s_mn = reinterpret_cast<float *>(slot_at(it, lay.mn));
            float *const s_R = reinterpret_cast<float *>(slot_at(it, lay.R));
            uint32_t *const s_key = reinterpret_cast<uint32_t *>(slot_at(it, lay.key));   // [level][group]

            // ---- budget arithmetic of the window
            uint32_t ell = a.full_ell, rem = a.full_rem, rem_after = a.full_rem_after;
            if (n != n_max) {                                     // ragged last window: work it out here
                rem = (uint32_t)((((uint64_t)a.beta_q8 * n) >> 8) - (uint64_t)a.S[0] * n);
                ell = 0;
                while (ell + 1 < a.m && (a.S[ell + 1] - a.S[0]) * n <= rem) ell++;
                rem_after = rem - (a.S[ell] - a.S[0]) * n;
            }
            const bool all_max = ell + 1 == a.m;
            const bool need_sep = !all_max && rem_after < a.cost[ell];   // the best raise out of level ell does not fit

            // ---- ranges and importance keys of the groups (group g: lane g % 32)
            const uint32_t upg = G > 256u ? G >> 8 : 1u;          // units per group
            uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;               // smallest key into level ell, largest key out of it
            for (uint32_t g = lane; g < n; g += 32u) {
                float lo = umn[g * upg], hi = umx[g * upg];
                for (uint32_t j = 1; j < upg; j++) {
                    lo = fmin2(lo, umn[g * upg + j]);
                    hi = fmax2(hi, umx[g * upg + j]);
                }
                float R = __fsub_rn(hi, lo);
                if (R < 0x1p-118f) R = 0.0f;                      // degenerate group: constant
                s_mn[g] = lo;
                s_R[g] = R;
                for (uint32_t k = 0; k < nl; k++) {
                    const uint32_t key = __float_as_uint(__fmul_rn(R, a.v[k]));
                    s_key[k * n_max + g] = key;
                    if (k + 1u == ell) kmin = min(kmin, key);
                    if (k == ell) kmax = max(kmax, key);
                }
            }
            __syncwarp();
            // One width for all: every group reaches level ell (by the definition of ell that fits) and no raise out of it
            // is taken, which needs every raise into level ell to sort ahead of every raise out of it (ties go to the lower
            // level; a group's raises appear in level order, so the levels below and above follow).
            bool uniform = all_max || need_sep;
            if (need_sep && ell > 0u) {
                kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
                kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
                uniform = kmin >= kmax;
            }

            DAF_GSTAMP(1);
            // ---- general choice (Sec. 3.4.1): the greedy accepts the longest prefix of the raises, sorted by (key
            // descending, level ascending, group ascending), whose summed cost fits.  F(t), the cost of all raises with
            // key >= t, falls as t grows, so the prefix is every raise with a key above Kp = max{t : F(t) > rem}, and then
            // the raises with key Kp in order while they fit.  Kp is built bit by bit from the top.
            uint32_t Kp = 0u, left = 0u;                          // left: budget after every raise with a key above Kp
            uint32_t fit[3] = {0u, 0u, 0u};                       // raises of level k with key Kp that are accepted
            uint32_t level_reg[4] = {0u, 0u, 0u, 0u};             // up to 128 groups: the levels come out of the register version
            const bool in_regs = !uniform && n <= 128u;
            if (in_regs) {
                // candidates in registers: slot k * Q + q is raise k of group q * 32 + lane
                auto run = [&](auto qtag) {
                    constexpr int Q = decltype(qtag)::value;
                    uint32_t key[3 * Q], cw[3 * Q], slot_cost[3 * Q];
                    bool take[3 * Q];
#pragma unroll
                    for (int k = 0; k < 3; k++)
#pragma unroll
                        for (int q = 0; q < Q; q++) {
                            const uint32_t g = (uint32_t)lane + 32u * q;
                            const bool on = (uint32_t)k < nl && g < n;
                            key[k * Q + q] = on ? s_key[k * n_max + g] : 0u;
                            cw[k * Q + q] = on ? a.cost[k] | 0x10000u : 0u;
                            slot_cost[k * Q + q] = a.cost[k];
                        }
                    accept_prefix<3 * Q, false>(key, cw, slot_cost, rem, 0u, 0u, lane, take);
#pragma unroll
                    for (int q = 0; q < Q; q++) level_reg[q] = (uint32_t)take[q] + take[Q + q] + take[2 * Q + q];
                };
                if (n <= 64u) run(std::integral_constant<int, 2>{});
                else run(std::integral_constant<int, 4>{});
            }
            if (!uniform && !in_regs) {
                auto from = [&](uint32_t t) -> uint32_t {         // F(t) | (number of raises with key >= t) << 16
                    uint32_t f = 0u;
                    for (uint32_t k = 0; k < nl; k++) {
                        const uint32_t cw = a.cost[k] | 0x10000u;
                        for (uint32_t g = lane; g < n; g += 32u) f += s_key[k * n_max + g] >= t ? cw : 0u;
                    }
                    return __reduce_add_sync(0xFFFFFFFFu, f);
                };
                uint32_t at_lo = from(0u), at_hi = 0u;            // F | N at the two ends of the interval that holds Kp
                if ((at_lo & 0xFFFFu) > rem) {
                    uint32_t khi = 0u, klo = 0xFFFFFFFFu;
                    for (uint32_t k = 0; k < nl; k++)
                        for (uint32_t g = lane; g < n; g += 32u) {
                            khi = max(khi, s_key[k * n_max + g]);
                            klo = min(klo, s_key[k * n_max + g]);
                        }
                    khi = __reduce_max_sync(0xFFFFFFFFu, khi);
                    klo = __reduce_min_sync(0xFFFFFFFFu, klo);
                    const uint32_t diff = khi ^ klo;
                    int bit = diff != 0u ? 31 - __clz(diff) : -1; // the interval is [Kp, Kp + 2^(bit+1))
                    Kp = diff != 0u ? khi & ~((2u << bit) - 1u) : khi;
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
                    if (bit >= 0) {                               // one raise left in the interval: Kp is its key
                        const uint32_t sh = (uint32_t)bit + 1u;
                        uint32_t only = 0u;
                        for (uint32_t k = 0; k < nl; k++)
                            for (uint32_t g = lane; g < n; g += 32u) {
                                const uint32_t key = s_key[k * n_max + g];
                                if (sh >= 32u || (key >> sh) == (Kp >> sh)) only = max(only, key);
                            }
                        Kp = __reduce_max_sync(0xFFFFFFFFu, only);
                    }
                } else {
                    at_hi = from(1u);                             // every raise with a positive key fits (Kp = 0)
                }
                left = rem - (at_hi & 0xFFFFu);
                // raises with key Kp: level by level, group by group, while they fit; the walk stops at the first that does not
                bool open = true;
                for (uint32_t k = 0; k < nl; k++) {
                    uint32_t ties = 0u;
                    for (uint32_t g = lane; g < n; g += 32u) ties += s_key[k * n_max + g] == Kp ? 1u : 0u;
                    ties = __reduce_add_sync(0xFFFFFFFFu, ties);
                    if (ties != 0u && open) {
                        fit[k] = min(ties, left / a.cost[k]);
                        left -= fit[k] * a.cost[k];
                        open = fit[k] == ties;
                    }
                }
            }

            DAF_GSTAMP(2);
            // ---- widths, byte offsets of the groups within the window (exclusive scan in group order), records
            uint32_t run = 0u;                                    // bytes of the groups before this round of 32
            uint32_t seen[3] = {0u, 0u, 0u};                      // raises with key Kp met so far, per level
            bool clamp_any = false;
            for (uint32_t g32 = 0; g32 < n; g32 += 32u) {
                const uint32_t g = g32 + (uint32_t)lane;
                const bool on = g < n;
                uint32_t level = ell;
                if (in_regs) {
                    level = level_reg[(g32 >> 5) & 3u];
                } else if (!uniform) {
                    level = 0u;
                    for (uint32_t k = 0; k < nl; k++) {
                        const uint32_t key = on ? s_key[k * n_max + g] : 0u;
                        const bool tie = on && key == Kp;
                        const uint32_t tmask = __ballot_sync(0xFFFFFFFFu, tie);
                        const uint32_t rank = seen[k] + (uint32_t)__popc(tmask & ((1u << lane) - 1u));
                        if (on && (key > Kp || (tie && rank < fit[k]))) level++;
                        seen[k] += (uint32_t)__popc(tmask);
                    }
                }
                const uint32_t b = a.S[level], size = on ? (G >> 3) * b : 0u;
                uint32_t incl = size;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (lane >= o) incl += y;
                }
                if (on) {
                    const float R = s_R[g], mn = s_mn[g];
                    const float Lf = (float)((1u << b) - 1u);
                    const bool pos = R > 0.0f;
                    const float inv = pos ? __fdiv_rn(Lf, R) : 0.0f;
                    const bool clamp = pos && inv < 0x1p-126f;    // 1/scale not a normal number: codes may pass 2^b - 1
                    clamp_any |= clamp;
                    GroupRec r;
                    r.mn = mn;
                    r.inv = inv;
                    r.b = b | (clamp ? 0x100u : 0u);
                    r.off = run + incl - size;
                    rec[g] = r;
                    td.bits[g0 + g] = (uint8_t)b;
                    td.mn[g0 + g] = mn;
                    td.scale[g0 + g] = pos ? __fdiv_rn(R, Lf) : 0.0f;
                }
                run += __shfl_sync(0xFFFFFFFFu, incl, 31);
            }
            const uint32_t total = run;                           // packed bytes of the window

            DAF_GSTAMP(3);
            // ---- publish the window's size at once; its place in the packed buffer is looked up when this warp comes
            // back for its next window, two iterations from now, when the windows before it have long published theirs
            if (lane == 0) st_relaxed_u64(a.flags2 + gw, ((w == 0u ? kFlagPrefix : kFlagAggregate) << kFlagShift) | total);
            if (BATCH && lane < 10) philox_store_round_keys(h.rkeys, td.seed, lane);
            if (lane == 0) {
                h.n_elems = n_elems;
                h.ti = ti;
            }
            pend_it = it;
            pend_gw = gw;
            pend_total = total;
            finish(false);                                        // (a tensor's first window, or windows before it that are all placed)
            (void)clamp_any;
        }
        return;
    }

    // ================================================================ worker warps
    const uint32_t strip0 = (uint32_t)warp * STRIP;               // the strip's first element within its window
    const uint32_t e0 = strip0 + (uint32_t)lane * 8u;             // the lane's first element of chunk 0
    uint32_t hist[kLag];                                          // windows of the last kLag iterations (hist[0]: the oldest)
#pragma unroll
    for (int j = 0; j < kLag; j++) hist[j] = 0xFFFFFFFFu;
    uint32_t drain = 0;                                           // iterations since the windows ran out
    for (uint32_t it = 0;; it++) {
        // ---- this iteration's window (drawn by the first worker that finished pass A of the iteration before)
        uint32_t gw = 0xFFFFFFFFu;
        if (drain == 0u) {
            unsigned polls = 0;
            while (ld_volatile_shared(&s_tag[it % kRing]) != it + 1u) {
                if (ld_volatile_shared(&s_abort) != 0u) break;
                if (++polls > a.poll_limit) {
                    if (lane == 0) record_error(DAF_ERR_TIMEOUT, 0xFFFFFFFFu, 15u);
                    st_volatile_shared(&s_abort, 1u);
                    break;
                }
                __nanosleep(32);
            }
            __threadfence_block();
            gw = ld_volatile_shared(&s_gw[it % kRing]);
        }
        const bool valid = gw < a.total_windows;
        if (ld_volatile_shared(&s_abort) != 0u) break;

        // ---- pass A: min / max of this window's strip into its slot
        if (valid) {
            const TensorDesc &td = a.t[tensor_index(gw)];
            const uint32_t w = gw - td.first_window;
            uint32_t n_elems = WE;
            if (w + 1u == td.n_windows) n_elems = (uint32_t)(td.numel - (uint64_t)w * WE);
            float *const umn = reinterpret_cast<float *>(slot_at(it, lay.umn));
            float *const umx = reinterpret_cast<float *>(slot_at(it, lay.umx));
            const char *const src = reinterpret_cast<const char *>(td.in) + ((uint64_t)w * WE + e0) * EB;
            float x[CHUNKS][8];
#pragma unroll
            for (int c = 0; c < CHUNKS; c++) {
#pragma unroll
                for (int i = 0; i < 8; i++) x[c][i] = 0.0f;
                if (e0 + 256u * c < n_elems) Elem<T>::load8_keep(src + 256u * EB * c, x[c]);
            }
#pragma unroll
            for (int c = 0; c < CHUNKS; c++) {
                if (RELU) {
#pragma unroll
                    for (int i = 0; i < 8; i++) x[c][i] = fmaxf(x[c][i], 0.0f);
                }
                float lo, hi;
                extremes8(x[c], lo, hi);
                if (G >= 256u) {
                    lo = warp_min(lo);
                    hi = warp_max(hi);
                    if (lane == 0) {
                        umn[warp * CHUNKS + c] = lo;
                        umx[warp * CHUNKS + c] = hi;
                    }
                } else {
                    const uint32_t lpg = G >> 3;                  // lanes per group
                    for (uint32_t off = 1; off < lpg; off <<= 1) {
                        lo = fmin2(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, off));
                        hi = fmax2(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, off));
                    }
                    if (((uint32_t)lane & (lpg - 1u)) == 0u) {
                        const uint32_t u = (strip0 + 256u * c + (uint32_t)lane * 8u) >> log2G;
                        umn[u] = lo;
                        umx[u] = hi;
                    }
                }
            }
        }
        __syncwarp();
        // (also for "no more windows": the decider then leaves; the other decider learns it one iteration later)
        if (lane == 0 && drain < 2u) bar_arrive(&head(it).stats_in);
        // ---- the next iteration's window: whoever gets here first draws the ticket (just in time, so that windows are
        // taken up in the order of their numbers, which the look-back relies on)
        if (lane == 0 && drain == 0u && atomicCAS(&s_claim, it, it + 1u) == it) {
            const uint32_t next = valid ? atomicAdd(&a.hdr->ticket2, 1u) : 0xFFFFFFFFu;   // (none once the windows have run out)
            st_volatile_shared(&s_gw[(it + 1u) % kRing], next);
            __threadfence_block();
            st_volatile_shared(&s_tag[(it + 1u) % kRing], it + 2u);
        }

        // ---- pass B: quantize, pack and store the strip of the window of kLag iterations ago with the records its
        // decider has left
        const uint32_t gw_prev = hist[0];
        if (gw_prev != 0xFFFFFFFFu) {
            WinHead &h = head(it - kLag);
            if (!wait(&h.ready, ((it - kLag) / kRing) & 1u, gw_prev, 14u)) break;
            const uint32_t n_elems = h.n_elems;
            if (h.store != 0u) {
                const TensorDesc &td = a.t[BATCH ? h.ti : 0u];
                const uint32_t w = gw_prev - td.first_window;
                const GroupRec *const rec = reinterpret_cast<const GroupRec *>(slot_at(it - kLag, lay.rec));
                unsigned char *const out = h.out;
                const char *const src = reinterpret_cast<const char *>(td.in) + ((uint64_t)w * WE + e0) * EB;
                char *const act = RELU ? reinterpret_cast<char *>(td.act) + ((uint64_t)w * WE + e0) * EB : nullptr;
                const uint64_t blk0 = (td.elem_base >> 3) + (uint64_t)w * (WE >> 3) + (e0 >> 3);
                float x[CHUNKS][8];
#pragma unroll
                for (int c = 0; c < CHUNKS; c++) {
#pragma unroll
                    for (int i = 0; i < 8; i++) x[c][i] = 0.0f;
                    if (e0 + 256u * c < n_elems) Elem<T>::load8(src + 256u * EB * c, x[c]);
                }
#pragma unroll
                for (int c = 0; c < CHUNKS; c++) {
                    const uint32_t e = e0 + 256u * c;
                    if (e >= n_elems) continue;                   // (groups are whole: the lane's group exists iff its elements do)
                    if (RELU) {
                        // fused producer: what is compressed (and written out) is max(x, +0); the lane stores what it loaded,
                        // and nobody reads this window's input again, so the output may be the input buffer
#pragma unroll
                        for (int i = 0; i < 8; i++) x[c][i] = fmaxf(x[c][i], 0.0f);
                        Elem<T>::store8(act + 256u * EB * c, x[c]);
                    }
                    const GroupRec r = rec[e >> log2G];
                    uint32_t o[4];
                    if (a.nearest) {
                        o[0] = o[1] = o[2] = o[3] = 0x80008000u;   // every 16-bit lane = 2 * 2^14: round half up
                    } else {
                        const uint64_t blk = blk0 + 32u * c;
                        if (BATCH) {
                            const PhiloxSharedKeys sk{reinterpret_cast<const uint4 *>(h.rkeys)};
                            philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), sk, o);
                        } else {
                            philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), a.keys, o);
                        }
                    }
                    const uint32_t b = r.b & 0xFFu;
                    unsigned char *const p = out + r.off + ((e & (G - 1u)) >> 3) * b;
                    if (r.b & 0x100u) quantize_store<true>(b, x[c], r.mn, r.inv, o, p, G >= 64u);
                    else quantize_store<false>(b, x[c], r.mn, r.inv, o, p, G >= 64u);
                }
            }
        }
#pragma unroll
        for (int j = 0; j + 1 < kLag; j++) hist[j] = hist[j + 1];
        hist[kLag - 1] = valid ? gw : 0xFFFFFFFFu;
        if (!valid && ++drain > (uint32_t)kLag) break;            // the last windows have been through pass B
    }
    // A CTA that leaves early poisons the windows it has drawn and not settled, so that nobody waits for them.
    if (tid == 0 && ld_volatile_shared(&s_abort) != 0u) {
        for (uint32_t r = 0; r < (uint32_t)kRing; r++) {
            const uint32_t g = ld_volatile_shared(&s_gw[r]);
            if (g < a.total_windows) atomicCAS(reinterpret_cast<unsigned long long *>(a.flags2 + g), 0ull, (unsigned long long)(kFlagPoison << kFlagShift));
        }
    }
}

template <typename T, int CHUNKS, bool BATCH, bool RELU>
static cudaError_t launch_general(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    const uint32_t units = args.G >= 256u ? (uint32_t)kWarps * CHUNKS : args.n_max;
    const int smem = (int)(general::kRing * general::slot_layout(args.n_max, units).bytes);
    int ctas = 0;
    const cudaError_t e = persistent_ctas(reinterpret_cast<const void *>(&general_compress_kernel<T, CHUNKS, BATCH, RELU>),
                                          general::kCtaThreads, smem, &ctas);
    if (e != cudaSuccess) return e;
    const uint32_t grid = args.total_windows < (uint32_t)ctas ? args.total_windows : (uint32_t)ctas;
    general_compress_kernel<T, CHUNKS, BATCH, RELU><<<grid, general::kCtaThreads, smem, stream>>>(args);
    return cudaGetLastError();
}

template <typename T, bool BATCH, bool RELU>
cudaError_t dispatch_general_t(uint32_t chunks, const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    if constexpr (RELU) {                                         // fused producer: single tensor, default window
        return launch_general<T, 4, false, true>(args, stream);
    } else {
        if (chunks == 1) return launch_general<T, 1, BATCH, false>(args, stream);
        if (chunks == 2) return launch_general<T, 2, BATCH, false>(args, stream);
        return launch_general<T, 4, BATCH, false>(args, stream);
    }
}

#define DAF_INSTANTIATE_GENERAL(T)                                                                                          \
    template cudaError_t dispatch_general_t<T, false, false>(uint32_t, const CompressArgs<1> &, cudaStream_t);              \
    template cudaError_t dispatch_general_t<T, true, false>(uint32_t, const CompressArgs<DAF_BATCH_MAX> &, cudaStream_t);   \
    template cudaError_t dispatch_general_t<T, false, true>(uint32_t, const CompressArgs<1> &, cudaStream_t);

}  // namespace daf
