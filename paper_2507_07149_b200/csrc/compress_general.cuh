// General compress kernel: any mix of widths within a window.  A persistent CTA (two per
// multiprocessor) processes one window (window_elems elements) at a time and reads the input from
// HBM exactly once.
//
//   - the next window is staged into shared memory by one bulk asynchronous copy (TMA,
//     completion on an mbarrier) while the current one is processed;
//   - staged window -> registers (8 consecutive elements per lane and chunk), per-group
//     min / max (3-input min/max, warp redux or segmented shuffles);
//   - per-window greedy bit-width choice (Sec. 3.4.1 of the paper: importance per bit): a quick
//     test recognises windows whose groups all end at the same width; the general case finds
//     the key at which the accepted prefix of the sorted raises ends without sorting them (a
//     bitwise search by one warp for up to 64 groups, a radix select by the owner warps above);
//   - intra-window exclusive scan of the group byte lengths; the window's byte count is
//     published at once in a 64-bit descriptor;
//   - Eq. 1 quantization with stochastic rounding (Philox4x32-10, 16 bits per element, the
//     float -> uint step done with the power-of-two offset of Eq. 5) and lane-local LSB-first
//     packing into a shared-memory buffer;
//   - the window's device-wide byte offset comes from a bounded decoupled look-back over the
//     descriptors, done one window later by a warp of its own, so that the compute warps never
//     wait for other CTAs; the packed window then leaves shared memory as one bulk asynchronous
//     store.
//
// Windows are handed out by an atomic ticket, so every window with a smaller index than the
// one a CTA holds is owned by a running (or finished) CTA and the look-back always makes
// progress; every wait is bounded all the same: on a timeout the status word is set, the
// window's descriptor is poisoned (so that the CTAs behind it stop too) and the CTA leaves.
//
// Calls whose windows all end with one width are served faster by the streaming kernel
// (compress_stream.cuh); this kernel runs behind it and returns at once unless it was asked for.
// This header is included by one translation unit per element type.
#pragma once
#include "compress_shared.cuh"

namespace daf {

// Staged window -> registers, then min / max per unit of LPU lanes (a full warp uses the
// redux instruction) written to shared memory.  Chunks past a ragged window's end read
// stale bytes; their results are never used.
template <typename T, int CHUNKS, int LPU, int ACT>
__device__ __forceinline__ void load_and_reduce(const unsigned char *stage, int warp, int lane, float (&x)[CHUNKS][8],
                                                float *s_umn, float *s_umx)
{
    constexpr int kChunkBytes = 256 * Elem<T>::kBytes;
#pragma unroll
    for (int c = 0; c < CHUNKS; c++) load8_staged<T>(stage + (warp * CHUNKS + c) * kChunkBytes, lane, x[c]);
    if (ACT == kActRelu || ACT == kActRelu6) {                   // fused producer: what is compressed is the activation
#pragma unroll
        for (int c = 0; c < CHUNKS; c++) {
            float y[8];
            activate8<ACT>(x[c], y);
        }
    }
#pragma unroll
    for (int c = 0; c < CHUNKS; c++) {
        float lo = fmin3(fmin3(x[c][0], x[c][1], x[c][2]), fmin3(x[c][3], x[c][4], x[c][5]), fmin2(x[c][6], x[c][7]));
        float hi = fmax3(fmax3(x[c][0], x[c][1], x[c][2]), fmax3(x[c][3], x[c][4], x[c][5]), fmax2(x[c][6], x[c][7]));
        if (LPU == 32) {
            asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(lo) : "f"(lo));
            asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(hi) : "f"(hi));
        } else if (LPU == 16) {
            // two units per chunk: a warp-wide reduction for each half, the other half's lanes holding the identity
            const bool upper = lane >= 16;
            const float inf = __uint_as_float(0x7F800000u), ninf = __uint_as_float(0xFF800000u);
            float lo_a = upper ? inf : lo, lo_b = upper ? lo : inf, hi_a = upper ? ninf : hi, hi_b = upper ? hi : ninf;
            asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(lo_a) : "f"(lo_a));
            asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(lo_b) : "f"(lo_b));
            asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(hi_a) : "f"(hi_a));
            asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(hi_b) : "f"(hi_b));
            lo = upper ? lo_b : lo_a;
            hi = upper ? hi_b : hi_a;
        } else {
#pragma unroll
            for (int off = 1; off < LPU; off <<= 1) {
                lo = fmin2(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, off));
                hi = fmax2(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, off));
            }
        }
        // every lane of a unit holds the unit's result and stores it (same address, same value):
        // cheaper than a divergent branch around the store
        const int u = (warp * CHUNKS + c) * (32 / LPU) + lane / LPU;
        s_umn[u] = lo;
        s_umx[u] = hi;
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

// The CTA is 16 compute warps, one control warp and one widths warp; two CTAs share an SM and
// cover each other's waits.  Hardware barrier 1 ("stage"; the control warp, the widths warp
// when it is in charge, else the owner warps wait, the rest only arrive): the compute warps have
// moved the staged window into registers, published its per-unit min / max, and finished the
// previous window's packed bytes.  Barrier 2 ("widths", compute warps wait): the verdict on the
// window's widths and the group records are in.  Barrier 3 is private to the warps that own
// group records (more than 64 groups per window); barrier 4 ends their general bit choice.
constexpr int kComputeWarps = kWarps;
constexpr int kCompressThreads = kThreads + 64;
constexpr uint32_t kBarStage = 1, kBarWidths = 2, kBarOwners = 3, kBarChoice = 4;
constexpr int kSelWords = kGeneralSelWords;

__device__ __forceinline__ void bar_sync(uint32_t id, uint32_t threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void bar_arrive(uint32_t id, uint32_t threads)
{
    __threadfence_block();                                        // this thread's shared-memory writes first
    asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// Quantize + pack one window whose groups all have width B (no clamp needed): no per-chunk
// decisions, packed position computed from the element index alone.
template <typename KEYS, int CHUNKS, int B>
__device__ __forceinline__ void quantize_uniform(const float (&x)[CHUNKS][8], const GroupRec *s_grp, uint32_t log2G,
                                                 uint32_t e0, uint64_t blk0, const KEYS &keys, unsigned char *s_out)
{
    unsigned char *const out = s_out + (e0 >> 3) * B;
#pragma unroll
    for (int c = 0; c < CHUNKS; c++) {
        const float2 mi = *reinterpret_cast<const float2 *>(&s_grp[(e0 + 256u * c) >> log2G]);   // mn, inv
        uint32_t o[4];
        const uint64_t blk = blk0 + 32u * c;
        philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), keys, o);
        uint32_t w0, w1;
        quantize8<B, false>(x[c], mi.x, mi.y, o, w0, w1);
        unsigned char *p = out + 32 * B * c;
        if (B == 1) *p = (unsigned char)w0;
        else if (B == 2) *reinterpret_cast<uint16_t *>(p) = (uint16_t)w0;
        else if (B == 4) *reinterpret_cast<uint32_t *>(p) = w0;
        else *reinterpret_cast<uint2 *>(p) = make_uint2(w0, w1);
    }
}

template <typename KEYS, int CHUNKS>
__device__ __forceinline__ void quantize_uniform_b(uint32_t b, const float (&x)[CHUNKS][8], const GroupRec *s_grp,
                                                   uint32_t log2G, uint32_t e0, uint64_t blk0, const KEYS &keys,
                                                   unsigned char *s_out)
{
    switch (b) {
    case 1: quantize_uniform<KEYS, CHUNKS, 1>(x, s_grp, log2G, e0, blk0, keys, s_out); break;
    case 2: quantize_uniform<KEYS, CHUNKS, 2>(x, s_grp, log2G, e0, blk0, keys, s_out); break;
    case 4: quantize_uniform<KEYS, CHUNKS, 4>(x, s_grp, log2G, e0, blk0, keys, s_out); break;
    default: quantize_uniform<KEYS, CHUNKS, 8>(x, s_grp, log2G, e0, blk0, keys, s_out); break;
    }
}

// Budget arithmetic of a window of n groups.
struct Budget {
    uint32_t ell;          // largest level every group can be raised to
    uint32_t rem;          // bit units left after the smallest width
    bool all_max;          // every group reaches the largest width
    bool need_sep;         // the best raise of level ell does not fit: uniform iff the levels separate
};

// WIDTHS: at most 64 groups per window (groups of 256 elements or more at the default window): the
// widths warp settles every window, of one width or mixed; otherwise the compute warps that own
// group records do (mixed windows: radix select on the keys).
template <typename T, int CHUNKS, bool BATCH, bool WIDTHS, int ACT>
__global__ void __launch_bounds__(kCompressThreads, 2)
compress_kernel(const __grid_constant__ CompressArgs<BATCH ? DAF_BATCH_MAX : 1> a)
{
    constexpr uint32_t WE = kThreads * kLaneElems * CHUNKS;

    extern __shared__ __align__(128) unsigned char smem[];       // [stage | out0 | out1 | group arrays]
    __shared__ uint32_t s_wtot[kComputeWarps];
    __shared__ __align__(8) uint64_t s_full;                     // mbarrier: staged window has landed (or there is none)
    __shared__ uint32_t s_next[2];                               // ticket of the window of iteration i (slot i & 1)
    __shared__ uint32_t s_lost;                                  // a staged copy did not land in time
    __shared__ __align__(16) uint32_t s_rkeys[2][20];            // batched calls: Philox round keys of the window's tensor
    __shared__ uint32_t s_tot[2];                                // packed bytes of the window of iteration i (slot i & 1)
    __shared__ uint32_t s_mode[2];                               // how that window's widths came out (see below)
    __shared__ uint32_t s_slow[2];                               // a group of that window needs the clamped quantizer
    __shared__ uint32_t s_kmin[2], s_kmax[2];                    // separation test of that window: key extremes over the owner warps

    unsigned char *const s_stage = smem;
    float *const s_umn = reinterpret_cast<float *>(smem + a.lay.umn);         // [2][units]
    float *const s_umx = reinterpret_cast<float *>(smem + a.lay.umx);
    // general bit choice with more than 64 groups: [8][16] bins, largest / smallest key, sum of all, the last key, [3][16] ties
    uint32_t *const s_sel = reinterpret_cast<uint32_t *>(smem + a.lay.sel);
    GroupRec *const s_grp = reinterpret_cast<GroupRec *>(smem + a.lay.grp);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t G = a.G, log2G = a.log2G;
    uint64_t *const flags = a.flags2;                             // (the first array belongs to the streaming kernel)
    unsigned int *const ticket = &a.hdr->ticket2;
    if (a.gated != 0u && *reinterpret_cast<volatile unsigned int *>(&a.hdr->retry) == 0u) return;   // nothing to redo

    auto tensor_of = [&](uint32_t gw) -> const TensorDesc & { return a.t[BATCH ? find_tensor(a, gw) : 0u]; };
    // Control lane: draws a ticket; starts the bulk copy of that window into the stage, or
    // completes the stage's barrier empty-handed when the windows have run out.
    auto draw_ticket = [&]() -> uint32_t { return atomicAdd(ticket, 1u); };
    auto stage_window = [&](uint32_t t, uint32_t iter) {
        s_next[iter & 1u] = t;                                    // ordered before the barrier's completion
        if (t < a.total_windows) {
            const TensorDesc &nd = tensor_of(t);
            const uint64_t base = (uint64_t)(t - nd.first_window) * WE;
            const uint64_t left = nd.numel - base;
            const uint32_t bytes = (uint32_t)(left < WE ? left : WE) * Elem<T>::kBytes;
            mbar_expect_tx(&s_full, bytes);
            bulk_load(s_stage, reinterpret_cast<const char *>(nd.in) + base * Elem<T>::kBytes, bytes, &s_full);
        } else {
            mbar_arrive(&s_full);
        }
    };
    auto record_error = [&](unsigned code, uint32_t window) {
        if (atomicCAS(&a.hdr->status, 0u, code) == 0u) a.hdr->fail_window = window;
    };
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

    if (tid == kThreads) {
        mbar_init(&s_full, 1);
        s_lost = 0u;
        s_slow[0] = s_slow[1] = 0u;
        s_kmin[0] = s_kmin[1] = 0xFFFFFFFFu;
        s_kmax[0] = s_kmax[1] = 0u;
        stage_window(draw_ticket(), 0u);
    }
    if (!WIDTHS && tid < kSelWords) s_sel[tid] = tid == 129 ? 0xFFFFFFFFu : 0u;   // rest state of the choice's counters
    __syncthreads();

    // With at most 64 groups per window (groups of 256 elements or more at the default window) a warp of its own, which
    // holds no window data, settles the windows whose groups all end at the same width: lane l
    // looks after groups l and l + 32.  See the compute warps' own version below for the test.
    constexpr bool ctl_widths = WIDTHS;
    const uint32_t stage_threads = ctl_widths ? kCompressThreads : kThreads + 32;   // who meets at the "stage" barrier
    auto uniform_widths = [&](uint32_t gw, uint32_t iter, bool &arrived) {
        arrived = false;
        const TensorDesc &td = tensor_of(gw);
        if (BATCH && lane < 10) philox_store_round_keys(s_rkeys[iter & 1u], td.seed, lane);
        const uint32_t w = gw - td.first_window;
        const uint64_t wbase = (uint64_t)w * WE;
        const uint64_t left = td.numel - wbase;
        const uint32_t n_elems = left < WE ? (uint32_t)left : WE;
        const uint32_t n = n_elems >> log2G;
        const uint32_t rr = G > 256u ? G >> 8 : 1u;               // units per group (a unit: one group, at most 256 elements)
        const uint64_t g0 = wbase >> log2G;
        const uint32_t units = WE >> (G < 256u ? log2G : 8u);
        const float *umn = s_umn + (iter & 1u) * units, *umx = s_umx + (iter & 1u) * units;
        const Budget bud = budget_of(n);
        const float vl = a.v[bud.ell > 0 ? bud.ell - 1 : 0], vh = a.v[bud.ell];
        float mn[2], R[2];
        uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
#pragma unroll
        for (int q = 0; q < 2; q++) {
            const uint32_t g = (uint32_t)lane + 32u * q;
            mn[q] = R[q] = 0.0f;
            if (g < n) {
                float lo = umn[g * rr], hi = umx[g * rr];
                for (uint32_t k = 1; k < rr; k++) {
                    lo = fmin2(lo, umn[g * rr + k]);
                    hi = fmax2(hi, umx[g * rr + k]);
                }
                float Rg = __fsub_rn(hi, lo);
                if (Rg < 0x1p-118f) Rg = 0.0f;                    // degenerate group: constant
                mn[q] = lo;
                R[q] = Rg;
                kmin = min(kmin, __float_as_uint(__fmul_rn(Rg, vl)));
                kmax = max(kmax, __float_as_uint(__fmul_rn(Rg, vh)));
            }
        }
        // 1/scale for the width all groups would share: the divisions overlap the reductions below
        float inv_ell[2];
        {
            const float Lf = (float)((1u << a.S[bud.ell]) - 1u);
#pragma unroll
            for (int q = 0; q < 2; q++) inv_ell[q] = R[q] > 0.0f ? __fdiv_rn(Lf, R[q]) : 0.0f;
        }
        bool same = bud.all_max || bud.need_sep;
        if (bud.need_sep && bud.ell > 0) {
            kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
            kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
            same = kmin >= kmax;
        }
        if (lane == 0) s_slow[(iter & 1u) ^ 1u] = 0u;             // reset the flag of the next window
        if (same) {
            const uint32_t b = a.S[bud.ell], size = (G >> 3) * b;
#pragma unroll
            for (int q = 0; q < 2; q++) {
                const uint32_t g = (uint32_t)lane + 32u * q;
                if (g < n) {
                    const float inv = inv_ell[q];
                    // 1/scale not a normal number: codes may need the clamp, take the careful quantizer
                    if (R[q] > 0.0f && inv < 0x1p-126f) s_slow[iter & 1u] = 1u;
                    GroupRec rec;
                    rec.mn = mn[q];
                    rec.inv = inv;
                    rec.b = b;
                    rec.off = g * size;
                    s_grp[g] = rec;
                }
            }
            if (lane == 0) {
                // the window's byte count is known: publish it at once
                const uint32_t total = n * size;
                st_relaxed_u64(flags + gw, ((w == 0u ? kFlagPrefix : kFlagAggregate) << kFlagShift) | total);
                s_tot[iter & 1u] = total;
            }
        }
        if (!same) {
            // ------------------------------------------------------------ general bit choice, by this warp alone
            // Lane l holds the keys fl(R v_k) of groups l and l + 32.  If every raise below level ell
            // sorts ahead of every raise of level ell, and every raise above it behind, the accepted
            // prefix is: all raises below ell (they fit by the definition of ell) and then raises of
            // level ell alone, so only those two keys per lane enter the search; otherwise all six do.
            const uint32_t nl = a.m - 1u;
            uint32_t key[6], cw[6], slot_cost[6];                 // slot 2k + q: raise k of group lane + 32 q
            uint32_t up_min = 0xFFFFFFFFu, dn_max = 0u, my_min = 0xFFFFFFFFu, my_max = 0u;
#pragma unroll
            for (int k = 0; k < 3; k++)
#pragma unroll
                for (int q = 0; q < 2; q++) {
                    const bool on = (uint32_t)k < nl && (uint32_t)lane + 32u * q < n;
                    const uint32_t kk = on ? __float_as_uint(__fmul_rn(R[q], a.v[k])) : 0u;
                    key[2 * k + q] = kk;
                    cw[2 * k + q] = on ? a.cost[k] | 0x10000u : 0u;   // cost in the low half, 1 in the high half; 0: no candidate
                    slot_cost[2 * k + q] = a.cost[k];
                    if (on) {
                        if ((uint32_t)k < bud.ell) up_min = min(up_min, kk);
                        else if ((uint32_t)k > bud.ell) dn_max = max(dn_max, kk);
                        else {
                            my_min = min(my_min, kk);
                            my_max = max(my_max, kk);
                        }
                    }
                }
            up_min = __reduce_min_sync(0xFFFFFFFFu, up_min);
            dn_max = __reduce_max_sync(0xFFFFFFFFu, dn_max);
            my_min = __reduce_min_sync(0xFFFFFFFFu, my_min);
            my_max = __reduce_max_sync(0xFFFFFFFFu, my_max);
            uint32_t lvl[2];
            if (up_min >= my_max && dn_max <= my_min) {           // ties go to the lower level: >= and <= are enough
                uint32_t key2[2], cw2[2], cost2[2];
                bool take[2];
#pragma unroll
                for (int q = 0; q < 2; q++) {
                    key2[q] = bud.ell == 0u ? key[q] : bud.ell == 1u ? key[2 + q] : key[4 + q];
                    cw2[q] = bud.ell == 0u ? cw[q] : bud.ell == 1u ? cw[2 + q] : cw[4 + q];
                    cost2[q] = a.cost[bud.ell];
                }
                accept_prefix<2, true>(key2, cw2, cost2, bud.rem - (a.S[bud.ell] - a.S[0]) * n, my_max, my_min, lane, take);
                lvl[0] = bud.ell + take[0];
                lvl[1] = bud.ell + take[1];
            } else {
                bool take[6];
                accept_prefix<6, false>(key, cw, slot_cost, bud.rem, 0u, 0u, lane, take);
                lvl[0] = (uint32_t)take[0] + take[2] + take[4];
                lvl[1] = (uint32_t)take[1] + take[3] + take[5];
            }
            // records: width, 1/scale, byte offset (exclusive scan of the sizes, both groups of a lane in one word)
            uint32_t bq[2], size[2];
#pragma unroll
            for (int q = 0; q < 2; q++) {
                bq[q] = a.S[lvl[q]];
                size[q] = (uint32_t)lane + 32u * q < n ? (G >> 3) * bq[q] : 0u;
            }
            uint32_t incl = size[0] | (size[1] << 16);
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += y;
            }
            const uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
            const uint32_t total = (tot & 0xFFFFu) + (tot >> 16);
#pragma unroll
            for (int q = 0; q < 2; q++) {
                const uint32_t g = (uint32_t)lane + 32u * q;
                if (g < n) {
                    const float Lf = (float)((1u << bq[q]) - 1u);
                    const float inv = R[q] > 0.0f ? __fdiv_rn(Lf, R[q]) : 0.0f;
                    if (R[q] > 0.0f && inv < 0x1p-126f) s_slow[iter & 1u] = 1u;
                    GroupRec rec;
                    rec.mn = mn[q];
                    rec.inv = inv;
                    rec.b = bq[q];
                    rec.off = q == 0 ? (incl & 0xFFFFu) - size[0] : (tot & 0xFFFFu) + (incl >> 16) - size[1];
                    s_grp[g] = rec;
                }
            }
            if (lane == 0) {
                st_relaxed_u64(flags + gw, ((w == 0u ? kFlagPrefix : kFlagAggregate) << kFlagShift) | total);
                s_tot[iter & 1u] = total;
                s_mode[iter & 1u] = 1u;                           // per-group records
            }
            bar_arrive(kBarWidths, kThreads + 32);
            arrived = true;
#pragma unroll
            for (int q = 0; q < 2; q++) {
                const uint32_t g = (uint32_t)lane + 32u * q;
                if (g < n) {
                    const float Lf = (float)((1u << bq[q]) - 1u);
                    td.bits[g0 + g] = (uint8_t)bq[q];
                    td.mn[g0 + g] = mn[q];
                    td.scale[g0 + g] = R[q] > 0.0f ? __fdiv_rn(R[q], Lf) : 0.0f;
                }
            }
            return;
        }
        if (lane == 0) s_mode[iter & 1u] = !a.nearest ? 1u + a.S[bud.ell] : 1u;
        // the compute warps have what they need: let them go, then write the groups' metadata
        bar_arrive(kBarWidths, kThreads + 32);
        arrived = true;
        const uint32_t b = a.S[bud.ell];
        const float Lf = (float)((1u << b) - 1u);
#pragma unroll
        for (int q = 0; q < 2; q++) {
            const uint32_t g = (uint32_t)lane + 32u * q;
            if (g < n) {
                td.bits[g0 + g] = (uint8_t)b;
                td.mn[g0 + g] = mn[q];
                td.scale[g0 + g] = R[q] > 0.0f ? __fdiv_rn(R[q], Lf) : 0.0f;
            }
        }
    };

    if (warp == kComputeWarps + 1) {
        // ============================================================ widths warp
        if (!ctl_widths) return;
        for (uint32_t iter = 0;; iter++) {
            bar_sync(kBarStage, stage_threads);                   // every unit's min / max is visible
            const uint32_t gw = s_next[iter & 1u];
            if (gw >= a.total_windows) break;
            bool arrived = false;
            if (s_lost == 0u) uniform_widths(gw, iter, arrived);
            if (!arrived) bar_arrive(kBarWidths, kThreads + 32);  // the verdict on the window is in
            if (s_lost != 0u) break;
        }
        return;
    }
    if (warp == kComputeWarps) {
        // ============================================================ control warp
        // Per window i: wait until the compute warps have consumed stage(i) and finished the
        // packed bytes of window i-1; start the copy of window i+1; then, off the compute
        // warps' critical path, find window i-1's byte offset by look-back, publish its
        // inclusive prefix, and send its packed bytes to global memory.
        uint32_t gw = s_next[0];
        bool have_prev = false;
        uint32_t p_gw = 0;
        for (uint32_t iter = 0;; iter++) {
            const bool valid = gw < a.total_windows;
            bar_sync(kBarStage, stage_threads);
            const bool lost = s_lost != 0u;
            uint32_t next = 0xFFFFFFFFu;
            if (valid && !lost) {
                if (lane == 0) stage_window(draw_ticket(), iter + 1u);
                __syncwarp();
                next = s_next[(iter + 1u) & 1u];
            }
            if (have_prev) {
                const TensorDesc &pd = tensor_of(p_gw);
                const uint32_t p_total = s_tot[(iter & 1u) ^ 1u];
                const unsigned char *src = smem + a.lay.out0 + ((iter & 1u) ^ 1u) * a.lay.out_stride;
                uint64_t excl = 0;
                int state = 1;
                if (p_gw != pd.first_window) {
                    state = lookback<kLookDepth>(flags, p_gw, pd.first_window, lane, true, a.poll_limit, &excl);
                    if (lane == 0) {
                        // a wait that ran out is reported before the descriptor is poisoned; the windows behind, which
                        // only meet the poison, stop without a report of their own
                        if (state == -2) {
                            record_error(DAF_ERR_TIMEOUT, p_gw);
                            __threadfence();
                        }
                        st_relaxed_u64(flags + p_gw, state == 1 ? ((kFlagPrefix << kFlagShift) | (excl + p_total))
                                                                    : (kFlagPoison << kFlagShift));
                    }
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
                    // no room: nothing of the window is stored (a failed wait has reported itself above)
                    if (lane == 0 && state == 1) record_error(DAF_ERR_CAPACITY, p_gw);
                } else if (a.bulk_store) {
                    if (lane == 0 && p_total) {
                        bulk_store(pd.packed + excl, src, p_total);
                        bulk_store_wait_read();                   // the buffer is packed into again two windows on
                    }
                } else {                                          // groups of 32 / 64: windows are only 4-byte aligned
                    uint32_t *dst = reinterpret_cast<uint32_t *>(pd.packed + excl);
                    const uint32_t *s32 = reinterpret_cast<const uint32_t *>(src);
                    for (uint32_t i = lane; i < (p_total >> 2); i += 32) dst[i] = s32[i];
                }
            }
            if (!valid) break;
            if (lost) {
                if (lane == 0) {
                    record_error(DAF_ERR_TIMEOUT, gw);
                    st_relaxed_u64(flags + gw, kFlagPoison << kFlagShift);
                    mbar_wait_bounded(&s_full, iter & 1u, a.poll_limit);        // one more bounded chance for the lost copy
                }
                break;
            }
            have_prev = true;
            p_gw = gw;
            gw = next;
        }
        if (lane == 0) bulk_store_wait_all();
        return;
    }

    // ================================================================ compute warps
    const uint32_t e0 = (uint32_t)(warp * CHUNKS * 256 + lane * 8);    // this lane's first element of chunk 0
    const uint32_t units = WE >> (G < 256u ? log2G : 8u);         // units per window
    const uint32_t n_max = a.n_max, nl = a.m - 1u;
    for (uint32_t iter = 0;; iter++) {
        // ---------------------------------------------------------------- the staged window has landed (or there is none)
        bool lost = false;
        if (!mbar_wait_bounded(&s_full, iter & 1u, a.poll_limit)) {
            s_lost = 1u;
            lost = true;
        }
        const uint32_t gw = lost ? 0u : s_next[iter & 1u];
        if (!lost && gw >= a.total_windows) break;
        unsigned char *const s_out = smem + a.lay.out0 + (iter & 1u) * a.lay.out_stride;
        const TensorDesc &td = tensor_of(gw);
        const uint32_t w = gw - td.first_window;
        const uint64_t wbase = (uint64_t)w * WE;
        const uint64_t left = td.numel - wbase;
        const uint32_t n_elems = left < WE ? (uint32_t)left : WE;
        const uint32_t n = n_elems >> log2G;                      // groups in this window
        float *const umn = s_umn + (iter & 1u) * units, *const umx = s_umx + (iter & 1u) * units;

        // ---------------------------------------------------------------- staged window -> registers, unit min / max
        float x[CHUNKS][8];
        if (G >= 256u) load_and_reduce<T, CHUNKS, 32, ACT>(s_stage, warp, lane, x, umn, umx);
        else if (G == 128u) load_and_reduce<T, CHUNKS, 16, ACT>(s_stage, warp, lane, x, umn, umx);
        else if (G == 64u) load_and_reduce<T, CHUNKS, 8, ACT>(s_stage, warp, lane, x, umn, umx);
        else load_and_reduce<T, CHUNKS, 4, ACT>(s_stage, warp, lane, x, umn, umx);
        if (ACT != kActNone && !lost) {
            // the activation goes out as it is compressed: one 8-element store per lane and chunk (the
            // window was staged whole before, so the output may be the input buffer)
            char *const act = reinterpret_cast<char *>(td.act) + wbase * Elem<T>::kBytes;
#pragma unroll
            for (int c = 0; c < CHUNKS; c++) {
                const uint32_t e = e0 + 256u * c;
                if (e < n_elems) {
                    if (ACT == kActGelu) {                        // x stays what is compressed; GELU(x) goes out
                        float keep[8], y[8];
#pragma unroll
                        for (int i = 0; i < 8; i++) keep[i] = x[c][i];
                        activate8<ACT>(keep, y);
                        Elem<T>::store8(act + (size_t)e * Elem<T>::kBytes, y);
                    } else {
                        Elem<T>::store8(act + (size_t)e * Elem<T>::kBytes, x[c]);
                    }
                }
            }
        }
        // ---------------------------------------------------------------- widths, first try: one width for all
        // The warps that own group records (thread g: group g) test whether every group ends at
        // level ell: every raise below level ell must sort ahead of every raise from level ell
        // upward (ties go to the lower level); they all fit and the next does not.  If so they
        // write the records at once; otherwise all compute warps share the general choice below.
        const Budget bud = budget_of(n);
        const uint64_t g0 = wbase >> log2G;                       // first group of the window in the tensor
        const uint32_t owners = (n + 31u) >> 5;
        const bool owner = (uint32_t)warp < owners, mine = (uint32_t)tid < n;
        const bool big = G > 256u;                                // a group spans several 256-element units
        float mn = 0.0f, Rg = 0.0f;
        // Owner threads: records, metadata, window total.  level_of: this thread's level.
        // (the group's metadata is written by write_metadata: at once, or after the other warps have
        // been let go when they wait for nothing but the records)
        auto write_metadata = [&](uint32_t level) {
            if (mine) {
                const uint32_t b = a.S[level];
                const float Lf = (float)((1u << b) - 1u);
                td.bits[g0 + tid] = (uint8_t)b;
                td.mn[g0 + tid] = mn;
                td.scale[g0 + tid] = Rg > 0.0f ? __fdiv_rn(Rg, Lf) : 0.0f;
            }
        };
        auto write_records = [&](uint32_t level, bool uniform_b) {
            uint32_t size = 0, b = 0;
            float inv = 0.0f;
            if (mine) {
                b = a.S[level];
                const float Lf = (float)((1u << b) - 1u);
                inv = Rg > 0.0f ? __fdiv_rn(Lf, Rg) : 0.0f;
                // 1/scale not a normal number: codes may need the clamp, take the careful quantizer
                if (Rg > 0.0f && inv < 0x1p-126f) s_slow[iter & 1u] = 1u;
                size = (G >> 3) * b;
            }
            uint32_t total, off;
            if (uniform_b) {
                off = (uint32_t)tid * size;
                total = n * (G >> 3) * a.S[level];
            } else {
                // byte offset of each group inside the window: exclusive scan of the sizes
                uint32_t incl = size, before = 0;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (lane >= o) incl += y;
                }
                total = __shfl_sync(0xFFFFFFFFu, incl, 31);
                if (owners > 1) {
                    if (lane == 0) s_wtot[warp] = total;
                    bar_sync(kBarOwners, owners * 32u);
                    total = 0;
                    for (uint32_t k = 0; k < owners; k++) {
                        const uint32_t t = s_wtot[k];
                        if (k < (uint32_t)warp) before += t;
                        total += t;
                    }
                }
                off = before + incl - size;
            }
            if (mine) {
                GroupRec rec;
                rec.mn = mn;
                rec.inv = inv;
                rec.b = b;
                rec.off = off;
                s_grp[tid] = rec;
            }
            if (tid == 0) {
                // the window's byte count is known: publish it at once
                st_relaxed_u64(flags + gw, ((w == 0u ? kFlagPrefix : kFlagAggregate) << kFlagShift) | total);
                s_tot[iter & 1u] = total;
            }
        };
        auto own_range = [&]() {
            if (mine) {
                float mx;
                if (big) {
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
            }
        };
        if (ctl_widths) {
            bar_arrive(kBarStage, stage_threads);              // unit min / max out, stage consumed, last window packed
            bar_sync(kBarWidths, kThreads + 32);                  // the widths warp's verdict (and records) visible
        } else {
            if (owner) {
                bar_sync(kBarStage, stage_threads);            // every unit's min / max is visible; the stage is free
                if (BATCH && tid < 10) philox_store_round_keys(s_rkeys[iter & 1u], td.seed, tid);
                if (tid == 0) {                                   // reset the next window's slots
                    s_slow[(iter & 1u) ^ 1u] = 0u;
                    s_kmin[(iter & 1u) ^ 1u] = 0xFFFFFFFFu;
                    s_kmax[(iter & 1u) ^ 1u] = 0u;
                }
                own_range();
                bool uniform = bud.all_max || bud.need_sep;
                if (bud.need_sep && bud.ell > 0) {
                    // each owner warp puts in the key extremes of its own groups; the owners meet once
                    uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
                    if (mine) {
                        kmin = __float_as_uint(__fmul_rn(Rg, a.v[bud.ell - 1]));
                        kmax = __float_as_uint(__fmul_rn(Rg, a.v[bud.ell]));
                    }
                    kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
                    kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
                    if (owners > 1) {
                        if (lane == 0) {
                            atomicMin(&s_kmin[iter & 1u], kmin);
                            atomicMax(&s_kmax[iter & 1u], kmax);
                        }
                        bar_sync(kBarOwners, owners * 32u);
                        kmin = s_kmin[iter & 1u];
                        kmax = s_kmax[iter & 1u];
                    }
                    uniform = kmin >= kmax;
                }
                if (s_lost == 0u) {
                    if (uniform) write_records(bud.ell, true);
                    if (tid == 0) s_mode[iter & 1u] = !uniform ? 0u : !a.nearest ? 1u + a.S[bud.ell] : 1u;
                }
            } else {
                bar_arrive(kBarStage, stage_threads);
            }
            bar_sync(kBarWidths, kThreads);                       // records (or the news that there are none yet) visible
            if (owner && s_lost == 0u && s_mode[iter & 1u] != 0u) write_metadata(bud.ell);
        }
        if (s_lost != 0u) break;
        const uint32_t mode = s_mode[iter & 1u];                  // 0: general choice needed; 1: records; 1 + b: one width b
        const uint64_t blk0 = ((td.elem_base + wbase) >> 3) + (e0 >> 3);

        const bool quick = mode >= 2u && s_slow[iter & 1u] == 0u; // one width, no clamp needed
        if (!ctl_widths && mode == 0u) {
            // -------------------------------------------------------------- general bit choice (more than 64 groups)
            // The greedy of Sec. 3.4.1 accepts the longest prefix of the candidate raises, sorted by
            // (key descending, level ascending, group ascending), whose summed cost fits the window's
            // budget.  F(t), the cost of all raises with key >= t, falls as t grows, so the prefix is
            // every raise with a key above Kp, the largest t with F(t) > rem, and then the raises with
            // key Kp in order while they fit.  Thread g holds the keys of group g; Kp is found four bits
            // at a time from the top (below the keys' common leading bits): the raises whose key lies in
            // the interval that still holds Kp are counted into sixteen bins by the next four bits
            // (cost and number), one meeting of the owner warps per step, and each of them reads off the
            // bin that holds Kp.  As soon as a single raise is left in the interval, its key is Kp.
            if (owner) {                                          // the warps that own group records; the others wait below
            uint32_t *const H = s_sel, *const s_hi = s_sel + 128, *const s_lo = s_sel + 129, *const s_all = s_sel + 130;
            uint32_t *const s_only = s_sel + 131, *const s_tie = s_sel + 132;
            uint32_t key[3], cwk[3];                              // cwk: cost | 1 << 16, or 0 for "no candidate"
            uint32_t whi = 0u, wlo = 0xFFFFFFFFu, wall = 0u;
#pragma unroll
            for (int k = 0; k < 3; k++) {
                const bool on = mine && (uint32_t)k < nl;
                key[k] = on ? __float_as_uint(__fmul_rn(Rg, a.v[k])) : 0u;
                cwk[k] = on ? a.cost[k] | 0x10000u : 0u;
                if (on) {
                    whi = max(whi, key[k]);
                    wlo = min(wlo, key[k]);
                    wall += cwk[k];
                }
            }
            whi = __reduce_max_sync(0xFFFFFFFFu, whi);
            wlo = __reduce_min_sync(0xFFFFFFFFu, wlo);
            wall = __reduce_add_sync(0xFFFFFFFFu, wall);
            if (lane == 0 && wall != 0u) {
                atomicMax(s_hi, whi);
                atomicMin(s_lo, wlo);
                atomicAdd(s_all, wall);
            }
            bar_sync(kBarOwners, owners * 32u);
            const uint32_t hi = *s_hi, lo = *s_lo, all = *s_all;
            const uint32_t below = (1u << lane) - 1u;
            uint32_t Kp = hi, above = 0u, ties = all >> 16;       // above: F | N << 16 of the raises beyond the interval
            const bool take_all = (all & 0xFFFFu) <= bud.rem;     // every raise fits
            if (!take_all && hi != lo) {
                uint32_t sh = (31u - (uint32_t)__clz(hi ^ lo)) & ~3u;   // the four bits sh .. sh + 3 come next
                Kp = sh >= 28u ? 0u : (hi >> (sh + 4u)) << (sh + 4u);
                for (uint32_t j = 0;; j++) {
                    uint32_t *const Hj = H + 16u * j;
#pragma unroll
                    for (int k = 0; k < 3; k++) {
                        const bool m = cwk[k] != 0u && (sh >= 28u || ((key[k] ^ Kp) >> (sh + 4u)) == 0u);
                        const uint32_t d = (key[k] >> sh) & 15u;
                        const uint32_t act = __ballot_sync(0xFFFFFFFFu, m);
                        if (act != 0u) {
                            const int leader = __ffs(act) - 1;
                            const uint32_t d0 = __shfl_sync(0xFFFFFFFFu, d, leader);
                            if (__all_sync(0xFFFFFFFFu, !m || d == d0)) {   // one bin for the whole warp: one atomic
                                const uint32_t sum = __reduce_add_sync(0xFFFFFFFFu, m ? cwk[k] : 0u);
                                if (lane == leader) atomicAdd(&Hj[d0], sum);
                            } else if (m) {
                                atomicAdd(&Hj[d], cwk[k]);
                            }
                        }
                    }
                    bar_sync(kBarOwners, owners * 32u);
                    const uint32_t h = lane < 16 ? Hj[lane] : 0u;
                    uint32_t S = h;                               // lanes 0..15: bins lane .. 15 summed
#pragma unroll
                    for (int o = 1; o < 16; o <<= 1) S += __shfl_down_sync(0xFFFFFFFFu, S, o);
                    const uint32_t over = __ballot_sync(0xFFFFFFFFu, ((above + S) & 0xFFFFu) > bud.rem) & 0xFFFFu;
                    const uint32_t dstar = 31u - (uint32_t)__clz(over | 1u);   // bin 0 always qualifies
                    above += __shfl_sync(0xFFFFFFFFu, S, (int)(dstar + 1u));   // lane 16 holds 0
                    ties = __shfl_sync(0xFFFFFFFFu, h, (int)dstar) >> 16;
                    Kp |= dstar << sh;
                    if (ties == 1u || sh == 0u) break;
                    sh -= 4u;
                }
                if (sh != 0u) {                                   // one raise left in [Kp, Kp + 2^sh): Kp is its key
#pragma unroll
                    for (int k = 0; k < 3; k++)
                        if (cwk[k] != 0u && ((key[k] ^ Kp) >> sh) == 0u) *s_only = key[k];
                    bar_sync(kBarOwners, owners * 32u);
                    Kp = *s_only;
                }
            }
            const uint32_t left = bud.rem - (above & 0xFFFFu);    // after every raise with a key above Kp
            uint32_t level = 0;
            if (take_all) {
                level = mine ? nl : 0u;
            } else if (ties <= 1u) {
#pragma unroll
                for (int k = 0; k < 3; k++)
                    if (cwk[k] != 0u) level += key[k] > Kp || (key[k] == Kp && a.cost[k] <= left);
            } else {
                // several raises share the key Kp: they are accepted level by level, group by group, while they fit
                uint32_t tb[3];
#pragma unroll
                for (int k = 0; k < 3; k++) {
                    tb[k] = __ballot_sync(0xFFFFFFFFu, cwk[k] != 0u && key[k] == Kp);
                    if (lane == 0) s_tie[16 * k + warp] = (uint32_t)__popc(tb[k]);
                }
                bar_sync(kBarOwners, owners * 32u);
#pragma unroll
                for (int k = 0; k < 3; k++) {
                    if (cwk[k] == 0u) continue;
                    if (key[k] > Kp) {
                        level++;
                    } else if (key[k] == Kp) {
                        uint32_t cum = 0;
                        for (int k2 = 0; k2 < k; k2++)
                            for (int wp = 0; wp < kComputeWarps; wp++) cum += s_tie[16 * k2 + wp] * a.cost[k2];
                        for (int wp = 0; wp < warp; wp++) cum += s_tie[16 * k + wp] * a.cost[k];
                        cum += ((uint32_t)__popc(tb[k] & below) + 1u) * a.cost[k];
                        level += cum <= left;
                    }
                }
            }
            write_records(level, false);
            write_metadata(level);
            }
            bar_sync(kBarChoice, kThreads);                       // group records visible to all compute warps
            if (tid < kSelWords) s_sel[tid] = tid == 129 ? 0xFFFFFFFFu : 0u;   // the counters go back to their rest state
        }

        if (quick) {
            // -------------------------------------------------------------- quantize + pack, one width, no clamp needed
            if (BATCH) {
                const PhiloxSharedKeys sk{reinterpret_cast<const uint4 *>(s_rkeys[iter & 1u])};
                quantize_uniform_b<PhiloxSharedKeys, CHUNKS>(mode - 1u, x, s_grp, log2G, e0, blk0, sk, s_out);
            } else {
                quantize_uniform_b<PhiloxKeys, CHUNKS>(mode - 1u, x, s_grp, log2G, e0, blk0, a.keys, s_out);
            }
        } else {
            // -------------------------------------------------------------- quantize + pack with per-group widths
            auto draw = [&](int c, uint32_t (&o)[4]) {
                if (a.nearest) {
                    o[0] = o[1] = o[2] = o[3] = 0x80008000u;       // every 16-bit lane = 2 * 2^14
                } else {
                    const uint64_t blk = blk0 + 32u * c;
                    if (BATCH) {
                        const PhiloxSharedKeys sk{reinterpret_cast<const uint4 *>(s_rkeys[iter & 1u])};
                        philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), sk, o);
                    } else {
                        philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), a.keys, o);
                    }
                }
            };
            if (G >= 64u && s_slow[iter & 1u] == 0u) {
                // no clamp needed: fixed-width packing chosen by the lane's width, 8-byte aligned stores.  With
                // G >= 256 a warp's chunk lies in one group; below, the warp splits by width (mostly into one part)
#pragma unroll
                for (int c = 0; c < CHUNKS; c++) {
                    const uint32_t e = e0 + 256u * c;
                    if (e >= n_elems) break;                      // ragged last window: whole chunks are missing
                    const GroupRec rec = s_grp[e >> log2G];
                    uint32_t o[4], t[8], w0, w1;
                    draw(c, o);
                    noisy_sums8(x[c], rec.mn, rec.inv, o, t);     // (the arithmetic all widths share stays outside the split)
                    unsigned char *p = s_out + rec.off + ((e & (G - 1u)) >> 3) * rec.b;
                    switch (rec.b) {
                    case 1:
                        close_codes8<1, false>(t, w0, w1);
                        *p = (unsigned char)w0;
                        break;
                    case 2:
                        close_codes8<2, false>(t, w0, w1);
                        *reinterpret_cast<uint16_t *>(p) = (uint16_t)w0;
                        break;
                    case 4:
                        close_codes8<4, false>(t, w0, w1);
                        *reinterpret_cast<uint32_t *>(p) = w0;
                        break;
                    default:
                        close_codes8<8, false>(t, w0, w1);
                        *reinterpret_cast<uint2 *>(p) = make_uint2(w0, w1);
                        break;
                    }
                }
            } else {
#pragma unroll
                for (int c = 0; c < CHUNKS; c++) {
                    const uint32_t e = e0 + 256u * c;
                    const GroupRec rec = s_grp[e >> log2G];
                    uint32_t o[4], w0, w1;
                    draw(c, o);
                    quantize8_any(x[c], rec.mn, rec.inv, o, rec.b, w0, w1);
                    unsigned char *p = s_out + rec.off + ((e & (G - 1u)) >> 3) * rec.b;
                    if (e < n_elems) {
                        if (rec.b == 1u) {
                            *p = (unsigned char)w0;
                        } else if (rec.b == 2u) {
                            *reinterpret_cast<uint16_t *>(p) = (uint16_t)w0;
                        } else if (rec.b == 4u) {
                            *reinterpret_cast<uint32_t *>(p) = w0;
                        } else if (G >= 64u) {
                            *reinterpret_cast<uint2 *>(p) = make_uint2(w0, w1);
                        } else {                                   // G = 32: groups are only 4-byte aligned
                            reinterpret_cast<uint32_t *>(p)[0] = w0;
                            reinterpret_cast<uint32_t *>(p)[1] = w1;
                        }
                    }
                }
            }
        }
        if (a.bulk_store) fence_async_shared();                   // packed bytes visible to the bulk store issued later
    }
    bar_arrive(kBarStage, stage_threads);                      // the last window's packed bytes are complete
}

// ------------------------------------------------------------------------------------------
// Launch
// ------------------------------------------------------------------------------------------
template <typename T, int CHUNKS, bool BATCH, bool WIDTHS, int ACT = kActNone>
static cudaError_t launch(const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    const int smem = (int)args.lay.total;
    int ctas = 0;
    const cudaError_t e = persistent_ctas(reinterpret_cast<const void *>(&compress_kernel<T, CHUNKS, BATCH, WIDTHS, ACT>),
                                          kCompressThreads, smem, &ctas);
    if (e != cudaSuccess) return e;
    const uint32_t grid = args.total_windows < (uint32_t)ctas ? args.total_windows : (uint32_t)ctas;
    compress_kernel<T, CHUNKS, BATCH, WIDTHS, ACT><<<grid, kCompressThreads, smem, stream>>>(args);
    return cudaGetLastError();
}


template <typename T, bool BATCH, int ACT>
cudaError_t dispatch_general_t(uint32_t chunks, const CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    const bool widths = args.n_max <= 64u;                        // few enough groups for the widths warp
    if constexpr (ACT != kActNone) {                              // fused producer: single tensor, default window (chunks == 4)
        static_assert(!BATCH, "the fused producer is compiled for single-tensor launches only");
        return widths ? launch<T, 4, false, true, ACT>(args, stream) : launch<T, 4, false, false, ACT>(args, stream);
    } else {
        switch (chunks) {
        case 1: return widths ? launch<T, 1, BATCH, true>(args, stream) : launch<T, 1, BATCH, false>(args, stream);
        case 2: return widths ? launch<T, 2, BATCH, true>(args, stream) : launch<T, 2, BATCH, false>(args, stream);
        default: return widths ? launch<T, 4, BATCH, true>(args, stream) : launch<T, 4, BATCH, false>(args, stream);
        }
    }
}

#define DAF_INSTANTIATE_GENERAL(T)                                                                                          \
    template cudaError_t dispatch_general_t<T, false, kActNone>(uint32_t, const CompressArgs<1> &, cudaStream_t);              \
    template cudaError_t dispatch_general_t<T, true, kActNone>(uint32_t, const CompressArgs<DAF_BATCH_MAX> &, cudaStream_t);   \
    template cudaError_t dispatch_general_t<T, false, kActRelu>(uint32_t, const CompressArgs<1> &, cudaStream_t);              \
    template cudaError_t dispatch_general_t<T, false, kActRelu6>(uint32_t, const CompressArgs<1> &, cudaStream_t);             \
    template cudaError_t dispatch_general_t<T, false, kActGelu>(uint32_t, const CompressArgs<1> &, cudaStream_t);

}  // namespace daf
