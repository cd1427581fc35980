// Host side of the compress entry points: argument checks, the launch plan, and the order of the
// kernels of one call.
//
//   daf_compress = [clear the workspace] -> streaming kernel -> verify kernel -> general kernel
//                                                                                (or widths -> offsets -> pack)
//
// The streaming kernel (compress_stream.cuh) assumes that every window ends with one width; the
// verify kernel checks that assumption window by window and writes the window offsets; what
// handles any mix of widths runs last and returns at once unless one of the two asked for it
// (hdr->retry), in which case it redoes the call: the general kernel (compress_general.cuh), or,
// for large calls on 16-bit elements, the three two-pass kernels (compress_twopass.cuh).
// When the parameters rule out windows of one width, or the call is small, the streaming kernel
// is not launched.
#include "compress_shared.cuh"

namespace daf {
// Runs behind the streaming kernel: one thread per window compares the key extremes gathered in
// the window's word, checks that a ragged last window's budget arithmetic asks for the same
// single width, and writes the window's offset (and the total behind a tensor's last window).
template <int NT>
__global__ void __launch_bounds__(256) verify_stream_kernel(const __grid_constant__ CompressArgs<NT> a, uint32_t we)
{
    const uint32_t gw = blockIdx.x * blockDim.x + threadIdx.x;
    if (gw >= a.total_windows) return;
    uint32_t lo = 0, hi = a.n_tensors - 1;                        // last tensor whose first window is <= gw
    while (lo < hi) {
        const uint32_t mid = (lo + hi + 1) >> 1;
        if (a.t[mid].first_window <= gw) lo = mid; else hi = mid - 1;
    }
    const TensorDesc &td = a.t[lo];
    const uint32_t w = gw - td.first_window, b = a.S[a.full_ell];
    const uint64_t wbytes = (uint64_t)(we >> 3) * b;
    bool ok = true;
    if (a.full_test != 0u) {
        const uint64_t word = a.flags[gw];
        ok = ~(uint32_t)word >= (uint32_t)(word >> 32);
    }
    td.woff[w] = (uint64_t)w * wbytes;
    if (w + 1u == td.n_windows) {
        const uint64_t n_elems = td.numel - (uint64_t)w * we;
        if (n_elems != we) {
            const uint32_t n = (uint32_t)(n_elems >> a.log2G);
            const uint32_t rem = (uint32_t)((((uint64_t)a.beta_q8 * n) >> 8) - (uint64_t)a.S[0] * n);
            uint32_t ell = 0;
            while (ell + 1 < a.m && (a.S[ell + 1] - a.S[0]) * n <= rem) ell++;
            const uint32_t rem_after = rem - (a.S[ell] - a.S[0]) * n;
            ok = ok && ell == a.full_ell && (ell + 1 == a.m || rem_after < a.cost[ell]);
        }
        td.woff[w + 1u] = (uint64_t)w * wbytes + (n_elems >> 3) * b;
    }
    if (!ok) atomicExch(&a.hdr->retry, 1u);
}

// Packed size of tensor t if every window ends with one width (what the streaming kernel assumes).
template <int NT> static uint64_t one_width_total(const CompressArgs<NT> &a, const TensorDesc &t, uint32_t we)
{
    const uint64_t full_bytes = (uint64_t)(we >> 3) * a.S[a.full_ell];
    const uint64_t last_elems = t.numel - (uint64_t)(t.n_windows - 1u) * we;
    uint32_t ell = a.full_ell;
    if (last_elems != we) {                                       // ragged last window: its own budget arithmetic
        const uint64_t n = last_elems >> a.log2G;
        const uint64_t rem = (((uint64_t)a.beta_q8 * n) >> 8) - (uint64_t)a.S[0] * n;
        ell = 0;
        while (ell + 1 < a.m && (uint64_t)(a.S[ell + 1] - a.S[0]) * n <= rem) ell++;
    }
    return (uint64_t)(t.n_windows - 1u) * full_bytes + (last_elems >> 3) * a.S[ell];
}

// One call = the streaming kernel, which assumes that every window ends with one width, followed
// by the general kernel, which returns at once unless the streaming one asked for it.  When the
// parameters rule out windows of one width (a budget that no single width meets exactly and that
// leaves room for raises, or round-to-nearest), when the packed buffer could not hold such a result
// (the general kernel then reports the overflow window by window), or when the call is small (it is
// launch-bound, and one launch is cheaper than two), only the general kernel is launched.
constexpr uint32_t kStreamMinWindows = 4096;                     // measured break-even
constexpr uint32_t kTwoPassMinWindows = 4096;                    // below, one launch of the general kernel beats three (measured: sets of
                                                                  // 16-bit tensors of 600 - 2400 windows each, one call per tensor, came out
                                                                  // 7 % faster when mixed and 17 % slower when of one width)

template <bool BATCH, int ACT = kActNone>
static cudaError_t dispatch(uint32_t dtype, uint32_t chunks, uint32_t flags, CompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args,
                            cudaStream_t stream)
{
    const bool all_max = args.full_ell + 1 == args.m;
    const bool need_sep = !all_max && args.full_rem_after < args.cost[args.full_ell];
    bool try_stream = !args.nearest && (all_max || need_sep) && !(flags & DAF_FLAG_STREAM_NEVER) &&
                      (args.total_windows > kStreamMinWindows || (flags & DAF_FLAG_STREAM_ALWAYS));
    // ReLU and ReLU6 in front make the call bandwidth-bound (a second full-size stream, the activation, goes out): the
    // general kernel, which moves whole windows with bulk copies, is then the faster one (1.48 against 1.70 ms on 2^30
    // binary32 elements); GELU is bound by arithmetic and stays with the streaming kernel
    if ((ACT == kActRelu || ACT == kActRelu6) && !(flags & DAF_FLAG_STREAM_ALWAYS)) try_stream = false;
    for (uint32_t i = 0; try_stream && i < args.n_tensors; i++)
        try_stream = one_width_total(args, args.t[i], chunks * 4096u) <= args.t[i].capacity;
    // A budget between two widths: the two-width streaming kernel, if the group size is one it handles and the packed
    // buffer holds what it would write (its sizes do not depend on the data).
    bool try_two = !args.nearest && ACT == kActNone && !all_max && !need_sep && chunks == 4u && args.G >= 256u && args.G <= 1024u &&
                   !(flags & DAF_FLAG_STREAM_NEVER) && (args.total_windows > kStreamMinWindows || (flags & DAF_FLAG_STREAM_ALWAYS));
    args.tw_k = 0u;
    if (try_two) {
        const uint32_t kk = args.full_rem_after / args.cost[args.full_ell];
        args.tw_k = kk < args.n_max ? kk : args.n_max;
        const uint64_t lo = (uint64_t)(args.G >> 3) * args.S[args.full_ell];
        const uint64_t up = (uint64_t)(args.G >> 3) * (args.S[args.full_ell + 1u] - args.S[args.full_ell]);
        const uint64_t we = chunks * 4096u, wb = args.n_max * lo + args.tw_k * up;   // elements and packed bytes of a whole window
        args.tw_blo = args.S[args.full_ell];
        args.tw_bhi = args.S[args.full_ell + 1u];
        args.tw_size_lo = (uint32_t)lo;
        args.tw_size_up = (uint32_t)up;
        args.tw_lf_lo = (float)((1u << args.tw_blo) - 1u);
        args.tw_lf_hi = (float)((1u << args.tw_bhi) - 1u);
        args.tw_wbytes = wb;
        args.tw_v_my = args.v[args.full_ell];
        args.tw_test_lo = args.full_ell > 0u;
        args.tw_test_hi = args.full_ell + 2u < args.m;
        args.tw_v_lo = args.tw_test_lo ? args.v[args.full_ell - 1u] : 0.0f;
        args.tw_v_hi = args.tw_test_hi ? args.v[args.full_ell + 1u] : 0.0f;
        for (uint32_t i = 0; try_two && i < args.n_tensors; i++) {
            const uint64_t tail = args.t[i].numel % we;           // elements of a ragged last window (0: none)
            uint64_t total = (uint64_t)(args.t[i].n_windows - (tail ? 1u : 0u)) * wb;
            if (tail) {                                           // its own budget arithmetic, as the kernel does it
                const uint64_t n = tail >> args.log2G, base = (uint64_t)(args.S[args.full_ell] - args.S[0]) * n;
                const uint64_t rem = (((uint64_t)args.beta_q8 * n) >> 8) - (uint64_t)args.S[0] * n;
                uint64_t kl = base <= rem ? (rem - base) / args.cost[args.full_ell] : 0u;   // (base > rem: the kernel gives the window up)
                if (kl > n) kl = n;
                total += n * lo + kl * up;
            }
            try_two = total <= args.t[i].capacity;
        }
    }
    args.flags2 = args.flags + args.total_windows;
    args.gated = (try_stream || try_two) ? 1u : 0u;
    if (try_two) {
        const cudaError_t e = dispatch_two_width<BATCH>(dtype, args, stream);
        if (e != cudaSuccess) return e;
    }
    if (try_stream) {
        cudaError_t e = dispatch_stream<BATCH, ACT>(dtype, chunks, args, stream);
        if (e != cudaSuccess) return e;
        verify_stream_kernel<BATCH ? DAF_BATCH_MAX : 1><<<(args.total_windows + 255u) / 256u, 256, 0, stream>>>(args, chunks * 4096u);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    // Windows of mixed widths.  The two-pass kernels (compress_twopass.cuh) read the input twice and never wait; the
    // general kernel reads it once, but its warps hold a window in registers while its widths are decided.  Measured
    // (B200, whole calls): 16-bit elements, groups of 128, mostly mixed windows: 0.86 ms two-pass against 1.10 ms
    // general on 581 M elements; the same with windows of one width throughout: 0.93 against 0.74 ms on 671 M; binary32,
    // groups of 256, budget between two widths: 0.73 against 0.70 ms on 466 M.  So: 16-bit elements, calls large enough
    // that three launches do not matter, unless the caller says otherwise.
    bool two_pass = ACT == kActNone && chunks == 4u && args.G >= 128u && args.G <= 1024u && !(flags & DAF_FLAG_ONE_PASS);
    if (!(flags & DAF_FLAG_TWO_PASS)) two_pass = two_pass && dtype != DAF_F32 && args.total_windows > kTwoPassMinWindows;
    if (two_pass) return dispatch_twopass<BATCH>(dtype, args, stream);
    return dispatch_general<BATCH, ACT>(dtype, chunks, args, stream);
}

// Shared-memory carve-up for one launch configuration.
static SmemLayout make_layout(uint32_t we, uint32_t elem_bytes, uint32_t G, uint32_t window_cap_bytes)
{
    auto up = [](uint32_t v) { return (v + 127u) & ~127u; };
    const uint32_t n_max = we / G, units = we / (G < 256u ? G : 256u);
    SmemLayout l;
    uint32_t at = up(we * elem_bytes);
    l.out0 = at;
    l.out_stride = up(window_cap_bytes < 16u ? 16u : window_cap_bytes);
    at += 2u * l.out_stride;
    l.umn = at; at += up(2u * 4u * units);
    l.umx = at; at += up(2u * 4u * units);
    l.sel = at; at += n_max > 64u ? up(4u * kGeneralSelWords) : 0u;
    l.grp = at; at += up(16u * n_max);
    l.total = at;
    return l;
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
    a.poll_limit = (p->flags >> 8) ? (p->flags >> 8) : kMaxPolls;
    a.n_max = pl.We / pl.G;
    a.bulk_store = pl.G >= 128u;                                  // every group is then a multiple of 16 bytes
    {
        const uint32_t n = a.n_max;
        a.full_rem = (uint32_t)((((uint64_t)pl.beta_q8 * n) >> 8) - (uint64_t)pl.S[0] * n);
        a.full_ell = 0;
        while (a.full_ell + 1 < pl.m && (pl.S[a.full_ell + 1] - pl.S[0]) * n <= a.full_rem) a.full_ell++;
        a.full_rem_after = a.full_rem - (pl.S[a.full_ell] - pl.S[0]) * n;
        a.full_test = a.full_ell + 1 < pl.m && a.full_rem_after < pl.cost[a.full_ell] && a.full_ell > 0;
        a.stream_v_lo = pl.v[a.full_ell > 0 ? a.full_ell - 1 : 0];
        a.stream_v_hi = pl.v[a.full_ell];
    }
    a.lay = make_layout(pl.We, p->dtype == DAF_F32 ? 4u : 2u, pl.G, (uint32_t)((((uint64_t)pl.beta_q8 * pl.W) >> 8) * pl.G / 8));
    for (int k = 0; k < kMaxLevels; k++) {
        a.S[k] = pl.S[k];
        a.cost[k] = pl.cost[k];
        a.v[k] = pl.v[k];
    }
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
// the input is read eight elements per lane: 32 bytes at a time for binary32, 16 for the 16-bit types
static bool aligned_in(const void *p, uint32_t dtype) { return (reinterpret_cast<uintptr_t>(p) & (dtype == DAF_F32 ? 31u : 15u)) == 0; }

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
    if (!aligned_in(d_in, params->dtype) || !aligned16(d_packed) || !aligned16(d_workspace) || (reinterpret_cast<uintptr_t>(d_min) & 3u) ||
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
    if (!(params->flags & DAF_FLAG_KEEP_WORKSPACE) && cudaMemsetAsync(d_workspace, 0, pl.workspace, s) != cudaSuccess) return DAF_ERR_CUDA;
    return dispatch<false>(params->dtype, pl.chunks, params->flags, a, s) == cudaSuccess ? DAF_OK : DAF_ERR_CUDA;
}

extern "C" daf_status daf_act_compress(const daf_params *params, uint32_t act, const void *d_in, void *d_act, void *d_packed,
                                       uint64_t packed_capacity, uint8_t *d_bits, float *d_min, float *d_scale,
                                       uint64_t *d_window_offsets, void *d_workspace, uint64_t workspace_bytes,
                                       daf_stream stream)
{
    if (act != DAF_ACT_RELU && act != DAF_ACT_RELU6 && act != DAF_ACT_GELU) return DAF_ERR_INVALID_ARG;
    // ReLU and ReLU6 may run in place (applying them twice changes nothing, so a second pass over the call still reads
    // what it needs); GELU may not: the input is what is compressed
    if (act == DAF_ACT_GELU && d_act == d_in) return DAF_ERR_INVALID_ARG;
    Plan pl;
    daf_status st = make_plan(params, &pl);
    if (st != DAF_OK) return st;
    if (!d_in || !d_act || !d_packed || !d_bits || !d_min || !d_scale || !d_window_offsets || !d_workspace)
        return DAF_ERR_INVALID_ARG;
    if (!aligned_in(d_in, params->dtype) || !aligned16(d_packed) || !aligned16(d_workspace) || (reinterpret_cast<uintptr_t>(d_act) & 31u) ||
        (reinterpret_cast<uintptr_t>(d_min) & 3u) || (reinterpret_cast<uintptr_t>(d_scale) & 3u) ||
        (reinterpret_cast<uintptr_t>(d_window_offsets) & 7u))
        return DAF_ERR_INVALID_ARG;
    if (workspace_bytes < pl.workspace) return DAF_ERR_CAPACITY;
    if (pl.n_windows > 0xFFFFFFF0ull || pl.chunks != 4) return DAF_ERR_UNSUPPORTED;   // default window only

    CompressArgs<1> a;
    fill_common(a, pl, params, d_workspace);
    a.total_windows = (uint32_t)pl.n_windows;
    a.n_tensors = 1;
    a.keys = philox_keys(params->seed);
    a.t[0] = TensorDesc{d_in, reinterpret_cast<uint8_t *>(d_packed), packed_capacity, d_bits, d_min, d_scale,
                        d_window_offsets, params->numel, params->elem_index_base, params->seed, 0u,
                        (uint32_t)pl.n_windows, d_act};
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (!(params->flags & DAF_FLAG_KEEP_WORKSPACE) && cudaMemsetAsync(d_workspace, 0, pl.workspace, s) != cudaSuccess) return DAF_ERR_CUDA;
    cudaError_t e;
    if (act == DAF_ACT_RELU) e = dispatch<false, kActRelu>(params->dtype, pl.chunks, params->flags, a, s);
    else if (act == DAF_ACT_RELU6) e = dispatch<false, kActRelu6>(params->dtype, pl.chunks, params->flags, a, s);
    else e = dispatch<false, kActGelu>(params->dtype, pl.chunks, params->flags, a, s);
    return e == cudaSuccess ? DAF_OK : DAF_ERR_CUDA;
}

extern "C" daf_status daf_relu_compress(const daf_params *params, const void *d_in, void *d_act, void *d_packed,
                                        uint64_t packed_capacity, uint8_t *d_bits, float *d_min, float *d_scale,
                                        uint64_t *d_window_offsets, void *d_workspace, uint64_t workspace_bytes,
                                        daf_stream stream)
{
    return daf_act_compress(params, DAF_ACT_RELU, d_in, d_act, d_packed, packed_capacity, d_bits, d_min, d_scale,
                            d_window_offsets, d_workspace, workspace_bytes, stream);
}

// ------------------------------------------------------------------------------------------
// Compress with the kernel's scratch in a fixed device array instead of a caller's workspace,
// for callers that cannot allocate one (see include/daf.h).  In host code the array's name is
// only a handle: the address a kernel can use comes from cudaGetSymbolAddress, looked up once
// per device with that device current.
// ------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(WorkspaceHeader) + 16ull * DAF_STATIC_MAX_WINDOWS];

extern "C" daf_status daf_compress_static(const daf_params *params, const void *d_in, void *d_packed,
                                          uint64_t packed_capacity, uint8_t *d_bits, float *d_min, float *d_scale,
                                          uint64_t *d_window_offsets, uint32_t *d_status, daf_stream stream)
{
    Plan pl;
    daf_status st = make_plan(params, &pl);
    if (st != DAF_OK) return st;
    if (!d_in || !d_packed || !d_bits || !d_min || !d_scale || !d_window_offsets) return DAF_ERR_INVALID_ARG;
    if (!aligned_in(d_in, params->dtype) || !aligned16(d_packed) || (reinterpret_cast<uintptr_t>(d_min) & 3u) ||
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
    if (dispatch<false>(params->dtype, pl.chunks, params->flags, a, s) != cudaSuccess) return DAF_ERR_CUDA;
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
    return sizeof(WorkspaceHeader) + 16ull * windows;
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
            pl.beta_q8 != pl0.beta_q8 || p->rounding != params[0].rounding || p->flags != params[0].flags)
            return DAF_ERR_INVALID_ARG;
        if (!d_in[i] || !d_packed[i] || !d_bits[i] || !d_min[i] || !d_scale[i] || !d_window_offsets[i] || !aligned_in(d_in[i], params[i].dtype) ||
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
    const uint64_t need = sizeof(WorkspaceHeader) + 16ull * windows;
    if (workspace_bytes < need) return DAF_ERR_CAPACITY;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (!(params[0].flags & DAF_FLAG_KEEP_WORKSPACE) && cudaMemsetAsync(d_workspace, 0, need, s) != cudaSuccess) return DAF_ERR_CUDA;
    return dispatch<true>(params[0].dtype, pl0.chunks, params[0].flags, a, s) == cudaSuccess ? DAF_OK : DAF_ERR_CUDA;
}
