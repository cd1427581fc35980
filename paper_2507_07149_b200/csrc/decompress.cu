// Decompress kernel: unpack + dequantize (Sec. 2.3 of the paper: stored activations return to
// their original precision before the gradient computation).  One CTA per window; no CTA
// depends on another because compress stored every window's byte offset.
//
//   bits of the window's groups -> intra-window exclusive scan of the group byte lengths
//   -> each lane reads the b bytes holding its 8 consecutive codes, widens them with the
//      power-of-two offset of Eq. 5 (bits | 0x4B000000 is the float 2^23 + code),
//      x_hat = fma(code, scale, min), rounds to the output type and stores 32 (or 16) bytes.
#include "common.cuh"

namespace daf {

struct DecTensor {
    const uint8_t *packed;
    const uint8_t *bits;
    const float *mn;
    const float *scale;
    const uint64_t *woff;
    void *out;
    uint64_t numel;
    uint32_t first_window;
    uint32_t n_windows;
    const void *grad;        // fused consumer (daf_decompress_relu_grad): the incoming gradient
};

template <int NT> struct DecompressArgs {
    uint32_t total_windows, n_tensors, G, log2G;
    DecTensor t[NT];
};

struct DecRec {
    float mn, scale;
    uint32_t b, off;
};

// The restored value as it would be stored in type T (round to nearest even), back in binary32.
template <typename T> __device__ __forceinline__ float as_stored(float y);
template <> __device__ __forceinline__ float as_stored<float>(float y) { return y; }
template <> __device__ __forceinline__ float as_stored<__half>(float y) { return __half2float(__float2half_rn(y)); }
template <> __device__ __forceinline__ float as_stored<__nv_bfloat16>(float y) { return __bfloat162float(__float2bfloat16_rn(y)); }

// MASK != 0: fused consumer.  Instead of the restored value the kernel stores the gradient of the activation
// whose producer stored it: ReLU, the incoming gradient where the restored output is positive, else +0; ReLU6, where
// it lies strictly between 0 and 6; GELU, the incoming gradient times GELU'(restored input).
template <typename T, int CHUNKS, bool BATCH, int MASK>
__global__ void __launch_bounds__(kThreads)
decompress_kernel(const __grid_constant__ DecompressArgs<BATCH ? DAF_BATCH_MAX : 1> a)
{
    constexpr uint32_t WE = kThreads * kLaneElems * CHUNKS;
    __shared__ __align__(16) DecRec s_grp[kMaxGroups];
    __shared__ uint32_t s_wtot[kWarps];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t G = a.G, log2G = a.log2G;
    const uint32_t gw = blockIdx.x;

    uint32_t ti = 0;
    if (BATCH) {
        uint32_t lo = 0, hi = a.n_tensors - 1;
        while (lo < hi) {
            uint32_t mid = (lo + hi + 1) >> 1;
            if (a.t[mid].first_window <= gw) lo = mid; else hi = mid - 1;
        }
        ti = lo;
    }
    const DecTensor &td = a.t[ti];
    const uint32_t w = gw - td.first_window;
    const uint64_t wbase = (uint64_t)w * WE;
    const uint64_t left = td.numel - wbase;
    const uint32_t n_elems = left < WE ? (uint32_t)left : WE;
    const uint32_t n = n_elems >> log2G;
    const uint64_t g0 = wbase >> log2G;

    const uint64_t window_offset = td.woff[w];                    // asked for now, needed after the two meetings below
    // group records: width, min, scale and the group's byte offset inside the window; built by the
    // warps whose threads map to groups (thread g: group g), the others only meet them
    const bool owner = (uint32_t)(warp * 32) < n;
    uint32_t b = 0, size = 0, incl = 0;
    float mn = 0.0f, scale = 0.0f;
    if (owner) {
        if ((uint32_t)tid < n) {
            b = td.bits[g0 + tid];
            mn = td.mn[g0 + tid];
            scale = td.scale[g0 + tid];
            size = (G >> 3) * b;
        }
        incl = size;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            uint32_t y = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += y;
        }
        if (lane == 31) s_wtot[warp] = incl;
    }
    __syncthreads();
    if ((uint32_t)tid < n) {
        uint32_t before = 0;
        for (int i = 0; i < warp; i++) before += s_wtot[i];
        DecRec rec;
        rec.mn = mn;
        rec.scale = scale;
        rec.b = b;
        rec.off = before + incl - size;
        s_grp[tid] = rec;
    }
    __syncthreads();

    const uint8_t *src = td.packed + window_offset;
    char *out = reinterpret_cast<char *>(td.out) + wbase * Elem<T>::kBytes;
#pragma unroll
    for (int c = 0; c < CHUNKS; c++) {
        const uint32_t e = (uint32_t)((warp * CHUNKS + c) * 256 + lane * 8);
        if (e >= n_elems) continue;
        const DecRec rec = s_grp[e >> log2G];
        const uint8_t *p = src + rec.off + ((e & (G - 1u)) >> 3) * rec.b;
        float y[8];
        switch (rec.b) {
        case 1: decode8<1>(*p, 0u, rec.mn, rec.scale, y); break;
        case 2: decode8<2>(*reinterpret_cast<const uint16_t *>(p), 0u, rec.mn, rec.scale, y); break;
        case 4: decode8<4>(*reinterpret_cast<const uint32_t *>(p), 0u, rec.mn, rec.scale, y); break;
        default: {
            uint32_t w0, w1;
            if (G >= 64u) {
                const uint2 v = *reinterpret_cast<const uint2 *>(p);
                w0 = v.x;
                w1 = v.y;
            } else {                                              // G = 32: groups are only 4-byte aligned
                w0 = reinterpret_cast<const uint32_t *>(p)[0];
                w1 = reinterpret_cast<const uint32_t *>(p)[1];
            }
            decode8<8>(w0, w1, rec.mn, rec.scale, y);
            break;
        }
        }
        if (MASK) {
            float g[8];
            Elem<T>::load8(reinterpret_cast<const char *>(td.grad) + (wbase + e) * Elem<T>::kBytes, g);
#pragma unroll
            for (int i = 0; i < 8; i++) {
                const float r = as_stored<T>(y[i]);
                if (MASK == kActRelu) y[i] = r > 0.0f ? g[i] : 0.0f;
                else if (MASK == kActRelu6) y[i] = (r > 0.0f && r < 6.0f) ? g[i] : 0.0f;
                else y[i] = g[i] * gelu_grad_f(r);
            }
        }
        Elem<T>::store8(out + (size_t)e * Elem<T>::kBytes, y);
    }
}

// The same for windows of at most 64 groups (groups of 256 elements or more at the default window): no shared memory
// and no meeting of the CTA's warps.  Every warp reads the widths of the window's groups itself (two per lane, 64 bytes
// that sit in L1 after the first warp), scans their byte lengths with shuffles and serves its own chunks; a chunk lies
// in one group, so width, offset, min and scale are the same for all its lanes.
template <typename T, int CHUNKS, bool BATCH, int MASK>
__global__ void __launch_bounds__(kThreads, MASK == kActGelu ? 3 : 4)   // (32 registers: four CTAs per SM; the GELU factor needs more)
decompress_few_groups_kernel(const __grid_constant__ DecompressArgs<BATCH ? DAF_BATCH_MAX : 1> a)
{
    constexpr uint32_t WE = kThreads * kLaneElems * CHUNKS;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t G = a.G, log2G = a.log2G;
    const uint32_t gw = blockIdx.x;
    uint32_t ti = 0;
    if (BATCH) {
        uint32_t lo = 0, hi = a.n_tensors - 1;
        while (lo < hi) {
            uint32_t mid = (lo + hi + 1) >> 1;
            if (a.t[mid].first_window <= gw) lo = mid; else hi = mid - 1;
        }
        ti = lo;
    }
    const DecTensor &td = a.t[ti];
    const uint32_t w = gw - td.first_window;
    const uint64_t wbase = (uint64_t)w * WE;
    const uint64_t left = td.numel - wbase;
    const uint32_t n_elems = left < WE ? (uint32_t)left : WE;
    const uint32_t n = n_elems >> log2G;
    const uint64_t g0 = wbase >> log2G;
    const uint32_t first_chunk = (uint32_t)warp * CHUNKS * 256u;
    if (first_chunk >= n_elems) return;                           // (a ragged window: nothing for this warp)

    const uint64_t window_offset = td.woff[w];
    const uint32_t b0 = (uint32_t)lane < n ? td.bits[g0 + lane] : 0u, b1 = (uint32_t)lane + 32u < n ? td.bits[g0 + lane + 32] : 0u;
    // min and scale of the warp's chunks' groups, asked for early
    float mn[CHUNKS], scale[CHUNKS];
#pragma unroll
    for (int c = 0; c < CHUNKS; c++) {
        const uint32_t cs = first_chunk + 256u * c;
        const uint32_t g = cs < n_elems ? cs >> log2G : 0u;
        mn[c] = td.mn[g0 + g];
        scale[c] = td.scale[g0 + g];
    }
    const uint32_t size0 = (G >> 3) * b0, size1 = (G >> 3) * b1;
    uint32_t incl0 = size0, incl1 = size1;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const uint32_t y0 = __shfl_up_sync(0xFFFFFFFFu, incl0, off), y1 = __shfl_up_sync(0xFFFFFFFFu, incl1, off);
        if (lane >= off) {
            incl0 += y0;
            incl1 += y1;
        }
    }
    const uint32_t excl0 = incl0 - size0, excl1 = __shfl_sync(0xFFFFFFFFu, incl0, 31) + incl1 - size1;

    const uint8_t *src = td.packed + window_offset;
    char *out = reinterpret_cast<char *>(td.out) + wbase * Elem<T>::kBytes;
#pragma unroll
    for (int c = 0; c < CHUNKS; c++) {
        const uint32_t cs = first_chunk + 256u * c;               // the chunk's first element: the same for all lanes
        if (cs >= n_elems) break;
        const uint32_t g = cs >> log2G, from = g & 31u;
        const uint32_t b = __shfl_sync(0xFFFFFFFFu, g < 32u ? b0 : b1, (int)from);
        const uint32_t goff = __shfl_sync(0xFFFFFFFFu, g < 32u ? excl0 : excl1, (int)from);
        const uint32_t e = cs + (uint32_t)lane * 8u;
        const uint8_t *p = src + goff + ((e & (G - 1u)) >> 3) * b;
        float y[8];
        switch (b) {
        case 1: decode8<1>(*p, 0u, mn[c], scale[c], y); break;
        case 2: decode8<2>(*reinterpret_cast<const uint16_t *>(p), 0u, mn[c], scale[c], y); break;
        case 4: decode8<4>(*reinterpret_cast<const uint32_t *>(p), 0u, mn[c], scale[c], y); break;
        default: {
            const uint2 v = *reinterpret_cast<const uint2 *>(p);
            decode8<8>(v.x, v.y, mn[c], scale[c], y);
            break;
        }
        }
        if (MASK != kActNone) {
            float gr[8];
            Elem<T>::load8(reinterpret_cast<const char *>(td.grad) + (wbase + e) * Elem<T>::kBytes, gr);
#pragma unroll
            for (int i = 0; i < 8; i++) {
                const float r = as_stored<T>(y[i]);
                if (MASK == kActRelu) y[i] = r > 0.0f ? gr[i] : 0.0f;
                else if (MASK == kActRelu6) y[i] = (r > 0.0f && r < 6.0f) ? gr[i] : 0.0f;
                else y[i] = gr[i] * gelu_grad_f(r);
            }
        }
        Elem<T>::store8(out + (size_t)e * Elem<T>::kBytes, y);
    }
}

template <typename T, int CHUNKS, bool BATCH, int MASK>
static cudaError_t launch(const DecompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args, cudaStream_t stream)
{
    if (args.G >= 256u)                                           // a chunk lies in one group, a window has at most 64
        decompress_few_groups_kernel<T, CHUNKS, BATCH, MASK><<<args.total_windows, kThreads, 0, stream>>>(args);
    else
        decompress_kernel<T, CHUNKS, BATCH, MASK><<<args.total_windows, kThreads, 0, stream>>>(args);
    return cudaGetLastError();
}

template <bool BATCH, int MASK = kActNone>
static cudaError_t dispatch(uint32_t dtype, uint32_t chunks, const DecompressArgs<BATCH ? DAF_BATCH_MAX : 1> &args,
                            cudaStream_t stream)
{
#define DAF_CASE(T)                                                     \
    switch (chunks) {                                                   \
    case 1: return launch<T, 1, BATCH, MASK>(args, stream);             \
    case 2: return launch<T, 2, BATCH, MASK>(args, stream);             \
    default: return launch<T, 4, BATCH, MASK>(args, stream);            \
    }
    if (dtype == DAF_F32) { DAF_CASE(float) }
    if (dtype == DAF_F16) { DAF_CASE(__half) }
    DAF_CASE(__nv_bfloat16)
#undef DAF_CASE
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static daf_status check_ptrs(const void *packed, const uint8_t *bits, const float *mn, const float *scale,
                             const uint64_t *woff, const void *out, uint32_t dtype)
{
    if (!packed || !bits || !mn || !scale || !woff || !out) return DAF_ERR_INVALID_ARG;
    const uintptr_t out_mask = dtype == DAF_F32 ? 31u : 15u;      // a lane stores its 8 elements at once
    if (!aligned16(packed) || (reinterpret_cast<uintptr_t>(out) & out_mask) || (reinterpret_cast<uintptr_t>(mn) & 3u) ||
        (reinterpret_cast<uintptr_t>(scale) & 3u) || (reinterpret_cast<uintptr_t>(woff) & 7u))
        return DAF_ERR_INVALID_ARG;
    return DAF_OK;
}

}  // namespace daf

using namespace daf;

extern "C" daf_status daf_decompress(const daf_params *params, const void *d_packed, const uint8_t *d_bits,
                                     const float *d_min, const float *d_scale, const uint64_t *d_window_offsets,
                                     void *d_out, void *d_workspace, uint64_t workspace_bytes, daf_stream stream)
{
    (void)d_workspace;
    (void)workspace_bytes;
    Plan pl;
    daf_status st = make_plan(params, &pl);
    if (st != DAF_OK) return st;
    st = check_ptrs(d_packed, d_bits, d_min, d_scale, d_window_offsets, d_out, params->dtype);
    if (st != DAF_OK) return st;
    if (pl.n_windows > 0x7FFFFFFFull) return DAF_ERR_UNSUPPORTED;
    DecompressArgs<1> a;
    a.total_windows = (uint32_t)pl.n_windows;
    a.n_tensors = 1;
    a.G = pl.G;
    a.log2G = pl.log2G;
    a.t[0] = DecTensor{reinterpret_cast<const uint8_t *>(d_packed), d_bits, d_min, d_scale, d_window_offsets, d_out,
                       params->numel, 0u, (uint32_t)pl.n_windows};
    return dispatch<false>(params->dtype, pl.chunks, a, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess ? DAF_OK
                                                                                                                 : DAF_ERR_CUDA;
}

extern "C" daf_status daf_decompress_act_grad(const daf_params *params, uint32_t act, const void *d_packed,
                                              const uint8_t *d_bits, const float *d_min, const float *d_scale,
                                              const uint64_t *d_window_offsets, const void *d_grad_out, void *d_grad_in,
                                              daf_stream stream)
{
    if (act != DAF_ACT_RELU && act != DAF_ACT_RELU6 && act != DAF_ACT_GELU) return DAF_ERR_INVALID_ARG;
    Plan pl;
    daf_status st = make_plan(params, &pl);
    if (st != DAF_OK) return st;
    st = check_ptrs(d_packed, d_bits, d_min, d_scale, d_window_offsets, d_grad_in, params->dtype);
    if (st != DAF_OK) return st;
    if (!d_grad_out || (reinterpret_cast<uintptr_t>(d_grad_out) & (params->dtype == DAF_F32 ? 31u : 15u))) return DAF_ERR_INVALID_ARG;
    if (pl.n_windows > 0x7FFFFFFFull) return DAF_ERR_UNSUPPORTED;
    DecompressArgs<1> a;
    a.total_windows = (uint32_t)pl.n_windows;
    a.n_tensors = 1;
    a.G = pl.G;
    a.log2G = pl.log2G;
    a.t[0] = DecTensor{reinterpret_cast<const uint8_t *>(d_packed), d_bits, d_min, d_scale, d_window_offsets, d_grad_in,
                       params->numel, 0u, (uint32_t)pl.n_windows, d_grad_out};
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (act == DAF_ACT_RELU) e = dispatch<false, kActRelu>(params->dtype, pl.chunks, a, s);
    else if (act == DAF_ACT_RELU6) e = dispatch<false, kActRelu6>(params->dtype, pl.chunks, a, s);
    else e = dispatch<false, kActGelu>(params->dtype, pl.chunks, a, s);
    return e == cudaSuccess ? DAF_OK : DAF_ERR_CUDA;
}

extern "C" daf_status daf_decompress_relu_grad(const daf_params *params, const void *d_packed, const uint8_t *d_bits,
                                               const float *d_min, const float *d_scale, const uint64_t *d_window_offsets,
                                               const void *d_grad_out, void *d_grad_in, daf_stream stream)
{
    return daf_decompress_act_grad(params, DAF_ACT_RELU, d_packed, d_bits, d_min, d_scale, d_window_offsets, d_grad_out,
                                   d_grad_in, stream);
}


extern "C" daf_status daf_decompress_batch(uint32_t n, const daf_params *params, const void *const *d_packed,
                                           const uint8_t *const *d_bits, const float *const *d_min,
                                           const float *const *d_scale, const uint64_t *const *d_window_offsets,
                                           void *const *d_out, daf_stream stream)
{
    if (n == 0 || n > DAF_BATCH_MAX || !params || !d_packed || !d_bits || !d_min || !d_scale || !d_window_offsets || !d_out)
        return DAF_ERR_INVALID_ARG;
    Plan pl0;
    daf_status st = make_plan(&params[0], &pl0);
    if (st != DAF_OK) return st;
    DecompressArgs<DAF_BATCH_MAX> a;
    a.n_tensors = n;
    a.G = pl0.G;
    a.log2G = pl0.log2G;
    uint64_t windows = 0;
    for (uint32_t i = 0; i < n; i++) {
        Plan pl;
        st = make_plan(&params[i], &pl);
        if (st != DAF_OK) return st;
        if (params[i].dtype != params[0].dtype || pl.G != pl0.G || pl.We != pl0.We) return DAF_ERR_INVALID_ARG;
        st = check_ptrs(d_packed[i], d_bits[i], d_min[i], d_scale[i], d_window_offsets[i], d_out[i], params[i].dtype);
        if (st != DAF_OK) return st;
        if (windows + pl.n_windows > 0x7FFFFFFFull) return DAF_ERR_UNSUPPORTED;
        a.t[i] = DecTensor{reinterpret_cast<const uint8_t *>(d_packed[i]), d_bits[i], d_min[i], d_scale[i],
                           d_window_offsets[i], d_out[i], params[i].numel, (uint32_t)windows, (uint32_t)pl.n_windows};
        windows += pl.n_windows;
    }
    a.total_windows = (uint32_t)windows;
    return dispatch<true>(params[0].dtype, pl0.chunks, a, reinterpret_cast<cudaStream_t>(stream)) == cudaSuccess
               ? DAF_OK
               : DAF_ERR_CUDA;
}
