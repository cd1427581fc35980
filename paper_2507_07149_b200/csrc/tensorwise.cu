// Per-tensor statistics and per-tensor quantization: Eq. 1 of the paper at the granularity the paper states it (one
// min, max and bit width per activation tensor), with the collective reduction of Sec. 3.2.1-3.2.2 behind it.
//
//   daf_tensor_minmax     one pass over the tensor: lane-local 3-input min / max on 256-bit loads, warp redux, a tree over
//                         the CTA's warps in shared memory, then ONE atomic per CTA and statistic on a monotone integer key
//                         of the float (the paper's hybrid of tree and atomic reduction; its compare-and-swap loop, Alg. 1,
//                         is replaced by the native integer atomic max on that key).  The CTA that finishes last turns the
//                         keys back into floats.  Bound: HBM reads.
//   daf_tensor_compress   Eq. 1 with the tensor's min and range: Philox4x32-10 stochastic rounding, fixed width, codes
//                         packed LSB-first.  Element-wise; bound: HBM reads.
//   daf_tensor_decompress the inverse: x_hat = fma(code, scale, min).
//
// The group-wise path (compress.cu) is the product's main line; this file is the special case "one group = the tensor".
#include "compress_shared.cuh"

namespace daf {

// Monotone map float -> uint32 under the total order in which -0 < +0 (and back).
__device__ __forceinline__ uint32_t ordered_key(float f)
{
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : u | 0x80000000u;
}
__device__ __forceinline__ float from_ordered_key(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? k & 0x7FFFFFFFu : ~k);
}

// d_stats words: [0] min, [1] max, [2] range (0 for a degenerate tensor), [3] unused, [4] key accumulator of the minimum
// (complemented, so that zero is its identity), [5] key accumulator of the maximum, [6] CTAs done.  Words 4-6 are zero on entry.
template <typename T>
__global__ void __launch_bounds__(kThreads) tensor_minmax_kernel(const void *in, uint64_t n_units, uint32_t *stats)
{
    __shared__ float s_lo[kWarps], s_hi[kWarps];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const char *const base = reinterpret_cast<const char *>(in);
    constexpr uint64_t UB = 8u * Elem<T>::kBytes;                 // bytes of a unit (8 elements, one load)
    float lo = __uint_as_float(0x7F800000u), hi = __uint_as_float(0xFF800000u);
    const uint64_t stride = (uint64_t)gridDim.x * kThreads;
    uint64_t u = (uint64_t)blockIdx.x * kThreads + tid;
    // four loads in flight per lane
    for (; u + 3u * stride < n_units; u += 4u * stride) {
        float x[4][8];
#pragma unroll
        for (int j = 0; j < 4; j++) Elem<T>::load8(base + (u + j * stride) * UB, x[j]);
#pragma unroll
        for (int j = 0; j < 4; j++) {
            lo = fmin3(lo, fmin3(x[j][0], x[j][1], x[j][2]), fmin3(x[j][3], x[j][4], x[j][5]));
            lo = fmin3(lo, x[j][6], x[j][7]);
            hi = fmax3(hi, fmax3(x[j][0], x[j][1], x[j][2]), fmax3(x[j][3], x[j][4], x[j][5]));
            hi = fmax3(hi, x[j][6], x[j][7]);
        }
    }
    for (; u < n_units; u += stride) {
        float x[8];
        Elem<T>::load8(base + u * UB, x);
        lo = fmin3(lo, fmin3(x[0], x[1], x[2]), fmin3(x[3], x[4], x[5]));
        lo = fmin3(lo, x[6], x[7]);
        hi = fmax3(hi, fmax3(x[0], x[1], x[2]), fmax3(x[3], x[4], x[5]));
        hi = fmax3(hi, x[6], x[7]);
    }
    asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(lo) : "f"(lo));
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(hi) : "f"(hi));
    if (lane == 0) {
        s_lo[warp] = lo;
        s_hi[warp] = hi;
    }
    __syncthreads();
    if (warp == 0) {
        lo = lane < kWarps ? s_lo[lane] : __uint_as_float(0x7F800000u);
        hi = lane < kWarps ? s_hi[lane] : __uint_as_float(0xFF800000u);
        asm volatile("redux.sync.min.f32 %0, %1, 0xffffffff;" : "=f"(lo) : "f"(lo));
        asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(hi) : "f"(hi));
        if (lane == 0) {
            atomicMax(&stats[4], ~ordered_key(lo));
            atomicMax(&stats[5], ordered_key(hi));
            __threadfence();
            if (atomicAdd(&stats[6], 1u) == gridDim.x - 1u) {     // the last CTA: every CTA's contribution is in
                __threadfence();
                const float mn = from_ordered_key(~atomicMax(&stats[4], 0u)), mx = from_ordered_key(atomicMax(&stats[5], 0u));
                float R = __fsub_rn(mx, mn);
                if (!(R >= 0x1p-118f)) R = 0.0f;                  // degenerate: treated as constant (as for groups)
                stats[0] = __float_as_uint(mn);
                stats[1] = __float_as_uint(mx);
                stats[2] = __float_as_uint(R);
            }
        }
    }
}

template <int B> __device__ __forceinline__ void store_codes(unsigned char *p, uint32_t w0, uint32_t w1)
{
    if (B == 1) *p = (unsigned char)w0;
    else if (B == 2) *reinterpret_cast<uint16_t *>(p) = (uint16_t)w0;
    else if (B == 4) *reinterpret_cast<uint32_t *>(p) = w0;
    else *reinterpret_cast<uint2 *>(p) = make_uint2(w0, w1);
}
template <int B> __device__ __forceinline__ void load_codes(const unsigned char *p, uint32_t &w0, uint32_t &w1)
{
    w1 = 0u;
    if (B == 1) w0 = *p;
    else if (B == 2) w0 = *reinterpret_cast<const uint16_t *>(p);
    else if (B == 4) w0 = *reinterpret_cast<const uint32_t *>(p);
    else {
        const uint2 v = *reinterpret_cast<const uint2 *>(p);
        w0 = v.x;
        w1 = v.y;
    }
}

// Eq. 1 with the tensor's statistics.  A warp takes chunks of 256 elements (8 per lane = one Philox block per lane).
template <typename T, int B>
__global__ void __launch_bounds__(kThreads, 2)
tensor_quantize_kernel(const void *in, uint64_t n_units, const uint32_t *stats, unsigned char *packed, float *min_scale,
                       PhiloxKeys keys, uint64_t blk_base, uint32_t nearest)
{
    const int lane = threadIdx.x & 31;
    constexpr float Lf = (float)((1u << B) - 1u);
    constexpr uint64_t UB = 8u * Elem<T>::kBytes;
    const float mn = __uint_as_float(stats[0]), R = __uint_as_float(stats[2]);
    const float inv = R > 0.0f ? __fdiv_rn(Lf, R) : 0.0f;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        min_scale[0] = mn;
        min_scale[1] = R > 0.0f ? __fdiv_rn(R, Lf) : 0.0f;
    }
    const char *const base = reinterpret_cast<const char *>(in);
    const uint64_t n_warps = (uint64_t)gridDim.x * kWarps, gwarp = (uint64_t)blockIdx.x * kWarps + (threadIdx.x >> 5);
    const uint64_t n_chunks = (n_units + 31u) >> 5;
    for (uint64_t c0 = gwarp * 4u; c0 < n_chunks; c0 += n_warps * 4u) {
        float x[4][8];
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const uint64_t u = (c0 + j) * 32u + lane;
#pragma unroll
            for (int i = 0; i < 8; i++) x[j][i] = mn;
            if (u < n_units) Elem<T>::load8(base + u * UB, x[j]);
        }
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const uint64_t u = (c0 + j) * 32u + lane;
            uint32_t o[4], w0, w1;
            if (nearest) {
                o[0] = o[1] = o[2] = o[3] = 0x80008000u;           // every 16-bit lane = 2 * 2^14: round half up
            } else {
                const uint64_t blk = blk_base + u;
                philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), keys, o);
            }
            // 1/scale is a normal number unless the range passes about 2^126: only then can a code pass L and need the clamp
            if (R > 0x1p125f) quantize8<B, true>(x[j], mn, inv, o, w0, w1);
            else quantize8<B, false>(x[j], mn, inv, o, w0, w1);
            if (u < n_units) store_codes<B>(packed + u * B, w0, w1);
        }
    }
}

template <typename T, int B>
__global__ void __launch_bounds__(kThreads, 4)
tensor_dequantize_kernel(const unsigned char *packed, uint64_t n_units, const float *min_scale, void *out)
{
    const int lane = threadIdx.x & 31;
    constexpr uint64_t UB = 8u * Elem<T>::kBytes;
    const float mn = min_scale[0], scale = min_scale[1];
    char *const base = reinterpret_cast<char *>(out);
    const uint64_t n_warps = (uint64_t)gridDim.x * kWarps, gwarp = (uint64_t)blockIdx.x * kWarps + (threadIdx.x >> 5);
    const uint64_t n_chunks = (n_units + 31u) >> 5;
    for (uint64_t c0 = gwarp * 4u; c0 < n_chunks; c0 += n_warps * 4u) {
        uint32_t w0[4], w1[4];
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const uint64_t u = (c0 + j) * 32u + lane;
            w0[j] = w1[j] = 0u;
            if (u < n_units) load_codes<B>(packed + u * B, w0[j], w1[j]);
        }
#pragma unroll
        for (int j = 0; j < 4; j++) {
            const uint64_t u = (c0 + j) * 32u + lane;
            float y[8];
            decode8<B>(w0[j], w1[j], mn, scale, y);
            if (u < n_units) Elem<T>::store8(base + u * UB, y);
        }
    }
}

static bool aligned_to(const void *p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1u)) == 0; }

static daf_status check_tensor(uint32_t dtype, const void *d_data, uint64_t numel)
{
    if (dtype > DAF_BF16 || !d_data || !aligned_to(d_data, dtype == DAF_F32 ? 32u : 16u)) return DAF_ERR_INVALID_ARG;
    if (numel == 0 || numel % 8u) return DAF_ERR_SHAPE;
    return DAF_OK;
}

template <typename K> static cudaError_t grid_for(K kernel, uint64_t work_items, uint32_t *grid)
{
    int ctas = 0;
    const cudaError_t e = persistent_ctas(reinterpret_cast<const void *>(kernel), kThreads, 0, &ctas);
    if (e != cudaSuccess) return e;
    *grid = (uint32_t)(work_items < (uint64_t)ctas ? (work_items ? work_items : 1u) : (uint64_t)ctas);
    return cudaSuccess;
}

}  // namespace daf

using namespace daf;

extern "C" daf_status daf_tensor_minmax(uint32_t dtype, const void *d_in, uint64_t numel, void *d_stats, daf_stream stream)
{
    daf_status st = check_tensor(dtype, d_in, numel);
    if (st != DAF_OK) return st;
    if (!d_stats || !aligned_to(d_stats, 16u)) return DAF_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    uint32_t *stats = reinterpret_cast<uint32_t *>(d_stats);
    if (cudaMemsetAsync(stats + 4, 0, 16, s) != cudaSuccess) return DAF_ERR_CUDA;
    const uint64_t n_units = numel / 8u, per_cta = (uint64_t)kThreads * 4u;
    uint32_t grid = 1;
    cudaError_t e;
#define DAF_MINMAX(T)                                                                         \
    e = grid_for(&tensor_minmax_kernel<T>, (n_units + per_cta - 1u) / per_cta, &grid);        \
    if (e == cudaSuccess) tensor_minmax_kernel<T><<<grid, kThreads, 0, s>>>(d_in, n_units, stats);
    if (dtype == DAF_F32) { DAF_MINMAX(float) }
    else if (dtype == DAF_F16) { DAF_MINMAX(__half) }
    else { DAF_MINMAX(__nv_bfloat16) }
#undef DAF_MINMAX
    return e == cudaSuccess && cudaGetLastError() == cudaSuccess ? DAF_OK : DAF_ERR_CUDA;
}

namespace {

template <typename T, int B>
cudaError_t launch_quantize(const void *d_in, uint64_t n_units, const uint32_t *stats, unsigned char *packed, float *min_scale,
                            const PhiloxKeys &keys, uint64_t blk_base, uint32_t nearest, cudaStream_t s)
{
    uint32_t grid = 1;
    const cudaError_t e = grid_for(&tensor_quantize_kernel<T, B>, (n_units + 2047u) / 2048u, &grid);
    if (e != cudaSuccess) return e;
    tensor_quantize_kernel<T, B><<<grid, kThreads, 0, s>>>(d_in, n_units, stats, packed, min_scale, keys, blk_base, nearest);
    return cudaGetLastError();
}
template <typename T, int B>
cudaError_t launch_dequantize(const unsigned char *packed, uint64_t n_units, const float *min_scale, void *out, cudaStream_t s)
{
    // one CTA per 16384 elements, as many CTAs as that takes (no CTA depends on another; measured faster than a
    // persistent grid: the hardware's block scheduler balances the write stream better)
    const uint64_t ctas = (n_units + 2047u) / 2048u;
    const uint32_t grid = (uint32_t)(ctas < 0x7FFFFFFFull ? ctas : 0x7FFFFFFFull);
    tensor_dequantize_kernel<T, B><<<grid, kThreads, 0, s>>>(packed, n_units, min_scale, out);
    return cudaGetLastError();
}

}  // namespace

#define DAF_BY_WIDTH(CALL, T)                    \
    switch (width) {                             \
    case 1: e = CALL(T, 1); break;               \
    case 2: e = CALL(T, 2); break;               \
    case 4: e = CALL(T, 4); break;               \
    default: e = CALL(T, 8); break;              \
    }
#define DAF_BY_TYPE(CALL)                                     \
    if (dtype == DAF_F32) { DAF_BY_WIDTH(CALL, float) }       \
    else if (dtype == DAF_F16) { DAF_BY_WIDTH(CALL, __half) } \
    else { DAF_BY_WIDTH(CALL, __nv_bfloat16) }

extern "C" daf_status daf_tensor_compress(uint32_t dtype, const void *d_in, uint64_t numel, uint32_t width, uint32_t rounding,
                                          uint64_t seed, uint64_t elem_index_base, const void *d_stats, void *d_packed,
                                          float *d_min_scale, daf_stream stream)
{
    daf_status st = check_tensor(dtype, d_in, numel);
    if (st != DAF_OK) return st;
    if ((width != 1 && width != 2 && width != 4 && width != 8) || rounding > DAF_ROUND_NEAREST || (elem_index_base & 7u) || !d_stats ||
        !aligned_to(d_stats, 16u) || !d_packed || !aligned_to(d_packed, 16u) || !d_min_scale || !aligned_to(d_min_scale, 4u))
        return DAF_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const uint64_t n_units = numel / 8u;
    const PhiloxKeys keys = philox_keys(seed);
    const uint32_t *stats = reinterpret_cast<const uint32_t *>(d_stats);
    unsigned char *packed = reinterpret_cast<unsigned char *>(d_packed);
    cudaError_t e;
#define DAF_Q(T, B) launch_quantize<T, B>(d_in, n_units, stats, packed, d_min_scale, keys, elem_index_base >> 3, rounding == DAF_ROUND_NEAREST, s)
    DAF_BY_TYPE(DAF_Q)
#undef DAF_Q
    return e == cudaSuccess ? DAF_OK : DAF_ERR_CUDA;
}

extern "C" daf_status daf_tensor_decompress(uint32_t dtype, const void *d_packed, uint64_t numel, uint32_t width,
                                            const float *d_min_scale, void *d_out, daf_stream stream)
{
    daf_status st = check_tensor(dtype, d_out, numel);
    if (st != DAF_OK) return st;
    if ((width != 1 && width != 2 && width != 4 && width != 8) || !d_packed || !aligned_to(d_packed, 16u) || !d_min_scale ||
        !aligned_to(d_min_scale, 4u))
        return DAF_ERR_INVALID_ARG;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const uint64_t n_units = numel / 8u;
    const unsigned char *packed = reinterpret_cast<const unsigned char *>(d_packed);
    cudaError_t e;
#define DAF_D(T, B) launch_dequantize<T, B>(packed, n_units, d_min_scale, d_out, s)
    DAF_BY_TYPE(DAF_D)
#undef DAF_D
    return e == cudaSuccess ? DAF_OK : DAF_ERR_CUDA;
}
