// Device-side helpers shared by the compress / decompress / scan kernels (sm_100a only).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/daf.h"

namespace daf {

constexpr int kThreads = 512;          // threads per CTA of the compress / decompress kernels
constexpr int kWarps = kThreads / 32;
constexpr int kLaneElems = 8;          // consecutive elements owned by one lane = one Philox block
constexpr int kMaxGroups = 512;        // groups per window at G = 32, window 16384
constexpr int kMaxLevels = 4;          // widths {1,2,4,8}

// ---------------------------------------------------------------------------------------------
// Workspace layout: a 256-byte header followed by two arrays of one 64-bit look-back descriptor
// per window (one array for the quick kernel, one for the full kernel that runs if the quick one
// gives up).  The header and the descriptors are zeroed by a memset enqueued ahead of the kernels.
// ---------------------------------------------------------------------------------------------
struct WorkspaceHeader {
    unsigned int status;        // daf_status recorded by the device (0 = OK)
    unsigned int ticket;        // next window to hand out
    unsigned int fail_window;   // first window that recorded an error (diagnostic)
    unsigned int fail_site;     // which wait or check recorded it (diagnostic)
    unsigned int retry;         // the quick kernel met a window it does not handle: the full kernel must run
    unsigned int ticket2;       // next window to hand out in the full kernel
    unsigned int pad[58];
};
static_assert(sizeof(WorkspaceHeader) == 256, "header is 256 bytes");

// Look-back descriptor: state in the top two bits, byte count in the low 62.
constexpr uint64_t kFlagShift = 62;
constexpr uint64_t kFlagEmpty = 0, kFlagAggregate = 1, kFlagPrefix = 2, kFlagPoison = 3;
constexpr uint64_t kFlagValueMask = (1ull << kFlagShift) - 1;
// A look-back wait polls at most this many times (with a short sleep between polls) before
// the kernel gives up, records DAF_ERR_TIMEOUT and poisons its own descriptor.
constexpr unsigned int kMaxPolls = 1u << 20;

__device__ __forceinline__ uint64_t ld_relaxed_u64(const uint64_t *p)
{
    uint64_t v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(uint64_t *p, uint64_t v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11).  Round keys are passed in precomputed, so that each
// round is two 32x32->64 multiplies and two three-input XORs.
// ---------------------------------------------------------------------------------------------
struct PhiloxKeys {
    uint32_t k0[10];
    uint32_t k1[10];
};

constexpr uint32_t kPhiloxM0 = 0xD2511F53u, kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u, kPhiloxW1 = 0xBB67AE85u;

__host__ __device__ inline PhiloxKeys philox_keys(uint64_t seed)
{
    PhiloxKeys k;
    uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; r++) {
        k.k0[r] = a;
        k.k1[r] = b;
        a += kPhiloxW0;
        b += kPhiloxW1;
    }
    return k;
}

// Counter (c0, c1, 0, 0): the third and fourth counter words are zero for every block this
// library draws, which removes one multiply from the first round.
template <typename Keys>
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, const Keys &keys, uint32_t (&o)[4])
{
    uint32_t c2 = 0u, c3 = 0u;
#pragma unroll
    for (int r = 0; r < 10; r++) {
        const uint64_t p0 = (uint64_t)kPhiloxM0 * c0, p1 = (uint64_t)kPhiloxM1 * c2;   // one wide multiply each
        c0 = (uint32_t)(p1 >> 32) ^ c1 ^ keys.k0[r];
        c1 = (uint32_t)p1;
        c2 = (uint32_t)(p0 >> 32) ^ c3 ^ keys.k1[r];
        c3 = (uint32_t)p0;
    }
    o[0] = c0; o[1] = c1; o[2] = c2; o[3] = c3;
}

// Round keys laid out in shared memory as {k0[r], k1[r]} pairs, r = 0 .. 9 (two rounds per
// 16-byte load): for kernels that serve tensors with different seeds.
struct PhiloxSharedKeys {
    const uint4 *pairs;
};
__device__ __forceinline__ void philox_store_round_keys(uint32_t *pairs, uint64_t seed, int r)
{
    pairs[2 * r] = (uint32_t)seed + (uint32_t)r * kPhiloxW0;
    pairs[2 * r + 1] = (uint32_t)(seed >> 32) + (uint32_t)r * kPhiloxW1;
}
template <>
__device__ __forceinline__ void philox4x32_10<PhiloxSharedKeys>(uint32_t c0, uint32_t c1, const PhiloxSharedKeys &s,
                                                                 uint32_t (&o)[4])
{
    uint32_t c2 = 0u, c3 = 0u;
#pragma unroll
    for (int i = 0; i < 5; i++) {
        const uint4 k = s.pairs[i];
        uint64_t p0 = (uint64_t)kPhiloxM0 * c0, p1 = (uint64_t)kPhiloxM1 * c2;
        c0 = (uint32_t)(p1 >> 32) ^ c1 ^ k.x;
        c1 = (uint32_t)p1;
        c2 = (uint32_t)(p0 >> 32) ^ c3 ^ k.y;
        c3 = (uint32_t)p0;
        p0 = (uint64_t)kPhiloxM0 * c0;
        p1 = (uint64_t)kPhiloxM1 * c2;
        c0 = (uint32_t)(p1 >> 32) ^ c1 ^ k.z;
        c1 = (uint32_t)p1;
        c2 = (uint32_t)(p0 >> 32) ^ c3 ^ k.w;
        c3 = (uint32_t)p0;
    }
    o[0] = c0; o[1] = c1; o[2] = c2; o[3] = c3;
}

// ---------------------------------------------------------------------------------------------
// Element types: 8 consecutive elements per lane, widened exactly to binary32.
// ---------------------------------------------------------------------------------------------
template <typename T> struct Elem;

template <> struct Elem<float> {
    static constexpr int kBytes = 4;
    // 32 bytes per lane in one 256-bit access (sm_100).
    static __device__ __forceinline__ void load8(const void *p, float (&x)[8])
    {
        asm volatile("ld.global.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=f"(x[0]), "=f"(x[1]), "=f"(x[2]), "=f"(x[3]), "=f"(x[4]), "=f"(x[5]), "=f"(x[6]), "=f"(x[7])
                     : "l"(p));
    }
    // the same load, but the line may stay in L1 for a second reader on this multiprocessor
    static __device__ __forceinline__ void load8_keep(const void *p, float (&x)[8])
    {
        asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=f"(x[0]), "=f"(x[1]), "=f"(x[2]), "=f"(x[3]), "=f"(x[4]), "=f"(x[5]), "=f"(x[6]), "=f"(x[7])
                     : "l"(p));
    }
    static __device__ __forceinline__ void widen8(const uint4 &v, float (&x)[8])   // 16 bytes = 4 elements
    {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
        x[4] = x[0]; x[5] = x[1]; x[6] = x[2]; x[7] = x[3];
    }
    static __device__ __forceinline__ void store8(void *p, const float (&x)[8])
    {
        asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(x[0]), "f"(x[1]), "f"(x[2]),
                     "f"(x[3]), "f"(x[4]), "f"(x[5]), "f"(x[6]), "f"(x[7])
                     : "memory");
    }
};

template <> struct Elem<__half> {
    static constexpr int kBytes = 2;
    static __device__ __forceinline__ void load8(const void *p, float (&x)[8])
    {
        uint4 v;
        asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; i++) {
            __half2 h = *reinterpret_cast<const __half2 *>(&w[i]);
            float2 f = __half22float2(h);
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    }
    static __device__ __forceinline__ void load8_keep(const void *p, float (&x)[8])
    {
        uint4 v;
        asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
        widen8(v, x);
    }
    static __device__ __forceinline__ void widen8(const uint4 &v, float (&x)[8])   // 16 bytes = 8 elements
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; i++) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    }
    static __device__ __forceinline__ void store8(void *p, const float (&x)[8])
    {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; i++) {
            __half2 h = __floats2half2_rn(x[2 * i], x[2 * i + 1]);   // round to nearest even
            w[i] = *reinterpret_cast<uint32_t *>(&h);
        }
        asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
    }
};

template <> struct Elem<__nv_bfloat16> {
    static constexpr int kBytes = 2;
    static __device__ __forceinline__ void load8(const void *p, float (&x)[8])
    {
        uint4 v;
        asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; i++) {
            x[2 * i] = __uint_as_float(w[i] << 16);              // bfloat16 is the top half of binary32
            x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    static __device__ __forceinline__ void load8_keep(const void *p, float (&x)[8])
    {
        uint4 v;
        asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
        widen8(v, x);
    }
    static __device__ __forceinline__ void widen8(const uint4 &v, float (&x)[8])   // 16 bytes = 8 elements
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; i++) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    static __device__ __forceinline__ void store8(void *p, const float (&x)[8])
    {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; i++) {
            __nv_bfloat162 h = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);   // round to nearest even
            w[i] = *reinterpret_cast<uint32_t *>(&h);
        }
        asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
    }
};

// min / max of three operands in one instruction (sm_100); -0.0 orders below +0.0.
__device__ __forceinline__ float fmin3(float a, float b, float c)
{
    float r;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
__device__ __forceinline__ float fmin2(float a, float b)
{
    float r;
    asm("min.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ float fmax2(float a, float b)
{
    float r;
    asm("max.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}

// Host-side description shared by the launchers.
struct Plan {
    uint32_t G, log2G, We, chunks, W;      // group size, its log2, window elements, chunks per thread, groups per window
    uint32_t beta_q8;
    uint32_t m;                            // number of allowed widths
    uint32_t S[kMaxLevels];                // allowed widths, ascending
    uint32_t cost[kMaxLevels];             // S[k+1] - S[k]
    float v[kMaxLevels];                   // importance-per-bit factor of the raise k -> k+1
    uint64_t n_groups, n_windows, capacity, workspace;
};

daf_status make_plan(const daf_params *p, Plan *plan);

// Grid of a persistent kernel on the current device: multiprocessors x resident CTAs per
// multiprocessor for `threads` threads and `dyn_smem` bytes of dynamic shared memory (the kernel's
// limit on dynamic shared memory is raised first when it has to be).  Both are properties of a
// (kernel, device) pair and are remembered per pair; safe to call from several host threads.
cudaError_t persistent_ctas(const void *kernel, int threads, int dyn_smem, int *ctas);

// Activations of the fused producers and consumers (Sec. 3.2.3 of the paper: the statistics are taken where the
// activation is produced, the restored value is used where the gradient is formed).
//   ReLU   y = max(x, +0)            what is compressed: y     gradient: g where restored y > 0
//   ReLU6  y = min(max(x, +0), 6)    what is compressed: y     gradient: g where 0 < restored y < 6
//   GELU   y = x Phi(x) = x/2 (1 + erf(x / sqrt 2))    what is compressed: x (the backward pass needs the input)
//          gradient: g * (Phi(x) + x phi(x)) at the restored x
// The GELU pair is bound by arithmetic, not by memory, so it takes the cheap forms: erf rather than erfc (the far
// negative tail, where x Phi(x) is below 2^-24 |x|, is then rounding noise around 0) and the fast exponential.
enum : int { kActNone = 0, kActRelu = 1, kActRelu6 = 2, kActGelu = 3 };
__device__ __forceinline__ float gelu_f(float x) { return (0.5f * x) * (1.0f + erff(0.70710678118654752f * x)); }
__device__ __forceinline__ float gelu_grad_f(float x)
{
    return 0.5f * (1.0f + erff(0.70710678118654752f * x)) + (x * 0.3989422804014327f) * __expf(-0.5f * (x * x));
}
// x: the chunk as loaded; afterwards x = what is compressed, y = what the producer writes out.
template <int ACT> __device__ __forceinline__ void activate8(float (&x)[8], float (&y)[8])
{
#pragma unroll
    for (int i = 0; i < 8; i++) {
        if (ACT == kActRelu) x[i] = fmaxf(x[i], 0.0f);
        if (ACT == kActRelu6) x[i] = fminf(fmaxf(x[i], 0.0f), 6.0f);
        y[i] = ACT == kActGelu ? gelu_f(x[i]) : x[i];
    }
}

// Eight codes of width B (LSB-first in w0, and w1 for B = 8) back to values: the code is widened with the power-of-two
// offset of Eq. 5 (bits | 0x4B000000 is the float 2^23 + code), then x_hat = fma(code, scale, min).
template <int B> __device__ __forceinline__ void decode8(uint32_t w0, uint32_t w1, float mn, float scale, float (&y)[8])
{
    constexpr uint32_t L = (1u << B) - 1u;
#pragma unroll
    for (int i = 0; i < 8; i++) {
        uint32_t f;
        if (B == 8) {
            // byte i of the pair of words into the low byte of 0x4B0000xx in one permute
            f = __byte_perm(i < 4 ? w0 : w1, 0x4B000000u, 0x7540u | (uint32_t)(i & 3));
        } else {
            f = ((w0 >> (B * i)) & L) | 0x4B000000u;
        }
        const float q = __fsub_rn(__uint_as_float(f), 8388608.0f);   // exact: f is the float 2^23 + code
        y[i] = __fmaf_rn(q, scale, mn);
    }
}

}  // namespace daf
