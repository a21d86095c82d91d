// Shared device helpers of the HiLoRe hot-path kernels (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/hilore.h"

#if defined(__CUDA_ARCH__) && (__CUDA_ARCH__ < 1000)
#error "these kernels are written for sm_100a (B200) only"
#endif

namespace hilore {

constexpr int kCodecThreads = 256;   // 8 warps per CTA in the streaming codec kernels
constexpr int kBlockSumSlots = 4096; // per-CTA shared slots for per-block sums of squares (16 KB)

// ---- 256-bit global accesses (sm_100: one instruction moves 32 bytes per lane) ----
__device__ __forceinline__ void ld_global_256(const void *p, uint32_t (&w)[8])
{
    asm volatile("ld.global.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                 : "l"(p));
}

__device__ __forceinline__ void st_global_256(void *p, const uint32_t (&w)[8])
{
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                 "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                 : "memory");
}

__device__ __forceinline__ uint4 ld_global_128_stream(const void *p)
{
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// ---- packed conversions ----
// Two fp32 -> two E4M3FN codes, round to nearest even, saturating at +-448; `lo` lands in the low byte.
__device__ __forceinline__ uint32_t cvt_e4m3x2(float hi, float lo)
{
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

// Two E4M3FN codes (low 16 bits of `c`) -> two fp16 (exact), packed.
__device__ __forceinline__ uint32_t cvt_e4m3x2_to_f16x2(uint32_t c)
{
    uint32_t r;
    uint16_t h = (uint16_t)c;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(h));
    return r;
}

__device__ __forceinline__ float f16_lo_to_f32(uint32_t h2)
{
    float f;
    uint16_t h = (uint16_t)(h2 & 0xFFFFu);
    asm("cvt.f32.f16 %0, %1;" : "=f"(f) : "h"(h));
    return f;
}

__device__ __forceinline__ float f16_hi_to_f32(uint32_t h2)
{
    float f;
    uint16_t h = (uint16_t)(h2 >> 16);
    asm("cvt.f32.f16 %0, %1;" : "=f"(f) : "h"(h));
    return f;
}

// Two fp32 -> packed bf16x2, round to nearest even; `lo` lands in the low half.
__device__ __forceinline__ uint32_t cvt_bf16x2(float hi, float lo)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// max over the sixteen |bf16| bit patterns held in w[0..7] (as unsigned 16-bit integers, so that
// Inf and NaN patterns (>= 0x7F80) compare above every finite value).
__device__ __forceinline__ uint32_t absmax_bits16(const uint32_t (&w)[8])
{
    const uint32_t M = 0x7FFF7FFFu;
    uint32_t a = __vimax3_u16x2(w[0] & M, w[1] & M, w[2] & M);
    uint32_t b = __vimax3_u16x2(w[3] & M, w[4] & M, w[5] & M);
    uint32_t c = __vimax3_u16x2(w[6] & M, w[7] & M, a);
    uint32_t m = __vmaxu2(b, c);
    return max(m & 0xFFFFu, m >> 16);
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

struct DeviceInfo {
    int sms;
};
// Number of SMs of the current device (queried each call; the library keeps no state).
inline int sm_count()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess)
        return 148;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return 148;
    return sms;
}

} // namespace hilore
