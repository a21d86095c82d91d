// Shared device helpers of the HiLoRe hot-path kernels (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/hilore.h"

#if defined(__CUDA_ARCH__) && (__CUDA_ARCH__ < 1000)
#error "these kernels are written for sm_100a (B200) only"
#endif

namespace hilore {

constexpr int kCodecThreads = 256;   // 8 warps per CTA in the streaming codec kernels
constexpr int kBlockSumSlots = 6144; // per-CTA shared slots for per-block sums of squares (24 KB)

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

__device__ __forceinline__ uint2 ld_global_64_stream(const void *p)
{
    uint2 v;
    asm volatile("ld.global.L1::no_allocate.v2.b32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

__device__ __forceinline__ uint4 ld_global_128_stream(const void *p)
{
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Ask the copy engine to pull `bytes` (a multiple of 16, 16-byte aligned) from HBM into L2, no register or
// shared-memory destination: the later plain loads of this range then hit L2.
__device__ __forceinline__ void prefetch_l2_bulk(const void *p, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

// Ask for the cache line that holds *p to be brought into L2; nothing waits for it.
__device__ __forceinline__ void prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// Programmatic dependent launch: block until the kernels this one depends on have completed and their writes are
// visible (a no-op when the kernel was launched without the attribute); and tell the next kernel of the stream that
// it may start to become resident.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- packed conversions ----
// Two fp32 -> two E4M3FN codes, round to nearest even, saturating at +-448; `lo` lands in the low byte.
__device__ __forceinline__ uint32_t cvt_e4m3x2(float hi, float lo)
{
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

// Four fp32 -> four E4M3FN codes in one word, x0 in the lowest byte.  The two 16-bit halves are joined inside
// the asm block, so no zero-extension of the halves is emitted.
__device__ __forceinline__ uint32_t cvt_e4m3x4(float x0, float x1, float x2, float x3)
{
    uint32_t r;
    asm("{\n\t.reg .b16 lo, hi;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
        "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
        "mov.b32 %0, {lo, hi};\n\t}"
        : "=r"(r)
        : "f"(x0), "f"(x1), "f"(x2), "f"(x3));
    return r;
}

// Four fp32 -> four int8 codes in one word (round to nearest even, saturating), x0 in the lowest byte.
__device__ __forceinline__ uint32_t cvt_s8x4(float x0, float x1, float x2, float x3)
{
    uint32_t hi, r;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(__float2int_rn(x3)), "r"(__float2int_rn(x2)), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(__float2int_rn(x1)), "r"(__float2int_rn(x0)), "r"(hi));
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

// ---- packed fp32 pairs (sm_100: one instruction per two fp32 lanes, each lane rounded as IEEE RN) ----
__device__ __forceinline__ uint64_t f32x2_pack(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}

__device__ __forceinline__ void f32x2_unpack(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}

__device__ __forceinline__ uint64_t f32x2_mul(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ uint64_t f32x2_fma(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

__device__ __forceinline__ uint64_t f32x2_add(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ uint64_t f32x2_sub(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ uint64_t u32x2_pack(uint32_t lo, uint32_t hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

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

// Launch with the programmatic-stream-serialization attribute: the kernel may become resident while the previous
// kernel of the stream drains.  Every kernel launched this way executes griddepcontrol.wait before its first
// access to global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Risk score and H / L / R gating of one unit (Eq. "token-weighted-risk", Eq. "available-recovery-actions"; the
// threshold rule stands in for the paper's allocator): psi = fl32(fl32(kappa E) ebar); desired = L below tau_lo, H
// from tau_hi on, else R (NaN -> R); outside the candidate set of q -> R.  `E` == nullptr: the desired action is
// action_io[u] as given.
struct PlanTail {
    const hilore_unit *units;
    const float *kappa, *ebar;
    float tau_lo, tau_hi;
    const uint8_t *avail;
    uint8_t *action_io;
    float *psi;
    uint8_t *recompute;
    uint64_t *retained_bytes;
};

__device__ __forceinline__ void decide_unit(const PlanTail &p, int u, const float *E)
{
    uint32_t want = p.action_io[u];
    if (E != nullptr) {
        const float v = __fmul_rn(__fmul_rn(p.kappa[u], *E), p.ebar[u]);
        if (p.psi) p.psi[u] = v;
        want = (v < p.tau_lo) ? HILORE_ACT_L : ((v >= p.tau_hi) ? HILORE_ACT_H : HILORE_ACT_R);
    }
    const uint32_t q = p.avail[u];
    const bool ok = (q == HILORE_ACT_H) || (q == HILORE_ACT_L && want != HILORE_ACT_H) || (want == HILORE_ACT_R);
    const uint32_t a = (ok && want <= HILORE_ACT_L) ? want : (uint32_t)HILORE_ACT_R;
    p.action_io[u] = (uint8_t)a;
    if (p.recompute) p.recompute[u] = (a == HILORE_ACT_R);
    if (p.retained_bytes) {
        const uint64_t n = (uint64_t)p.units[u].rows * (uint64_t)p.units[u].cols;
        uint64_t b = 0;
        if (a == HILORE_ACT_H) b = 2 * n;
        else if (a == HILORE_ACT_L) b = n + (p.units[u].fmt == HILORE_FMT_E4M3FN_RAW ? 0 : 4 * (n / HILORE_BLOCK));
        p.retained_bytes[u] = b;
    }
}

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Immutable properties of the devices, looked up once per device and process (no device memory involved).
struct LaunchCache {
    static constexpr int kMaxDevices = 64, kMaxKernels = 64;
    std::mutex mu;
    int sms[kMaxDevices] = {};
    struct Entry {
        const void *kernel;
        int device, per_sm;
    } occ[kMaxKernels] = {};
    int n_occ = 0;
};
inline LaunchCache &launch_cache()
{
    static LaunchCache c;
    return c;
}

inline int current_device()
{
    int dev = 0;
    return cudaGetDevice(&dev) == cudaSuccess ? dev : 0;
}

// Number of SMs of the current device.
inline int sm_count()
{
    const int dev = current_device();
    LaunchCache &c = launch_cache();
    if (dev >= 0 && dev < LaunchCache::kMaxDevices && c.sms[dev] > 0)
        return c.sms[dev];
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return 148;
    if (dev >= 0 && dev < LaunchCache::kMaxDevices) {
        std::lock_guard<std::mutex> lock(c.mu);
        c.sms[dev] = sms;
    }
    return sms;
}

// Resident CTAs per SM of `kernel` at `threads` threads and `smem` bytes of dynamic shared memory.
template <typename K> inline int ctas_per_sm(K kernel, int threads, size_t smem, int fallback)
{
    const int dev = current_device();
    LaunchCache &c = launch_cache();
    const void *key = reinterpret_cast<const void *>(kernel);
    {
        std::lock_guard<std::mutex> lock(c.mu);
        for (int i = 0; i < c.n_occ; ++i)
            if (c.occ[i].kernel == key && c.occ[i].device == dev)
                return c.occ[i].per_sm;
    }
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem) != cudaSuccess || per_sm <= 0)
        return fallback;
    std::lock_guard<std::mutex> lock(c.mu);
    if (c.n_occ < LaunchCache::kMaxKernels)
        c.occ[c.n_occ++] = {key, dev, per_sm};
    return per_sm;
}

} // namespace hilore
