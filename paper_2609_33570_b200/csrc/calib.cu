// Calibration statistics of the L codec: e^L = ||x_hat - x||_2 / (||x||_2 + 1e-8) of one unit
// (Eq. "calibration-metrics" / "app-calibration-error": operands widened to fp32 before the subtraction and
// the norms) and the closed-form susceptibility fit (Eq. "susceptibility").  Used at initialisation on the
// calibration microbatches, not in the per-microbatch hot loop.
#include "common.cuh"
#include "codec.cuh"

namespace hilore {

constexpr int kErrThreads = 256;
constexpr int kErrMaxGrid = 2048; // partial slots in the workspace

__device__ __forceinline__ void err16(const uint32_t (&a)[8], const uint32_t (&b)[8], float &err2, float &x2)
{
    float e = 0.0f, n = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float xl = bf16_lo(a[i]), xh = bf16_hi(a[i]);
        const float dl = bf16_lo(b[i]) - xl, dh = bf16_hi(b[i]) - xh;
        e = fmaf(dl, dl, e);
        e = fmaf(dh, dh, e);
        n = fmaf(xl, xl, n);
        n = fmaf(xh, xh, n);
    }
    err2 = e;
    x2 = n;
}

// Every CTA sums a contiguous share of the 16-element chunks (fp32 per chunk, fp64 across chunks) and leaves
// one pair of partial sums in its own slot: no atomics, the result does not depend on scheduling.
__global__ void __launch_bounds__(kErrThreads) relerr_partial_kernel(const uint16_t *__restrict__ x, const uint16_t *__restrict__ xh,
                                                                     int64_t rows, int64_t cols, int64_t ld, int64_t ldh,
                                                                     double *__restrict__ partial)
{
    const int64_t cpr = cols >> 4, n = rows * cpr;
    const int64_t c0 = (n / gridDim.x) * blockIdx.x + ((n % gridDim.x) * blockIdx.x) / gridDim.x;
    const int64_t c1 = (n / gridDim.x) * (blockIdx.x + 1) + ((n % gridDim.x) * (blockIdx.x + 1)) / gridDim.x;
    double err = 0.0, nrm = 0.0;
    for (int64_t c = c0 + threadIdx.x; c < c1; c += kErrThreads) {
        const int64_t r = c / cpr, cc = c - r * cpr;
        uint32_t a[8], b[8];
        ld_global_256(x + r * ld + cc * 16, a);
        ld_global_256(xh + r * ldh + cc * 16, b);
        float e, m;
        err16(a, b, e, m);
        err += (double)e;
        nrm += (double)m;
    }
    __shared__ double sm[kErrThreads / 32][2];
    err = warp_sum(err);
    nrm = warp_sum(nrm);
    if ((threadIdx.x & 31) == 0) {
        sm[threadIdx.x >> 5][0] = err;
        sm[threadIdx.x >> 5][1] = nrm;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double e = 0.0, m = 0.0;
        for (int w = 0; w < kErrThreads / 32; ++w) {
            e += sm[w][0];
            m += sm[w][1];
        }
        partial[2 * blockIdx.x] = e;
        partial[2 * blockIdx.x + 1] = m;
    }
}

__global__ void __launch_bounds__(32) relerr_final_kernel(const double *partial, int nparts, double *e_out, double *norms2)
{
    double e = 0.0, m = 0.0;
    for (int i = threadIdx.x; i < nparts; i += 32) {
        e += partial[2 * i];
        m += partial[2 * i + 1];
    }
    e = warp_sum(e);
    m = warp_sum(m);
    if (threadIdx.x == 0) {
        *e_out = sqrt(e) / (sqrt(m) + 1e-8);
        if (norms2) {
            norms2[0] = e;
            norms2[1] = m;
        }
    }
}

// e^L of format FMT on x without materialising codes or x_hat: each thread encodes its two 16-element chunks with
// the compress kernel's own routine, decodes them with the recover kernel's own routine (so x_hat is bit for
// bit what hilore_recover would write) and accumulates both norms.  x is read once: 2 B per element.
template <int FMT>
__global__ void __launch_bounds__(kCodecThreads) codec_relerr_kernel(const uint16_t *__restrict__ x, int64_t rows, int64_t cols,
                                                                    int64_t ld, double *__restrict__ partial)
{
    const int tid = threadIdx.x, lane = tid & 31;
    const int64_t cpr = cols >> 4, n = rows * cpr; // chunks; a multiple of 4 (cols % 64 == 0)
    const int64_t steps = (n + 2 * kCodecThreads - 1) / (2 * kCodecThreads);
    const int64_t s_begin = (steps / gridDim.x) * blockIdx.x + ((steps % gridDim.x) * blockIdx.x) / gridDim.x;
    const int64_t s_end = (steps / gridDim.x) * (blockIdx.x + 1) + ((steps % gridDim.x) * (blockIdx.x + 1)) / gridDim.x;
    double err = 0.0, nrm = 0.0;
    for (int64_t st = s_begin; st < s_end; ++st) { // the trip count is uniform over the CTA (shuffles inside)
        const int64_t ca = st * 2 * kCodecThreads + tid, cb = ca + kCodecThreads;
        uint32_t wa[8], wb[8];
        zero8(wa); // a chunk past the end reads as zeros: code 0, x_hat 0, no contribution
        zero8(wb);
        if (ca < n) {
            const int64_t r = ca / cpr;
            ld_global_256(x + r * ld + (ca - r * cpr) * 16, wa);
        }
        if (cb < n) {
            const int64_t r = cb / cpr;
            ld_global_256(x + r * ld + (cb - r * cpr) * 16, wb);
        }
        uint4 qa, qb;
        float s, unused;
        bool careful_unused;
        process_pair<FMT, true, false>(wa, wb, lane, qa, qb, s, unused, careful_unused);
        float sa = 1.0f, sb = 1.0f;
        if (FMT != HILORE_FMT_E4M3FN_RAW) { // the scale of chunk a's block sits in lane 0 of the quad, of chunk b's in lane 2
            sa = __shfl_sync(0xFFFFFFFFu, s, (lane & 28));
            sb = __shfl_sync(0xFFFFFFFFu, s, (lane & 28) | 2);
        }
        uint32_t oa[8], ob[8];
        decode16<FMT>(qa, sa, oa);
        decode16<FMT>(qb, sb, ob);
        float e0, m0, e1, m1;
        err16(wa, oa, e0, m0);
        err16(wb, ob, e1, m1);
        err += (double)e0 + (double)e1;
        nrm += (double)m0 + (double)m1;
    }
    __shared__ double sm[kCodecThreads / 32][2];
    err = warp_sum(err);
    nrm = warp_sum(nrm);
    if (lane == 0) {
        sm[tid >> 5][0] = err;
        sm[tid >> 5][1] = nrm;
    }
    __syncthreads();
    if (tid == 0) {
        double e = 0.0, m = 0.0;
        for (int w = 0; w < kCodecThreads / 32; ++w) {
            e += sm[w][0];
            m += sm[w][1];
        }
        partial[2 * blockIdx.x] = e;
        partial[2 * blockIdx.x + 1] = m;
    }
}

} // namespace hilore

using namespace hilore;

extern "C" int hilore_codec_relative_error(const void *x, int64_t rows, int64_t cols, int64_t ld, int32_t fmt, int32_t block,
                                           double *e_out, double *norms2, void *workspace, size_t workspace_bytes,
                                           void *stream)
{
    if (rows < 0 || cols <= 0 || !e_out || !workspace || (rows > 0 && !x))
        return HILORE_INVALID_ARG;
    if (fmt != HILORE_FMT_E4M3FN_RAW && fmt != HILORE_FMT_E4M3FN_BLK && fmt != HILORE_FMT_INT8_BLK)
        return HILORE_INVALID_ARG;
    if (cols % 64 != 0 || ld < cols || (fmt == HILORE_FMT_E4M3FN_RAW ? block != 0 : block != 64))
        return HILORE_SHAPE;
    if (ld % 16 != 0 || !aligned(x, 32) || !aligned(e_out, 8) || !aligned(norms2, 8) || !aligned(workspace, 16))
        return HILORE_ALIGN;
    if (workspace_bytes < hilore_relative_error_workspace_bytes())
        return HILORE_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t steps = (rows * (cols / 16) + 2 * kCodecThreads - 1) / (2 * kCodecThreads);
    int64_t grid = (int64_t)sm_count() * 4;
    if (grid > kErrMaxGrid) grid = kErrMaxGrid;
    if (grid > steps) grid = steps;
    if (grid < 1) grid = 1;
    double *partial = static_cast<double *>(workspace);
    const uint16_t *xp = static_cast<const uint16_t *>(x);
    if (fmt == HILORE_FMT_E4M3FN_RAW)
        codec_relerr_kernel<HILORE_FMT_E4M3FN_RAW><<<(unsigned)grid, kCodecThreads, 0, st>>>(xp, rows, cols, ld, partial);
    else if (fmt == HILORE_FMT_E4M3FN_BLK)
        codec_relerr_kernel<HILORE_FMT_E4M3FN_BLK><<<(unsigned)grid, kCodecThreads, 0, st>>>(xp, rows, cols, ld, partial);
    else
        codec_relerr_kernel<HILORE_FMT_INT8_BLK><<<(unsigned)grid, kCodecThreads, 0, st>>>(xp, rows, cols, ld, partial);
    relerr_final_kernel<<<1, 32, 0, st>>>(partial, (int)grid, e_out, norms2);
    return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
}

extern "C" size_t hilore_relative_error_workspace_bytes(void) { return (size_t)kErrMaxGrid * 2 * sizeof(double); }

extern "C" int hilore_relative_error(const void *x, const void *xhat, int64_t rows, int64_t cols, int64_t ld, int64_t ld_hat,
                                     double *e_out, double *norms2, void *workspace, size_t workspace_bytes, void *stream)
{
    if (rows < 0 || cols <= 0 || !e_out || !workspace)
        return HILORE_INVALID_ARG;
    if (rows > 0 && (!x || !xhat))
        return HILORE_INVALID_ARG;
    if (cols % 16 != 0 || ld < cols || ld_hat < cols)
        return HILORE_SHAPE;
    if (ld % 16 != 0 || ld_hat % 16 != 0 || !aligned(x, 32) || !aligned(xhat, 32) || !aligned(e_out, 8) || !aligned(norms2, 8) ||
        !aligned(workspace, 16))
        return HILORE_ALIGN;
    if (workspace_bytes < hilore_relative_error_workspace_bytes())
        return HILORE_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t chunks = rows * (cols / 16);
    int64_t grid = (int64_t)sm_count() * ctas_per_sm(relerr_partial_kernel, kErrThreads, 0, 4);
    if (grid > kErrMaxGrid) grid = kErrMaxGrid;
    if (grid > (chunks + kErrThreads - 1) / kErrThreads) grid = (chunks + kErrThreads - 1) / kErrThreads;
    if (grid < 1) grid = 1;
    double *partial = static_cast<double *>(workspace);
    relerr_partial_kernel<<<(unsigned)grid, kErrThreads, 0, st>>>(static_cast<const uint16_t *>(x), static_cast<const uint16_t *>(xhat),
                                                                 rows, cols, ld, ld_hat, partial);
    relerr_final_kernel<<<1, 32, 0, st>>>(partial, (int)grid, e_out, norms2);
    return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
}

// kappa = argmin_{kappa >= 0} sum (y - kappa x)^2 = max(0, sum x y / sum x^2); host arrays, host arithmetic
// (a handful of calibration pairs per unit class).
extern "C" double hilore_fit_kappa(const double *x, const double *y, int64_t n)
{
    double sxy = 0.0, sxx = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        sxy += x[i] * y[i];
        sxx += x[i] * x[i];
    }
    if (!(sxx > 0.0))
        return 0.0;
    const double k = sxy / sxx;
    return k > 0.0 ? k : 0.0;
}
