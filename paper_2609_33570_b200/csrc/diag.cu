// Structural-sparsity diagnostics of the update coefficients (diagnostic paragraph "Structural sparsity in
// diagnostic replays", Eq. "diagnostic-clipping"): exclusive cause counts of zero policy-gradient slots and the
// share of sum |omega| carried by the top decile of slots.  The k-th largest |omega| is found exactly by a
// three-pass radix select on the fp32 bit patterns (integer histograms: deterministic); the sums are per-CTA
// fp64 partials in fixed workspace slots, added in a fixed order.
#include "common.cuh"

namespace hilore {

constexpr int kDiagThreads = 256;
constexpr int kDiagMaxGrid = 1184;
constexpr int kBins = 2048;

struct DiagState {
    unsigned long long hist[3][kBins];
    unsigned long long counts[5];      // padding, zero advantage, clipped, zero omega, slots
    unsigned long long k, remaining, greater;
    uint32_t prefix;                   // bits of the k-th largest |omega| found so far (high bits first)
    double partial[2 * kDiagMaxGrid];  // per CTA: sum |omega|, sum of |omega| above the threshold
};

struct DiagArgs {
    const float *adv, *ratio, *omega;
    const uint8_t *mask;
    int64_t n_rows, T, n;
    float clip_eps;
    DiagState *st;
};

// |omega| bit patterns of four consecutive slots starting at k (k % 4 == 0 when `vec`), padding reads as zero.
__device__ __forceinline__ void abs_bits4(const DiagArgs &a, int64_t k, bool vec, uint32_t (&b)[4], int &cnt)
{
    if (vec && k + 4 <= a.n) {
        const uint4 w = ld_global_128_stream(a.omega + k);
        const uint32_t m = *reinterpret_cast<const uint32_t *>(a.mask + k);
        b[0] = (m & 0xFFu) ? (w.x & 0x7FFFFFFFu) : 0u;
        b[1] = (m & 0xFF00u) ? (w.y & 0x7FFFFFFFu) : 0u;
        b[2] = (m & 0xFF0000u) ? (w.z & 0x7FFFFFFFu) : 0u;
        b[3] = (m & 0xFF000000u) ? (w.w & 0x7FFFFFFFu) : 0u;
        cnt = 4;
    } else {
        cnt = (int)((a.n - k) < 4 ? (a.n - k) : 4);
        for (int j = 0; j < 4; ++j)
            b[j] = (j < cnt && a.mask[k + j]) ? (__float_as_uint(a.omega[k + j]) & 0x7FFFFFFFu) : 0u;
    }
}

// One shared-memory increment per distinct bin among the lanes of a warp that have a value (`active`); every lane of
// the warp calls this.  (Plain atomics measure 10 % slower on B200 for the top digits of |omega|, which take a dozen
// values per warp; electing the bins one by one with a shuffle and a ballot each, twice slower.)
__device__ __forceinline__ void hist_add(unsigned int *sh, uint32_t bin, bool active)
{
    const unsigned peers = __match_any_sync(0xFFFFFFFFu, active ? bin : 0xFFFFFFFFu);
    if (active && (int)(__ffs(peers) - 1) == (int)(threadIdx.x & 31))
        atomicAdd(&sh[bin], (unsigned)__popc(peers));
}

__device__ __forceinline__ bool vec_ok(const DiagArgs &a)
{
    return ((reinterpret_cast<uintptr_t>(a.omega) | reinterpret_cast<uintptr_t>(a.ratio)) % 16 == 0) &&
           (reinterpret_cast<uintptr_t>(a.mask) % 4 == 0);
}

// pass 0: cause counts, sum |omega|, histogram of bits 30..20
__global__ void __launch_bounds__(kDiagThreads) diag_count_kernel(const __grid_constant__ DiagArgs a)
{
    __shared__ unsigned int sh[kBins];
    __shared__ unsigned long long sc[4];
    __shared__ double ssum[kDiagThreads / 32];
    for (int i = threadIdx.x; i < kBins; i += kDiagThreads) sh[i] = 0;
    if (threadIdx.x < 4) sc[threadIdx.x] = 0;
    __syncthreads();
    const float hi = 1.0f + a.clip_eps, lo = 1.0f - a.clip_eps;
    const bool vec = vec_ok(a);
    unsigned int c0 = 0, c1 = 0, c2 = 0, c3 = 0;
    double sum = 0.0;
    const int64_t quads = (a.n + 3) / 4, stride = (int64_t)gridDim.x * kDiagThreads;
    // whole warps stay in the loop together (hist_add is a warp-wide call); a lane beyond the end has no value
    for (int64_t q0 = (int64_t)blockIdx.x * kDiagThreads + (threadIdx.x & ~31); q0 < quads; q0 += stride) {
        const int64_t q = q0 + (threadIdx.x & 31);
        const bool in = q < quads;
        const int64_t k = in ? 4 * q : 0;
        uint32_t b[4] = {0, 0, 0, 0};
        int cnt = 0;
        float r[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        uint32_t mword = 0; // the four mask bytes, one per slot
        if (in) {
            abs_bits4(a, k, vec, b, cnt);
            if (vec && cnt == 4) {
                const uint4 w = ld_global_128_stream(a.ratio + k);
                r[0] = __uint_as_float(w.x), r[1] = __uint_as_float(w.y), r[2] = __uint_as_float(w.z), r[3] = __uint_as_float(w.w);
                mword = *reinterpret_cast<const uint32_t *>(a.mask + k);
            } else {
                for (int j = 0; j < cnt; ++j) {
                    r[j] = a.ratio[k + j];
                    mword |= (uint32_t)(a.mask[k + j] != 0) << (8 * j);
                }
            }
        }
        int64_t row = k / a.T, col = k - row * a.T;
        float A = in ? a.adv[row] : 0.0f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const bool act = j < cnt;
            if (act) {
                const bool m = ((mword >> (8 * j)) & 0xFFu) != 0;
                if (!m) ++c0;
                else if (A == 0.0f) ++c1;
                else if ((A > 0.0f && r[j] > hi) || (A < 0.0f && r[j] < lo)) ++c2;
                if (b[j] == 0) ++c3;
                sum += (double)__uint_as_float(b[j]);
                if (++col == a.T && k + j + 1 < a.n) {
                    col = 0;
                    A = a.adv[++row];
                }
            }
            hist_add(sh, b[j] >> 20, act);
        }
    }
    atomicAdd(&sc[0], (unsigned long long)c0);
    atomicAdd(&sc[1], (unsigned long long)c1);
    atomicAdd(&sc[2], (unsigned long long)c2);
    atomicAdd(&sc[3], (unsigned long long)c3);
    sum = warp_sum(sum);
    if ((threadIdx.x & 31) == 0) ssum[threadIdx.x >> 5] = sum;
    __syncthreads();
    for (int i = threadIdx.x; i < kBins; i += kDiagThreads)
        if (sh[i]) atomicAdd(&a.st->hist[0][i], (unsigned long long)sh[i]);
    if (threadIdx.x < 4 && sc[threadIdx.x]) atomicAdd(&a.st->counts[threadIdx.x], sc[threadIdx.x]);
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < kDiagThreads / 32; ++w) t += ssum[w];
        a.st->partial[2 * blockIdx.x] = t;
    }
}

// From the histogram of the current digit, pick the bin that holds the k-th largest value: the largest bin b with
// (number of values in bins above b) < remaining.  One CTA of 1024 threads, two bins each, suffix sums by scan.
__global__ void __launch_bounds__(1024) diag_select_kernel(DiagState *st, int pass, int64_t n)
{
    __shared__ unsigned long long above[kBins + 1];   // above[b] = count in bins >= b
    __shared__ unsigned long long wsum[32];
    const int t = threadIdx.x;
    // reversed order: position p holds bin kBins - 1 - p, so an inclusive prefix scan gives counts in bins >= b
    const unsigned long long v0 = st->hist[pass][kBins - 1 - 2 * t], v1 = st->hist[pass][kBins - 2 - 2 * t];
    unsigned long long x = v0 + v1;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, x, o);
        if ((t & 31) >= o) x += y;
    }
    if ((t & 31) == 31) wsum[t >> 5] = x;
    __syncthreads();
    if (t < 32) {
        unsigned long long w = wsum[t];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, w, o);
            if (t >= o) w += y;
        }
        wsum[t] = w;
    }
    __syncthreads();
    const unsigned long long incl = x + ((t >> 5) ? wsum[(t >> 5) - 1] : 0ull);
    above[kBins - 1 - 2 * t] = incl - v1;
    above[kBins - 2 - 2 * t] = incl;
    if (t == 0) above[kBins] = 0;
    __syncthreads();
    const unsigned long long k = (unsigned long long)((n + 9) / 10); // ceil(0.1 n)
    const unsigned long long rem = pass == 0 ? k : st->remaining;
    __syncthreads();
    for (int b = 2 * t; b < 2 * t + 2; ++b) {
        // bin b holds the k-th largest when above[b + 1] < rem <= above[b] (no bin when the record is empty)
        if (above[b + 1] < rem && rem <= above[b]) {
            st->remaining = rem - above[b + 1];
            st->greater = (pass == 0 ? 0ull : st->greater) + above[b + 1];
            st->prefix = (pass == 0 ? 0u : st->prefix) | (uint32_t)b << (pass == 0 ? 20 : (pass == 1 ? 9 : 0));
            if (pass == 0) {
                st->counts[4] = (unsigned long long)n;
                st->k = k;
            }
        }
    }
}

// passes 1, 2: histogram of the next digit among the values that share the prefix found so far
__global__ void __launch_bounds__(kDiagThreads) diag_hist_kernel(const __grid_constant__ DiagArgs a, int pass)
{
    __shared__ unsigned int sh[kBins];
    for (int i = threadIdx.x; i < kBins; i += kDiagThreads) sh[i] = 0;
    __syncthreads();
    const uint32_t prefix = a.st->prefix;
    const bool vec = vec_ok(a);
    const int64_t quads = (a.n + 3) / 4, stride = (int64_t)gridDim.x * kDiagThreads;
    for (int64_t q = (int64_t)blockIdx.x * kDiagThreads + threadIdx.x; q < quads; q += stride) {
        uint32_t b[4];
        int cnt;
        abs_bits4(a, 4 * q, vec, b, cnt);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (j < cnt) {
                if (pass == 1) {
                    if ((b[j] >> 20) == (prefix >> 20)) atomicAdd(&sh[(b[j] >> 9) & 0x7FFu], 1u);
                } else {
                    if ((b[j] >> 9) == (prefix >> 9)) atomicAdd(&sh[b[j] & 0x1FFu], 1u);
                }
            }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kBins; i += kDiagThreads)
        if (sh[i]) atomicAdd(&a.st->hist[pass][i], (unsigned long long)sh[i]);
}

// sum of the values strictly above the k-th largest
__global__ void __launch_bounds__(kDiagThreads) diag_topsum_kernel(const __grid_constant__ DiagArgs a)
{
    __shared__ double ssum[kDiagThreads / 32];
    const uint32_t thr = a.st->prefix;
    const bool vec = vec_ok(a);
    double sum = 0.0;
    const int64_t quads = (a.n + 3) / 4, stride = (int64_t)gridDim.x * kDiagThreads;
    for (int64_t q = (int64_t)blockIdx.x * kDiagThreads + threadIdx.x; q < quads; q += stride) {
        uint32_t b[4];
        int cnt;
        abs_bits4(a, 4 * q, vec, b, cnt);
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (j < cnt && b[j] > thr) sum += (double)__uint_as_float(b[j]);
    }
    sum = warp_sum(sum);
    if ((threadIdx.x & 31) == 0) ssum[threadIdx.x >> 5] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < kDiagThreads / 32; ++w) t += ssum[w];
        a.st->partial[2 * blockIdx.x + 1] = t;
    }
}

__global__ void __launch_bounds__(32) diag_final_kernel(const DiagState *st, int nparts, int64_t *counts, double *top_share,
                                                        double *sum_abs)
{
    double tot = 0.0, top = 0.0;
    for (int i = threadIdx.x; i < nparts; i += 32) {
        tot += st->partial[2 * i];
        top += st->partial[2 * i + 1];
    }
    tot = warp_sum(tot);
    top = warp_sum(top);
    if (threadIdx.x == 0) {
        for (int c = 0; c < 5; ++c) counts[c] = (int64_t)st->counts[c];
        // the slots above the threshold, plus as many copies of the threshold value as the decile still needs
        top += (double)(st->k - st->greater) * (double)__uint_as_float(st->prefix);
        if (top_share) *top_share = tot > 0.0 ? top / tot : 0.0;
        if (sum_abs) *sum_abs = tot;
    }
}

} // namespace hilore

using namespace hilore;

extern "C" size_t hilore_omega_diagnostics_workspace_bytes(void) { return sizeof(DiagState); }

extern "C" int hilore_omega_diagnostics(const float *adv, const float *ratio, const uint8_t *mask, const float *omega,
                                        int64_t n_rows, int64_t T, float clip_eps, int64_t *counts, double *top_share,
                                        double *sum_abs, void *workspace, size_t workspace_bytes, void *stream)
{
    if (n_rows < 0 || T < 0 || !counts || !workspace)
        return HILORE_INVALID_ARG;
    const int64_t n = n_rows * T;
    if (n > 0 && (!adv || !ratio || !mask || !omega))
        return HILORE_INVALID_ARG;
    if (!aligned(workspace, 16) || !aligned(counts, 8) || !aligned(top_share, 8) || !aligned(sum_abs, 8) || !aligned(adv, 4) ||
        !aligned(ratio, 4) || !aligned(omega, 4))
        return HILORE_ALIGN;
    if (workspace_bytes < sizeof(DiagState))
        return HILORE_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DiagState *ds = static_cast<DiagState *>(workspace);
    if (cudaMemsetAsync(ds, 0, sizeof(DiagState), st) != cudaSuccess)
        return HILORE_CUDA;
    DiagArgs a{adv, ratio, omega, mask, n_rows, T, n, clip_eps, ds};
    int64_t grid = (int64_t)sm_count() * 8;
    if (grid > kDiagMaxGrid) grid = kDiagMaxGrid;
    if (grid > (n + kDiagThreads - 1) / kDiagThreads) grid = (n + kDiagThreads - 1) / kDiagThreads;
    if (grid < 1) grid = 1;
    diag_count_kernel<<<(unsigned)grid, kDiagThreads, 0, st>>>(a);
    diag_select_kernel<<<1, 1024, 0, st>>>(ds, 0, n);
    diag_hist_kernel<<<(unsigned)grid, kDiagThreads, 0, st>>>(a, 1);
    diag_select_kernel<<<1, 1024, 0, st>>>(ds, 1, n);
    diag_hist_kernel<<<(unsigned)grid, kDiagThreads, 0, st>>>(a, 2);
    diag_select_kernel<<<1, 1024, 0, st>>>(ds, 2, n);
    diag_topsum_kernel<<<(unsigned)grid, kDiagThreads, 0, st>>>(a);
    diag_final_kernel<<<1, 32, 0, st>>>(ds, (int)grid, counts, top_share, sum_abs);
    return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
}
