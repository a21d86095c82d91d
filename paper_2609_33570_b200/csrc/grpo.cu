// GRPO loss coefficients and update exposure: hilore_mask_count, hilore_grpo_coeffs,
// hilore_unit_exposure.  Paper: Eq. "grpo-objective", Eq. "update-coefficient", the K3 derivative in
// the proof of Prop. 1, Eq. "activation-token-weights" and Eq. "mlp-weighted-exposure".
#include "common.cuh"

#include <cooperative_groups.h>

#include <cstdlib>

namespace hilore {

// ------------------------------------------------------------------ N = sum of the update mask
__global__ void __launch_bounds__(256) mask_count_kernel(const uint8_t *mask, int64_t n, unsigned long long *count)
{
    // vector part: 16 bytes per step when the base is 16-byte aligned; the rest byte by byte
    const bool vec = (reinterpret_cast<uintptr_t>(mask) & 15) == 0;
    const int64_t nvec = vec ? (n >> 4) : 0;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x, gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned int local = 0;
    const uint4 *m4 = reinterpret_cast<const uint4 *>(mask);
    for (int64_t i = gid; i < nvec; i += stride) {
        const uint4 v = ld_global_128_stream(m4 + i);
        local += __popc(__vcmpne4(v.x, 0) & 0x01010101u) + __popc(__vcmpne4(v.y, 0) & 0x01010101u) +
                 __popc(__vcmpne4(v.z, 0) & 0x01010101u) + __popc(__vcmpne4(v.w, 0) & 0x01010101u);
    }
    for (int64_t i = (nvec << 4) + gid; i < n; i += stride)
        local += mask[i] != 0;
    __shared__ unsigned int sm[8];
    unsigned int w = local;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
        w += __shfl_xor_sync(0xFFFFFFFFu, w, o);
    if ((threadIdx.x & 31) == 0)
        sm[threadIdx.x >> 5] = w;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long t = 0;
        for (int i = 0; i < 8; ++i)
            t += sm[i];
        if (t)
            atomicAdd(count, t); // integer addition: the total does not depend on the order
    }
}

// ------------------------------------------------------------------ coefficients
struct CoeffArgs {
    const float *rewards;
    int64_t n_resp_total;
    int G;
    int64_t resp_offset, n_rows, T;
    const float *logp_new, *logp_old, *logp_ref;
    const uint8_t *mask;
    int64_t N_norm;
    const long long *N_norm_dev;
    float clip_eps, beta, adv_eps;
    float *adv_out, *omega, *ratio;
    uint8_t *clip_mask;
    int tiles_per_row;
};

constexpr int kCoeffThreads = 128;
constexpr int kCoeffVec = 2;                                  // float4 groups per thread
constexpr int kCoeffTile = kCoeffThreads * kCoeffVec * 4;     // 1024 slots of one response per CTA (generic kernel)

// Mean and population standard deviation of the G rewards of one prompt group, in fp64 (one warp; every lane
// returns the same values).  One pass over the rewards shifted by the group's first one, d_j = R_j - R_0 (exact
// in fp64): mean = R_0 + S1 / G, variance = (S2 - S1^2 / G) / G with S1 = sum d_j, S2 = sum d_j^2.  Because
// d_0 = 0 the subtraction loses at most a factor G of the 2^-53 relative precision; and all rewards are the same
// number exactly when S2 == 0, which is the test for an equal-reward group.
struct GroupStats {
    double r0, mu, sigma; // mu is the mean of the shifted rewards
    bool equal;
};

__device__ __forceinline__ GroupStats group_stats(const float *R, int G, int lane)
{
    GroupStats g;
    g.r0 = (double)__ldg(R);
    double s1 = 0.0, s2 = 0.0;
    for (int j = lane; j < G; j += 32) {
        const double d = (double)__ldg(R + j) - g.r0;
        s1 += d;
        s2 = fma(d, d, s2);
    }
    s1 = warp_sum(s1);
    s2 = warp_sum(s2);
    g.equal = s2 == 0.0;
    g.mu = 0.0;
    g.sigma = 0.0;
    if (g.equal)
        return g;
    g.mu = s1 / (double)G;
    g.sigma = sqrt(fmax((s2 - s1 * g.mu) / (double)G, 0.0));
    return g;
}

// Advantage of a response with reward `r`: exactly zero in an equal-reward group, whatever the rounding of the mean.
__device__ __forceinline__ float advantage_of(const GroupStats &g, float r, float adv_eps)
{
    return g.equal ? 0.0f : (float)((((double)r - g.r0) - g.mu) / (g.sigma + (double)adv_eps));
}

// Advantage of response `resp`, from the G rewards of its prompt group (one warp).
__device__ __forceinline__ float group_advantage(const float *rewards, int64_t resp, int G, float adv_eps, int lane)
{
    const GroupStats g = group_stats(rewards + (resp / G) * G, G, lane);
    return advantage_of(g, __ldg(rewards + resp), adv_eps);
}

constexpr float kLog2e = 1.4426950408889634f;

// exp(d) for the importance ratio: one multiplication and one ex2.approx (relative error |d| * 2^-24 + 2^-22:
// 3e-7 for the |d| < 1 of an actor update, below 6e-6 over the whole range where the result is a normal number).
__device__ __forceinline__ float ex2_approx(float x)
{
    float r;
    asm("ex2.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float exp_ratio(float d) { return ex2_approx(__fmul_rn(d, kLog2e)); }

// exp(d) - 1 for the K3 term.  |d| <= 0.25 (an actor a few updates away from its reference): the Taylor series to
// degree 6 by FMAs (the first dropped term is d^6 / 5040 of the result: 5e-8), no cancellation; beyond that
// exp_ratio(d) - 1, whose relative error 2^-22 e^d / |e^d - 1| stays below 9e-7 there.
constexpr float kK3Switch = 0.25f;
__device__ __forceinline__ float expm1_k3(float d)
{
    if (fabsf(d) > kK3Switch)
        return exp_ratio(d) - 1.0f;
    float p = 1.3888889e-3f;        // 1/6!
    p = fmaf(p, d, 8.3333333e-3f);  // 1/5!
    p = fmaf(p, d, 4.1666667e-2f);  // 1/4!
    p = fmaf(p, d, 1.6666667e-1f);  // 1/3!
    p = fmaf(p, d, 0.5f);           // 1/2!
    return fmaf(__fmul_rn(p, d), d, d);
}
// The same polynomial for two values at once (each lane rounded like the scalar form, so the bits agree).
__device__ __forceinline__ uint64_t expm1_k3_poly_x2(uint64_t d)
{
    uint64_t p = f32x2_pack(1.3888889e-3f, 1.3888889e-3f);
    p = f32x2_fma(p, d, f32x2_pack(8.3333333e-3f, 8.3333333e-3f));
    p = f32x2_fma(p, d, f32x2_pack(4.1666667e-2f, 4.1666667e-2f));
    p = f32x2_fma(p, d, f32x2_pack(1.6666667e-1f, 1.6666667e-1f));
    p = f32x2_fma(p, d, f32x2_pack(0.5f, 0.5f));
    return f32x2_fma(f32x2_mul(p, d), d, d);
}

// One coefficient, the defining sequence of operations (every kernel of this file produces these bits):
//   r = exp_ratio(s - o);  chi = A >= 0 ? r <= hi : r >= lo;  policy = chi ? coef * r : 0   (coef = -A / N)
//   omega = m ? fma(-beta / N, expm1_k3(s_ref - s), policy) : 0                              (K3 term if beta != 0)
// VAR selects the score variants of the component ablations: 0 = the coefficient omega itself; 1 = chi_t r_t
// replaced by 1 in the policy contribution; 2 = the advantage-only signal m_t A.
template <int VAR = 0>
__device__ __forceinline__ float omega_scalar(float s, float o, float rf, bool m, bool kl_on, float A, float coef, float nkl,
                                              float hi, float lo, float &r, bool &c)
{
    r = exp_ratio(s - o);
    c = (A >= 0.0f) ? (r <= hi) : (r >= lo);
    float v = VAR == 2 ? A : (VAR == 1 ? coef : (c ? __fmul_rn(coef, r) : 0.0f));
    if (kl_on && VAR != 2)
        v = fmaf(nkl, expm1_k3(rf - s), v);
    return m ? v : 0.0f;
}

// Generic kernel: one CTA of 128 threads per 1024 slots of one response, 128-bit accesses (T % 4 == 0, 16-byte
// alignment).  Takes the shapes the warp-tile kernel below does not.
template <bool KL, bool EXTRA, int VAR>
__global__ void __launch_bounds__(kCoeffThreads) grpo_coeffs_kernel(const __grid_constant__ CoeffArgs a)
{
    // 32-bit index arithmetic (the host checks that the grid fits)
    const uint32_t tpr = (uint32_t)a.tiles_per_row;
    const uint32_t row32 = tpr == 1 ? blockIdx.x : blockIdx.x / tpr;
    const int tt = (int)(blockIdx.x - row32 * tpr);
    const int64_t row = row32;
    const int tid = threadIdx.x, lane = tid & 31;
    const int64_t rowbase = row * a.T;
    grid_dependency_wait();

    // issue the token loads first; the group statistics below overlap with them
    float4 sn[kCoeffVec], so[kCoeffVec], sr[kCoeffVec];
    uint32_t mk[kCoeffVec];
    int64_t t0[kCoeffVec];
#pragma unroll
    for (int j = 0; j < kCoeffVec; ++j) {
        t0[j] = (int64_t)tt * kCoeffTile + (int64_t)(j * kCoeffThreads + tid) * 4;
        if (t0[j] < a.T) {
            const int64_t k = rowbase + t0[j];
            sn[j] = __ldcs(reinterpret_cast<const float4 *>(a.logp_new + k));
            so[j] = __ldcs(reinterpret_cast<const float4 *>(a.logp_old + k));
            if (KL) sr[j] = __ldcs(reinterpret_cast<const float4 *>(a.logp_ref + k));
            mk[j] = __ldcs(reinterpret_cast<const unsigned int *>(a.mask + k));
        }
    }
    grid_dependency_release();

    __shared__ float s_adv, s_coef, s_nkl;
    if (tid < 32) { // the per-response scalars, fp64 arithmetic once per CTA
        const float A = group_advantage(a.rewards, a.resp_offset + row, a.G, a.adv_eps, lane);
        if (lane == 0) {
            const long long N = a.N_norm_dev ? *a.N_norm_dev : (long long)a.N_norm;
            const double invN = N > 0 ? 1.0 / (double)N : 0.0;
            s_adv = A;
            s_coef = (float)(-(double)A * invN); // omega = coef * r on the unclipped branch
            s_nkl = -(float)((double)a.beta * invN);
            if (tt == 0 && a.adv_out)
                a.adv_out[row] = A;
        }
    }
    __syncthreads();
    const float A = s_adv, coef = s_coef, nkl = s_nkl;
    const float hi = 1.0f + a.clip_eps, lo = 1.0f - a.clip_eps;

#pragma unroll
    for (int j = 0; j < kCoeffVec; ++j) {
        if (t0[j] >= a.T)
            continue;
        const float s[4] = {sn[j].x, sn[j].y, sn[j].z, sn[j].w};
        const float o[4] = {so[j].x, so[j].y, so[j].z, so[j].w};
        const float rf[4] = {sr[j].x, sr[j].y, sr[j].z, sr[j].w};
        float w[4], r[4];
        uint32_t chi = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const bool m = ((mk[j] >> (8 * i)) & 0xFFu) != 0;
            bool c;
            w[i] = omega_scalar<VAR>(s[i], o[i], KL ? rf[i] : 0.0f, m, KL, A, coef, nkl, hi, lo, r[i], c);
            chi |= (uint32_t)c << (8 * i);
        }
        const int64_t k = rowbase + t0[j];
        __stcs(reinterpret_cast<float4 *>(a.omega + k), make_float4(w[0], w[1], w[2], w[3]));
        if (EXTRA) {
            if (a.ratio) __stcs(reinterpret_cast<float4 *>(a.ratio + k), make_float4(r[0], r[1], r[2], r[3]));
            if (a.clip_mask) __stcs(reinterpret_cast<unsigned int *>(a.clip_mask + k), chi);
        }
    }
}

// ---- the fast path: one WARP per tile of kWarpIters * 256 slots of one response, no CTA barrier
// Tile and register budget, measured on B200 at 2^24 slots (13 B/slot; 17 with the K3 term): two pieces of 256
// slots per warp and at most 80 registers (six CTAs per SM) give 34.0 / 44.3 us (6.4 TB/s both); one piece 39.7 /
// 48.4, four pieces 34.3 / 48.1, the unconstrained 87-register build 36.1 / 47.4.
#ifndef HILORE_COEFF_IT
#define HILORE_COEFF_IT 2
#endif
#ifndef HILORE_COEFF_MINB
#define HILORE_COEFF_MINB 6
#endif
#ifndef HILORE_COEFF_MINB_KL
#define HILORE_COEFF_MINB_KL 6
#endif
constexpr int kWarpIters = HILORE_COEFF_IT;
constexpr int kWarpTile = kWarpIters * 256;

// Eight consecutive slots of one lane.  The subtractions, the scaling by log2(e), the product with -A / N and the
// K3 polynomial run on packed fp32 pairs (one instruction per two slots, each lane rounded as the scalar
// operation would be); ex2.approx, the clip compare and the selects are per slot.  Results are bit for bit those
// of omega_scalar.  POS: the sign of the advantage (uniform over the warp), which fixes the side of the clip test.
template <bool KL, bool EXTRA, int VAR, bool POS>
__device__ __forceinline__ void coeffs8(const uint32_t (&sn)[8], const uint32_t (&so)[8], const uint32_t (&sr)[8], uint2 mk,
                                        float A, float coef, float nkl, float hi, float lo, uint32_t (&w)[8],
                                        uint32_t (&rr)[8], uint2 &chi)
{
    const uint64_t l2e = f32x2_pack(kLog2e, kLog2e), coef2 = f32x2_pack(coef, coef);
    float v[8];
    uint32_t cb[8];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const uint64_t s2 = u32x2_pack(sn[2 * e], sn[2 * e + 1]), o2 = u32x2_pack(so[2 * e], so[2 * e + 1]);
        float x0, x1;
        f32x2_unpack(f32x2_mul(f32x2_sub(s2, o2), l2e), x0, x1);
        const float r0 = ex2_approx(x0), r1 = ex2_approx(x1);
        const bool c0 = POS ? (r0 <= hi) : (r0 >= lo), c1 = POS ? (r1 <= hi) : (r1 >= lo);
        if (VAR == 0) {
            float p0, p1;
            f32x2_unpack(f32x2_mul(coef2, f32x2_pack(r0, r1)), p0, p1);
            v[2 * e] = c0 ? p0 : 0.0f;
            v[2 * e + 1] = c1 ? p1 : 0.0f;
        } else {
            v[2 * e] = v[2 * e + 1] = VAR == 2 ? A : coef;
        }
        if (EXTRA) {
            rr[2 * e] = __float_as_uint(r0);
            rr[2 * e + 1] = __float_as_uint(r1);
            cb[2 * e] = c0;
            cb[2 * e + 1] = c1;
        }
    }
    if (KL && VAR != 2) {
        const uint64_t nkl2 = f32x2_pack(nkl, nkl);
        float big = 0.0f; // largest |s_ref - s| of the eight
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const uint64_t d2 = f32x2_sub(u32x2_pack(sr[2 * e], sr[2 * e + 1]), u32x2_pack(sn[2 * e], sn[2 * e + 1]));
            float d0, d1;
            f32x2_unpack(d2, d0, d1);
            big = fmaxf(big, fmaxf(fabsf(d0), fabsf(d1)));
            f32x2_unpack(f32x2_fma(nkl2, expm1_k3_poly_x2(d2), f32x2_pack(v[2 * e], v[2 * e + 1])), v[2 * e], v[2 * e + 1]);
        }
        if (!(big <= kK3Switch)) { // rare (also taken for NaN): some slot is beyond the polynomial's range
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                float r;
                bool c;
                v[e] = omega_scalar<VAR>(__uint_as_float(sn[e]), __uint_as_float(so[e]), __uint_as_float(sr[e]), true, true, A,
                                         coef, nkl, hi, lo, r, c);
            }
        }
    }
    if (mk.x != 0x01010101u || mk.y != 0x01010101u) { // some slot of the eight is masked out
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const uint32_t byte = ((e < 4 ? mk.x : mk.y) >> (8 * (e & 3))) & 0xFFu;
            v[e] = byte != 0 ? v[e] : 0.0f;
        }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) w[e] = __float_as_uint(v[e]);
    if (EXTRA) {
        chi.x = cb[0] | (cb[1] << 8) | (cb[2] << 16) | (cb[3] << 24);
        chi.y = cb[4] | (cb[5] << 8) | (cb[6] << 16) | (cb[7] << 24);
    }
}

// Each warp owns one tile: its loads (256-bit per lane and tensor) are issued first, the group statistics of its
// response follow while they are in flight, then the arithmetic and the 256-bit stores.  Warps never wait for one
// another.  Needs T % 8 == 0 and 32-byte aligned tensors (8-byte for the masks); launched with the
// programmatic-serialization attribute, so a following launch of this library becomes resident while this one drains.
template <bool KL, bool EXTRA, int VAR>
__global__ void __launch_bounds__(kCoeffThreads, KL ? HILORE_COEFF_MINB_KL : HILORE_COEFF_MINB)
    grpo_coeffs_warp_kernel(const __grid_constant__ CoeffArgs a, uint32_t total_tiles)
{
    const int lane = threadIdx.x & 31;
    const uint32_t wt = blockIdx.x * (kCoeffThreads / 32) + (threadIdx.x >> 5);
    if (wt >= total_tiles)
        return;
    const uint32_t tpr = (uint32_t)a.tiles_per_row;
    const uint32_t row32 = tpr == 1 ? wt : wt / tpr;
    const int tt = (int)(wt - row32 * tpr);
    const int64_t row = row32, rowbase = row * a.T;
    grid_dependency_wait();
    uint32_t sn[kWarpIters][8], so[kWarpIters][8], sr[KL ? kWarpIters : 1][8];
    uint2 mk[kWarpIters];
    int64_t t0[kWarpIters];
#pragma unroll
    for (int i = 0; i < kWarpIters; ++i) {
        t0[i] = (int64_t)tt * kWarpTile + i * 256 + lane * 8;
        if (t0[i] < a.T) {
            const int64_t k = rowbase + t0[i];
            ld_global_256(a.logp_new + k, sn[i]);
            ld_global_256(a.logp_old + k, so[i]);
            if (KL) ld_global_256(a.logp_ref + k, sr[i]);
            mk[i] = ld_global_64_stream(a.mask + k);
        }
    }
    grid_dependency_release();
    const float A = group_advantage(a.rewards, a.resp_offset + row, a.G, a.adv_eps, lane);
    const long long N = a.N_norm_dev ? *a.N_norm_dev : (long long)a.N_norm;
    const double invN = N > 0 ? 1.0 / (double)N : 0.0;
    const float coef = (float)(-(double)A * invN);
    const float nkl = -(float)((double)a.beta * invN);
    if (tt == 0 && lane == 0 && a.adv_out)
        a.adv_out[row] = A;
    const float hi = 1.0f + a.clip_eps, lo = 1.0f - a.clip_eps;
#pragma unroll
    for (int i = 0; i < kWarpIters; ++i) {
        if (t0[i] >= a.T)
            continue;
        uint32_t w[8], rr[8];
        uint2 chi;
        if (A >= 0.0f) coeffs8<KL, EXTRA, VAR, true>(sn[i], so[i], sr[KL ? i : 0], mk[i], A, coef, nkl, hi, lo, w, rr, chi);
        else coeffs8<KL, EXTRA, VAR, false>(sn[i], so[i], sr[KL ? i : 0], mk[i], A, coef, nkl, hi, lo, w, rr, chi);
        const int64_t k = rowbase + t0[i];
        st_global_256(a.omega + k, w);
        if (EXTRA) {
            if (a.ratio) st_global_256(a.ratio + k, rr);
            if (a.clip_mask) *reinterpret_cast<uint2 *>(a.clip_mask + k) = chi;
        }
    }
}

// ------------------------------------------------------------------ coefficients, packed layout
// Sequences lie back to back (no padding slots); sequence i owns tokens cu[i] .. cu[i+1]-1.
// Index of the sequence that owns token k: the largest i < n_seq with cu[i] <= k.  Bounded for any contents.
__device__ __forceinline__ int owner_sequence(const int32_t *cu, int n_seq, int64_t k, int lo = 0)
{
    int hi = n_seq; // invariant: cu[lo] <= k (cu[0] = 0), answer in [lo, hi)
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if ((int64_t)__ldg(cu + mid) <= k) lo = mid;
        else hi = mid;
    }
    return lo;
}

// The same search by one whole warp: 32 probes per step, so a table of a million sequences takes four dependent
// loads instead of twenty.  All lanes return the answer.
__device__ __forceinline__ int owner_sequence_warp(const int32_t *cu, int n_seq, int64_t k, int lane)
{
    int lo = 0, hi = n_seq;
    while (hi - lo > 1) {
        const int64_t span = hi - lo;
        const int p = lo + (int)((span * (lane + 1)) / 33); // lo <= p < hi
        const int nle = __popc(__ballot_sync(0xFFFFFFFFu, (int64_t)__ldg(cu + p) <= k));
        const int new_lo = lo + (int)((span * nle) / 33);
        const int new_hi = nle < 32 ? lo + (int)((span * (nle + 1)) / 33) : hi;
        lo = new_lo;
        hi = new_hi;
    }
    return lo;
}

// One warp per prompt group that meets the microbatch: the statistics once, then the members' advantages.
__global__ void __launch_bounds__(128) packed_advantage_kernel(const float *rewards, int64_t resp_offset, int64_t n_seq, int G,
                                                                float adv_eps, float *adv)
{
    const int lane = threadIdx.x & 31;
    const int64_t g = resp_offset / G + (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    // Launched as a programmatic dependent: first everything ahead in the stream must be complete (a kernel of this
    // library may still be reading the advantage array this kernel rewrites).  Then the coefficient kernel behind
    // this one may start: it reads its token data and finds its sequences while this kernel runs, and waits for the
    // advantages (griddepcontrol.wait) before it uses them.
    grid_dependency_wait();
    grid_dependency_release();
    if (g * G >= resp_offset + n_seq) return;
    const GroupStats st = group_stats(rewards + g * G, G, lane);
    for (int j = lane; j < G; j += 32) {
        const int64_t resp = g * G + j;
        if (resp >= resp_offset && resp < resp_offset + n_seq)
            adv[resp - resp_offset] = advantage_of(st, __ldg(rewards + resp), adv_eps);
    }
}

struct PackedArgs {
    const int32_t *cu;
    int n_seq;
    int64_t n_tok;
    const float *adv, *logp_new, *logp_old, *logp_ref;
    const uint8_t *mask;
    int64_t N_norm;
    const long long *N_norm_dev;
    float clip_eps, beta;
    float *omega, *ratio;
    uint8_t *clip_mask;
};

template <bool KL, bool EXTRA>
__global__ void __launch_bounds__(kCoeffThreads) grpo_coeffs_packed_kernel(const __grid_constant__ PackedArgs a)
{
    const int tid = threadIdx.x;
    float4 sn[kCoeffVec], so[kCoeffVec], sr[kCoeffVec];
    uint32_t mk[kCoeffVec];
    int64_t k0[kCoeffVec];
    int cnt[kCoeffVec];
#pragma unroll
    for (int j = 0; j < kCoeffVec; ++j) {
        k0[j] = (int64_t)blockIdx.x * kCoeffTile + (int64_t)(j * kCoeffThreads + tid) * 4;
        const int64_t left = a.n_tok - k0[j];
        cnt[j] = left >= 4 ? 4 : (left > 0 ? (int)left : 0);
        if (cnt[j] == 4) {
            sn[j] = __ldcs(reinterpret_cast<const float4 *>(a.logp_new + k0[j]));
            so[j] = __ldcs(reinterpret_cast<const float4 *>(a.logp_old + k0[j]));
            if (KL) sr[j] = __ldcs(reinterpret_cast<const float4 *>(a.logp_ref + k0[j]));
            mk[j] = __ldcs(reinterpret_cast<const unsigned int *>(a.mask + k0[j]));
        } else if (cnt[j] > 0) { // ragged end of the microbatch: element by element
            float tn[4] = {0, 0, 0, 0}, to[4] = {0, 0, 0, 0}, tr[4] = {0, 0, 0, 0};
            uint32_t m = 0;
            for (int i = 0; i < cnt[j]; ++i) {
                tn[i] = a.logp_new[k0[j] + i];
                to[i] = a.logp_old[k0[j] + i];
                if (KL) tr[i] = a.logp_ref[k0[j] + i];
                m |= (uint32_t)(a.mask[k0[j] + i] != 0) << (8 * i);
            }
            sn[j] = make_float4(tn[0], tn[1], tn[2], tn[3]);
            so[j] = make_float4(to[0], to[1], to[2], to[3]);
            sr[j] = make_float4(tr[0], tr[1], tr[2], tr[3]);
            mk[j] = m;
        }
    }
    // the sequences that meet this tile: found once per CTA (two searches over the whole table, in parallel with
    // the token loads), then each group searches that short range only
    __shared__ int s_range[2];
    __shared__ int64_t s_first_end;
    __shared__ float s_first_adv;
    __shared__ double s_invN;
    if (tid == 64) { // the fp64 reciprocal of the normaliser once per CTA
        const long long N = a.N_norm_dev ? *a.N_norm_dev : (long long)a.N_norm;
        s_invN = N > 0 ? 1.0 / (double)N : 0.0;
    }
    if (tid < 64) {
        const int64_t first = (int64_t)blockIdx.x * kCoeffTile;
        const int64_t last = min(first + kCoeffTile, a.n_tok) - 1;
        const int own = owner_sequence_warp(a.cu, a.n_seq, tid < 32 ? first : last, tid & 31);
        if ((tid & 31) == 0) s_range[tid >> 5] = own;
        if (tid == 0) { // most groups of a tile lie in its first sequence: its end and advantage go to shared memory
            s_first_end = (int64_t)__ldg(a.cu + own + 1);
            s_first_adv = __ldg(a.adv + own);
        }
    }
    __syncthreads();
    const int seq_first = s_range[0], seq_end = s_range[1] + 1;
    const double invN = s_invN;
    const float nkl = -(float)((double)a.beta * invN);
    const float hi = 1.0f + a.clip_eps, lo = 1.0f - a.clip_eps;

#pragma unroll
    for (int j = 0; j < kCoeffVec; ++j) {
        if (cnt[j] == 0)
            continue;
        int seq = seq_first;
        int64_t end = s_first_end;
        float A = s_first_adv;
        if (k0[j] >= end) {
            seq = owner_sequence(a.cu, seq_end, k0[j], seq_first);
            end = (int64_t)__ldg(a.cu + seq + 1);
            A = __ldg(a.adv + seq);
        }
        float coef = (float)(-(double)A * invN);
        const float s[4] = {sn[j].x, sn[j].y, sn[j].z, sn[j].w};
        const float o[4] = {so[j].x, so[j].y, so[j].z, so[j].w};
        const float rf[4] = {sr[j].x, sr[j].y, sr[j].z, sr[j].w};
        float w[4], r[4];
        uint32_t chi = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (k0[j] + i >= end && i < cnt[j]) { // the group crosses into the next non-empty sequence
                while (seq + 1 < a.n_seq && k0[j] + i >= end) {
                    ++seq;
                    end = (int64_t)__ldg(a.cu + seq + 1);
                }
                A = __ldg(a.adv + seq);
                coef = (float)(-(double)A * invN);
            }
            const bool m = ((mk[j] >> (8 * i)) & 0xFFu) != 0;
            bool c;
            w[i] = omega_scalar<0>(s[i], o[i], KL ? rf[i] : 0.0f, m, KL, A, coef, nkl, hi, lo, r[i], c);
            chi |= (uint32_t)c << (8 * i);
        }
        if (cnt[j] == 4) {
            __stcs(reinterpret_cast<float4 *>(a.omega + k0[j]), make_float4(w[0], w[1], w[2], w[3]));
            if (EXTRA) {
                if (a.ratio) __stcs(reinterpret_cast<float4 *>(a.ratio + k0[j]), make_float4(r[0], r[1], r[2], r[3]));
                if (a.clip_mask) __stcs(reinterpret_cast<unsigned int *>(a.clip_mask + k0[j]), chi);
            }
        } else {
            for (int i = 0; i < cnt[j]; ++i) {
                a.omega[k0[j] + i] = w[i];
                if (EXTRA) {
                    if (a.ratio) a.ratio[k0[j] + i] = r[i];
                    if (a.clip_mask) a.clip_mask[k0[j] + i] = (uint8_t)((chi >> (8 * i)) & 1u);
                }
            }
        }
    }
}

// The packed fast path: one WARP per tile of kWarpTile tokens, as in the dense warp kernel (no CTA barrier, 256-bit
// accesses, packed fp32 pairs).  The warp finds the owner of its first token with one cooperative search, then reads
// the 32 sequence boundaries that follow it with one coalesced load: those that fall inside the tile tell every lane
// its sequence by counting, without further loads (sequences of 1-3 K tokens: zero or one boundary per tile).  A lane
// whose eight tokens lie in one sequence takes the packed arithmetic; one that straddles a boundary, or the ragged
// end of the microbatch, walks its tokens one by one.  Same bits as the generic kernel.  Needs 32-byte aligned
// tensors (8-byte masks).
template <bool KL, bool EXTRA>
__global__ void __launch_bounds__(kCoeffThreads, 6) grpo_coeffs_packed_warp_kernel(const __grid_constant__ PackedArgs a,
                                                                                    uint32_t total_tiles)
{
    constexpr uint32_t kFull = 0xFFFFFFFFu;
    const int lane = threadIdx.x & 31;
    const uint32_t wt = blockIdx.x * (kCoeffThreads / 32) + (threadIdx.x >> 5);
    if (wt >= total_tiles)
        return;
    const int64_t first = (int64_t)wt * kWarpTile;
    // The kernel ahead in the stream computes the advantages and nothing else, and it lets this one start only after
    // everything before it in the stream is complete: token data, masks, sequence boundaries and N are final already.
    uint32_t sn[kWarpIters][8], so[kWarpIters][8], sr[KL ? kWarpIters : 1][8];
    uint2 mk[kWarpIters];
    int64_t k0[kWarpIters];
    int cnt[kWarpIters];
#pragma unroll
    for (int i = 0; i < kWarpIters; ++i) {
        k0[i] = first + i * 256 + lane * 8;
        const int64_t left = a.n_tok - k0[i];
        cnt[i] = left >= 8 ? 8 : (left > 0 ? (int)left : 0);
        if (cnt[i] == 8) {
            ld_global_256(a.logp_new + k0[i], sn[i]);
            ld_global_256(a.logp_old + k0[i], so[i]);
            if (KL) ld_global_256(a.logp_ref + k0[i], sr[i]);
            mk[i] = ld_global_64_stream(a.mask + k0[i]);
        } else { // ragged end of the microbatch: element by element, zeros beyond it
            uint32_t m[2] = {0, 0};
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const bool in = e < cnt[i];
                sn[i][e] = in ? __float_as_uint(a.logp_new[k0[i] + e]) : 0u;
                so[i][e] = in ? __float_as_uint(a.logp_old[k0[i] + e]) : 0u;
                if (KL) sr[i][e] = in ? __float_as_uint(a.logp_ref[k0[i] + e]) : 0u;
                if (in && a.mask[k0[i] + e] != 0) m[e >> 2] |= 1u << (8 * (e & 3));
            }
            mk[i] = make_uint2(m[0], m[1]);
        }
    }
    const int64_t last = min(first + kWarpTile, a.n_tok) - 1;
    const int own = owner_sequence_warp(a.cu, a.n_seq, first, lane);
    // lane j: the first token of sequence own + 1 + j (past the table: a value no token reaches)
    const int bi = own + 1 + lane;
    const int bound = bi <= a.n_seq ? __ldg(a.cu + bi) : 0x7FFFFFFF;
    const int nle = __popc(__ballot_sync(kFull, (int64_t)bound <= last)); // sequences that begin inside the tile
    const long long N = a.N_norm_dev ? *a.N_norm_dev : (long long)a.N_norm;
    const double invN = N > 0 ? 1.0 / (double)N : 0.0;
    const float nkl = -(float)((double)a.beta * invN);
    const float hi = 1.0f + a.clip_eps, lo = 1.0f - a.clip_eps;
    grid_dependency_wait(); // the advantages are complete from here on
    grid_dependency_release();
#pragma unroll
    for (int i = 0; i < kWarpIters; ++i) {
        int seq;
        int64_t end;
        if (nle < 32) { // the owner of this lane's first token: `own` plus the boundaries at or below it
            int c = 0;
            for (int j = 0; j < nle; ++j) c += (int64_t)__shfl_sync(kFull, bound, j) <= k0[i];
            seq = own + c;
            end = (int64_t)__shfl_sync(kFull, bound, c);
        } else {        // more than 32 sequences in 512 tokens: every lane searches
            seq = owner_sequence(a.cu, a.n_seq, min(k0[i], last), own);
            end = (int64_t)__ldg(a.cu + seq + 1);
        }
        if (cnt[i] == 0)
            continue;
        float A = __ldg(a.adv + seq);
        float coef = (float)(-(double)A * invN);
        uint32_t w[8], rr[8];
        uint2 chi = make_uint2(0u, 0u);
        if (cnt[i] == 8 && k0[i] + 8 <= end) {
            if (A >= 0.0f) coeffs8<KL, EXTRA, 0, true>(sn[i], so[i], sr[KL ? i : 0], mk[i], A, coef, nkl, hi, lo, w, rr, chi);
            else coeffs8<KL, EXTRA, 0, false>(sn[i], so[i], sr[KL ? i : 0], mk[i], A, coef, nkl, hi, lo, w, rr, chi);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                if (e < cnt[i] && k0[i] + e >= end) { // into the next non-empty sequence
                    while (seq + 1 < a.n_seq && k0[i] + e >= end) {
                        ++seq;
                        end = (int64_t)__ldg(a.cu + seq + 1);
                    }
                    A = __ldg(a.adv + seq);
                    coef = (float)(-(double)A * invN);
                }
                const bool m = (((e < 4 ? mk[i].x : mk[i].y) >> (8 * (e & 3))) & 0xFFu) != 0;
                float r;
                bool c;
                w[e] = __float_as_uint(omega_scalar<0>(__uint_as_float(sn[i][e]), __uint_as_float(so[i][e]),
                                                       KL ? __uint_as_float(sr[KL ? i : 0][e]) : 0.0f, m, KL, A, coef, nkl, hi,
                                                       lo, r, c));
                rr[e] = __float_as_uint(r);
                if (e < 4) chi.x |= (uint32_t)c << (8 * e);
                else chi.y |= (uint32_t)c << (8 * (e - 4));
            }
        }
        if (cnt[i] == 8) {
            st_global_256(a.omega + k0[i], w);
            if (EXTRA) {
                if (a.ratio) st_global_256(a.ratio + k0[i], rr);
                if (a.clip_mask) *reinterpret_cast<uint2 *>(a.clip_mask + k0[i]) = chi;
            }
        } else {
            for (int e = 0; e < cnt[i]; ++e) {
                a.omega[k0[i] + e] = __uint_as_float(w[e]);
                if (EXTRA) {
                    if (a.ratio) a.ratio[k0[i] + e] = __uint_as_float(rr[e]);
                    if (a.clip_mask) a.clip_mask[k0[i] + e] = (uint8_t)(((e < 4 ? chi.x : chi.y) >> (8 * (e & 3))) & 1u);
                }
            }
        }
    }
}

// ------------------------------------------------------------------ exposure
constexpr int kExpThreads = 256;
constexpr int kExpTile = kExpThreads * 4; // slots per CTA
constexpr int kExpUnits = 8;              // units per CTA (omega and mask are read once for all of them)
constexpr int kMaxClusterTiles = 16;      // CTAs (tiles of tokens) of a unit group in the cluster form

// One warp adds the per-tile partials of unit u in a fixed order and applies the closed form
//   E_u = (S2_u + eps * S3) / (S1_u / |T_b| + eps),  S1 = sum a, S2 = sum |omega| a, S3 = sum |omega|.
// Every lane returns E_u; *s3_out gets S3.
// The closed form from the per-lane sums over the tiles (lane t holds the sums of tiles t, t + 32, ...).
__device__ __forceinline__ float exposure_from_lane_sums(double s1, double s2, double s3, double cnt, float eps_alpha, double *s3_out)
{
    s1 = warp_sum(s1);
    s2 = warp_sum(s2);
    s3 = warp_sum(s3);
    cnt = warp_sum(cnt);
    double E = 0.0;
    if (cnt > 0.0)
        E = (s2 + (double)eps_alpha * s3) / (s1 / cnt + (double)eps_alpha);
    *s3_out = s3;
    return (float)E;
}

__device__ __forceinline__ float exposure_of_unit(const double *part, int tok_row, int ntiles, int u, float eps_alpha, int lane,
                                                  double *s3_out)
{
    double s1 = 0.0, s2 = 0.0, s3 = 0.0, cnt = 0.0;
    for (int t = lane; t < ntiles; t += 32) { // tok_row: the row of partials that holds sum |omega| and |T_b|
        s1 += __ldcg(part + ((int64_t)u * ntiles + t) * 2);
        s2 += __ldcg(part + ((int64_t)u * ntiles + t) * 2 + 1);
        s3 += __ldcg(part + ((int64_t)tok_row * ntiles + t) * 2);
        cnt += __ldcg(part + ((int64_t)tok_row * ntiles + t) * 2 + 1);
    }
    return exposure_from_lane_sums(s1, s2, s3, cnt, eps_alpha, s3_out);
}

// Inputs of the coefficient pass when it is fused into the exposure reduction (hilore_coeffs_exposure).
constexpr int kFusedRows = 64; // responses one CTA's slots may span
struct FusedCoeff {
    const float *rewards;
    int G;
    int64_t resp_offset;
    const float *logp_new, *logp_old, *logp_ref;
    int64_t N_norm;
    const long long *N_norm_dev;
    float clip_eps, beta, adv_eps;
    float *omega_out;
};

struct ExpArgs {
    const float *omega;
    const uint8_t *mask;
    int64_t n_rows, T, n_tok;
    const float *row_rms;
    int U;
    int64_t rms_ld;
    int row_shift;
    double *part; // [(U + 1), ntiles, 2]
    int ntiles;
    const int32_t *cu; // packed layout: sequence boundaries (else nullptr: rows of T slots)
    int n_seq;
    int steps;         // pieces of kExpTile slots per CTA
    FusedCoeff f;      // used by the fused kernel only
    // single-launch form: the CTA that finishes last adds the partials and, if asked, takes the plan decisions
    unsigned int *done; // counter of finished CTAs (zero before the launch), or nullptr: a second kernel finishes
    int cluster;        // 1: the CTAs of a unit group form one thread-block cluster and reduce through its shared memory
    float eps_alpha;
    float *exposure, *sum_abs_omega;
    PlanTail plan;      // plan.avail == nullptr: no decisions
};

// A CTA covers `steps` consecutive pieces of kExpTile slots for kExpUnits units: every thread accumulates its
// slots of all pieces in registers (fp32) and the warp / CTA reduction runs once per CTA, so that the reduction
// no longer costs more than the loads on large token grids.
// One coefficient, exactly as grpo_coeffs_kernel computes it (same expressions, same rounding).
__device__ __forceinline__ float fused_omega(float s, float o, float rf, bool m, float A, float coef, float kl, float hi, float lo)
{
    float r;
    bool c;
    return omega_scalar<0>(s, o, rf, m, kl != 0.0f, A, coef, -kl, hi, lo, r, c);
}

// FUSED: omega is not read but computed here from the log-probabilities (and written once, by the CTAs of the
// first unit group): the coefficient pass and its reduction to exposure scores in one sweep.
template <bool VEC, bool FUSED = false>
__global__ void __launch_bounds__(kExpThreads) exposure_partial_kernel(const __grid_constant__ ExpArgs a)
{
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int tile = blockIdx.x;
    const int u0 = blockIdx.y * kExpUnits, nu = min(kExpUnits, a.U - u0);
    __shared__ double sm[kExpThreads / 32][2 * (kExpUnits + 1)];
    namespace cg = cooperative_groups;
    cg::cluster_group cl = cg::this_cluster();
    if (a.cluster)
        cl.barrier_arrive(); // first phase of the cluster barrier: once all have arrived, every CTA of the cluster runs
    grid_dependency_wait();
    grid_dependency_release(); // the final reduction may become resident; it waits for this grid to complete
    __shared__ float s_A[FUSED ? kFusedRows : 1], s_coef[FUSED ? kFusedRows : 1];
    int64_t row_lo = 0;
    float f_kl = 0.0f, f_hi = 0.0f, f_lo = 0.0f;
    bool pre = false; // FUSED: this thread's slots of the CTA's only piece are in registers already
    uint32_t pre_m = 0;
    float4 pre_sn = make_float4(0.0f, 0.0f, 0.0f, 0.0f), pre_so = pre_sn, pre_sr = pre_sn;
    float4 pre_av[FUSED ? kExpUnits : 1];
    if (FUSED) { // the per-response scalars of the responses this CTA's slots belong to
        // This form runs at microbatch size, where the kernel is a chain of dependent memory latencies: ask for the
        // first piece's token data, the units' magnitudes and the plan inputs now, so that they arrive while the
        // group statistics (rewards -> fp64 sums -> shuffles) are worked out.
        {
            const int64_t k = (int64_t)tile * a.steps * kExpTile + (int64_t)tid * 4;
            if (k < a.n_tok && !(VEC && a.steps == 1)) { // (the one-piece form loads them into registers below)
                prefetch_l2(a.f.logp_new + k);
                prefetch_l2(a.f.logp_old + k);
                if (a.f.logp_ref) prefetch_l2(a.f.logp_ref + k);
                prefetch_l2(a.mask + k);
                for (int j = 0; j < nu; ++j) prefetch_l2(a.row_rms + (int64_t)(u0 + j) * a.rms_ld + k);
            }
            if ((a.done != nullptr || a.cluster) && a.plan.avail != nullptr && tid < nu) {
                prefetch_l2(a.plan.kappa + u0 + tid);
                prefetch_l2(a.plan.ebar + u0 + tid);
                prefetch_l2(a.plan.avail + u0 + tid);
                prefetch_l2(&a.plan.units[u0 + tid].rows);
            }
        }
        const int64_t slot_lo = (int64_t)tile * a.steps * kExpTile;
        const int64_t slot_hi = min(a.n_tok, slot_lo + (int64_t)a.steps * kExpTile);
        row_lo = slot_lo / a.T;
        const int nrows = (int)((slot_hi - 1) / a.T - row_lo) + 1;
        const long long N = a.f.N_norm_dev ? *a.f.N_norm_dev : (long long)a.f.N_norm;
        const double invN = N > 0 ? 1.0 / (double)N : 0.0;
        f_kl = (float)((double)a.f.beta * invN);
        // One piece per CTA (the microbatch form): its token data and the units' magnitudes are loaded into
        // registers now, so that only arithmetic is left once the statistics are known.
        if (VEC && a.steps == 1) {
            const int64_t k = slot_lo + (int64_t)tid * 4;
            if (k < a.n_tok) {
                pre = true;
                pre_m = *reinterpret_cast<const unsigned int *>(a.mask + k);
                pre_sn = *reinterpret_cast<const float4 *>(a.f.logp_new + k);
                pre_so = *reinterpret_cast<const float4 *>(a.f.logp_old + k);
                if (f_kl != 0.0f) pre_sr = *reinterpret_cast<const float4 *>(a.f.logp_ref + k);
#pragma unroll
                for (int j = 0; j < kExpUnits; ++j)
                    if (j < nu) pre_av[j] = *reinterpret_cast<const float4 *>(a.row_rms + (int64_t)(u0 + j) * a.rms_ld + k);
            }
        }
        for (int r = wid; r < nrows; r += kExpThreads / 32) {
            const float A = group_advantage(a.f.rewards, a.f.resp_offset + row_lo + r, a.f.G, a.f.adv_eps, lane);
            if (lane == 0) {
                s_A[r] = A;
                s_coef[r] = (float)(-(double)A * invN);
            }
        }
        f_hi = 1.0f + a.f.clip_eps;
        f_lo = 1.0f - a.f.clip_eps;
        __syncthreads();
    }
    // per-thread partials in fp32 (four terms per piece), warp tree in fp32, across warps and tiles in fp64
    float acc[2 * (kExpUnits + 1)];
#pragma unroll
    for (int q = 0; q < 2 * (kExpUnits + 1); ++q) acc[q] = 0.0f;
    // Large token grids (the plain vector path): two pieces per trip, all their loads issued before the first
    // use, so that a thread has twenty 16-byte loads in flight instead of ten; the sums are taken in the order of
    // the one-piece loop below, whose results they equal bit for bit.
    for (int st = 0; VEC && !FUSED && st < a.steps; st += 2) {
        int64_t k[2];
        bool ok[2];
        uint32_t m[2] = {0, 0};
        uint4 w[2], av[2][kExpUnits];
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            k[p] = ((int64_t)tile * a.steps + st + p) * kExpTile + (int64_t)tid * 4;
            ok[p] = st + p < a.steps && k[p] < a.n_tok; // n_tok % 4 == 0: a group is valid as a whole
            if (ok[p]) {
                m[p] = __ldcs(reinterpret_cast<const unsigned int *>(a.mask + k[p]));
                w[p] = ld_global_128_stream(a.omega + k[p]);
#pragma unroll
                for (int j = 0; j < kExpUnits; ++j)
                    if (j < nu) av[p][j] = ld_global_128_stream(a.row_rms + (int64_t)(u0 + j) * a.rms_ld + k[p]);
            }
        }
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            if (!ok[p])
                continue;
            const float wv[4] = {__uint_as_float(w[p].x), __uint_as_float(w[p].y), __uint_as_float(w[p].z), __uint_as_float(w[p].w)};
            bool mk[4];
            float wabs[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                mk[i] = ((m[p] >> (8 * i)) & 0xFFu) != 0;
                wabs[i] = mk[i] ? fabsf(wv[i]) : 0.0f;
            }
            acc[2 * kExpUnits] += (wabs[0] + wabs[1]) + (wabs[2] + wabs[3]);
            acc[2 * kExpUnits + 1] += (float)((int)mk[0] + (int)mk[1] + (int)mk[2] + (int)mk[3]);
#pragma unroll
            for (int j = 0; j < kExpUnits; ++j) {
                float s1 = 0.0f, s2 = 0.0f;
                if (j < nu) {
                    const float t[4] = {__uint_as_float(av[p][j].x), __uint_as_float(av[p][j].y), __uint_as_float(av[p][j].z),
                                        __uint_as_float(av[p][j].w)};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        s1 += mk[i] ? t[i] : 0.0f;
                        s2 = fmaf(wabs[i], mk[i] ? t[i] : 0.0f, s2);
                    }
                }
                acc[2 * j] += s1;
                acc[2 * j + 1] += s2;
            }
        }
    }
    for (int st = 0; !(VEC && !FUSED) && st < a.steps; ++st) {
        const int64_t piece = (int64_t)tile * a.steps + st;
        if (piece * kExpTile >= a.n_tok)
            break;
        float wabs[4];   // |omega| at valid slots, else 0
        bool mk[4];      // slot is in T_b
        bool has[4];     // ... and its activation row exists (t - row_shift >= 0)
        int64_t slot[4];
        if (VEC) {
            const int64_t k = piece * kExpTile + (int64_t)tid * 4;
#pragma unroll
            for (int i = 0; i < 4; ++i) slot[i] = k + i;
            if (k < a.n_tok) { // n_tok % 4 == 0: a group is valid as a whole
                const uint32_t m = (FUSED && pre) ? pre_m : *reinterpret_cast<const unsigned int *>(a.mask + k);
                float wv[4];
                if (FUSED) { // T % 4 == 0: the four slots belong to one response
                    float4 sn = pre_sn, so = pre_so, sr = pre_sr;
                    if (!pre) {
                        sn = *reinterpret_cast<const float4 *>(a.f.logp_new + k);
                        so = *reinterpret_cast<const float4 *>(a.f.logp_old + k);
                        if (f_kl != 0.0f) sr = *reinterpret_cast<const float4 *>(a.f.logp_ref + k);
                    }
                    const int ri = (int)(k / a.T - row_lo);
                    const float A = s_A[ri], coef = s_coef[ri];
                    wv[0] = fused_omega(sn.x, so.x, sr.x, (m & 0xFFu) != 0, A, coef, f_kl, f_hi, f_lo);
                    wv[1] = fused_omega(sn.y, so.y, sr.y, (m & 0xFF00u) != 0, A, coef, f_kl, f_hi, f_lo);
                    wv[2] = fused_omega(sn.z, so.z, sr.z, (m & 0xFF0000u) != 0, A, coef, f_kl, f_hi, f_lo);
                    wv[3] = fused_omega(sn.w, so.w, sr.w, (m & 0xFF000000u) != 0, A, coef, f_kl, f_hi, f_lo);
                    if (a.f.omega_out && blockIdx.y == 0)
                        *reinterpret_cast<float4 *>(a.f.omega_out + k) = make_float4(wv[0], wv[1], wv[2], wv[3]);
                } else {
                    const float4 w = *reinterpret_cast<const float4 *>(a.omega + k);
                    wv[0] = w.x; wv[1] = w.y; wv[2] = w.z; wv[3] = w.w;
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    mk[i] = ((m >> (8 * i)) & 0xFFu) != 0;
                    has[i] = mk[i];
                    wabs[i] = mk[i] ? fabsf(wv[i]) : 0.0f;
                }
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    mk[i] = false;
                    has[i] = false;
                    wabs[i] = 0.0f;
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int64_t k = piece * kExpTile + i * kExpThreads + tid;
                slot[i] = k;
                mk[i] = false;
                has[i] = false;
                wabs[i] = 0.0f;
                if (FUSED && k < a.n_tok) { // every slot gets its coefficient, masked ones a zero
                    const int ri = (int)(k / a.T - row_lo);
                    const float w = fused_omega(a.f.logp_new[k], a.f.logp_old[k], f_kl != 0.0f ? a.f.logp_ref[k] : 0.0f,
                                                a.mask[k] != 0, s_A[ri], s_coef[ri], f_kl, f_hi, f_lo);
                    if (a.f.omega_out && blockIdx.y == 0) a.f.omega_out[k] = w;
                    wabs[i] = fabsf(w);
                }
                if (k < a.n_tok && a.mask[k] != 0) {
                    mk[i] = true;
                    if (!FUSED) wabs[i] = fabsf(a.omega[k]);
                    // a slot whose source row lies before the start of its response has no activation term
                    if (a.row_shift == 0) has[i] = true;
                    else if (a.cu) has[i] = k - (int64_t)__ldg(a.cu + owner_sequence(a.cu, a.n_seq, k)) >= a.row_shift;
                    else has[i] = (k % a.T) >= a.row_shift;
                }
            }
        }
        acc[2 * kExpUnits] += (wabs[0] + wabs[1]) + (wabs[2] + wabs[3]);
        // the weights average to one over the slots of T_b that have an activation row: those are counted
        acc[2 * kExpUnits + 1] += (float)((int)has[0] + (int)has[1] + (int)has[2] + (int)has[3]);
#pragma unroll
        for (int j = 0; j < kExpUnits; ++j) {
            float s1 = 0.0f, s2 = 0.0f;
            if (j < nu) {
                const float *ar = a.row_rms + (int64_t)(u0 + j) * a.rms_ld;
                float av[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                if (VEC) {
                    if (slot[0] < a.n_tok) {
                        const float4 t = (FUSED && pre) ? pre_av[FUSED ? j : 0] : *reinterpret_cast<const float4 *>(ar + slot[0]);
                        av[0] = t.x; av[1] = t.y; av[2] = t.z; av[3] = t.w;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (has[i]) av[i] = ar[slot[i] - a.row_shift];
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    s1 += has[i] ? av[i] : 0.0f;
                    s2 = fmaf(wabs[i], has[i] ? av[i] : 0.0f, s2);
                }
            }
            acc[2 * j] += s1;
            acc[2 * j + 1] += s2;
        }
    }
#pragma unroll
    for (int q = 0; q < 2 * (kExpUnits + 1); ++q) {
        const float v = warp_sum(acc[q]);
        if (lane == 0) sm[wid][q] = (double)v;
    }
    __syncthreads();
    // cluster form: the partial sums of the cluster's CTAs, tile by tile, in the shared memory of its first CTA
    __shared__ double s_all[kMaxClusterTiles][2 * (kExpUnits + 1)];
    if (a.cluster)
        cl.barrier_wait(); // (long since complete) the first CTA's shared memory may be written now
    if (tid < 2 * (kExpUnits + 1)) {
        double t = 0.0;
        for (int w = 0; w < kExpThreads / 32; ++w) t += sm[w][tid];
        const int j = tid >> 1, which = tid & 1;
        if (a.cluster) {
            cl.map_shared_rank(&s_all[0][0], 0)[cl.block_rank() * (2 * (kExpUnits + 1)) + tid] = t;
        } else if (j < kExpUnits) {
            if (j < nu) a.part[((int64_t)(u0 + j) * a.ntiles + tile) * 2 + which] = t;
        } else if (a.done != nullptr) { // single-launch form: every unit group keeps its own copy of the token sums
            a.part[((int64_t)(a.U + blockIdx.y) * a.ntiles + tile) * 2 + which] = t;
        } else if (blockIdx.y == 0) {
            a.part[((int64_t)a.U * a.ntiles + tile) * 2 + which] = t;
        }
    }
    if (a.cluster) {
        // Cluster form of the single launch (microbatch sizes): the CTAs of a unit group -- one per tile of tokens --
        // are one thread-block cluster.  Every CTA has written its partial sums into the first CTA's shared memory
        // (distributed shared memory) and arrives at the cluster barrier (release); the first CTA waits for all
        // (acquire) and goes on alone, lane t taking tile t as the final kernel does, so the results are those of
        // the other forms bit for bit.  No partial sum goes through global memory, nothing is counted, nothing needs
        // clearing, and the other CTAs are gone as soon as they have arrived: nobody reads their shared memory.
        cl.barrier_arrive();
        if (cl.block_rank() != 0)
            return;
        cl.barrier_wait();
        if (wid < nu) {
            double s1 = 0.0, s2 = 0.0, s3 = 0.0, cnt = 0.0;
            if (lane < (int)gridDim.x) {
                s1 = s_all[lane][2 * wid];
                s2 = s_all[lane][2 * wid + 1];
                s3 = s_all[lane][2 * kExpUnits];
                cnt = s_all[lane][2 * kExpUnits + 1];
            }
            double s3_all;
            const float E = exposure_from_lane_sums(s1, s2, s3, cnt, a.eps_alpha, &s3_all);
            if (lane == 0) {
                const int u = u0 + wid;
                a.exposure[u] = E;
                if (u == 0 && a.sum_abs_omega) *a.sum_abs_omega = (float)s3_all;
                if (a.plan.avail) decide_unit(a.plan, u, &E);
            }
        }
        return;
    }
    if (a.done == nullptr)
        return;
    // Single-launch form.  Every CTA publishes its partials and counts itself on its unit group's counter; the one
    // that counts last has all partials of the group in view: its eight warps add those of the group's eight units
    // in the order of exposure_final_kernel (so the results do not depend on which CTA that is) and take the units'
    // plan decisions.  It leaves the counter at zero.
    __shared__ bool s_last;
    __threadfence();
    __syncthreads();
    if (tid == 0)
        s_last = atomicAdd(a.done + blockIdx.y, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!s_last)
        return;
    __threadfence();
    if (wid < nu) {
        const int u = u0 + wid;
        double s3;
        const float E = exposure_of_unit(a.part, a.U + blockIdx.y, a.ntiles, u, a.eps_alpha, lane, &s3);
        if (lane == 0) {
            a.exposure[u] = E;
            if (u == 0 && a.sum_abs_omega) *a.sum_abs_omega = (float)s3;
            if (a.plan.avail) decide_unit(a.plan, u, &E);
        }
    }
    if (tid == 0)
        a.done[blockIdx.y] = 0;
}

// One warp per unit adds the per-tile partials in a fixed order and applies the closed form
//   E_u = (S2_u + eps * S3) / (S1_u / |T_b| + eps),  S1 = sum a, S2 = sum |omega| a, S3 = sum |omega|.
__global__ void __launch_bounds__(32) exposure_final_kernel(const double *part, int U, int ntiles, float eps_alpha,
                                                            float *exposure, float *sum_abs_omega)
{
    const int u = blockIdx.x, lane = threadIdx.x;
    grid_dependency_wait();
    grid_dependency_release();
    double s3;
    const float E = exposure_of_unit(part, U, ntiles, u, eps_alpha, lane, &s3);
    if (lane == 0) {
        exposure[u] = E;
        if (u == 0 && sum_abs_omega) *sum_abs_omega = (float)s3;
    }
}

} // namespace hilore

using namespace hilore;

extern "C" int hilore_mask_count(const uint8_t *mask, int64_t n, int64_t *count, void *stream)
{
    if (count == nullptr || n < 0 || (n > 0 && mask == nullptr))
        return HILORE_INVALID_ARG;
    if (!aligned(count, 8))
        return HILORE_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(count, 0, sizeof(int64_t), st) != cudaSuccess)
        return HILORE_CUDA;
    if (n == 0)
        return HILORE_OK;
    int64_t blocks = (n / 16 + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    mask_count_kernel<<<(unsigned)blocks, 256, 0, st>>>(mask, n, reinterpret_cast<unsigned long long *>(count));
    return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
}

static int launch_coeffs(const float *rewards, int64_t n_resp_total, int32_t G, int64_t resp_offset, int64_t n_rows,
                         int64_t T, const float *logp_new, const float *logp_old, const float *logp_ref, const uint8_t *mask,
                         int64_t N_norm, const int64_t *N_norm_dev, float clip_eps, float beta, float adv_eps, int variant,
                         float *adv_out, float *omega, float *ratio, uint8_t *clip_mask, void *stream)
{
    if (variant < 0 || variant > 2)
        return HILORE_INVALID_ARG;
    if (rewards == nullptr || n_resp_total < 0 || G <= 0 || resp_offset < 0 || n_rows < 0 || T < 0)
        return HILORE_INVALID_ARG;
    if (n_resp_total % G != 0 || resp_offset + n_rows > n_resp_total || T % 4 != 0)
        return HILORE_SHAPE;
    if (beta != 0.0f && logp_ref == nullptr)
        return HILORE_INVALID_ARG;
    if (N_norm_dev == nullptr && N_norm <= 0)
        return HILORE_ZERO_NORM;
    if (n_rows == 0 || T == 0)
        return HILORE_OK;
    if (logp_new == nullptr || logp_old == nullptr || mask == nullptr || omega == nullptr)
        return HILORE_INVALID_ARG;
    if (!aligned(logp_new, 16) || !aligned(logp_old, 16) || !aligned(logp_ref, 16) || !aligned(omega, 16) ||
        !aligned(ratio, 16) || !aligned(mask, 4) || !aligned(clip_mask, 4) || !aligned(rewards, 4) ||
        !aligned(adv_out, 4) || !aligned(N_norm_dev, 8))
        return HILORE_ALIGN;
    CoeffArgs a{};
    a.rewards = rewards;
    a.n_resp_total = n_resp_total;
    a.G = G;
    a.resp_offset = resp_offset;
    a.n_rows = n_rows;
    a.T = T;
    a.logp_new = logp_new;
    a.logp_old = logp_old;
    a.logp_ref = (beta != 0.0f) ? logp_ref : nullptr;
    a.mask = mask;
    a.N_norm = N_norm;
    a.N_norm_dev = reinterpret_cast<const long long *>(N_norm_dev);
    a.clip_eps = clip_eps;
    a.beta = beta;
    a.adv_eps = adv_eps;
    a.adv_out = adv_out;
    a.omega = omega;
    a.ratio = ratio;
    a.clip_mask = clip_mask;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool kl = beta != 0.0f, extra = (ratio != nullptr) || (clip_mask != nullptr);
    // programmatic dependent launch: the kernels wait (griddepcontrol.wait) before their first global access
    cudaLaunchConfig_t cfg{};
    cfg.blockDim = dim3(kCoeffThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const bool wide = T % 8 == 0 && aligned(logp_new, 32) && aligned(logp_old, 32) && aligned(a.logp_ref, 32) &&
                      aligned(omega, 32) && aligned(ratio, 32) && aligned(mask, 8) && aligned(clip_mask, 8);
    if (wide) { // one warp per tile of kWarpTile slots
        const int64_t tpr = (T + kWarpTile - 1) / kWarpTile;
        const int64_t tiles = tpr * n_rows;
        if (tpr > 0x7FFFFFFF || tiles > 0x7FFFFFFF)
            return HILORE_SHAPE;
        a.tiles_per_row = (int)tpr;
        void (*kernel)(CoeffArgs, uint32_t) = nullptr;
#define HILORE_PICK(V)                                                                                                  \
    kernel = kl ? (extra ? grpo_coeffs_warp_kernel<true, true, V> : grpo_coeffs_warp_kernel<true, false, V>)            \
                : (extra ? grpo_coeffs_warp_kernel<false, true, V> : grpo_coeffs_warp_kernel<false, false, V>)
        if (variant == 0) { HILORE_PICK(0); }
        else if (variant == 1) { HILORE_PICK(1); }
        else { HILORE_PICK(2); }
#undef HILORE_PICK
        constexpr int kWarps = kCoeffThreads / 32;
        cfg.gridDim = dim3((unsigned)((tiles + kWarps - 1) / kWarps));
        if (cudaLaunchKernelEx(&cfg, kernel, a, (uint32_t)tiles) != cudaSuccess)
            return HILORE_CUDA;
        return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
    }
    const int64_t tpr = (T + kCoeffTile - 1) / kCoeffTile;
    const int64_t tiles = tpr * n_rows;
    if (tpr > 0x7FFFFFFF || tiles > 0x7FFFFFFF)
        return HILORE_SHAPE;
    a.tiles_per_row = (int)tpr;
    void (*kernel)(CoeffArgs) = nullptr;
#define HILORE_PICK(V)                                                                                                  \
    kernel = kl ? (extra ? grpo_coeffs_kernel<true, true, V> : grpo_coeffs_kernel<true, false, V>)                      \
                : (extra ? grpo_coeffs_kernel<false, true, V> : grpo_coeffs_kernel<false, false, V>)
    if (variant == 0) { HILORE_PICK(0); }
    else if (variant == 1) { HILORE_PICK(1); }
    else { HILORE_PICK(2); }
#undef HILORE_PICK
    cfg.gridDim = dim3((unsigned)tiles);
    if (cudaLaunchKernelEx(&cfg, kernel, a) != cudaSuccess)
        return HILORE_CUDA;
    return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
}

extern "C" int hilore_grpo_coeffs(const float *rewards, int64_t n_resp_total, int32_t G, int64_t resp_offset,
                                  int64_t n_rows, int64_t T, const float *logp_new, const float *logp_old,
                                  const float *logp_ref, const uint8_t *mask, int64_t N_norm,
                                  const int64_t *N_norm_dev, float clip_eps, float beta, float adv_eps,
                                  float *adv_out, float *omega, float *ratio, uint8_t *clip_mask, void *stream)
{
    return launch_coeffs(rewards, n_resp_total, G, resp_offset, n_rows, T, logp_new, logp_old, logp_ref, mask, N_norm,
                         N_norm_dev, clip_eps, beta, adv_eps, 0, adv_out, omega, ratio, clip_mask, stream);
}

extern "C" int hilore_grpo_coeffs_variant(const float *rewards, int64_t n_resp_total, int32_t G, int64_t resp_offset,
                                          int64_t n_rows, int64_t T, const float *logp_new, const float *logp_old,
                                          const float *logp_ref, const uint8_t *mask, int64_t N_norm,
                                          const int64_t *N_norm_dev, float clip_eps, float beta, float adv_eps,
                                          int32_t variant, float *adv_out, float *omega, float *ratio, uint8_t *clip_mask,
                                          void *stream)
{
    return launch_coeffs(rewards, n_resp_total, G, resp_offset, n_rows, T, logp_new, logp_old, logp_ref, mask, N_norm,
                         N_norm_dev, clip_eps, beta, adv_eps, variant, adv_out, omega, ratio, clip_mask, stream);
}

extern "C" size_t hilore_workspace_bytes(int32_t U, int64_t n_tok)
{
    if (U < 0 || n_tok < 0)
        return 0;
    const int64_t ntiles = (n_tok + kExpTile - 1) / kExpTile;
    return (size_t)(U + 1) * (size_t)(ntiles > 0 ? ntiles : 1) * 2 * sizeof(double);
}

// Whether `kernel` may be launched with clusters of `size` CTAs on the current device (sizes above 8 need an opt-in
// and enough SMs per GPC); asked once per kernel, size and device.
template <typename K> static bool cluster_launch_ok(K kernel, int size)
{
    static std::mutex mu;
    static struct { const void *k; int size, dev, ok; } seen[64];
    static int n_seen = 0;
    const int dev = current_device();
    const void *key = reinterpret_cast<const void *>(kernel);
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < n_seen; ++i)
        if (seen[i].k == key && seen[i].size == size && seen[i].dev == dev)
            return seen[i].ok != 0;
    int ok = 1;
    if (size > 8 && cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
        ok = 0;
    if (ok) {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)size, 1);
        cfg.blockDim = dim3(kExpThreads);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)size;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg) != cudaSuccess || clusters < 1)
            ok = 0;
    }
    (void)cudaGetLastError();
    if (n_seen < 64)
        seen[n_seen++] = {key, size, dev, ok};
    return ok != 0;
}

// Single-launch form: partial sums of the U units and one row of token sums per unit group, then the counters.
static size_t scores_plan_partial_bytes(int32_t U, int64_t n_tok)
{
    const int64_t ntiles = (n_tok + kExpTile - 1) / kExpTile;
    const size_t groups = ((size_t)U + kExpUnits - 1) / kExpUnits;
    return ((size_t)U + groups) * (size_t)(ntiles > 0 ? ntiles : 1) * 2 * sizeof(double);
}
extern "C" size_t hilore_scores_plan_workspace_bytes(int32_t U, int64_t n_tok);

// fused: compute omega inside the reduction (hilore_coeffs_exposure); *fused_done tells the caller whether that was
// possible for this shape (otherwise nothing has been launched and the caller runs the two passes in turn).
static int launch_exposure(const float *omega, const uint8_t *mask, int64_t n_rows, int64_t T, int64_t n_tok,
                           const int32_t *cu, int64_t n_seq, const float *row_rms, int32_t U, int64_t rms_ld,
                           int32_t row_shift, float eps_alpha, float *exposure, float *sum_abs_omega, void *workspace,
                           size_t workspace_bytes, void *stream, const FusedCoeff *fused = nullptr, bool *fused_done = nullptr,
                           const PlanTail *plan = nullptr, bool single_launch = false)
{
    if (n_rows < 0 || T < 0 || n_tok < 0 || U < 0 || row_shift < 0 || row_shift > 1)
        return HILORE_INVALID_ARG;
    if (U == 0)
        return HILORE_OK;
    if (exposure == nullptr || row_rms == nullptr || workspace == nullptr)
        return HILORE_INVALID_ARG;
    if (n_tok > 0 && (omega == nullptr || mask == nullptr))
        return HILORE_INVALID_ARG;
    if (rms_ld < n_tok)
        return HILORE_SHAPE;
    if (!aligned(workspace, 16) || !aligned(omega, 4) || !aligned(row_rms, 4) || !aligned(exposure, 4) ||
        !aligned(sum_abs_omega, 4) || !aligned(cu, 4))
        return HILORE_ALIGN;
    const size_t part_bytes = single_launch ? scores_plan_partial_bytes(U, n_tok) : hilore_workspace_bytes(U, n_tok);
    if (workspace_bytes < (single_launch ? hilore_scores_plan_workspace_bytes(U, n_tok) : part_bytes))
        return HILORE_WORKSPACE;
    const int64_t pieces = (n_tok + kExpTile - 1) / kExpTile;
    const int64_t groups = (U + kExpUnits - 1) / kExpUnits;
    if (pieces > 0x7FFFFFFF || groups > 65535)
        return HILORE_SHAPE;
    // pieces per CTA: as many (up to 8) as still leave two full waves of CTAs
    int steps = 1;
    while (steps < 8 && (pieces / (2 * steps)) * groups >= 2ll * sm_count() * 8)
        steps *= 2;
    const int64_t ntiles64 = (pieces + steps - 1) / steps;
    if (fused) { // a CTA keeps the scalars of the responses its slots span in shared memory; recomputing omega in
                 // every unit group only pays while the call is launch-bound
        const bool ok = T > 0 && ((int64_t)steps * kExpTile) / T + 2 <= kFusedRows && n_tok <= (1ll << 18);
        *fused_done = ok;
        if (!ok)
            return HILORE_OK;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ExpArgs a{};
    if (fused) a.f = *fused;
    a.omega = omega;
    a.mask = mask;
    a.n_rows = n_rows;
    a.T = T;
    a.n_tok = n_tok;
    a.row_rms = row_rms;
    a.U = U;
    a.rms_ld = rms_ld;
    a.row_shift = row_shift;
    a.part = static_cast<double *>(workspace);
    a.ntiles = (int)ntiles64;
    a.cu = cu;
    a.n_seq = (int)n_seq;
    a.steps = steps;
    a.eps_alpha = eps_alpha;
    a.exposure = exposure;
    a.sum_abs_omega = sum_abs_omega;
    // Microbatch sizes (up to 16 tiles): one thread-block cluster per unit group, one CTA per tile, reduction through
    // the cluster's shared memory; no counters, no memset.  More tiles (or a device that refuses the launch) take the
    // forms below.
    // Every caller of the reduction takes this form at these sizes (it needs no workspace and no second launch).
    // HILORE_DISABLE_CLUSTER_LAUNCH in the environment (any value but "0") sends every call through the workspace
    // forms instead: same bits, for comparing the forms and for tools that cannot follow cluster launches.
    const char *no_cluster = std::getenv("HILORE_DISABLE_CLUSTER_LAUNCH");
    const bool clusters_on = no_cluster == nullptr || no_cluster[0] == '\0' || (no_cluster[0] == '0' && no_cluster[1] == '\0');
    // A tile count that is not a power of two takes the next one: the CTAs beyond the last tile add zeros.
    int csize = 1;
    while (csize < a.ntiles) csize *= 2;
    if (clusters_on && a.ntiles >= 1 && a.ntiles <= kMaxClusterTiles && steps == 1) {
        const bool vec = row_shift == 0 && (n_tok % 4 == 0) && (rms_ld % 4 == 0) && aligned(omega, 16) &&
                         aligned(mask, 4) && aligned(row_rms, 16);
        void (*kernel)(ExpArgs) = nullptr;
        if (fused) {
            const bool fvec = vec && aligned(fused->logp_new, 16) && aligned(fused->logp_old, 16) && aligned(fused->logp_ref, 16) &&
                              aligned(fused->omega_out, 16);
            kernel = fvec ? exposure_partial_kernel<true, true> : exposure_partial_kernel<false, true>;
        } else {
            kernel = vec ? exposure_partial_kernel<true, false> : exposure_partial_kernel<false, false>;
        }
        if (cluster_launch_ok(kernel, csize)) {
            a.cluster = 1;
            if (plan) a.plan = *plan;
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3((unsigned)csize, (unsigned)groups);
            cfg.blockDim = dim3(kExpThreads);
            cfg.stream = st;
            cudaLaunchAttribute attr[2];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = (unsigned)csize;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[1].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 2;
            if (cudaLaunchKernelEx(&cfg, kernel, a) == cudaSuccess && cudaGetLastError() == cudaSuccess)
                return HILORE_OK;
            (void)cudaGetLastError(); // refused: fall through to the counter form
            a.cluster = 0;
        }
    }
    if (single_launch && a.ntiles > 0) { // the counter of finished CTAs sits behind the partials and starts at zero
        a.done = reinterpret_cast<unsigned int *>(static_cast<unsigned char *>(workspace) + part_bytes);
        if (plan) a.plan = *plan;
        if (cudaMemsetAsync(a.done, 0, sizeof(unsigned int) * (size_t)groups, st) != cudaSuccess)
            return HILORE_CUDA;
    }
    if (a.ntiles > 0) {
        const dim3 grid((unsigned)a.ntiles, (unsigned)((U + kExpUnits - 1) / kExpUnits));
        const bool vec = row_shift == 0 && (n_tok % 4 == 0) && (rms_ld % 4 == 0) && aligned(omega, 16) &&
                         aligned(mask, 4) && aligned(row_rms, 16);
        void (*kernel)(ExpArgs) = nullptr;
        if (fused) {
            const bool fvec = vec && aligned(fused->logp_new, 16) && aligned(fused->logp_old, 16) && aligned(fused->logp_ref, 16) &&
                              aligned(fused->omega_out, 16);
            kernel = fvec ? exposure_partial_kernel<true, true> : exposure_partial_kernel<false, true>;
        } else {
            kernel = vec ? exposure_partial_kernel<true, false> : exposure_partial_kernel<false, false>;
        }
        if (launch_dependent(kernel, grid, dim3(kExpThreads), 0, st, a) != cudaSuccess || cudaGetLastError() != cudaSuccess)
            return HILORE_CUDA;
    }
    if (a.done != nullptr) // the partial kernel's last CTA has finished the reduction (and the plan)
        return HILORE_OK;
    if (launch_dependent(exposure_final_kernel, dim3((unsigned)U), dim3(32), 0, st, (const double *)a.part, (int)U, a.ntiles, eps_alpha,
                         exposure, sum_abs_omega) != cudaSuccess)
        return HILORE_CUDA;
    return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
}

extern "C" int hilore_unit_exposure(const float *omega, const uint8_t *mask, int64_t n_rows, int64_t T,
                                    const float *row_rms, int32_t U, int64_t rms_ld, int32_t row_shift,
                                    float eps_alpha, float *exposure, float *sum_abs_omega, void *workspace,
                                    size_t workspace_bytes, void *stream)
{
    if (n_rows < 0 || T < 0)
        return HILORE_INVALID_ARG;
    return launch_exposure(omega, mask, n_rows, T, n_rows * T, nullptr, 0, row_rms, U, rms_ld, row_shift, eps_alpha,
                           exposure, sum_abs_omega, workspace, workspace_bytes, stream);
}

extern "C" int hilore_coeffs_exposure(const float *rewards, int64_t n_resp_total, int32_t G, int64_t resp_offset, int64_t n_rows,
                                      int64_t T, const float *logp_new, const float *logp_old, const float *logp_ref,
                                      const uint8_t *mask, int64_t N_norm, const int64_t *N_norm_dev, float clip_eps, float beta,
                                      float adv_eps, const float *row_rms, int32_t U, int64_t rms_ld, int32_t row_shift,
                                      float eps_alpha, float *omega, float *exposure, float *sum_abs_omega, void *workspace,
                                      size_t workspace_bytes, void *stream)
{
    // the argument rules of the two calls it stands for
    if (rewards == nullptr || n_resp_total < 0 || G <= 0 || resp_offset < 0 || n_rows < 0 || T < 0 || U < 0)
        return HILORE_INVALID_ARG;
    if (n_resp_total % G != 0 || resp_offset + n_rows > n_resp_total || T % 4 != 0)
        return HILORE_SHAPE;
    if (beta != 0.0f && logp_ref == nullptr)
        return HILORE_INVALID_ARG;
    if (N_norm_dev == nullptr && N_norm <= 0)
        return HILORE_ZERO_NORM;
    const int64_t n_tok = n_rows * T;
    if (n_tok > 0 && (logp_new == nullptr || logp_old == nullptr || mask == nullptr || omega == nullptr))
        return HILORE_INVALID_ARG;
    if (!aligned(logp_new, 16) || !aligned(logp_old, 16) || !aligned(logp_ref, 16) || !aligned(omega, 16) || !aligned(mask, 4) ||
        !aligned(rewards, 4) || !aligned(N_norm_dev, 8))
        return HILORE_ALIGN;
    FusedCoeff f{};
    f.rewards = rewards;
    f.G = G;
    f.resp_offset = resp_offset;
    f.logp_new = logp_new;
    f.logp_old = logp_old;
    f.logp_ref = beta != 0.0f ? logp_ref : nullptr;
    f.N_norm = N_norm;
    f.N_norm_dev = reinterpret_cast<const long long *>(N_norm_dev);
    f.clip_eps = clip_eps;
    f.beta = beta;
    f.adv_eps = adv_eps;
    f.omega_out = omega;
    bool fused_done = false;
    if (U > 0 && n_tok > 0) {
        const int st = launch_exposure(omega, mask, n_rows, T, n_tok, nullptr, 0, row_rms, U, rms_ld, row_shift, eps_alpha,
                                       exposure, sum_abs_omega, workspace, workspace_bytes, stream, &f, &fused_done);
        if (st != HILORE_OK || fused_done)
            return st;
    }
    // shapes the fused kernel does not take (and U = 0): the two passes one after the other
    const int st = launch_coeffs(rewards, n_resp_total, G, resp_offset, n_rows, T, logp_new, logp_old, logp_ref, mask, N_norm,
                                 N_norm_dev, clip_eps, beta, adv_eps, 0, nullptr, omega, nullptr, nullptr, stream);
    if (st != HILORE_OK)
        return st;
    return launch_exposure(omega, mask, n_rows, T, n_tok, nullptr, 0, row_rms, U, rms_ld, row_shift, eps_alpha, exposure,
                           sum_abs_omega, workspace, workspace_bytes, stream);
}

extern "C" size_t hilore_scores_plan_workspace_bytes(int32_t U, int64_t n_tok)
{
    if (U < 0 || n_tok < 0)
        return 0;
    const size_t groups = ((size_t)U + kExpUnits - 1) / kExpUnits;
    return scores_plan_partial_bytes(U, n_tok) + ((groups * sizeof(unsigned int) + 15) & ~(size_t)15);
}

extern "C" int hilore_scores_plan(const float *rewards, int64_t n_resp_total, int32_t G, int64_t resp_offset, int64_t n_rows,
                                  int64_t T, const float *logp_new, const float *logp_old, const float *logp_ref,
                                  const uint8_t *mask, int64_t N_norm, const int64_t *N_norm_dev, float clip_eps, float beta,
                                  float adv_eps, const float *row_rms, int32_t U, int64_t rms_ld, int32_t row_shift,
                                  float eps_alpha, float *omega, float *exposure, float *sum_abs_omega,
                                  const hilore_unit *units_dev, const float *kappa, const float *ebar, float tau_lo, float tau_hi,
                                  const uint8_t *avail, uint8_t *action_io, float *psi, uint8_t *recompute,
                                  uint64_t *retained_bytes, void *workspace, size_t workspace_bytes, void *stream)
{
    // the argument rules of the calls it stands for
    if (rewards == nullptr || n_resp_total < 0 || G <= 0 || resp_offset < 0 || n_rows < 0 || T < 0 || U <= 0)
        return HILORE_INVALID_ARG;
    if (n_resp_total % G != 0 || resp_offset + n_rows > n_resp_total || T % 4 != 0)
        return HILORE_SHAPE;
    if (beta != 0.0f && logp_ref == nullptr)
        return HILORE_INVALID_ARG;
    if (N_norm_dev == nullptr && N_norm <= 0)
        return HILORE_ZERO_NORM;
    const int64_t n_tok = n_rows * T;
    if (n_tok <= 0 || logp_new == nullptr || logp_old == nullptr || mask == nullptr || omega == nullptr)
        return HILORE_INVALID_ARG;
    if (units_dev == nullptr || kappa == nullptr || ebar == nullptr || avail == nullptr || action_io == nullptr)
        return HILORE_INVALID_ARG;
    if (!aligned(logp_new, 16) || !aligned(logp_old, 16) || !aligned(logp_ref, 16) || !aligned(omega, 16) || !aligned(mask, 4) ||
        !aligned(rewards, 4) || !aligned(N_norm_dev, 8) || !aligned(units_dev, 8) || !aligned(kappa, 4) || !aligned(ebar, 4) ||
        !aligned(psi, 4) || !aligned(retained_bytes, 8))
        return HILORE_ALIGN;
    FusedCoeff f{};
    f.rewards = rewards;
    f.G = G;
    f.resp_offset = resp_offset;
    f.logp_new = logp_new;
    f.logp_old = logp_old;
    f.logp_ref = beta != 0.0f ? logp_ref : nullptr;
    f.N_norm = N_norm;
    f.N_norm_dev = reinterpret_cast<const long long *>(N_norm_dev);
    f.clip_eps = clip_eps;
    f.beta = beta;
    f.adv_eps = adv_eps;
    f.omega_out = omega;
    PlanTail plan{};
    plan.units = units_dev;
    plan.kappa = kappa;
    plan.ebar = ebar;
    plan.tau_lo = tau_lo;
    plan.tau_hi = tau_hi;
    plan.avail = avail;
    plan.action_io = action_io;
    plan.psi = psi;
    plan.recompute = recompute;
    plan.retained_bytes = retained_bytes;
    bool fused_done = false;
    int st = launch_exposure(omega, mask, n_rows, T, n_tok, nullptr, 0, row_rms, U, rms_ld, row_shift, eps_alpha, exposure,
                             sum_abs_omega, workspace, workspace_bytes, stream, &f, &fused_done, &plan, true);
    if (st != HILORE_OK || fused_done)
        return st;
    // shapes the one-sweep kernel does not take: the coefficient pass, then the reduction and the plan in one launch
    st = launch_coeffs(rewards, n_resp_total, G, resp_offset, n_rows, T, logp_new, logp_old, logp_ref, mask, N_norm, N_norm_dev,
                       clip_eps, beta, adv_eps, 0, nullptr, omega, nullptr, nullptr, stream);
    if (st != HILORE_OK)
        return st;
    return launch_exposure(omega, mask, n_rows, T, n_tok, nullptr, 0, row_rms, U, rms_ld, row_shift, eps_alpha, exposure,
                           sum_abs_omega, workspace, workspace_bytes, stream, nullptr, nullptr, &plan, true);
}

extern "C" int hilore_unit_exposure_packed(const float *omega, const uint8_t *mask, int64_t n_tok,
                                           const int32_t *cu_seqlens, int64_t n_seq, const float *row_rms, int32_t U,
                                           int64_t rms_ld, int32_t row_shift, float eps_alpha, float *exposure,
                                           float *sum_abs_omega, void *workspace, size_t workspace_bytes, void *stream)
{
    if (n_tok < 0 || n_tok > 0x7FFFFFFF || n_seq < 0 || n_seq > 0x7FFFFFFE || (n_tok > 0 && (cu_seqlens == nullptr || n_seq == 0)))
        return HILORE_INVALID_ARG;
    return launch_exposure(omega, mask, 1, n_tok, n_tok, n_tok > 0 ? cu_seqlens : nullptr, n_seq, row_rms, U, rms_ld,
                           row_shift, eps_alpha, exposure, sum_abs_omega, workspace, workspace_bytes, stream);
}

extern "C" int hilore_grpo_coeffs_packed(const float *rewards, int64_t n_resp_total, int32_t G, int64_t resp_offset,
                                         int64_t n_seq, const int32_t *cu_seqlens, int64_t n_tok, const float *logp_new,
                                         const float *logp_old, const float *logp_ref, const uint8_t *mask,
                                         int64_t N_norm, const int64_t *N_norm_dev, float clip_eps, float beta,
                                         float adv_eps, float *adv_out, float *omega, float *ratio, uint8_t *clip_mask,
                                         void *stream)
{
    if (rewards == nullptr || n_resp_total < 0 || G <= 0 || resp_offset < 0 || n_seq < 0 || n_tok < 0)
        return HILORE_INVALID_ARG;
    if (n_resp_total % G != 0 || resp_offset + n_seq > n_resp_total || n_tok > 0x7FFFFFFF || n_seq > 0x7FFFFFFE)
        return HILORE_SHAPE;
    if (beta != 0.0f && logp_ref == nullptr)
        return HILORE_INVALID_ARG;
    if (N_norm_dev == nullptr && N_norm <= 0)
        return HILORE_ZERO_NORM;
    if (n_seq == 0)
        return n_tok == 0 ? HILORE_OK : HILORE_SHAPE;
    if (cu_seqlens == nullptr || adv_out == nullptr)
        return HILORE_INVALID_ARG;
    if (n_tok > 0 && (logp_new == nullptr || logp_old == nullptr || mask == nullptr || omega == nullptr))
        return HILORE_INVALID_ARG;
    if (!aligned(logp_new, 16) || !aligned(logp_old, 16) || !aligned(logp_ref, 16) || !aligned(omega, 16) ||
        !aligned(ratio, 16) || !aligned(mask, 4) || !aligned(clip_mask, 4) || !aligned(rewards, 4) ||
        !aligned(adv_out, 4) || !aligned(N_norm_dev, 8) || !aligned(cu_seqlens, 4))
        return HILORE_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t n_groups = (resp_offset + n_seq + G - 1) / G - resp_offset / G;
    if (launch_dependent(packed_advantage_kernel, dim3((unsigned)((n_groups + 3) / 4)), dim3(128), 0, st, rewards, resp_offset,
                         n_seq, (int)G, adv_eps, adv_out) != cudaSuccess || cudaGetLastError() != cudaSuccess)
        return HILORE_CUDA;
    if (n_tok == 0)
        return HILORE_OK;
    PackedArgs a{};
    a.cu = cu_seqlens;
    a.n_seq = (int)n_seq;
    a.n_tok = n_tok;
    a.adv = adv_out;
    a.logp_new = logp_new;
    a.logp_old = logp_old;
    a.logp_ref = (beta != 0.0f) ? logp_ref : nullptr;
    a.mask = mask;
    a.N_norm = N_norm;
    a.N_norm_dev = reinterpret_cast<const long long *>(N_norm_dev);
    a.clip_eps = clip_eps;
    a.beta = beta;
    a.omega = omega;
    a.ratio = ratio;
    a.clip_mask = clip_mask;
    const bool kl = beta != 0.0f, extra = (ratio != nullptr) || (clip_mask != nullptr);
    if (aligned(logp_new, 32) && aligned(logp_old, 32) && aligned(a.logp_ref, 32) && aligned(omega, 32) && aligned(ratio, 32) &&
        aligned(mask, 8) && aligned(clip_mask, 8)) { // the warp-tile kernel, as a programmatic dependent of the advantages
        const int64_t wtiles = (n_tok + kWarpTile - 1) / kWarpTile;
        const int64_t grid = (wtiles + kCoeffThreads / 32 - 1) / (kCoeffThreads / 32);
        void (*wk)(PackedArgs, uint32_t) =
            kl ? (extra ? grpo_coeffs_packed_warp_kernel<true, true> : grpo_coeffs_packed_warp_kernel<true, false>)
               : (extra ? grpo_coeffs_packed_warp_kernel<false, true> : grpo_coeffs_packed_warp_kernel<false, false>);
        if (launch_dependent(wk, dim3((unsigned)grid), dim3(kCoeffThreads), 0, st, a, (uint32_t)wtiles) != cudaSuccess)
            return HILORE_CUDA;
        return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
    }
    const int64_t tiles = (n_tok + kCoeffTile - 1) / kCoeffTile;
    void (*kernel)(PackedArgs) = kl ? (extra ? grpo_coeffs_packed_kernel<true, true> : grpo_coeffs_packed_kernel<true, false>)
                                    : (extra ? grpo_coeffs_packed_kernel<false, true> : grpo_coeffs_packed_kernel<false, false>);
    kernel<<<(unsigned)tiles, kCoeffThreads, 0, st>>>(a);
    return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
}

extern "C" const char *hilore_status_string(int status)
{
    switch (status) {
    case HILORE_OK: return "ok";
    case HILORE_INVALID_ARG: return "invalid argument";
    case HILORE_SHAPE: return "shape not supported";
    case HILORE_ALIGN: return "pointer or leading dimension misaligned";
    case HILORE_ZERO_NORM: return "normaliser N is not positive";
    case HILORE_CUDA: return "CUDA launch failed";
    case HILORE_WORKSPACE: return "workspace too small";
    default: return "unknown status";
    }
}

extern "C" int hilore_abi_version(void) { return 1000; }

// ------------------------------------------------------------------ exposure without caller scratch
// Some callers cannot hand over a workspace: a saved-tensor hook that runs while the framework's
// caching allocator must not be entered, a host that has given every byte of device memory to
// another pool, or a latency-critical loop in which cudaMalloc (which may synchronise the whole
// device) is forbidden.  For them the partial sums of the exposure reduction live in a fixed array
// that is part of the library image: every GPU context that loads the library holds these bytes
// until it exits.
#include <mutex>

namespace hilore {
constexpr size_t kStaticScratchBytes = size_t(1) << 20; // 1 MiB: (U + 1) * ceil(n_tok / 1024) <= 65536
static __device__ __align__(256) unsigned char g_exposure_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static std::mutex g_scratch_mutex;
static void *g_scratch_addr[kMaxDevices] = {};

// Device address of g_exposure_scratch on the current device.  In host code the array's name is only
// a handle for the runtime, not an address a kernel could use: the address is asked for once per
// device, with that device current, and cached.
static int static_scratch_address(void **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
        return HILORE_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_exposure_scratch) != cudaSuccess || p == nullptr)
            return HILORE_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return HILORE_OK;
}
} // namespace hilore

extern "C" size_t hilore_static_scratch_bytes(void) { return hilore::kStaticScratchBytes; }

extern "C" int hilore_unit_exposure_static(const float *omega, const uint8_t *mask, int64_t n_rows, int64_t T,
                                           const float *row_rms, int32_t U, int64_t rms_ld, int32_t row_shift,
                                           float eps_alpha, float *exposure, float *sum_abs_omega, void *stream)
{
    if (n_rows < 0 || T < 0 || U < 0)
        return HILORE_INVALID_ARG;
    if (hilore_workspace_bytes(U, n_rows * T) > hilore::kStaticScratchBytes)
        return HILORE_WORKSPACE; // beyond the built-in scratch: use hilore_unit_exposure with a workspace
    void *scratch = nullptr;
    const int st = hilore::static_scratch_address(&scratch);
    if (st != HILORE_OK)
        return st;
    return hilore_unit_exposure(omega, mask, n_rows, T, row_rms, U, rms_ld, row_shift, eps_alpha, exposure,
                                sum_abs_omega, scratch, hilore::kStaticScratchBytes, stream);
}
