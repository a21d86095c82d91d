/*
 * CPU oracle for the HiLoRe actor-update hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, scalar C that writes out what the paper defines, in the paper's
 * order and notation, in double precision wherever the paper does not fix the
 * precision.  It shares no code with the CUDA library and must never be called
 * from the product path: only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may load it.
 *
 * What is pinned by what (see tests/test_oracle_*.py):
 *   orc_group_advantages  closed forms for Bernoulli groups, hand-worked groups,
 *                         zero-sum / unit-variance invariants, equal-reward rule
 *   orc_grpo_coeffs       hand-worked slots of Eq. "update-coefficient", central
 *                         finite differences of orc_grpo_objective (Prop. 1),
 *                         the r = 1 special case, Remark 1 invariants
 *   orc_row_rms,
 *   orc_unit_exposure     mean-one weights, constant-|omega| closed form, scale
 *                         invariance, Cor. 1 (all-zero omega), brute force by hand
 *   orc_compress/recover  fmt RAW: the routine the paper names (torch's
 *                         float8_e4m3fn cast) on all 65 536 bf16 patterns and all
 *                         256 codes; nearest-grid-point brute force.
 *                         fmt BLK (E4M3FN or INT8 with per-block scale): the
 *                         block-scaled format is NOT in the paper (its codec is
 *                         unscaled); it is pinned by the worked block, by the
 *                         reduction to fmt RAW for power-of-two scales, by the
 *                         error bounds and by brute force -- "parity unpinned"
 *                         with respect to the paper itself.
 *   orc_plan              the availability table of Eq. "available-recovery-
 *                         actions" (exhaustive), hand example.  The threshold
 *                         rule that picks the desired action is NOT in the paper
 *                         (its allocator is a knapsack DP): "parity unpinned".
 *   orc_relative_error,
 *   orc_fit_kappa         e^L against NumPy fp64 norms and its expected size on Gaussian data; kappa
 *                         against a brute-force minimisation over a grid and exact lines
 *   orc_grpo_coeffs_variant, orc_omega_diagnostics   hand-worked record, identities of Remark 1 (beta = 0:
 *                         zero-omega slots = padding + zero-advantage + clipped), NumPy sort for the
 *                         top-decile share, closed forms for uniform / one-hot |omega|
 *   orc_grpo_coeffs_packed, orc_unit_exposure_packed   the dense functions above on the same tokens laid
 *                         out with padding (every valid token equal, bit for bit), hand-worked two-sequence
 *                         record, zero-length sequences, first-token rule of row_shift
 *   orc_allocate          the paper's allocator (knapsack DP on the conservative grid): exhaustive
 *                         enumeration of all 3^U assignments of the discretised problem, the
 *                         feasibility guarantee of upward rounding, the tie rules and the
 *                         boundary cases, on hand examples
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_OK 0
#define ORC_INVALID 1
#define ORC_SHAPE 2
#define ORC_ZERO_NORM 4

enum { FMT_E4M3FN_RAW = 0, FMT_E4M3FN_BLK = 1, FMT_INT8_BLK = 2 };
enum { ACT_R = 0, ACT_H = 1, ACT_L = 2 };

/* ------------------------------------------------------------------ bf16 */

static float bf16_value(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* fp32 -> bf16, round to nearest, ties to even; NaN -> quiet NaN keeping the sign. */
static uint16_t bf16_from_float(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u)
        return (uint16_t)(((u >> 16) & 0x8000u) | 0x7FC0u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* ------------------------------------------------- FP8 E4M3FN (1-4-3, bias 7) */
/* Grid: normal values (8+M) * 2^(E-10) for E = 1..15 (E = 15, M = 7 is NaN, so the
 * largest finite value is 448); subnormals M * 2^-9; no infinities.               */

static double e4m3fn_value(uint8_t code)
{
    int E = (code >> 3) & 0xF, M = code & 7;
    double v;
    if (E == 0xF && M == 7)
        return NAN;
    if (E == 0)
        v = ldexp((double)M, -9);
    else
        v = ldexp((double)(8 + M), E - 10);
    return (code & 0x80) ? -v : v;
}

/* Round |v| to the nearest grid point (ties to the even mantissa).  v finite.
 * Returns the 7-bit magnitude code, or 0x100 when the rounded value exceeds 448. */
static unsigned e4m3fn_round_magnitude(double a)
{
    if (a == 0.0)
        return 0;
    int ex;
    (void)frexp(a, &ex);           /* a = f * 2^ex, f in [0.5, 1)  =>  floor(log2 a) = ex - 1 */
    int e = ex - 1;
    if (e < -6)
        e = -6;                    /* subnormal binade shares the spacing of 2^-6 */
    double step = ldexp(1.0, e - 3);
    double n = nearbyint(a / step);    /* default rounding mode: ties to even; a/step is exact */
    double q = n * step;
    if (q > 448.0)
        return 0x100;
    if (q < ldexp(1.0, -6))
        return (unsigned)n;        /* E = 0, M = n  (n in 0..7) */
    (void)frexp(q, &ex);
    e = ex - 1;                    /* may have moved up one binade */
    unsigned M = (unsigned)(q / ldexp(1.0, e - 3)) - 8u;
    return ((unsigned)(e + 7) << 3) | M;
}

/* Encode one real value.  overflow_to_nan: 1 = values that round above 448 become
 * NaN (the behaviour of the cast the paper names), 0 = they saturate to +-448.
 * NaN input always becomes the NaN code; +-Inf follows the overflow rule.        */
static uint8_t e4m3fn_encode(double v, int overflow_to_nan)
{
    uint8_t sign = signbit(v) ? 0x80 : 0x00;
    if (isnan(v))
        return sign | 0x7F;
    unsigned m = isinf(v) ? 0x100u : e4m3fn_round_magnitude(fabs(v));
    if (m == 0x100u)
        m = overflow_to_nan ? 0x7Fu : 0x7Eu;
    return sign | (uint8_t)m;
}

/* ------------------------------------------------------------ a1: advantages */
/* Group-relative advantage: (R - mean) / (population std + eps); a group whose
 * rewards are all equal has advantage exactly zero (GRPO setup paragraph).       */
int orc_group_advantages(const float *rewards, int64_t n_resp, int32_t G, float adv_eps, float *adv)
{
    if (!rewards || !adv || n_resp < 0 || G <= 0)
        return ORC_INVALID;
    if (n_resp % G)
        return ORC_SHAPE;
    for (int64_t g = 0; g < n_resp / G; ++g) {
        const float *R = rewards + g * G;
        float lo = R[0], hi = R[0];
        for (int j = 1; j < G; ++j) {
            if (R[j] < lo) lo = R[j];
            if (R[j] > hi) hi = R[j];
        }
        if (lo == hi) {
            for (int j = 0; j < G; ++j)
                adv[g * G + j] = 0.0f;
            continue;
        }
        double mu = 0.0;
        for (int j = 0; j < G; ++j)
            mu += (double)R[j];
        mu /= (double)G;
        double var = 0.0;
        for (int j = 0; j < G; ++j)
            var += ((double)R[j] - mu) * ((double)R[j] - mu);
        var /= (double)G;
        double sigma = sqrt(var);
        for (int j = 0; j < G; ++j)
            adv[g * G + j] = (float)(((double)R[j] - mu) / (sigma + (double)adv_eps));
    }
    return ORC_OK;
}

/* ------------------------------------------------------ a2: coefficients omega */
/* Eq. "update-coefficient" with the K3 derivative of the proof of Prop. 1.
 * adv holds one advantage per row (response).  N_norm <= 0 => N = sum of mask.
 * The clip decision is taken on the fp32-rounded ratio against fp32 bounds
 * 1 +- clip_eps, inclusive exactly as printed.                                   */
int orc_grpo_coeffs(const float *adv, const float *logp_new, const float *logp_old, const float *logp_ref,
                    const uint8_t *mask, int64_t n_rows, int64_t T, int64_t N_norm, float clip_eps, float beta,
                    float *omega, float *ratio, uint8_t *clip_mask)
{
    if (!adv || !logp_new || !logp_old || !mask || !omega || n_rows < 0 || T < 0)
        return ORC_INVALID;
    if (beta != 0.0f && !logp_ref)
        return ORC_INVALID;
    int64_t N = N_norm;
    if (N <= 0) {
        N = 0;
        for (int64_t i = 0; i < n_rows * T; ++i)
            N += mask[i] ? 1 : 0;
    }
    if (N <= 0)
        return ORC_ZERO_NORM;
    const float hi = 1.0f + clip_eps, lo = 1.0f - clip_eps;
    for (int64_t i = 0; i < n_rows; ++i) {
        const float A = adv[i];
        for (int64_t t = 0; t < T; ++t) {
            int64_t k = i * T + t;
            double r = exp((double)logp_new[k] - (double)logp_old[k]);
            float r32 = (float)r;
            int chi = (A >= 0.0f && r32 <= hi) || (A < 0.0f && r32 >= lo);
            double m = mask[k] ? 1.0 : 0.0;
            double w = -(m / (double)N) * (chi ? 1.0 : 0.0) * r * (double)A;
            if (beta != 0.0f)
                w += (double)beta * (m / (double)N) * (1.0 - exp((double)logp_ref[k] - (double)logp_new[k]));
            omega[k] = (float)w;
            if (ratio) ratio[k] = r32;
            if (clip_mask) clip_mask[k] = (uint8_t)chi;
        }
    }
    return ORC_OK;
}

/* Eq. "grpo-objective" plus beta times the K3 regulariser, with s in double so that a
 * test can difference it.  Used only to pin omega = dL/ds (Prop. 1).              */
double orc_grpo_objective(const float *adv, const double *s, const float *logp_old, const float *logp_ref,
                          const uint8_t *mask, int64_t n_rows, int64_t T, int64_t N, float clip_eps, float beta)
{
    const double hi = (double)(1.0f + clip_eps), lo = (double)(1.0f - clip_eps);
    double L = 0.0;
    for (int64_t i = 0; i < n_rows; ++i)
        for (int64_t t = 0; t < T; ++t) {
            int64_t k = i * T + t;
            if (!mask[k])
                continue;
            double r = exp(s[k] - (double)logp_old[k]);
            double rc = r < lo ? lo : (r > hi ? hi : r);
            double a = r * (double)adv[i], b = rc * (double)adv[i];
            L -= (a < b ? a : b) / (double)N;
            if (beta != 0.0f) {
                double d = (double)logp_ref[k] - s[k];
                L += (double)beta * (exp(d) - d - 1.0) / (double)N;
            }
        }
    return L;
}

/* ----------------------------------------------- a3: tokenwise activation RMS */
/* a_t = sqrt(mean_j X_{t,j}^2), Eq. "activation-token-weights" (left part).     */
int orc_row_rms(const uint16_t *x, int64_t rows, int64_t cols, int64_t ld, float *rms)
{
    if (!x || !rms || rows < 0 || cols <= 0)
        return ORC_INVALID;
    if (ld < cols)
        return ORC_SHAPE;
    for (int64_t r = 0; r < rows; ++r) {
        double acc = 0.0;
        for (int64_t j = 0; j < cols; ++j) {
            double v = (double)bf16_value(x[r * ld + j]);
            acc += v * v;
        }
        rms[r] = (float)sqrt(acc / (double)cols);
    }
    return ORC_OK;
}

/* ------------------------------------------------------ a4: update exposure */
/* alpha_t = (a_t + eps) / (mean_{s in T_b} a_s + eps);  E_u = sum_{t in T_b} |omega_t| alpha_t
 * (Eqs. "activation-token-weights", "mlp-weighted-exposure").  T_b = slots with mask = 1.
 * The activation row of slot (i, t) is (i, t - row_shift); a slot whose row would lie before the start of
 * its response carries no weight: it counts neither in the mean nor in E_u (so the weights of the slots
 * that do have a row average to one, as Eq. "activation-token-weights" requires).  No such slot => E_u = 0. */
int orc_unit_exposure(const float *omega, const uint8_t *mask, int64_t n_rows, int64_t T, const float *row_rms,
                      int32_t U, int64_t rms_ld, int32_t row_shift, float eps_alpha, float *exposure,
                      float *sum_abs_omega)
{
    if (!omega || !mask || !row_rms || !exposure || n_rows < 0 || T < 0 || U < 0)
        return ORC_INVALID;
    if (row_shift < 0 || row_shift > 1)
        return ORC_INVALID;
    if (rms_ld < n_rows * T)
        return ORC_SHAPE;
    int64_t cnt = 0; /* tokens of T_b that have an activation row: the weights average to one over these */
    double sw = 0.0;
    for (int64_t i = 0; i < n_rows; ++i)
        for (int64_t t = 0; t < T; ++t)
            if (mask[i * T + t]) {
                if (t - row_shift >= 0)
                    ++cnt;
                sw += fabs((double)omega[i * T + t]);
            }
    if (sum_abs_omega)
        *sum_abs_omega = (float)sw;
    for (int32_t u = 0; u < U; ++u) {
        const float *a = row_rms + (int64_t)u * rms_ld;
        if (cnt == 0) {
            exposure[u] = 0.0f;
            continue;
        }
        double abar = 0.0;
        for (int64_t i = 0; i < n_rows; ++i)
            for (int64_t t = 0; t < T; ++t)
                if (mask[i * T + t] && t - row_shift >= 0)
                    abar += (double)a[i * T + t - row_shift];
        abar /= (double)cnt;
        double E = 0.0;
        for (int64_t i = 0; i < n_rows; ++i)
            for (int64_t t = 0; t < T; ++t)
                if (mask[i * T + t] && t - row_shift >= 0) {
                    double alpha = ((double)a[i * T + t - row_shift] + (double)eps_alpha) / (abar + (double)eps_alpha);
                    E += fabs((double)omega[i * T + t]) * alpha;
                }
        exposure[u] = (float)E;
    }
    return ORC_OK;
}

/* ---------------------------------------------------------- a5 / a6: codec */
/* fmt RAW: Eq. "fp8-roundtrip" -- code = cast_E4M3FN(x) exactly as the named cast does
 *          it (single RNE rounding, overflow and non-finite inputs become NaN).
 * fmt BLK: per block of `block` consecutive elements of a row:
 *          amax = max |x_i| over the finite elements; if amax == 0 or the block has no
 *          finite element, s = inv = 1; else s = fl32(amax / Q), inv = fl32(Q / amax)
 *          with Q = 448 (E4M3FN) or 127 (INT8) (and s = inv = 1 if Q / amax overflows);  q_i = fl32(fl32(x_i) * inv);
 *          E4M3FN: code_i = RNE(q_i) saturating at +-448; INT8: code_i = RNE(q_i) clamped
 *          to +-127.  NaN input -> NaN code (sign|0x7F, resp. 0x80); +-Inf saturates.   */

static int finite_bf16(uint16_t b) { return (b & 0x7F80u) != 0x7F80u; }

int orc_compress(const uint16_t *x, int64_t rows, int64_t cols, int64_t ld, int32_t fmt, int32_t block,
                 uint8_t *codes, float *scales)
{
    if (!x || !codes || rows < 0 || cols <= 0)
        return ORC_INVALID;
    if (ld < cols)
        return ORC_SHAPE;
    if (fmt == FMT_E4M3FN_RAW) {
        for (int64_t r = 0; r < rows; ++r)
            for (int64_t j = 0; j < cols; ++j)
                codes[r * cols + j] = e4m3fn_encode((double)bf16_value(x[r * ld + j]), 1);
        return ORC_OK;
    }
    if (fmt != FMT_E4M3FN_BLK && fmt != FMT_INT8_BLK)
        return ORC_INVALID;
    if (block <= 0 || !scales)
        return ORC_INVALID;
    if (cols % block)
        return ORC_SHAPE;
    const float Q = (fmt == FMT_E4M3FN_BLK) ? 448.0f : 127.0f;
    const int64_t nb = cols / block;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t b = 0; b < nb; ++b) {
            const uint16_t *xb = x + r * ld + b * block;
            float amax = 0.0f;
            for (int i = 0; i < block; ++i)
                if (finite_bf16(xb[i])) {
                    float a = fabsf(bf16_value(xb[i]));
                    if (a > amax) amax = a;
                }
            float s = 1.0f, inv = 1.0f;
            if (amax > 0.0f) {
                s = amax / Q;
                inv = Q / amax;
                if (isinf(inv)) {          /* amax so small that Q / amax overflows fp32 */
                    s = 1.0f;
                    inv = 1.0f;
                }
            }
            scales[r * nb + b] = s;
            for (int i = 0; i < block; ++i) {
                float xv = bf16_value(xb[i]);
                float q = xv * inv;
                uint8_t c;
                if (fmt == FMT_E4M3FN_BLK) {
                    c = e4m3fn_encode((double)q, 0);
                } else if (isnan(q)) {
                    c = 0x80;
                } else {
                    double n = nearbyint((double)q);
                    if (n > 127.0) n = 127.0;
                    if (n < -127.0) n = -127.0;
                    c = (uint8_t)(int8_t)n;
                }
                codes[r * cols + b * block + i] = c;
            }
        }
    return ORC_OK;
}

/* Recover: RAW: x_hat = cast_BF16(code) (exact; NaN code -> bf16 quiet NaN).
 * BLK: x_hat = bf16_rne(fl32(value(code) * s)).                                 */
int orc_recover(const uint8_t *codes, const float *scales, int64_t rows, int64_t cols, int32_t fmt, int32_t block,
                uint16_t *out, int64_t ld_out)
{
    if (!codes || !out || rows < 0 || cols <= 0)
        return ORC_INVALID;
    if (ld_out < cols)
        return ORC_SHAPE;
    if (fmt == FMT_E4M3FN_RAW) {
        for (int64_t r = 0; r < rows; ++r)
            for (int64_t j = 0; j < cols; ++j)
                out[r * ld_out + j] = bf16_from_float((float)e4m3fn_value(codes[r * cols + j]));
        return ORC_OK;
    }
    if (fmt != FMT_E4M3FN_BLK && fmt != FMT_INT8_BLK)
        return ORC_INVALID;
    if (block <= 0 || !scales)
        return ORC_INVALID;
    if (cols % block)
        return ORC_SHAPE;
    const int64_t nb = cols / block;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t j = 0; j < cols; ++j) {
            uint8_t c = codes[r * cols + j];
            float v;
            if (fmt == FMT_E4M3FN_BLK)
                v = (float)e4m3fn_value(c);
            else
                v = (c == 0x80) ? NAN : (float)(int8_t)c;
            float s = scales[r * nb + j / block];
            float y = v * s;
            out[r * ld_out + j] = bf16_from_float(y);
        }
    return ORC_OK;
}

/* Pre-rounding reconstruction fl32(value(code) * s), for the error-bound pins. */
int orc_dequant_f32(const uint8_t *codes, const float *scales, int64_t rows, int64_t cols, int32_t fmt,
                    int32_t block, float *out)
{
    if (!codes || !out || rows < 0 || cols <= 0)
        return ORC_INVALID;
    const int64_t nb = (fmt == FMT_E4M3FN_RAW) ? 0 : cols / block;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t j = 0; j < cols; ++j) {
            uint8_t c = codes[r * cols + j];
            float v = (fmt == FMT_INT8_BLK) ? ((c == 0x80) ? NAN : (float)(int8_t)c) : (float)e4m3fn_value(c);
            float s = (fmt == FMT_E4M3FN_RAW) ? 1.0f : scales[r * nb + j / block];
            out[r * cols + j] = v * s;
        }
    return ORC_OK;
}

/* Calibration statistic e^L = ||x_hat - x||_2 / (||x||_2 + 1e-8), operands widened before the
 * subtraction and the norms (Eq. "app-calibration-error", left part).            */
double orc_relative_error(const uint16_t *x, const uint16_t *xhat, int64_t rows, int64_t cols, int64_t ld,
                          int64_t ld_hat)
{
    double num = 0.0, den = 0.0;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t j = 0; j < cols; ++j) {
            double a = (double)bf16_value(x[r * ld + j]);
            double b = (double)bf16_value(xhat[r * ld_hat + j]);
            num += (b - a) * (b - a);
            den += a * a;
        }
    return sqrt(num) / (sqrt(den) + 1e-8);
}

/* ------------------------------------------------------- a7: risk and gating */
/* psi_u = kappa_u * E_u * ebar_u (Eq. "token-weighted-risk"), evaluated in fp32 as
 * fl32(fl32(kappa * E) * ebar).  Desired action by thresholds (a stand-in for the
 * paper's knapsack allocator): psi < tau_lo -> L, psi >= tau_hi -> H, else R; NaN -> R.
 * If exposure is NULL the desired action is action_io[u] as given.
 * Availability (Eq. "available-recovery-actions"): q = H allows {H, L, R}, q = L allows
 * {L, R}, q = R allows {R}; a desired action that is not available becomes R.
 * retained_bytes: H keeps rows*cols*2, L keeps rows*cols (+ 4 bytes per block when
 * scaled), R keeps nothing.                                                      */
int orc_plan(const float *exposure, const float *kappa, const float *ebar, int32_t U, float tau_lo, float tau_hi,
             const uint8_t *avail, const int64_t *rows, const int64_t *cols, const int32_t *fmt,
             const int32_t *block, uint8_t *action_io, float *psi, uint8_t *recompute, uint64_t *retained_bytes)
{
    if (U < 0 || !avail || !action_io)
        return ORC_INVALID;
    if (exposure && (!kappa || !ebar))
        return ORC_INVALID;
    for (int32_t u = 0; u < U; ++u) {
        uint8_t want = action_io[u];
        if (exposure) {
            float t = kappa[u] * exposure[u];
            float p = t * ebar[u];
            if (psi) psi[u] = p;
            if (p < tau_lo) want = ACT_L;
            else if (p >= tau_hi) want = ACT_H;
            else want = ACT_R;          /* also reached when p is NaN */
        }
        if (want > ACT_L || avail[u] > ACT_L)
            return ORC_INVALID;
        int ok = (avail[u] == ACT_H) || (avail[u] == ACT_L && want != ACT_H) || (want == ACT_R);
        uint8_t a = ok ? want : ACT_R;
        action_io[u] = a;
        if (recompute) recompute[u] = (a == ACT_R);
        if (retained_bytes) {
            uint64_t n = (uint64_t)rows[u] * (uint64_t)cols[u];
            if (a == ACT_H) retained_bytes[u] = 2u * n;
            else if (a == ACT_L) retained_bytes[u] = n + ((fmt[u] == FMT_E4M3FN_RAW) ? 0u : 4u * (n / (uint64_t)block[u]));
            else retained_bytes[u] = 0;
        }
    }
    return ORC_OK;
}

/* ---------------------------------------------- joint H/L/R allocation (two-constraint knapsack) */
/* The paper's allocator (Appendix "Joint Allocation and Schedule Validation"): maximise sum_u dtau_u(a_u)
 * subject to sum_u dmem_u(a_u) <= M_res, sum_u d_u(a_u) <= delta_b with d(H) = d(R) = 0, d(L) = psi_u, and
 * a_u in A_u(q_u), solved exactly on a grid of N intervals per axis with costs rounded UP:
 *   h_B = M_res / N, h_d = delta_b / N, b_u(a) = ceil(dmem_u(a) / h_B), r_u(a) = ceil(d_u(a) / h_d);
 *   F_0(0,0) = 0, else -inf;  F_i(j,k) = max over available a with b <= j, r <= k of
 *   F_{i-1}(j - b, k - r) + dtau_i(a), candidates tried in the order R, H, L (the first maximum wins);
 *   terminal state: the largest F_U(j,k); ties go to the lower risk state k, then the lower memory state j.
 * Boundary cases: M_res == 0 leaves one memory state (only actions without memory cost);
 * delta_b == 0 disables L and leaves one risk state.  R always has utility 0 and costs 0.
 * dtau, dmem: [U][3] indexed by the action code (R = 0, H = 1, L = 2); column R is ignored.
 * A NaN or negative psi makes L unavailable for that unit; negative memory costs count as 0.
 * Plain triple loop over (unit, j, k) with a full predecessor table: O(U * (N+1)^2) time and memory.
 * Pinned by exhaustive enumeration of all 3^U assignments (tests/test_oracle_allocate.py).           */
int orc_allocate(int32_t U, const float *psi, const double *dtau, const double *dmem, const uint8_t *avail,
                 double M_res, double delta_b, int32_t N, uint8_t *action, double *totals)
{
    if (U < 0 || N <= 0 || !psi || !dtau || !dmem || !avail || !action)
        return ORC_INVALID;
    if (!(M_res >= 0.0) || !(delta_b >= 0.0))
        return ORC_INVALID;
    const int KB = (M_res > 0.0) ? N + 1 : 1, KD = (delta_b > 0.0) ? N + 1 : 1;
    const double hB = M_res / (double)N, hD = delta_b / (double)N;
    const size_t S = (size_t)KB * (size_t)KD;
    int *bc = (int *)malloc(sizeof(int) * 3 * (size_t)(U > 0 ? U : 1));
    int *rc = (int *)malloc(sizeof(int) * 3 * (size_t)(U > 0 ? U : 1));
    double *F0 = (double *)malloc(sizeof(double) * S), *F1 = (double *)malloc(sizeof(double) * S);
    uint8_t *pred = (uint8_t *)malloc(S * (size_t)(U > 0 ? U : 1));
    if (!bc || !rc || !F0 || !F1 || !pred) {
        free(bc); free(rc); free(F0); free(F1); free(pred);
        return ORC_INVALID;
    }
    /* integer costs; -1 marks an action that cannot be taken */
    for (int u = 0; u < U; ++u) {
        if (avail[u] > ACT_L) {
            free(bc); free(rc); free(F0); free(F1); free(pred);
            return ORC_INVALID;
        }
        for (int a = 0; a < 3; ++a) {
            int ok = (a == ACT_R) || (avail[u] == ACT_H) || (avail[u] == ACT_L && a == ACT_L);
            double dm = (a == ACT_R) ? 0.0 : dmem[u * 3 + a];
            double d = (a == ACT_L) ? (double)psi[u] : 0.0;
            if (dm < 0.0) dm = 0.0;
            if (a == ACT_L && (!(d >= 0.0) || delta_b == 0.0)) ok = 0;   /* NaN / negative risk; zero budget */
            if (!(dm == dm)) ok = 0;
            long b = 0, r = 0;
            if (ok) {
                if (M_res > 0.0) b = (long)ceil(dm / hB); else if (dm > 0.0) ok = 0;
                if (delta_b > 0.0) r = (long)ceil(d / hD);
                if (b > N || r > N || b < 0 || r < 0) ok = 0;
            }
            bc[u * 3 + a] = ok ? (int)b : -1;
            rc[u * 3 + a] = ok ? (int)r : -1;
        }
    }
    for (size_t s = 0; s < S; ++s) F0[s] = -INFINITY;
    F0[0] = 0.0;
    for (int u = 0; u < U; ++u) {
        for (int j = 0; j < KB; ++j)
            for (int k = 0; k < KD; ++k) {
                double best = -INFINITY;
                uint8_t arg = 255;
                for (int a = 0; a < 3; ++a) {            /* order R, H, L: the first maximum wins */
                    int b = bc[u * 3 + a], r = rc[u * 3 + a];
                    if (b < 0 || b > j || r > k) continue;
                    double prev = F0[(size_t)(j - b) * KD + (k - r)];
                    if (prev == -INFINITY) continue;
                    double v = prev + ((a == ACT_R) ? 0.0 : dtau[u * 3 + a]);
                    if (arg == 255 || v > best) {
                        best = v;
                        arg = (uint8_t)a;
                    }
                }
                F1[(size_t)j * KD + k] = best;
                pred[(size_t)u * S + (size_t)j * KD + k] = arg;
            }
        double *t = F0; F0 = F1; F1 = t;
    }
    /* terminal state: largest utility; ties: lower risk, then lower memory */
    int bj = 0, bk = 0;
    double bestF = -INFINITY;
    int have = 0;
    for (int k = 0; k < KD; ++k)
        for (int j = 0; j < KB; ++j) {
            double v = F0[(size_t)j * KD + k];
            if (v == -INFINITY) continue;
            if (!have || v > bestF) { bestF = v; bj = j; bk = k; have = 1; }
        }
    double tot_m = 0.0, tot_r = 0.0;
    int j = bj, k = bk;
    for (int u = U - 1; u >= 0; --u) {
        uint8_t a = pred[(size_t)u * S + (size_t)j * KD + k];
        if (a > ACT_L) a = ACT_R;                        /* cannot happen: R is always available */
        action[u] = a;
        j -= bc[u * 3 + a];
        k -= rc[u * 3 + a];
        if (a != ACT_R) tot_m += (dmem[u * 3 + a] < 0.0 ? 0.0 : dmem[u * 3 + a]);
        if (a == ACT_L) tot_r += (double)psi[u];
    }
    if (totals) { totals[0] = bestF; totals[1] = tot_m; totals[2] = tot_r; }
    free(bc); free(rc); free(F0); free(F1); free(pred);
    return ORC_OK;
}

/* Microbatch risk budget delta_b = delta * N_b / sum_b' N_b' (Appendix "Online Scheduling"). */
double orc_risk_budget(double delta, int64_t N_b, int64_t N_total)
{
    return (N_total > 0) ? delta * (double)N_b / (double)N_total : 0.0;
}

/* Susceptibility fit kappa_c = argmin_{kappa >= 0} sum (y - kappa x)^2 (Eq. "susceptibility"): the closed
 * form max(0, sum x y / sum x^2); 0 when every x is 0. */
double orc_fit_kappa(const double *x, const double *y, int64_t n)
{
    double sxy = 0.0, sxx = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        sxy += x[i] * y[i];
        sxx += x[i] * x[i];
    }
    if (!(sxx > 0.0))
        return 0.0;
    double k = sxy / sxx;
    return k > 0.0 ? k : 0.0;
}

/* ------------------------------------------------ packed (padding-removed) layout */
/* The padding-removal execution setting of the paper's DSR-sub configuration: the sequences of a microbatch
 * (prompt followed by response, no padding slots) lie back to back; sequence i owns tokens
 * cu_seqlens[i] .. cu_seqlens[i+1]-1 and carries the advantage of response i.  The arithmetic per token is
 * that of orc_grpo_coeffs; the mask now excludes prompt tokens only. */
int orc_grpo_coeffs_packed(const float *adv, const int32_t *cu_seqlens, int64_t n_seq, const float *logp_new,
                           const float *logp_old, const float *logp_ref, const uint8_t *mask, int64_t N_norm,
                           float clip_eps, float beta, float *omega, float *ratio, uint8_t *clip_mask)
{
    if (!adv || !cu_seqlens || n_seq < 0 || !logp_new || !logp_old || !mask || !omega)
        return ORC_INVALID;
    if (beta != 0.0f && !logp_ref)
        return ORC_INVALID;
    if (cu_seqlens[0] != 0)
        return ORC_SHAPE;
    for (int64_t i = 0; i < n_seq; ++i)
        if (cu_seqlens[i + 1] < cu_seqlens[i])
            return ORC_SHAPE;
    const int64_t n_tok = cu_seqlens[n_seq];
    int64_t N = N_norm;
    if (N <= 0) {
        N = 0;
        for (int64_t k = 0; k < n_tok; ++k) N += mask[k] ? 1 : 0;
    }
    if (N <= 0)
        return ORC_ZERO_NORM;
    const float hi = 1.0f + clip_eps, lo = 1.0f - clip_eps;
    for (int64_t i = 0; i < n_seq; ++i) {
        const float A = adv[i];
        for (int64_t k = cu_seqlens[i]; k < cu_seqlens[i + 1]; ++k) {
            double r = exp((double)logp_new[k] - (double)logp_old[k]);
            float r32 = (float)r;
            int chi = (A >= 0.0f && r32 <= hi) || (A < 0.0f && r32 >= lo);
            double m = mask[k] ? 1.0 : 0.0;
            double w = -(m / (double)N) * (chi ? 1.0 : 0.0) * r * (double)A;
            if (beta != 0.0f)
                w += (double)beta * (m / (double)N) * (1.0 - exp((double)logp_ref[k] - (double)logp_new[k]));
            omega[k] = (float)w;
            if (ratio) ratio[k] = r32;
            if (clip_mask) clip_mask[k] = (uint8_t)chi;
        }
    }
    return ORC_OK;
}

/* orc_unit_exposure on the packed layout: the activation row of token k is k - row_shift, taken only when it
 * lies inside the token's own sequence; a token without such a row carries no weight (see orc_unit_exposure). */
int orc_unit_exposure_packed(const float *omega, const uint8_t *mask, const int32_t *cu_seqlens, int64_t n_seq,
                             const float *row_rms, int32_t U, int64_t rms_ld, int32_t row_shift, float eps_alpha,
                             float *exposure, float *sum_abs_omega)
{
    if (!omega || !mask || !cu_seqlens || !row_rms || !exposure || n_seq < 0 || U < 0)
        return ORC_INVALID;
    if (row_shift < 0 || row_shift > 1)
        return ORC_INVALID;
    const int64_t n_tok = cu_seqlens[n_seq];
    if (rms_ld < n_tok)
        return ORC_SHAPE;
    int64_t cnt = 0; /* tokens of T_b whose activation row lies inside their own sequence */
    double sw = 0.0;
    for (int64_t i = 0; i < n_seq; ++i)
        for (int64_t k = cu_seqlens[i]; k < cu_seqlens[i + 1]; ++k)
            if (mask[k]) {
                if (k - row_shift >= cu_seqlens[i])
                    ++cnt;
                sw += fabs((double)omega[k]);
            }
    if (sum_abs_omega)
        *sum_abs_omega = (float)sw;
    for (int32_t u = 0; u < U; ++u) {
        const float *a = row_rms + (int64_t)u * rms_ld;
        if (cnt == 0) {
            exposure[u] = 0.0f;
            continue;
        }
        double abar = 0.0;
        for (int64_t i = 0; i < n_seq; ++i)
            for (int64_t k = cu_seqlens[i]; k < cu_seqlens[i + 1]; ++k)
                if (mask[k] && k - row_shift >= cu_seqlens[i])
                    abar += (double)a[k - row_shift];
        abar /= (double)cnt;
        double E = 0.0;
        for (int64_t i = 0; i < n_seq; ++i)
            for (int64_t k = cu_seqlens[i]; k < cu_seqlens[i + 1]; ++k)
                if (mask[k] && k - row_shift >= cu_seqlens[i]) {
                    double alpha = ((double)a[k - row_shift] + (double)eps_alpha) / (abar + (double)eps_alpha);
                    E += fabs((double)omega[k]) * alpha;
                }
        exposure[u] = (float)E;
    }
    return ORC_OK;
}

/* ------------------------------------------------ diagnostics and score variants on omega */
/* Score variants of the component ablations: bit 0 replaces chi_t r_t by 1 in the policy contribution
 * ("removing ratio/clipping"); bit 1 writes the advantage-only signal m_t A instead of omega (the summand of
 * the advantage-only exposure sum_t |A_t| alpha_t).  "Removing KL" is beta = 0.  Ratio and clip indicator are
 * reported as in orc_grpo_coeffs. */
int orc_grpo_coeffs_variant(const float *adv, const float *logp_new, const float *logp_old, const float *logp_ref,
                            const uint8_t *mask, int64_t n_rows, int64_t T, int64_t N_norm, float clip_eps, float beta,
                            int32_t variant, float *omega, float *ratio, uint8_t *clip_mask)
{
    int st = orc_grpo_coeffs(adv, logp_new, logp_old, logp_ref, mask, n_rows, T, N_norm, clip_eps, beta, omega, ratio,
                             clip_mask);
    if (st != ORC_OK || variant == 0)
        return st;
    int64_t N = N_norm;
    if (N <= 0) {
        N = 0;
        for (int64_t i = 0; i < n_rows * T; ++i) N += mask[i] ? 1 : 0;
    }
    for (int64_t i = 0; i < n_rows; ++i)
        for (int64_t t = 0; t < T; ++t) {
            int64_t k = i * T + t;
            double m = mask[k] ? 1.0 : 0.0;
            if (variant & 2) {
                omega[k] = (float)(m * (double)adv[i]);
                continue;
            }
            double w = -(m / (double)N) * (double)adv[i];               /* chi r -> 1 */
            if (beta != 0.0f)
                w += (double)beta * (m / (double)N) * (1.0 - exp((double)logp_ref[k] - (double)logp_new[k]));
            omega[k] = (float)w;
        }
    return ORC_OK;
}

static int cmp_desc_float(const void *a, const void *b)
{
    float x = *(const float *)a, y = *(const float *)b;
    return (x < y) - (x > y);
}

/* Structural sparsity of one record (diagnostic paragraph "Structural sparsity", Eq. "diagnostic-clipping"):
 * counts[0] = padding slots (m = 0); counts[1] = valid slots with zero advantage; counts[2] = valid slots with
 * nonzero advantage on a flat clipped branch, (A > 0 and r > 1 + eps) or (A < 0 and r < 1 - eps); counts[3] =
 * slots with omega == 0; counts[4] = all padded response slots (the common denominator).  top_share = share of
 * sum |omega| carried by the ceil(0.1 n) slots of largest |omega| (padding counts with zero coefficient). */
int orc_omega_diagnostics(const float *adv, const float *ratio, const uint8_t *mask, const float *omega, int64_t n_rows,
                          int64_t T, float clip_eps, int64_t *counts, double *top_share, double *sum_abs)
{
    if (!adv || !ratio || !mask || !omega || !counts || n_rows < 0 || T < 0)
        return ORC_INVALID;
    const int64_t n = n_rows * T;
    const float hi = 1.0f + clip_eps, lo = 1.0f - clip_eps;
    for (int c = 0; c < 5; ++c) counts[c] = 0;
    counts[4] = n;
    float *absw = (float *)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
    if (!absw)
        return ORC_INVALID;
    double total = 0.0;
    for (int64_t i = 0; i < n_rows; ++i)
        for (int64_t t = 0; t < T; ++t) {
            int64_t k = i * T + t;
            float A = adv[i], r = ratio[k];
            if (!mask[k]) counts[0]++;
            else if (A == 0.0f) counts[1]++;
            else if ((A > 0.0f && r > hi) || (A < 0.0f && r < lo)) counts[2]++;
            float w = mask[k] ? fabsf(omega[k]) : 0.0f;
            if (w == 0.0f) counts[3]++;
            absw[k] = w;
            total += (double)w;
        }
    qsort(absw, (size_t)n, sizeof(float), cmp_desc_float);
    int64_t kk = (n * 1 + 9) / 10;                     /* ceil(0.1 n) */
    double top = 0.0;
    for (int64_t i = 0; i < kk; ++i) top += (double)absw[i];
    free(absw);
    if (top_share) *top_share = total > 0.0 ? top / total : 0.0;
    if (sum_abs) *sum_abs = total;
    return ORC_OK;
}
