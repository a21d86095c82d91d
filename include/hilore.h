/*
 * hilore.h -- C ABI of the B200 (sm_100a) hot path of HiLoRe's GRPO actor update.
 *
 * Two parts (paper: Algorithm 1, lines "Coefficients", "Exposure", risk score, and the
 * capture / recovery of L units):
 *   1. the fused GRPO loss-coefficient pass and its reduction to one update-exposure score
 *      per recovery unit, available before backward (Prop. 1, Eq. "update-coefficient",
 *      Eq. "mlp-weighted-exposure");
 *   2. the low-precision store / recover path for saved bf16 activations
 *      (Eq. "fp8-roundtrip"), gated by the per-unit H / L / R plan
 *      (Eq. "available-recovery-actions").
 *
 * Conventions for every entry point
 *   - Returns an int status (HILORE_OK = 0).  Never throws, aborts or traps.
 *   - Every pointer is a DEVICE pointer owned by the caller, valid until the work enqueued
 *     by the call has finished, unless its comment says "host".
 *   - The library allocates nothing and keeps no data between calls (the one exception is stated at
 *     its declaration); it only remembers immutable device properties (SM count, CTAs per SM of its
 *     kernels) after the first call on a device.  Work is enqueued on `stream` (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream) and the call returns without synchronising.
 *     HILORE_CUDA reports a launch error seen by cudaGetLastError, nothing asynchronous.
 *   - Tensors are row-major.  bf16 tensors are passed as void* (16-bit patterns).
 *   - Output buffers must not overlap inputs or each other.
 *   - Optional pointers say "opt" and may be NULL.
 */
#ifndef HILORE_H
#define HILORE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ---- */
enum {
    HILORE_OK = 0,
    HILORE_INVALID_ARG = 1, /* NULL where data is required, negative size, unknown enum value          */
    HILORE_SHAPE = 2,       /* cols % 16 != 0, cols % block != 0, n_resp % G != 0, ld < cols, ...       */
    HILORE_ALIGN = 3,       /* a pointer or leading dimension misses the alignment stated below       */
    HILORE_ZERO_NORM = 4,   /* the normaliser N is not positive and no device-side N was given         */
    HILORE_CUDA = 5,        /* kernel launch failed                                                    */
    HILORE_WORKSPACE = 6    /* workspace too small; see hilore_workspace_bytes                         */
};

/* ---- storage formats of the L (compress) action ---- */
enum {
    HILORE_FMT_E4M3FN_RAW = 0, /* the paper's codec, Eq. "fp8-roundtrip": unscaled cast to FP8 E4M3FN,
                                  one byte per element, no scales; values that round above 448 and
                                  non-finite values become the NaN code, as the cast the paper names does */
    HILORE_FMT_E4M3FN_BLK = 1, /* E4M3FN payload + one fp32 absmax scale per block of 64 elements of a
                                  row (the benchmark's block-scaled generalisation; not in the paper)    */
    HILORE_FMT_INT8_BLK = 2    /* INT8 payload (+-127) + one fp32 absmax scale per block of 64            */
};
#define HILORE_BLOCK 64 /* the only block size of the scaled formats */

/* ---- recovery actions; the numeric order is the paper's tie order R, H, L ---- */
enum { HILORE_ACT_R = 0, HILORE_ACT_H = 1, HILORE_ACT_L = 2 };

/* ---- phases of hilore_plan_apply ---- */
enum {
    HILORE_PHASE_DECIDE = 0,  /* risk score, threshold rule, availability -> action / recompute / bytes  */
    HILORE_PHASE_CAPTURE = 1, /* forward-time capture by candidate plan q: q = L compress (+ token RMS),
                                 q = H token RMS only (bf16 kept), q = R nothing                          */
    HILORE_PHASE_ENCODE = 2,  /* post-forward encoding: units with q = H that were assigned L           */
    HILORE_PHASE_RECOVER = 3  /* backward-time recovery: units with action L are decoded to bf16         */
};

struct hilore_unit; /* one recovery unit of a microbatch; defined with hilore_plan_apply below */

const char *hilore_status_string(int status);
/* Version of this ABI (major * 1000 + minor). */
int hilore_abi_version(void);

/*
 * N = sum_t m_t, the learner's normaliser (Eq. "grpo-objective": N = sum of the update mask; the
 * setup section normalises by all valid response tokens of the complete rollout batch).
 *   mask   [n] u8, 0 or 1.            count  one int64 on the device, overwritten with the sum.
 * The sum is an integer, so the result does not depend on the order of the additions.
 */
int hilore_mask_count(const uint8_t *mask, int64_t n, int64_t *count, void *stream);

/*
 * Group-relative advantages and per-token update coefficients omega_t = dL/ds_t
 * (Eq. "grpo-objective", Eq. "update-coefficient", K3 derivative in the proof of Prop. 1):
 *     A_j     = (R_j - mean_g) / (population_std_g + adv_eps); a group whose rewards are all equal
 *               has A = +0 exactly (setup section, "GRPO and optimization")
 *     r_t     = exp(s_t - s_old_t)
 *     chi_t   = 1[(A >= 0 and r_t <= 1 + clip_eps) or (A < 0 and r_t >= 1 - clip_eps)]   (fp32 compare)
 *     omega_t = -(m_t / N) chi_t r_t A  +  beta (m_t / N) (1 - exp(s_ref_t - s_t))
 * Group statistics are evaluated in fp64 per response, the per-token part in fp32.
 *
 *   rewards      [n_resp_total] fp32; the G responses of prompt p are rewards[p*G .. p*G+G-1].
 *                n_resp_total % G must be 0 (HILORE_SHAPE).
 *   resp_offset, n_rows   this call covers responses [resp_offset, resp_offset + n_rows), a microbatch
 *                of the rollout batch; a prompt group may straddle two calls.
 *   logp_new, logp_old, logp_ref   [n_rows, T] fp32, 16-byte aligned; logp_ref may be NULL iff beta == 0.
 *   mask         [n_rows, T] u8 (0 / 1), 4-byte aligned.  T % 4 must be 0 (HILORE_SHAPE).  With T % 8 == 0, the fp32
 *                tensors 32-byte aligned and the byte tensors 8-byte aligned the call takes its fast path (256-bit
 *                accesses, one warp per 512 slots); the results do not depend on the path.
 *   N_norm, N_norm_dev   the normaliser N: if N_norm_dev (one int64 on the device, e.g. written by
 *                hilore_mask_count earlier on the same stream) is not NULL it is read by the kernel and
 *                N_norm is ignored; a device value <= 0 yields omega = 0 everywhere.  Otherwise N_norm
 *                (host value) must be > 0 (HILORE_ZERO_NORM).
 *   adv_out      opt [n_rows] fp32, advantage of each response of this call.
 *   omega        [n_rows, T] fp32, 16-byte aligned.  Masked slots get 0.
 *   ratio        opt [n_rows, T] fp32 (r_t as computed, also at masked slots), 16-byte aligned.
 *   clip_mask    opt [n_rows, T] u8 (chi_t), 4-byte aligned.
 */
int hilore_grpo_coeffs(const float *rewards, int64_t n_resp_total, int32_t G, int64_t resp_offset,
                       int64_t n_rows, int64_t T, const float *logp_new, const float *logp_old,
                       const float *logp_ref, const uint8_t *mask, int64_t N_norm,
                       const int64_t *N_norm_dev, float clip_eps, float beta, float adv_eps, float *adv_out,
                       float *omega, float *ratio, uint8_t *clip_mask, void *stream);

/*
 * hilore_grpo_coeffs followed by hilore_unit_exposure as ONE sweep (Algorithm 1, "coefficients" and "exposure"
 * lines; Eqs. "update-coefficient", "mlp-weighted-exposure"): the coefficients are computed inside the exposure
 * reduction instead of being written and read back, which saves launches and the round trip of omega when the
 * microbatch is small enough for the call to be launch-bound (n_rows * T <= 2^18 slots and at most 62 responses
 * per 1024 slots; other shapes run the two passes in turn inside this call).  Results are bit for bit those of
 * the two calls: omega [n_rows, T] (REQUIRED here, it is written either way), exposure [U], sum_abs_omega (opt).
 * Arguments, status codes and workspace as in the two calls; adv_out, ratio and clip_mask are not produced.
 */
int hilore_coeffs_exposure(const float *rewards, int64_t n_resp_total, int32_t G, int64_t resp_offset, int64_t n_rows,
                           int64_t T, const float *logp_new, const float *logp_old, const float *logp_ref,
                           const uint8_t *mask, int64_t N_norm, const int64_t *N_norm_dev, float clip_eps, float beta,
                           float adv_eps, const float *row_rms, int32_t U, int64_t rms_ld, int32_t row_shift,
                           float eps_alpha, float *omega, float *exposure, float *sum_abs_omega, void *workspace,
                           size_t workspace_bytes, void *stream);

/*
 * The score refresh of one microbatch in ONE kernel launch: hilore_coeffs_exposure followed by
 * hilore_plan_apply(HILORE_PHASE_DECIDE) (Algorithm 1, lines "coefficients", "exposure", risk score and allocation;
 * Eqs. "update-coefficient", "mlp-weighted-exposure", "token-weighted-risk", "available-recovery-actions").  The CTAs of
 * a group of eight units -- one per tile of 1024 tokens -- add their partial sums in the fixed order of the two-kernel
 * form and one of them takes the plan decisions of the group's units, so omega, exposure, psi, action_io, recompute and
 * retained_bytes are bit for bit those of the separate calls.  At microbatch size (up to 16 tiles of 1024 tokens;
 * the cluster is the next power of two) the CTAs of a group are one thread-block cluster and hand the sums to its
 * first CTA through distributed shared memory; otherwise through the workspace, the CTA that finishes last (a
 * counter per group, cleared by a memset inside the call) doing the rest.  Between forward and backward of a
 * microbatch this is one launch instead of four.
 *   Arguments as in hilore_coeffs_exposure (omega REQUIRED, U > 0, n_rows * T > 0) and in the DECIDE phase of
 *   hilore_plan_apply (units_dev, kappa, ebar, avail, action_io REQUIRED; psi, recompute, retained_bytes opt; the
 *   unit table is only read for rows, cols and fmt, on the device).
 *   workspace   at least hilore_scores_plan_workspace_bytes(U, n_rows * T) bytes, 16-byte aligned: the partial sums
 *               and, behind them, the counters of finished CTAs (unused by the cluster form).
 *   Microbatches beyond the one-sweep form's limits (see hilore_coeffs_exposure) run the coefficient pass first and
 *   then the reduction + plan launch.
 */
int hilore_scores_plan(const float *rewards, int64_t n_resp_total, int32_t G, int64_t resp_offset, int64_t n_rows,
                       int64_t T, const float *logp_new, const float *logp_old, const float *logp_ref,
                       const uint8_t *mask, int64_t N_norm, const int64_t *N_norm_dev, float clip_eps, float beta,
                       float adv_eps, const float *row_rms, int32_t U, int64_t rms_ld, int32_t row_shift,
                       float eps_alpha, float *omega, float *exposure, float *sum_abs_omega,
                       const struct hilore_unit *units_dev, const float *kappa, const float *ebar, float tau_lo,
                       float tau_hi, const uint8_t *avail, uint8_t *action_io, float *psi, uint8_t *recompute,
                       uint64_t *retained_bytes, void *workspace, size_t workspace_bytes, void *stream);
size_t hilore_scores_plan_workspace_bytes(int32_t U, int64_t n_tok);

/*
 * The coefficient and exposure passes on the packed (padding-removed) layout of the paper's DSR-sub execution
 * setting (Table "execution-configurations": "padding removal").  The sequences of a microbatch -- prompt
 * followed by the generated response, no padding slots -- lie back to back: sequence i (response
 * resp_offset + i of the rollout batch) owns tokens cu_seqlens[i] .. cu_seqlens[i+1]-1; the activation
 * tensors of the microbatch have one row per packed token.  Arithmetic per token exactly as in
 * hilore_grpo_coeffs / hilore_unit_exposure; mask = 1 on generated response tokens, 0 on prompt tokens.
 *
 *   cu_seqlens   [n_seq + 1] int32 on the device, cu_seqlens[0] = 0, non-decreasing (empty sequences allowed),
 *                cu_seqlens[n_seq] = n_tok.  The contents are the caller's responsibility (they are not read on
 *                the host); whatever they hold, no kernel indexes outside [0, n_seq] or [0, n_tok).
 *   logp_*, omega, ratio [n_tok] fp32, 16-byte aligned;  mask, clip_mask [n_tok] u8, 4-byte aligned; n_tok need
 *                not be a multiple of 4 (n_tok < 2^31).  With 32-byte aligned fp32 tensors and 8-byte aligned masks
 *                the call takes its fast kernel (one warp per 512 tokens); the results are the same bits either way.
 *   adv_out      [n_seq] fp32, REQUIRED here: the per-sequence advantages are written by a first launch and read
 *                by the token kernel (2 launches; the second starts while the first runs and waits for it only
 *                before it uses an advantage).
 *   Exposure: the activation row of token k is k - row_shift; with row_shift = 1 a token whose source row
 *   would fall before the start of its own sequence carries no weight (it counts neither in the mean nor in E_u).
 *   Other arguments, status codes and workspace as in the dense calls.
 */
int hilore_grpo_coeffs_packed(const float *rewards, int64_t n_resp_total, int32_t G, int64_t resp_offset,
                              int64_t n_seq, const int32_t *cu_seqlens, int64_t n_tok, const float *logp_new,
                              const float *logp_old, const float *logp_ref, const uint8_t *mask, int64_t N_norm,
                              const int64_t *N_norm_dev, float clip_eps, float beta, float adv_eps, float *adv_out,
                              float *omega, float *ratio, uint8_t *clip_mask, void *stream);
int hilore_unit_exposure_packed(const float *omega, const uint8_t *mask, int64_t n_tok, const int32_t *cu_seqlens,
                                int64_t n_seq, const float *row_rms, int32_t U, int64_t rms_ld, int32_t row_shift,
                                float eps_alpha, float *exposure, float *sum_abs_omega, void *workspace,
                                size_t workspace_bytes, void *stream);

/*
 * Score variants of the component ablations (paragraph "Component ablations"): hilore_grpo_coeffs with one
 * more argument.  variant 0: omega as above.  variant 1 ("removing ratio/clipping"): chi_t r_t replaced by 1 in
 * the policy contribution, omega_t = -(m_t / N) A + beta (m_t / N)(1 - exp(s_ref - s)).  variant 2: the
 * advantage-only signal omega_t := m_t A, whose exposure is sum_t |A_t| alpha_t.  "Removing KL" is beta = 0;
 * "removing activation weighting" is the sum_abs_omega output of hilore_unit_exposure; "removing
 * susceptibility" is kappa = 1.  ratio and clip_mask are reported as in hilore_grpo_coeffs.
 */
int hilore_grpo_coeffs_variant(const float *rewards, int64_t n_resp_total, int32_t G, int64_t resp_offset,
                               int64_t n_rows, int64_t T, const float *logp_new, const float *logp_old,
                               const float *logp_ref, const uint8_t *mask, int64_t N_norm,
                               const int64_t *N_norm_dev, float clip_eps, float beta, float adv_eps, int32_t variant,
                               float *adv_out, float *omega, float *ratio, uint8_t *clip_mask, void *stream);

/*
 * Structural sparsity of one record of coefficients (paragraph "Structural sparsity in diagnostic replays",
 * Eq. "diagnostic-clipping").  Over the n = n_rows * T padded response slots:
 *   counts[0] padding slots (m = 0);  counts[1] valid slots with zero advantage;  counts[2] valid slots with
 *   nonzero advantage on a flat clipped branch, (A > 0 and r > 1 + eps) or (A < 0 and r < 1 - eps);
 *   counts[3] slots whose coefficient is zero (padding counts as zero);  counts[4] = n, the common denominator.
 *   top_share = share of sum |omega| carried by the ceil(0.1 n) slots of largest |omega| (exact: the k-th largest
 *   value is found by a radix select on the bit patterns; ties at the threshold contribute as many copies as the
 *   decile still needs).   sum_abs = sum |omega| over valid slots.
 *   adv [n_rows], ratio / omega [n_rows, T] fp32, mask [n_rows, T] u8 (device); counts [5] int64, top_share,
 *   sum_abs (opt) fp64 on the device, 8-byte aligned; workspace hilore_omega_diagnostics_workspace_bytes() bytes.
 * Integer histograms and fixed-slot fp64 partial sums: the result is deterministic.
 */
int hilore_omega_diagnostics(const float *adv, const float *ratio, const uint8_t *mask, const float *omega,
                             int64_t n_rows, int64_t T, float clip_eps, int64_t *counts, double *top_share,
                             double *sum_abs, void *workspace, size_t workspace_bytes, void *stream);
size_t hilore_omega_diagnostics_workspace_bytes(void);

/*
 * Operational update exposure of U units over one microbatch
 * (Eq. "activation-token-weights", Eq. "mlp-weighted-exposure"):
 *     T_b = slots with mask = 1;  abar_u = mean_{t in T_b} a_{t,u}
 *     alpha_{t,u} = (a_{t,u} + eps_alpha) / (abar_u + eps_alpha)
 *     E_u = sum_{t in T_b} |omega_t| alpha_{t,u};       |T_b| = 0  =>  E_u = 0
 * a_{t,u} is row_rms[u*rms_ld + i*T + t - row_shift] for slot (i, t): row_shift = 1 takes the
 * activation row of the source position that predicts token t (the paper's wording), 0 the
 * token's own row.  A slot with t - row_shift < 0 has no activation row in this grid and carries no
 * weight: it counts neither in abar_u nor in E_u (the weights of the other slots of T_b average to
 * one); sum_abs_omega still covers all of T_b.
 *
 *   omega, mask   [n_rows, T] fp32 / u8 of the microbatch.    row_rms  [U, rms_ld] fp32, rms_ld >= n_rows*T.
 *   exposure      [U] fp32.     sum_abs_omega  opt, one fp32: sum_{t in T_b} |omega_t|.
 *   workspace     scratch of at least hilore_workspace_bytes(U, n_rows*T) bytes, 16-byte aligned; its
 *                 contents are overwritten (HILORE_WORKSPACE if too small).  Partial sums are kept in fp64
 *                 in fixed slots and added in a fixed order: the result is run-to-run deterministic.
 *   Launches: up to 16 tiles of 1024 tokens the call is ONE launch (the CTAs of a group of eight units are a
 *   thread-block cluster and add their sums through its shared memory; the workspace is not touched); larger
 *   microbatches take a second, small launch that adds the partial sums of the workspace.  Same bits either way.  With
 *   HILORE_DISABLE_CLUSTER_LAUNCH set in the environment (to anything but "0") no call of this library launches
 *   thread-block clusters.
 */
int hilore_unit_exposure(const float *omega, const uint8_t *mask, int64_t n_rows, int64_t T,
                         const float *row_rms, int32_t U, int64_t rms_ld, int32_t row_shift, float eps_alpha,
                         float *exposure, float *sum_abs_omega, void *workspace, size_t workspace_bytes,
                         void *stream);
size_t hilore_workspace_bytes(int32_t U, int64_t n_tok);

/*
 * hilore_unit_exposure for callers that cannot provide a workspace.  (The paper has no counterpart:
 * this is a packaging variant of the same reduction, with the same results.)
 *
 * Who needs it: code that must not allocate at the point where the exposure refresh runs -- for example
 * a saved-tensor hook running where the framework's caching allocator may not be re-entered, a process
 * whose device memory is wholly owned by another pool, or a latency-critical loop in which cudaMalloc
 * (which may synchronise the device) is ruled out.  The call allocates nothing on host or device: the
 * fp64 partial sums go to a fixed 1 MiB array inside the library image (hilore_static_scratch_bytes()),
 * which every GPU context that loads the library holds until it exits.
 *
 *   Arguments and results as hilore_unit_exposure, minus the workspace.
 *   Limit: hilore_workspace_bytes(U, n_rows*T) must not exceed the built-in array, i.e.
 *   (U + 1) * ceil(n_rows*T / 1024) <= 65536; larger problems return HILORE_WORKSPACE and nothing is
 *   launched (use hilore_unit_exposure with your own workspace).
 *   First call on a device: looks up the array's device address (once per device, with that device
 *   current) -- make this first call outside any stream capture.
 *   The array is shared by all calls and keeps the previous call's contents; every slot a call reads it
 *   has written first, so nothing needs clearing.  Two calls that overlap on the GPU (different streams
 *   without ordering, or several host threads) race on the array: order them.
 */
int hilore_unit_exposure_static(const float *omega, const uint8_t *mask, int64_t n_rows, int64_t T,
                                const float *row_rms, int32_t U, int64_t rms_ld, int32_t row_shift,
                                float eps_alpha, float *exposure, float *sum_abs_omega, void *stream);
size_t hilore_static_scratch_bytes(void);

/*
 * Compress one bf16 unit (the L action at capture time; Eq. "fp8-roundtrip" for fmt RAW) and, fused
 * into the same pass, the tokenwise activation magnitude a_t = sqrt(mean_j X_{t,j}^2) of
 * Eq. "activation-token-weights" (fp32 accumulation per block of 64, fp64 across the blocks of a row;
 * a row whose squares leave the fp32 range yields Inf).
 *   fmt RAW : code = cast_E4M3FN(x): one RNE rounding from the bf16 value; |x| up to 464 -> at most 448,
 *             larger, +-Inf and NaN -> sign | 0x7F.  block must be 0, scales NULL.
 *   fmt BLK : per block of 64 consecutive elements of a row: amax = max |x_i| over its finite elements;
 *             s = inv = 1 if amax == 0, if no element is finite, or if Q / amax overflows fp32;
 *             else s = fl32(amax / Q), inv = fl32(Q / amax), Q = 448 (E4M3FN) or 127 (INT8);
 *             q_i = fl32(x_i * inv); E4M3FN: code_i = RNE(q_i) saturating at +-448, NaN -> sign|0x7F;
 *             INT8: code_i = RNE(q_i) clamped to +-127, NaN -> 0x80.  block must be 64.
 *
 *   x        [rows, ld] bf16, ld >= cols, 32-byte aligned, ld % 16 == 0.    cols % 16 == 0 (RAW),
 *            cols % 64 == 0 (BLK).
 *   codes    [rows, cols] u8, 16-byte aligned; NULL => statistics only (row_rms must then be given).
 *   scales   [rows, cols/64] fp32 (BLK only).          row_rms  opt [rows] fp32.
 */
int hilore_compress(const void *x, int64_t rows, int64_t cols, int64_t ld, int32_t fmt, int32_t block,
                    uint8_t *codes, float *scales, float *row_rms, void *stream);

/*
 * Recover a compressed unit to bf16 (the L action at backward time).
 *   fmt RAW : x_hat = cast_BF16(code), exact; the NaN codes become a bf16 NaN.
 *   fmt BLK : x_hat = bf16_rne(fl32(value(code) * s)).
 *   codes [rows, cols] u8, 16-byte aligned;  scales [rows, cols/64] fp32 (BLK);
 *   out   [rows, ld_out] bf16, 32-byte aligned, ld_out % 16 == 0, ld_out >= cols.
 */
int hilore_recover(const uint8_t *codes, const float *scales, int64_t rows, int64_t cols, int32_t fmt,
                   int32_t block, void *out, int64_t ld_out, void *stream);

/*
 * Joint H / L / R allocation: the paper's allocator (Section "Joint H/L/R Allocation", Eq. "joint-allocation";
 * Appendix "Joint Allocation and Schedule Validation", Eqs. "allocation-grid", "allocation-integer-costs",
 * "allocation-dp").  Maximise sum_u dtau_u(a_u) subject to sum_u dmem_u(a_u) <= M_res,
 * sum_u d_u(a_u) <= delta_b with d(H) = d(R) = 0 and d(L) = psi_u, and a_u in A_u(q_u), exactly on the
 * conservative grid: h_B = M_res / N, h_d = delta_b / N, b_u(a) = ceil(dmem_u(a) / h_B),
 * r_u(a) = ceil(d_u(a) / h_d) (costs rounded up, so every grid-feasible assignment is feasible);
 * F_0(0,0) = 0, F_i(j,k) = max_a F_{i-1}(j - b, k - r) + dtau_i(a), candidates in the order R, H, L (first
 * maximum wins); terminal ties favour the lower risk state, then the lower memory state.  M_res == 0 leaves
 * one memory state (only actions without memory cost); delta_b == 0 disables L.  A NaN or negative psi_u makes
 * L unavailable for unit u; negative memory costs count as 0; R always has utility 0 and costs 0.
 * FP64 utilities as in the paper.  Layer i of the DP is one data-parallel pass over the (N+1)^2 states.
 *
 *   psi      [U] fp32 (device), e.g. written by hilore_plan_apply(PHASE_DECIDE).
 *   dtau, dmem   [U, 3] fp64 (device), indexed by the action code (R, H, L); column R is ignored.
 *   avail    [U] u8: the candidate plan q_u.        M_res, delta_b  host scalars, >= 0 (else INVALID_ARG).
 *   n_intervals  N; the paper uses 1024.
 *   action   [U] u8 out.   recompute  opt [U] u8 (1 iff R).   totals  opt [3] fp64: utility, memory, risk of the
 *            selection (8-byte aligned).
 *   workspace    hilore_allocate_workspace_bytes(U, N) bytes, 256-byte aligned (two value tables and the
 *            predecessor table; 105 MB for U = 84, N = 1024).
 * hilore_risk_budget: the microbatch budget delta_b = delta * N_b / sum_b' N_b' (host arithmetic).
 */
int hilore_allocate(int32_t U, const float *psi, const double *dtau, const double *dmem, const uint8_t *avail,
                    double M_res, double delta_b, int32_t n_intervals, uint8_t *action, uint8_t *recompute,
                    double *totals, void *workspace, size_t workspace_bytes, void *stream);
size_t hilore_allocate_workspace_bytes(int32_t U, int32_t n_intervals);
double hilore_risk_budget(double delta, int64_t N_b, int64_t N_total);

/*
 * Calibration of the L action (initialisation time, on the calibration microbatches).
 *   hilore_relative_error: e^L = ||x_hat - x||_2 / (||x||_2 + 1e-8) of one unit, operands widened to fp32 before
 *   the subtraction and the norms (Eq. "calibration-metrics"); fp32 per 16 elements, fp64 across them, per-CTA
 *   partial sums in fixed workspace slots, added in a fixed order (deterministic).
 *     x, xhat  [rows, ld] / [rows, ld_hat] bf16, 32-byte aligned, ld % 16 == 0; cols % 16 == 0.
 *     e_out    one fp64 on the device.    norms2   opt [2] fp64 on the device: ||x_hat - x||^2, ||x||^2.
 *     workspace  hilore_relative_error_workspace_bytes() bytes, 16-byte aligned.
 *   The mean reconstruction error ebar_u^L is the plain average of e^L over the calibration microbatches.
 *   hilore_fit_kappa: kappa_c = argmin_{kappa >= 0} sum_i (y_i - kappa x_i)^2 = max(0, sum x y / sum x^2)
 *   (Eq. "susceptibility"), x_i = E_{u,b} e^L_{u,b}; HOST arrays, host arithmetic; 0 if every x_i is 0.
 */
int hilore_relative_error(const void *x, const void *xhat, int64_t rows, int64_t cols, int64_t ld, int64_t ld_hat,
                          double *e_out, double *norms2, void *workspace, size_t workspace_bytes, void *stream);
size_t hilore_relative_error_workspace_bytes(void);
/*
 * The same e^L for x_hat = recover(compress(x)) in format fmt, fused: x is read once (2 B per element), encoded
 * and decoded in registers with the routines of hilore_compress / hilore_recover (x_hat is bit for bit what
 * they would produce), nothing else is written.  Shape and alignment rules of hilore_compress; workspace,
 * outputs and determinism as hilore_relative_error.  A unit with NaN codes gives e^L = NaN.
 */
int hilore_codec_relative_error(const void *x, int64_t rows, int64_t cols, int64_t ld, int32_t fmt, int32_t block,
                                double *e_out, double *norms2, void *workspace, size_t workspace_bytes, void *stream);
double hilore_fit_kappa(const double *x, const double *y, int64_t n);

/* One recovery unit of a microbatch: where its bf16 bundle lives and where its L representation goes.
 * A DEVICE array of these is passed to hilore_plan_apply.  Field rules as in hilore_compress /
 * hilore_recover; `out` may equal `x` only if the caller no longer needs the original. */
typedef struct hilore_unit {
    const void *x;   /* [rows, ld] bf16 saved activation                         */
    uint8_t *codes;  /* [rows, cols] u8                                          */
    float *scales;   /* [rows, cols/64] fp32, NULL for fmt RAW                   */
    void *out;       /* [rows, ld] bf16 reconstruction target of RECOVER         */
    float *row_rms;  /* opt [rows] fp32 token magnitudes written by CAPTURE      */
    int64_t rows, cols, ld;
    int32_t fmt, block;
} hilore_unit;

/*
 * Risk score, H / L / R gating and the batched capture / encode / recover of all units of a microbatch
 * in ONE launch per phase and 96 units (a longer table runs as consecutive launches over slices of 96)
 * (Eq. "token-weighted-risk": psi_u = kappa_c(u) E_u ebar_u; Eq. "available-recovery-actions").  All decisions
 * stay on the device: the gating arrays are read by the kernels, so no phase needs a host synchronisation.
 *
 *   units_dev   [U] hilore_unit on the DEVICE.     units_host  the same table on the HOST (read during
 *               the call for validation and launch sizing; must match units_dev).
 *   avail       [U] u8: the candidate plan q_u in {R, H, L} fixed before forward.
 *   action_io   [U] u8: DECIDE writes it; the other phases read it.
 *   DECIDE:  if exposure != NULL: psi_u = fl32(fl32(kappa_u * E_u) * ebar_u); desired = L if psi < tau_lo,
 *            H if psi >= tau_hi, else R (NaN -> R) -- a threshold stand-in for the paper's knapsack
 *            allocator; if exposure == NULL the desired action is action_io[u] as given.
 *            Then action = desired if it is in A_u(q_u) (q = H: {H,L,R}; q = L: {L,R}; q = R: {R}), else R.
 *            Writes psi (opt), action_io, recompute[u] = (action == R), retained_bytes[u] = 2*rows*cols (H),
 *            rows*cols + 4*rows*cols/64 (L; no scale term for fmt RAW), 0 (R).
 *   CAPTURE: q = L: compress into codes / scales and write row_rms; q = H: row_rms only; q = R: untouched.
 *   ENCODE:  units with q = H and action = L are compressed (post-forward encoding).
 *   RECOVER: units with action = L are decoded into `out`; H and R units are untouched (H keeps its
 *            exact bundle, Prop. "exact recovery equivalence"; R is recomputed by the caller).
 */
int hilore_plan_apply(const hilore_unit *units_dev, const hilore_unit *units_host, int32_t U, int32_t phase,
                      const float *exposure, const float *kappa, const float *ebar, float tau_lo,
                      float tau_hi, const uint8_t *avail, uint8_t *action_io, float *psi, uint8_t *recompute,
                      uint64_t *retained_bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* HILORE_H */
