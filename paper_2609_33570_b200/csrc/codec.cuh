// Streaming codec of the L action: bf16 -> FP8 E4M3FN / INT8 codes (+ per-block scales, + token RMS)
// and back.  Paper: Eq. "fp8-roundtrip" (unscaled cast) and Eq. "activation-token-weights" (a_t).
//
// Work split.  A CTA owns a contiguous range of rows of a unit.  A thread owns 16 consecutive
// elements ("chunk": one 256-bit load, one 128-bit store of codes) and handles chunks in pairs; four
// neighbouring lanes own one 64-element block, so the block absmax and the block sum of squares are
// xor-shuffles inside a quad.  Rows are swept in batches small enough that the per-block sums of
// squares of a batch fit in shared memory; at the end of a batch each warp adds the blocks of whole
// rows in a fixed order, so the token RMS is deterministic (no floating-point atomics anywhere).
// The instruction budget matters: at 6.5 TB/s the SM has about 8 issue slots per element, so the hot
// loop uses packed bf16x2 maxima, packed f32x2 multiplies / FMAs, a 128-entry table in place of the two IEEE
// divisions of a block, one conversion block per four codes, a rare-path repair after the stores instead of
// calls inside the loop, and pointer increments instead of index arithmetic.
#pragma once

#include "common.cuh"

namespace hilore {

enum CodecOp { OP_NONE = 0, OP_COMPRESS = 1, OP_STATS = 2, OP_RECOVER = 3 };

struct CodecWork {
    const hilore_unit *units; // device table, or nullptr => `single`
    hilore_unit single;
    int U;
    int phase;                // HILORE_PHASE_* for table mode; CodecOp for single mode
    const uint8_t *avail;     // q_u
    const uint8_t *action;    // a_u
    int64_t seg_bytes;        // scale of the windows all CTAs sweep together (see plan_unit)
    uint64_t share_m;         // 2^32 = share_m * grid + share_rem
    uint32_t share_rem;
    uint32_t rot_step;        // rotation of the CTA index per window (0 for grids of one or two CTAs)
};

__device__ __forceinline__ int unit_op(const CodecWork &wk, int u)
{
    if (wk.units == nullptr)
        return wk.phase;
    switch (wk.phase) {
    case HILORE_PHASE_CAPTURE: {
        const uint8_t q = wk.avail[u];
        return q == HILORE_ACT_L ? OP_COMPRESS : (q == HILORE_ACT_H ? OP_STATS : OP_NONE);
    }
    case HILORE_PHASE_ENCODE:
        return (wk.avail[u] == HILORE_ACT_H && wk.action[u] == HILORE_ACT_L) ? OP_COMPRESS : OP_NONE;
    case HILORE_PHASE_RECOVER:
        return wk.action[u] == HILORE_ACT_L ? OP_RECOVER : OP_NONE;
    default:
        return OP_NONE;
    }
}


// ---- work split ----
// What the CTAs of a launch share is a list of ITEMS per unit; CTA c' takes items [n*c'/nC, n*(c'+1)/nC) of every
// window of n items, so that all CTAs work inside one window of memory at a time (measured faster on B200 than
// one large private slice per CTA).  An item is a 16 KB piece (512 chunks: one iteration of the hot loops) of a
// contiguous unit when no per-row result is wanted (encode without token RMS, recover): every CTA then runs whole
// iterations only; otherwise a row (ragged ends of a CTA's rows take the predicated path).
// c' is the CTA index rotated by a fixed step per window.  Without the rotation the same CTAs take the same
// relative share of every unit of a microbatch; with it the shares move from unit to unit (measured on the 7B-shaped
// table of 84 units: token-RMS capture 5.8 -> 7.1 TB/s, recovery 5.9 -> 6.3 TB/s; the size of the step does not
// matter).  Nothing synchronises the CTAs between units, so only the total per CTA counts for the balance.
// A CTA's share of n items is (n * K(c')) >> 32 with K(c) = floor(c * 2^32 / nC) = c * M + floor(c * rem / nC)
// (M, rem from the host): one multiplication and a 32-bit division instead of two 64-bit divisions per window.
constexpr int kStageUnits = 96;
constexpr int kIterChunks = 2 * kCodecThreads;       // chunks one iteration of a CTA covers (16 KB of bf16)
constexpr int kFlatCols = kIterChunks * 16;          // a 16 KB piece seen as one row of 8192 elements

struct UnitPlan {
    int64_t items;     // rows or 16 KB pieces
    int64_t seg_items; // items per window
    bool flat;         // items are 16 KB pieces
    int tail_chunks;   // flat: chunks beyond the last whole piece
};

// `per_row`: a per-row result (token RMS) is wanted.
__device__ __forceinline__ UnitPlan plan_unit(const CodecWork &wk, const hilore_unit &u, bool per_row, bool recover)
{
    UnitPlan p;
    int64_t item_bytes = u.cols * 2;
    p.items = u.rows;
    p.flat = false;
    p.tail_chunks = 0;
    if (u.ld == u.cols && !per_row) {
        const int64_t chunks = u.rows * (u.cols >> 4);
        p.items = chunks / kIterChunks;
        p.tail_chunks = (int)(chunks - p.items * kIterChunks);
        p.flat = true;
        item_bytes = kFlatCols * 2;
    }
    // Units up to 1.5 x seg_bytes in one piece (see below for the exception); larger ones in equal windows: of seg_bytes where the items are 16 KB
    // pieces, of two thirds of it where they are rows, but of at least four to five rows per CTA (rows of 18944
    // elements are 37 KB each).  Measured on B200 with seg_bytes = 96 MiB, row windows of 96 -> 64 MiB: units
    // [., 4096] of 0.25 / 0.5 / 4 GiB compress at 5.92 -> 6.14, 6.34 -> 6.45, 6.41 -> 6.53 TB/s, a [65536, 8960] unit
    // 6.23 -> 6.59, while the 7B-shaped capture with codes loses 1.5 % unless its [16384, 18944] units keep the larger
    // windows; for 16 KB pieces the two sizes measure within 1 % of each other, either way round by shape.
    const int64_t nC = gridDim.x;
    const int64_t unit_bytes = p.items * item_bytes;
    p.seg_items = p.items;
    // (a single unit shared by rows is cut from seg_bytes on: units of 128-141 MiB compress 3-5 % faster in two
    // windows when they are alone in the launch, and 3 % slower when they are part of a table; below seg_bytes two
    // windows lose up to 7 %)
    // A unit alone in its launch and shared by 16 KB pieces is cut from 1.5 x seg_bytes on like the others, but into
    // windows of half of seg_bytes (E4M3FN + scales: recover at 0.5 / 1 / 4 GiB 6.11 -> 6.21, 6.23 -> 6.31, 6.39 -> 6.44
    // TB/s, compress without token RMS 2-4 % faster); the recover pass of the unscaled and the INT8 format keeps the
    // larger windows (1-3 % faster with them).
    const bool alone = wk.units == nullptr;
    const bool small_pieces = alone && p.flat && !(recover && u.fmt != HILORE_FMT_E4M3FN_BLK);
    const int64_t uncut = (alone && !p.flat) ? wk.seg_bytes : wk.seg_bytes + wk.seg_bytes / 2;
    if (unit_bytes >= uncut) {
        const int64_t window = small_pieces ? wk.seg_bytes / 2 : p.flat ? wk.seg_bytes : max(wk.seg_bytes * 2 / 3, 9 * nC * item_bytes / 2);
        const int64_t nseg = max((int64_t)1, (unit_bytes + window / 2) / window);
        p.seg_items = (p.items + nseg - 1) / nseg;
    }
    // a whole number of items per CTA and window, so that only a unit's last window is shared unevenly; rounded up,
    // so that the last window is never a sliver (rounded to nearest, a 0.5-1 GiB unit could end in a window of less
    // than one row per CTA: compress 6.1 -> 6.3 TB/s)
    p.seg_items = max((int64_t)1, (p.seg_items + nC - 1) / nC) * nC;
    return p;
}

struct UnitStage {
    hilore_unit u[kStageUnits];
    int op[kStageUnits];
    UnitPlan plan[kStageUnits]; // how each unit is shared among the CTAs (worked out once per kernel, not per CTA visit)
};

// Stage the launch's units: what to do with each (OP_NONE if the launch is not gated into it or it lacks a
// buffer the operation needs), its descriptor and its sharing plan.  `recover`: which of the two kernels is asking.
__device__ __forceinline__ void stage_units(const CodecWork &wk, bool recover, UnitStage &st)
{
    for (int t = threadIdx.x; t < wk.U; t += blockDim.x) {
        int op = unit_op(wk, t);
        if (recover ? (op != OP_RECOVER) : (op != OP_COMPRESS && op != OP_STATS))
            op = OP_NONE;
        if (op != OP_NONE) {
            hilore_unit u = wk.units ? wk.units[t] : wk.single;
            const bool scaled = u.fmt != HILORE_FMT_E4M3FN_RAW;
            if ((op == OP_COMPRESS && (!u.x || !u.codes || (scaled && !u.scales))) || (op == OP_STATS && (!u.x || !u.row_rms)) ||
                (op == OP_RECOVER && (!u.out || !u.codes || (scaled && !u.scales))))
                op = OP_NONE; // the unit lacks a buffer this operation needs: leave it untouched
            if (op == OP_COMPRESS && wk.units && wk.phase == HILORE_PHASE_ENCODE)
                u.row_rms = nullptr; // token magnitudes were collected at capture time
            st.u[t] = u;
            st.plan[t] = plan_unit(wk, u, !recover && u.row_rms != nullptr, recover);
        }
        st.op[t] = op;
    }
}

__device__ __forceinline__ uint64_t share_multiplier(const CodecWork &wk, uint32_t c) // floor(c * 2^32 / nC), c <= nC
{
    return (uint64_t)c * wk.share_m + (c * wk.share_rem) / gridDim.x;
}

// One piece of work of a CTA: rows [r0, r1) of a unit (or of the 16 KB-piece view of it), in batches of
// `rows_per_batch` rows where per-row sums are collected.
struct Job {
    hilore_unit u;
    int op;
    int64_t r0, r1;
    int rows_per_batch;
};

struct JobCursor {
    int ui = 0;           // current unit
    int64_t seg_item = 0; // first item of its next window
    uint32_t rot = 0;     // rotation of the CTA index, advanced per window
    bool tail_done = false;
};

// The next piece of work of this CTA, from the staged descriptors, gates and sharing plans of the launch.
__device__ __forceinline__ bool next_job(const CodecWork &wk, const UnitStage &st, JobCursor &cur, Job &j, int slots)
{
    const uint32_t nC = gridDim.x;
    for (; cur.ui < wk.U; ++cur.ui, cur.seg_item = 0, cur.tail_done = false) {
        j.op = st.op[cur.ui];
        if (j.op == OP_NONE)
            continue;
        j.u = st.u[cur.ui];
        const UnitPlan p = st.plan[cur.ui];
        const int nb = (int)(j.u.cols >> 6);
        while (cur.seg_item < p.items) {
            const int64_t s0 = cur.seg_item, n = min(p.seg_items, p.items - s0);
            cur.seg_item += n;
            uint32_t c = blockIdx.x + cur.rot;
            c = c >= nC ? c - nC : c;
            cur.rot += wk.rot_step;
            cur.rot = cur.rot >= nC ? cur.rot - nC : cur.rot;
            int64_t i0, i1;
            if (n < (1ll << 31)) {
                i0 = s0 + (int64_t)(((uint64_t)n * share_multiplier(wk, c)) >> 32);
                i1 = s0 + (int64_t)(((uint64_t)n * share_multiplier(wk, c + 1)) >> 32);
            } else {
                i0 = s0 + (n * (int64_t)c) / nC;
                i1 = s0 + (n * (int64_t)(c + 1)) / nC;
            }
            if (i0 >= i1)
                continue;
            j.r0 = i0;
            j.r1 = i1;
            if (p.flat) { // the unit as rows of 8192 contiguous elements
                j.u.rows = p.items;
                j.u.cols = j.u.ld = kFlatCols;
                j.rows_per_batch = 32;
            } else {
                j.rows_per_batch = max(1, slots / max(1, nb));
            }
            return true; // the cursor already points at the next window
        }
        if (p.flat && p.tail_chunks > 0 && !cur.tail_done) { // the last, partial piece: one short row
            cur.tail_done = true;
            uint32_t c = blockIdx.x + cur.rot;
            c = c >= nC ? c - nC : c;
            if (c == 0) {
                const int64_t done = p.items * kFlatCols; // elements in whole pieces
                j.u.x = static_cast<const uint16_t *>(j.u.x) + done;
                j.u.out = static_cast<uint16_t *>(j.u.out) + done;
                j.u.codes += done;
                j.u.scales += done >> 6;
                j.u.rows = 1;
                j.u.cols = j.u.ld = (int64_t)p.tail_chunks * 16;
                j.r0 = 0;
                j.r1 = 1;
                j.rows_per_batch = 1;
                return true;
            }
        }
    }
    return false;
}

template <int FMT> struct QMax {
    static constexpr float value = (FMT == HILORE_FMT_INT8_BLK) ? 127.0f : 448.0f;
};

// Largest |bf16| pattern whose reciprocal scale Q / amax no longer fits fp32 (it rounds to Inf):
// 448 / (1.75 * 2^-120) = 2^128 and 127 / (1.984375 * 2^-122) = 2^128.  At or below it (zero included)
// the block takes s = inv = 1.
template <int FMT> struct UnitScaleBelow {
    static constexpr uint32_t value = (FMT == HILORE_FMT_INT8_BLK) ? 0x02FEu : 0x03E0u;
};

// Smallest |bf16| pattern for which both s = amax / Q and inv = Q / amax are normal fp32 numbers
// (Q = 448: amax >= 1.75 * 2^-118; Q = 127: amax >= 1.984375 * 2^-120).  From here up to the largest finite
// pattern the two quotients follow from the 7 mantissa bits alone (scale table below).
template <int FMT> struct TableScaleFrom {
    static constexpr uint32_t value = (FMT == HILORE_FMT_INT8_BLK) ? 0x03FEu : 0x04E0u;
};

// Scale table.  amax is a bf16 number v * 2^E with v = 1 + m / 128, so fl32(amax / Q) = fl32(v / Q) * 2^E and
// fl32(Q / amax) = fl32(Q / v) * 2^-E exactly while the results stay normal: the correctly rounded quotient
// depends on m only, and the power of two is an integer addition to the exponent field.  Entry m holds the
// bit patterns of fl32(v / Q) and fl32(Q / v) with the exponent bias folded in, so that
//     bits(s) = tab[m] + (amax_bits & 0x7F80) * 65536,    bits(inv) = tab[128 + m] - (amax_bits & 0x7F80) * 65536.
// Two IEEE divisions per block become one shared-memory load and one integer multiply-add per lane.
constexpr int kScaleTableWords = 256; // per format family: [0,128) for s, [128,256) for inv

template <int FMT> __device__ __forceinline__ void fill_scale_table(uint32_t *tab)
{
    constexpr float Q = QMax<FMT>::value;
    for (int i = threadIdx.x; i < 128; i += blockDim.x) {
        const float v = 1.0f + (float)i * 0.0078125f;
        tab[i] = __float_as_uint(__fdiv_rn(v, Q)) - (127u << 23);
        tab[128 + i] = __float_as_uint(__fdiv_rn(Q, v)) + (127u << 23);
    }
}

__device__ __forceinline__ uint32_t int8_code(float q)
{
    int v = __float2int_rn(q);
    v = max(-127, min(127, v));
    return (uint32_t)v & 0xFFu;
}

// max.NaN.xorsign.abs.bf16x2: per half, magnitude = max(|a|, |b|) (NaN if either is NaN), sign = junk
__device__ __forceinline__ uint32_t maxabs_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.NaN.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

__device__ __forceinline__ uint32_t maxnan_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// |bf16| bit pattern of the largest magnitude among sixteen elements; 0x7FFF if any of them is NaN,
// 0x7F80 if any is Inf (and none NaN): one compare against 0x7F80 finds every block that needs care.
__device__ __forceinline__ uint32_t absmax16(const uint32_t (&w)[8])
{
    uint32_t a = maxabs_bf16x2(w[0], w[1]), b = maxabs_bf16x2(w[2], w[3]);
    uint32_t c = maxabs_bf16x2(w[4], w[5]), d = maxabs_bf16x2(w[6], w[7]);
    a = maxabs_bf16x2(a, b);
    c = maxabs_bf16x2(c, d);
    a = maxabs_bf16x2(a, c);
    a = maxabs_bf16x2(a, a >> 16);
    return a & 0x7FFFu;
}

// One element with the full rule set (overflow, Inf, NaN).  Rare path.
template <int FMT> __device__ __forceinline__ uint32_t encode1_careful(uint32_t bits, float inv)
{
    const uint32_t a = bits & 0x7FFFu, sign = (bits >> 8) & 0x80u;
    const float x = __uint_as_float(bits << 16);
    if (FMT == HILORE_FMT_E4M3FN_RAW) {
        if (a > 0x43E8u) // above 464: rounds past 448, or Inf / NaN
            return sign | 0x7Fu;
        return cvt_e4m3x2(0.0f, x) & 0xFFu;
    }
    if (FMT == HILORE_FMT_E4M3FN_BLK) {
        if (a > 0x7F80u)
            return sign | 0x7Fu;
        if (a == 0x7F80u)
            return sign | 0x7Eu;
        return cvt_e4m3x2(0.0f, __fmul_rn(x, inv)) & 0xFFu;
    }
    if (a > 0x7F80u)
        return 0x80u;
    if (a == 0x7F80u)
        return sign ? 0x81u : 0x7Fu;
    return int8_code(__fmul_rn(x, inv));
}

// Rare path, kept out of line and fed by value so that the common path keeps its data in registers.
template <int FMT> __device__ __forceinline__ uint4 encode16_careful_inl(uint4 lo, uint4 hi, float inv)
{
    const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    uint32_t c[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        c[i] = encode1_careful<FMT>(w[2 * i] & 0xFFFFu, inv) | (encode1_careful<FMT>(w[2 * i] >> 16, inv) << 8) |
               (encode1_careful<FMT>(w[2 * i + 1] & 0xFFFFu, inv) << 16) |
               (encode1_careful<FMT>(w[2 * i + 1] >> 16, inv) << 24);
    }
    return make_uint4(c[0], c[1], c[2], c[3]);
}

template <int FMT> __device__ __noinline__ uint4 encode16_careful(uint4 lo, uint4 hi, float inv)
{
    return encode16_careful_inl<FMT>(lo, hi, inv);
}

// max |bits| over the finite elements only (rare path, by value)
__device__ __forceinline__ uint32_t absmax16_finite_inl(uint4 lo, uint4 hi)
{
    const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    uint32_t m = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        uint32_t l = w[i] & 0x7FFFu, h = (w[i] >> 16) & 0x7FFFu;
        if (l < 0x7F80u) m = max(m, l);
        if (h < 0x7F80u) m = max(m, h);
    }
    return m;
}

static __device__ __noinline__ uint32_t absmax16_finite(uint4 lo, uint4 hi) { return absmax16_finite_inl(lo, hi); }

#define HILORE_LO4(w) make_uint4((w)[0], (w)[1], (w)[2], (w)[3])
#define HILORE_HI4(w) make_uint4((w)[4], (w)[5], (w)[6], (w)[7])

// One pass over a chunk: unpack each bf16 pair once, feed it to the sum of squares (SUMS) and to the
// scaled conversion (CODES).  Elements must be finite (BLK) / at most 464 in magnitude (RAW).
template <int FMT, bool CODES, bool SUMS>
__device__ __forceinline__ void chunk_pass(const uint32_t (&w)[8], float inv, uint4 &codes, float &sumsq)
{
    const uint64_t inv2 = f32x2_pack(inv, inv);
    uint64_t acc = 0; // {0.0f, 0.0f}
    uint32_t cw[4];   // four codes per word
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint64_t xa = f32x2_pack(bf16_lo(w[2 * i]), bf16_hi(w[2 * i]));
        uint64_t xb = f32x2_pack(bf16_lo(w[2 * i + 1]), bf16_hi(w[2 * i + 1]));
        if (SUMS) {
            acc = f32x2_fma(xa, xa, acc);
            acc = f32x2_fma(xb, xb, acc);
        }
        if (CODES) {
            if (FMT != HILORE_FMT_E4M3FN_RAW) { // fl32(x * inv), each lane rounded to nearest even
                xa = f32x2_mul(xa, inv2);
                xb = f32x2_mul(xb, inv2);
            }
            float a0, a1, b0, b1;
            f32x2_unpack(xa, a0, a1);
            f32x2_unpack(xb, b0, b1);
            if (FMT == HILORE_FMT_INT8_BLK)
                cw[i] = cvt_s8x4(a0, a1, b0, b1); // |q| <= 127 (1 + 2^-23) here, so saturation at -128 cannot occur
            else
                cw[i] = cvt_e4m3x4(a0, a1, b0, b1);
        }
    }
    if (CODES)
        codes = make_uint4(cw[0], cw[1], cw[2], cw[3]);
    if (SUMS) {
        float lo, hi;
        f32x2_unpack(acc, lo, hi);
        sumsq = lo + hi;
    }
}

// Everything a thread does with the two chunks it holds.  All 32 lanes must call this together
// (xor-shuffles inside).  The four lanes of a quad hold one 64-element block per chunk.
//   CODES: the two quotients of a block (s = amax / Q, inv = Q / amax; IEEE divisions, or with LATER the scale
//          table) are spread over the quad: lanes 0 / 1 compute s / inv of chunk 0's block, lanes 2 / 3 those
//          of chunk 1's block -- one per thread instead of four.  `s_store` is the scale of chunk 0's block in lanes with
//          (lane & 3) == 0 and of chunk 1's block in lanes with (lane & 3) == 2.
//   SUMS:  `bsum` is the block sum of squares of chunk 0's block in even lanes, of chunk 1's in odd lanes.
//   LATER: blocks that need the careful rules (Inf, NaN, overflow of the unscaled cast) are only reported in
//          `careful`; their codes and scales come out wrong here and the caller repairs them with
//          careful_pair_fixup after its stores.  This keeps calls and their register traffic out of the loop.
//   `tab` (LATER only): the scale table of this format in shared memory; blocks whose amax lies outside the
//          table's range and is not a unit-scale block are reported as careful too.
template <int FMT, bool CODES, bool SUMS, bool LATER = false>
__device__ __forceinline__ void process_pair(const uint32_t (&w0)[8], const uint32_t (&w1)[8], int lane, uint4 &c0,
                                             uint4 &c1, float &s_store, float &bsum, bool &careful,
                                             const uint32_t *tab = nullptr)
{
    constexpr float Q = QMax<FMT>::value;
    float inv0 = 1.0f, inv1 = 1.0f;
    bool careful0 = false, careful1 = false;
    s_store = 1.0f;
    if (CODES) {
        uint32_t m0 = absmax16(w0), m1 = absmax16(w1);
        if (FMT == HILORE_FMT_E4M3FN_RAW) {
            careful0 = m0 > 0x43E8u;
            careful1 = m1 > 0x43E8u;
        } else {
            uint32_t mp = m0 | (m1 << 16); // both blocks' maxima ride in one register through the quad
            mp = maxnan_bf16x2(mp, __shfl_xor_sync(0xFFFFFFFFu, mp, 1));
            mp = maxnan_bf16x2(mp, __shfl_xor_sync(0xFFFFFFFFu, mp, 2));
            m0 = mp & 0xFFFFu;
            m1 = mp >> 16;
            if (!LATER) careful0 = careful1 = (m0 >= 0x7F80u) || (m1 >= 0x7F80u); // uniform over the quad
            if (!LATER && careful0) { // Inf or NaN in one of the two blocks: absmax over the finite elements only
                const uint32_t quad_mask = 0xFu << (lane & 28);
                uint32_t f0 = absmax16_finite(HILORE_LO4(w0), HILORE_HI4(w0));
                uint32_t f1 = absmax16_finite(HILORE_LO4(w1), HILORE_HI4(w1));
                f0 = max(f0, __shfl_xor_sync(quad_mask, f0, 1));
                f1 = max(f1, __shfl_xor_sync(quad_mask, f1, 1));
                m0 = max(f0, __shfl_xor_sync(quad_mask, f0, 2));
                m1 = max(f1, __shfl_xor_sync(quad_mask, f1, 2));
            }
            const int q = lane & 3;
            const bool unit0 = m0 <= UnitScaleBelow<FMT>::value, unit1 = m1 <= UnitScaleBelow<FMT>::value;
            float r; // s in even lanes, inv in odd lanes
            if (LATER) {
                constexpr uint32_t kFrom = TableScaleFrom<FMT>::value, kSpan = 0x7F80u - kFrom;
                careful0 = careful1 = (!unit0 && (m0 - kFrom) >= kSpan) || (!unit1 && (m1 - kFrom) >= kSpan);
                const uint32_t m = (q & 2) ? m1 : m0;
                const uint32_t t = tab[((q & 1) << 7) + (m & 0x7Fu)];
                r = __uint_as_float(t + (m & 0x7F80u) * ((q & 1) ? 0xFFFF0000u : 0x00010000u));
            } else {
                const float a = __uint_as_float(((q & 2) ? m1 : m0) << 16);
                r = __fdiv_rn((q & 1) ? Q : a, (q & 1) ? a : Q);
            }
            inv0 = __shfl_sync(0xFFFFFFFFu, r, (lane & 28) | 1);
            inv1 = __shfl_sync(0xFFFFFFFFu, r, (lane & 28) | 3);
            inv0 = unit0 ? 1.0f : inv0;
            inv1 = unit1 ? 1.0f : inv1;
            s_store = ((q & 2) ? unit1 : unit0) ? 1.0f : r;
        }
    }
    float ss0 = 0.0f, ss1 = 0.0f;
    chunk_pass<FMT, CODES, SUMS>(w0, inv0, c0, ss0);
    chunk_pass<FMT, CODES, SUMS>(w1, inv1, c1, ss1);
    if (CODES && !LATER) {
        if (careful0) c0 = encode16_careful<FMT>(HILORE_LO4(w0), HILORE_HI4(w0), inv0);
        if (careful1) c1 = encode16_careful<FMT>(HILORE_LO4(w1), HILORE_HI4(w1), inv1);
    }
    if (CODES && LATER)
        careful = careful0 || careful1;
    if (SUMS) { // quad reduction of both blocks' sums with two shuffles
        const bool odd = lane & 1;
        float keep = odd ? ss1 : ss0;
        keep += __shfl_xor_sync(0xFFFFFFFFu, odd ? ss0 : ss1, 1);
        keep += __shfl_xor_sync(0xFFFFFFFFu, keep, 2);
        bsum = keep;
    }
}

__device__ __forceinline__ void zero8(uint32_t (&w)[8])
{
#pragma unroll
    for (int i = 0; i < 8; ++i) w[i] = 0;
}

// Redo the two chunks of a thread with the full rule set and overwrite what the fast path stored for them.
// Rare (a block holds Inf or NaN; the unscaled cast meets a magnitude above 464), so it re-reads the chunks
// instead of keeping them alive.  For the block formats the condition is uniform over a quad and all four lanes
// come here together; xa / xb is nullptr where the thread has no chunk.  The scale slots are written by the
// same lanes as on the fast path (lane 0 of the quad for chunk a's block, lane 2 for chunk b's).
template <int FMT>
__device__ __forceinline__ void careful_pair_fixup(const uint16_t *xa, const uint16_t *xb, uint8_t *ca, uint8_t *cb, float *sa,
                                                float *sb, int lane)
{
    constexpr float Q = QMax<FMT>::value;
    uint32_t w0[8], w1[8];
    if (xa) ld_global_256(xa, w0);
    else zero8(w0);
    if (xb) ld_global_256(xb, w1);
    else zero8(w1);
    float inv0 = 1.0f, inv1 = 1.0f;
    if (FMT != HILORE_FMT_E4M3FN_RAW) {
        const uint32_t quad_mask = 0xFu << (lane & 28);
        uint32_t f0 = absmax16_finite_inl(HILORE_LO4(w0), HILORE_HI4(w0));
        uint32_t f1 = absmax16_finite_inl(HILORE_LO4(w1), HILORE_HI4(w1));
        f0 = max(f0, __shfl_xor_sync(quad_mask, f0, 1));
        f1 = max(f1, __shfl_xor_sync(quad_mask, f1, 1));
        f0 = max(f0, __shfl_xor_sync(quad_mask, f0, 2));
        f1 = max(f1, __shfl_xor_sync(quad_mask, f1, 2));
        const float a0 = __uint_as_float(f0 << 16), a1 = __uint_as_float(f1 << 16);
        const bool unit0 = f0 <= UnitScaleBelow<FMT>::value, unit1 = f1 <= UnitScaleBelow<FMT>::value;
        inv0 = unit0 ? 1.0f : __fdiv_rn(Q, a0);
        inv1 = unit1 ? 1.0f : __fdiv_rn(Q, a1);
        const int q = lane & 3;
        if (q == 0 && xa) *sa = unit0 ? 1.0f : __fdiv_rn(a0, Q);
        if (q == 2 && xb) *sb = unit1 ? 1.0f : __fdiv_rn(a1, Q);
    }
    if (xa) *reinterpret_cast<uint4 *>(ca) = encode16_careful_inl<FMT>(HILORE_LO4(w0), HILORE_HI4(w0), inv0);
    if (xb) *reinterpret_cast<uint4 *>(cb) = encode16_careful_inl<FMT>(HILORE_LO4(w1), HILORE_HI4(w1), inv1);
}

// Compress (CODES) and / or collect the token RMS (SUMS) of rows [r0, r1) of one unit.
template <int FMT, bool CODES, bool SUMS>
__device__ __forceinline__ void compress_rows(const uint16_t *__restrict__ x, uint8_t *__restrict__ codes,
                                              float *__restrict__ scales, float *__restrict__ row_rms, int64_t cols,
                                              int64_t ld, int64_t r0, int64_t r1, int rows_per_batch, float *sm_blocksum,
                                              int prefetch, const uint32_t *tab)
{
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, q = lane & 3;
    const uint32_t nb = (uint32_t)(cols >> 6), cpr = (uint32_t)(cols >> 4);
    const uint32_t magic = (uint32_t)((0x100000000ull + cpr - 1) / cpr); // chunk index (< 2^16) / cpr, exactly
    const float inv_cols = 1.0f / (float)cols;
    const bool contig = ld == cols;

    for (int64_t rb0 = r0; rb0 < r1; rb0 += rows_per_batch) {
        const int rb = (int)min((int64_t)rows_per_batch, r1 - rb0);
        const uint32_t n = (uint32_t)rb * cpr; // chunks of this batch (a multiple of 4), <= 4 * kBlockSumSlots
        const uint16_t *xb = x + rb0 * ld;
        uint8_t *cb_ = codes + rb0 * cols;
        float *sb = scales + rb0 * (int64_t)nb;
        uint32_t base = 0;
        if (contig) { // whole iterations: no predicates, pointer increments only
            const uint16_t *xp = xb + (size_t)tid * 16;
            uint8_t *cp = cb_ + (size_t)tid * 16;
            float *sp = sb + (tid >> 2);
            float *bp = sm_blocksum + (tid >> 2);
            // One iteration of the CTA reads 16 KB contiguously.  An elected thread keeps the copy engine
            // `prefetch` iterations ahead, pulling those 16 KB pieces from HBM into L2, so that the warps'
            // own loads find their data in L2 and HBM traffic no longer waits for warp progress.
            constexpr uint32_t kIterBytes = 2 * kCodecThreads * 32;
            const uint32_t full_iters = n / (2 * kCodecThreads);
            const uint8_t *pf = reinterpret_cast<const uint8_t *>(xb);
            if (tid == 0)
                for (uint32_t k = 0; k < (uint32_t)prefetch && k < full_iters; ++k) prefetch_l2_bulk(pf + (size_t)k * kIterBytes, kIterBytes);
            // In a long batch the warps of a CTA drift apart and away from the elected thread's run-ahead; a barrier
            // every four iterations holds them together (+3 to +6 % on units of 0.5 GiB and more; short batches, as
            // in a microbatch of many units, are better off without it).
            const uint32_t sync_mask = full_iters >= 16 ? 3u : 0xFFFFFFFFu;
            uint32_t iter = 0;
            for (; base + 2 * kCodecThreads <= n; base += 2 * kCodecThreads, ++iter) {
                if (tid == 0 && prefetch > 0 && iter + prefetch < full_iters)
                    prefetch_l2_bulk(pf + (size_t)(iter + prefetch) * kIterBytes, kIterBytes);
                uint32_t wa[8], wb[8];
                ld_global_256(xp, wa);
                ld_global_256(xp + kCodecThreads * 16, wb);
                uint4 qa, qb;
                float s, ss;
                bool careful = false;
                process_pair<FMT, CODES, SUMS, true>(wa, wb, lane, qa, qb, s, ss, careful, tab);
                if (CODES) {
                    __stcs(reinterpret_cast<uint4 *>(cp), qa);
                    __stcs(reinterpret_cast<uint4 *>(cp + kCodecThreads * 16), qb);
                    if (FMT != HILORE_FMT_E4M3FN_RAW) {
                        if (q == 0) sp[0] = s;
                        if (q == 2) sp[kCodecThreads / 4] = s;
                    }
                    if (careful)
                        careful_pair_fixup<FMT>(xp, xp + kCodecThreads * 16, cp, cp + kCodecThreads * 16, sp,
                                                sp + kCodecThreads / 4, lane);
                }
                if (SUMS) {
                    if (q == 0) bp[0] = ss;
                    if (q == 1) bp[kCodecThreads / 4] = ss;
                }
                if ((iter & sync_mask) == 3u) __syncthreads(); // long batch: keep the warps behind the run-ahead
                xp += 2 * kCodecThreads * 16;
                cp += 2 * kCodecThreads * 16;
                sp += 2 * kCodecThreads / 4;
                bp += 2 * kCodecThreads / 4;
            }
        }
        for (; base < n; base += 2 * kCodecThreads) { // ragged end of a batch, or rows with a leading dimension
            const uint32_t ca = base + tid, cb = ca + kCodecThreads;
            const bool va = ca < n, vb = cb < n; // quads are valid as a whole (n is a multiple of 4)
            uint32_t wa[8], wb[8];
            zero8(wa);
            zero8(wb);
            const uint16_t *xa_ptr = nullptr, *xb_ptr = nullptr;
            if (va) {
                const uint32_t r = __umulhi(ca, magic);
                xa_ptr = xb + (int64_t)r * ld + (int64_t)(ca - r * cpr) * 16;
                ld_global_256(xa_ptr, wa);
            }
            if (vb) {
                const uint32_t r = __umulhi(cb, magic);
                xb_ptr = xb + (int64_t)r * ld + (int64_t)(cb - r * cpr) * 16;
                ld_global_256(xb_ptr, wb);
            }
            uint4 qa, qb;
            float s, ss;
            bool careful = false;
            process_pair<FMT, CODES, SUMS, true>(wa, wb, lane, qa, qb, s, ss, careful, tab);
            if (CODES) {
                if (va) *reinterpret_cast<uint4 *>(cb_ + (size_t)ca * 16) = qa;
                if (vb) *reinterpret_cast<uint4 *>(cb_ + (size_t)cb * 16) = qb;
                if (FMT != HILORE_FMT_E4M3FN_RAW) {
                    if (q == 0 && va) sb[ca >> 2] = s;
                    if (q == 2 && vb) sb[cb >> 2] = s;
                }
                if (careful)
                    careful_pair_fixup<FMT>(va ? xa_ptr : nullptr, vb ? xb_ptr : nullptr, cb_ + (size_t)ca * 16,
                                            cb_ + (size_t)cb * 16, sb + (ca >> 2), sb + (cb >> 2), lane);
            }
            if (SUMS) {
                if (q == 0 && va) sm_blocksum[ca >> 2] = ss;
                if (q == 1 && vb) sm_blocksum[cb >> 2] = ss;
            }
        }
        if (SUMS) {
            __syncthreads();
            for (int r = wid; r < rb; r += kCodecThreads / 32) {
                double acc = 0.0;
                for (uint32_t b = lane; b < nb; b += 32)
                    acc += (double)sm_blocksum[(uint32_t)r * nb + b];
                acc = warp_sum(acc);
                if (lane == 0)
                    row_rms[rb0 + r] = sqrtf((float)acc * inv_cols);
            }
            __syncthreads();
        } else {
            // Without the row reduction nothing else holds the warps of a CTA together, and they drift away from
            // the elected thread's run-ahead: one barrier per batch keeps them behind it (+25 % on multi-GB units).
            __syncthreads();
        }
    }
}

// Sixteen codes -> sixteen bf16 (eight words).
template <int FMT> __device__ __forceinline__ void decode16(const uint4 cd, float s, uint32_t (&o)[8])
{
    const uint64_t s2 = f32x2_pack(s, s);
    const uint32_t cw[4] = {cd.x, cd.y, cd.z, cd.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int p = 0; p < 2; ++p) {
            const uint32_t two = p ? (cw[i] >> 16) : (cw[i] & 0xFFFFu); // two codes
            float f0, f1;
            if (FMT == HILORE_FMT_INT8_BLK) {
                f0 = (float)(int)(int8_t)(two & 0xFF);
                f1 = (float)(int)(int8_t)(two >> 8);
            } else {
                const uint32_t hh = cvt_e4m3x2_to_f16x2(two);
                f0 = f16_lo_to_f32(hh);
                f1 = f16_hi_to_f32(hh);
            }
            if (FMT != HILORE_FMT_E4M3FN_RAW) {
                const uint64_t y = f32x2_mul(f32x2_pack(f0, f1), s2); // fl32(value * s) per lane
                f32x2_unpack(y, f0, f1);
            }
            o[2 * i + p] = cvt_bf16x2(f1, f0);
        }
        if (FMT == HILORE_FMT_INT8_BLK) { // code 0x80 is the reserved NaN: rare, patched per word
            const uint32_t is_nan = __vcmpeq4(cw[i], 0x80808080u); // 0xFF in every byte that holds 0x80
            if (is_nan) {
                const uint32_t lo = __byte_perm(is_nan, 0, 0x1100), hi = __byte_perm(is_nan, 0, 0x3322);
                o[2 * i] = (o[2 * i] & ~lo) | (0x7FC07FC0u & lo);
                o[2 * i + 1] = (o[2 * i + 1] & ~hi) | (0x7FC07FC0u & hi);
            }
        }
    }
}

// Decode rows [r0, r1) of one unit.
template <int FMT>
__device__ __forceinline__ void recover_rows(const uint8_t *__restrict__ codes, const float *__restrict__ scales,
                                             uint16_t *__restrict__ out, int64_t cols, int64_t ld, int64_t r0, int64_t r1,
                                             int prefetch)
{
    constexpr int UNR = 4;
    const int tid = threadIdx.x;
    const int64_t nb = cols >> 6, cpr = cols >> 4;
    const int64_t n = (r1 - r0) * cpr; // chunks of this CTA's rows
    const uint8_t *cb_ = codes + r0 * cols;
    const float *sb = scales + r0 * nb;
    int64_t base = 0;
    if (ld == cols) {
        const uint8_t *cp = cb_ + (size_t)tid * 16;
        const float *sp = sb + (tid >> 2);
        uint16_t *op = out + r0 * ld + (size_t)tid * 16;
        constexpr uint32_t kIterBytes = UNR * kCodecThreads * 16; // codes read per iteration of the CTA
        const int64_t full_iters = n / (UNR * kCodecThreads);
        if (tid == 0)
            for (int64_t k = 0; k < prefetch && k < full_iters; ++k) prefetch_l2_bulk(cb_ + k * kIterBytes, kIterBytes);
        int64_t iter = 0;
        for (; base + UNR * kCodecThreads <= n; base += UNR * kCodecThreads, ++iter) {
            if (tid == 0 && prefetch > 0 && iter + prefetch < full_iters)
                prefetch_l2_bulk(cb_ + (iter + prefetch) * kIterBytes, kIterBytes);
            uint4 cd[UNR];
            float s[UNR];
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                cd[j] = ld_global_128_stream(cp + (size_t)j * kCodecThreads * 16);
                s[j] = (FMT != HILORE_FMT_E4M3FN_RAW) ? __ldg(sp + j * (kCodecThreads / 4)) : 1.0f;
            }
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                uint32_t o[8];
                decode16<FMT>(cd[j], s[j], o);
                st_global_256(op + (size_t)j * kCodecThreads * 16, o);
            }
            cp += UNR * kCodecThreads * 16;
            sp += UNR * kCodecThreads / 4;
            op += UNR * kCodecThreads * 16;
        }
    }
    for (; base < n; base += kCodecThreads) {
        const int64_t c = base + tid;
        if (c < n) {
            const uint4 cd = ld_global_128_stream(cb_ + c * 16);
            const float s = (FMT != HILORE_FMT_E4M3FN_RAW) ? __ldg(sb + (c >> 2)) : 1.0f;
            uint32_t o[8];
            decode16<FMT>(cd, s, o);
            const int64_t r = c / cpr;
            st_global_256(out + (r0 + r) * ld + (c - r * cpr) * 16, o);
        }
    }
}


// ---- bulk stores (copy engine): shared memory -> global, tracked in per-thread groups ----
__device__ __forceinline__ void bulk_s2g(void *dst_gmem, const void *src_smem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst_gmem),
                 "r"((uint32_t)__cvta_generic_to_shared(src_smem)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all but the newest N bulk-store groups of this thread have finished reading shared memory
template <int N> __device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// make this thread's shared-memory writes visible to the copy engine
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

constexpr int kRecoverTileChunks = 2 * kCodecThreads;        // 512 chunks = 8192 elements per tile
constexpr int kRecoverTileBytes = kRecoverTileChunks * 32;   // 16 KB of bf16
constexpr int kRecoverStageBytes = 2 * kRecoverTileBytes;    // two tiles in shared memory

// Decode rows [r0, r1) of a unit (contiguous, or rows of at least 2 KB with a leading dimension).  The pass
// writes twice what it reads, and HBM takes writes best in large contiguous bursts: each tile of 8192 reconstructed values is assembled in
// shared memory and sent with one 16 KB bulk store while the threads work on the next tile (two buffers;
// a buffer is refilled only after the store that read it has finished reading).
// `tile` counts this CTA's tiles across calls, so the two buffers keep alternating from unit to unit.
template <int FMT>
__device__ __forceinline__ void recover_rows_bulk(const uint8_t *__restrict__ codes, const float *__restrict__ scales,
                                                  uint16_t *__restrict__ out, int64_t cols, int64_t ld, int64_t r0,
                                                  int64_t r1, uint8_t *sm_out, uint32_t &tile, int prefetch)
{
    const int tid = threadIdx.x;
    const int64_t nb = cols >> 6, cpr = cols >> 4;
    const int64_t n = (r1 - r0) * cpr; // chunks of this CTA's rows
    const uint8_t *cb_ = codes + r0 * cols;
    const float *sb = scales + r0 * nb;
    uint8_t *ob = reinterpret_cast<uint8_t *>(out + r0 * ld);
    const int64_t ntiles = (n + kRecoverTileChunks - 1) / kRecoverTileChunks;
    if (tid == 0)
        for (int64_t k = 0; k < prefetch && k < ntiles; ++k)
            prefetch_l2_bulk(cb_ + k * kRecoverTileChunks * 16, (uint32_t)min((int64_t)kRecoverTileChunks, n - k * kRecoverTileChunks) * 16);
    for (int64_t t = 0; t < ntiles; ++t, ++tile) {
        const int64_t base = t * kRecoverTileChunks;
        if (tid == 0 && prefetch > 0 && t + prefetch < ntiles)
            prefetch_l2_bulk(cb_ + (t + prefetch) * kRecoverTileChunks * 16,
                             (uint32_t)min((int64_t)kRecoverTileChunks, n - (t + prefetch) * kRecoverTileChunks) * 16);
        const int64_t ca = base + tid, cb = ca + kCodecThreads;
        const bool va = ca < n, vb = cb < n;
        uint4 cda = make_uint4(0, 0, 0, 0), cdb = cda;
        float sa = 1.0f, sb_ = 1.0f;
        if (va) {
            cda = ld_global_128_stream(cb_ + ca * 16);
            if (FMT != HILORE_FMT_E4M3FN_RAW) sa = __ldg(sb + (ca >> 2));
        }
        if (vb) {
            cdb = ld_global_128_stream(cb_ + cb * 16);
            if (FMT != HILORE_FMT_E4M3FN_RAW) sb_ = __ldg(sb + (cb >> 2));
        }
        uint32_t oa[8], ob2[8];
        decode16<FMT>(cda, sa, oa);
        decode16<FMT>(cdb, sb_, ob2);
        uint8_t *buf = sm_out + (tile & 1u) * kRecoverTileBytes;
        if (tid == 0)
            bulk_wait_read<1>(); // the store issued two tiles ago (same buffer) has finished reading it
        __syncthreads();
        uint4 *pa = reinterpret_cast<uint4 *>(buf + (size_t)tid * 32);
        uint4 *pb = reinterpret_cast<uint4 *>(buf + (size_t)(tid + kCodecThreads) * 32);
        pa[0] = make_uint4(oa[0], oa[1], oa[2], oa[3]);
        pa[1] = make_uint4(oa[4], oa[5], oa[6], oa[7]);
        pb[0] = make_uint4(ob2[0], ob2[1], ob2[2], ob2[3]);
        pb[1] = make_uint4(ob2[4], ob2[5], ob2[6], ob2[7]);
        fence_async_smem();
        __syncthreads();
        if (tid == 0) {
            const int64_t cnt = min((int64_t)kRecoverTileChunks, n - base);
            if (ld == cols) {
                bulk_s2g(ob + base * 32, buf, (uint32_t)cnt * 32u);
            } else { // rows with a leading dimension: one store per piece of a row inside the tile, one group per tile
                for (int64_t c = base; c < base + cnt;) {
                    const int64_t row = c / cpr, col = c - row * cpr;
                    const int64_t seg = min(cpr - col, base + cnt - c);
                    bulk_s2g(ob + (row * ld + col * 16) * 2, buf + (c - base) * 32, (uint32_t)seg * 32u);
                    c += seg;
                }
            }
            bulk_commit();
        }
    }
}

} // namespace hilore
