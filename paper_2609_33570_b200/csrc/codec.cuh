// Streaming codec of the L action: bf16 -> FP8 E4M3FN / INT8 codes (+ per-block scales, + token RMS)
// and back.  Paper: Eq. "fp8-roundtrip" (unscaled cast) and Eq. "activation-token-weights" (a_t).
//
// Work split.  A CTA owns a contiguous range of rows of a unit.  A thread owns 16 consecutive
// elements ("chunk": one 256-bit load, one 128-bit store of codes); four neighbouring lanes own one
// 64-element block, so the block absmax and the block sum of squares are two xor-shuffles.  Rows
// are swept in batches small enough that the per-block sums of squares of a batch fit in shared
// memory; at the end of a batch each warp adds the blocks of whole rows in a fixed order, so the
// token RMS is deterministic (no floating-point atomics anywhere).
#pragma once

#include "common.cuh"

namespace hilore {

enum CodecOp { OP_NONE = 0, OP_COMPRESS = 1, OP_STATS = 2, OP_RECOVER = 3 };

template <int FMT> struct QMax {
    static constexpr float value = (FMT == HILORE_FMT_INT8_BLK) ? 127.0f : 448.0f;
};

__device__ __forceinline__ uint32_t int8_code(float q)
{
    int v = __float2int_rn(q);
    v = max(-127, min(127, v));
    return (uint32_t)v & 0xFFu;
}

// Sixteen elements, every one finite (BLK) / none above 464 in magnitude (RAW).
template <int FMT> __device__ __forceinline__ uint4 encode16_fast(const uint32_t (&w)[8], float inv)
{
    uint32_t c[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float e0 = bf16_lo(w[2 * i]), e1 = bf16_hi(w[2 * i]);
        float e2 = bf16_lo(w[2 * i + 1]), e3 = bf16_hi(w[2 * i + 1]);
        if (FMT != HILORE_FMT_E4M3FN_RAW) {
            e0 = __fmul_rn(e0, inv);
            e1 = __fmul_rn(e1, inv);
            e2 = __fmul_rn(e2, inv);
            e3 = __fmul_rn(e3, inv);
        }
        if (FMT == HILORE_FMT_INT8_BLK)
            c[i] = int8_code(e0) | (int8_code(e1) << 8) | (int8_code(e2) << 16) | (int8_code(e3) << 24);
        else
            c[i] = cvt_e4m3x2(e1, e0) | (cvt_e4m3x2(e3, e2) << 16);
    }
    return make_uint4(c[0], c[1], c[2], c[3]);
}

// One element with the full rule set (overflow, Inf, NaN).  Rare path.
template <int FMT> __device__ __noinline__ uint32_t encode1_careful(uint32_t bits, float inv)
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

template <int FMT> __device__ __noinline__ uint4 encode16_careful(const uint32_t (&w)[8], float inv)
{
    uint32_t c[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        c[i] = encode1_careful<FMT>(w[2 * i] & 0xFFFFu, inv) | (encode1_careful<FMT>(w[2 * i] >> 16, inv) << 8) |
               (encode1_careful<FMT>(w[2 * i + 1] & 0xFFFFu, inv) << 16) |
               (encode1_careful<FMT>(w[2 * i + 1] >> 16, inv) << 24);
    }
    return make_uint4(c[0], c[1], c[2], c[3]);
}

// max |bits| over the finite elements only
__device__ __noinline__ uint32_t absmax_bits16_finite(const uint32_t (&w)[8])
{
    uint32_t m = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        uint32_t lo = w[i] & 0x7FFFu, hi = (w[i] >> 16) & 0x7FFFu;
        if (lo < 0x7F80u) m = max(m, lo);
        if (hi < 0x7F80u) m = max(m, hi);
    }
    return m;
}

__device__ __forceinline__ float sumsq16(const uint32_t (&w)[8])
{
    float a = 0.0f, b = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float lo = bf16_lo(w[i]), hi = bf16_hi(w[i]);
        a = fmaf(lo, lo, a);
        b = fmaf(hi, hi, b);
    }
    return a + b;
}

struct RowGeom {
    int64_t cols, ld;   // elements
    uint32_t cpr;       // 16-element chunks per row
    uint32_t nb;        // 64-element blocks per row
    uint32_t magic;     // ceil(2^32 / cpr): exact division of chunk indices < 2^16 by cpr
    int rows_per_batch; // rows swept between two row reductions
};

__device__ __forceinline__ RowGeom make_geom(int64_t cols, int64_t ld)
{
    RowGeom g;
    g.cols = cols;
    g.ld = ld;
    g.cpr = (uint32_t)(cols >> 4);
    g.nb = (uint32_t)(cols >> 6);
    g.magic = (uint32_t)((0x100000000ull + g.cpr - 1) / g.cpr);
    g.rows_per_batch = max(1, kBlockSumSlots / (int)g.nb);
    return g;
}

// Element offset of chunk c (within a batch that starts at row `row0`) in a [rows, ld] tensor.
__device__ __forceinline__ int64_t chunk_offset(const RowGeom &g, int64_t row0, uint32_t c, int64_t ld)
{
    if (ld == g.cols)
        return row0 * ld + (int64_t)c * 16;
    uint32_t r = __umulhi(c, g.magic);
    uint32_t cc = c - r * g.cpr;
    return (row0 + r) * ld + (int64_t)cc * 16;
}

// Compress (CODES) and / or collect the token RMS of rows [r0, r1) of one unit.
template <int FMT, bool CODES, int UNR>
__device__ void compress_rows(const hilore_unit &u, int64_t r0, int64_t r1, float *sm_blocksum)
{
    const RowGeom g = make_geom(u.cols, u.ld);
    const uint16_t *x = static_cast<const uint16_t *>(u.x);
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const uint32_t quad_mask = 0xFu << (lane & 28);
    const bool want_rms = (u.row_rms != nullptr);
    constexpr float Q = QMax<FMT>::value;

    for (int64_t rb0 = r0; rb0 < r1; rb0 += g.rows_per_batch) {
        const int rb = (int)min((int64_t)g.rows_per_batch, r1 - rb0);
        const uint32_t n = (uint32_t)rb * g.cpr; // chunks of this batch, <= 4 * kBlockSumSlots
        for (uint32_t base = 0; base < n; base += kCodecThreads * UNR) {
            uint32_t w[UNR][8];
            bool valid[UNR];
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                const uint32_t c = base + j * kCodecThreads + tid;
                valid[j] = c < n;
                if (valid[j]) {
                    ld_global_256(x + chunk_offset(g, rb0, c, g.ld), w[j]);
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) w[j][i] = 0;
                }
            }
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                const uint32_t c = base + j * kCodecThreads + tid;
                // n is a multiple of 4 and quads start at multiples of 4: a quad is valid as a whole
                if (CODES) {
                    uint32_t mm = absmax_bits16(w[j]);
                    float s = 1.0f, inv = 1.0f;
                    bool careful;
                    if (FMT == HILORE_FMT_E4M3FN_RAW) {
                        careful = mm > 0x43E8u;
                    } else {
                        mm = max(mm, __shfl_xor_sync(0xFFFFFFFFu, mm, 1));
                        mm = max(mm, __shfl_xor_sync(0xFFFFFFFFu, mm, 2));
                        careful = mm >= 0x7F80u;
                        if (careful) { // the block holds Inf or NaN: absmax over its finite elements
                            mm = absmax_bits16_finite(w[j]);
                            mm = max(mm, __shfl_xor_sync(quad_mask, mm, 1));
                            mm = max(mm, __shfl_xor_sync(quad_mask, mm, 2));
                        }
                        if (mm != 0) {
                            const float amax = __uint_as_float(mm << 16);
                            s = __fdiv_rn(amax, Q);
                            inv = __fdiv_rn(Q, amax);
                            if (isinf(inv)) {
                                s = 1.0f;
                                inv = 1.0f;
                            }
                        }
                    }
                    if (valid[j]) {
                        const uint4 codes = careful ? encode16_careful<FMT>(w[j], inv) : encode16_fast<FMT>(w[j], inv);
                        const int64_t flat = rb0 * g.cols + (int64_t)c * 16;
                        *reinterpret_cast<uint4 *>(u.codes + flat) = codes;
                        if (FMT != HILORE_FMT_E4M3FN_RAW && (lane & 3) == 0)
                            u.scales[rb0 * g.nb + (c >> 2)] = s;
                    }
                }
                if (want_rms) {
                    float ss = sumsq16(w[j]);
                    ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 1);
                    ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 2);
                    if (valid[j] && (lane & 3) == 0)
                        sm_blocksum[c >> 2] = ss;
                }
            }
        }
        if (want_rms) {
            __syncthreads();
            for (int r = wid; r < rb; r += kCodecThreads / 32) {
                double acc = 0.0;
                for (uint32_t b = lane; b < g.nb; b += 32)
                    acc += (double)sm_blocksum[(uint32_t)r * g.nb + b];
                acc = warp_sum(acc);
                if (lane == 0)
                    u.row_rms[rb0 + r] = (float)sqrt(acc / (double)g.cols);
            }
            __syncthreads();
        }
    }
}

// Decode rows [r0, r1) of one unit into u.out.
template <int FMT, int UNR> __device__ void recover_rows(const hilore_unit &u, int64_t r0, int64_t r1)
{
    const RowGeom g = make_geom(u.cols, u.ld);
    uint16_t *out = static_cast<uint16_t *>(u.out);
    const int tid = threadIdx.x;
    for (int64_t rb0 = r0; rb0 < r1; rb0 += g.rows_per_batch) {
        const int rb = (int)min((int64_t)g.rows_per_batch, r1 - rb0);
        const uint32_t n = (uint32_t)rb * g.cpr;
        for (uint32_t base = 0; base < n; base += kCodecThreads * UNR) {
            uint4 cd[UNR];
            float s[UNR];
            bool valid[UNR];
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                const uint32_t c = base + j * kCodecThreads + tid;
                valid[j] = c < n;
                s[j] = 1.0f;
                cd[j] = make_uint4(0, 0, 0, 0);
                if (valid[j]) {
                    cd[j] = ld_global_128_stream(u.codes + rb0 * g.cols + (int64_t)c * 16);
                    if (FMT != HILORE_FMT_E4M3FN_RAW)
                        s[j] = __ldg(u.scales + rb0 * g.nb + (c >> 2));
                }
            }
#pragma unroll
            for (int j = 0; j < UNR; ++j) {
                if (!valid[j])
                    continue;
                const uint32_t c = base + j * kCodecThreads + tid;
                const uint32_t cw[4] = {cd[j].x, cd[j].y, cd[j].z, cd[j].w};
                uint32_t o[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float f0, f1, f2, f3;
                    if (FMT == HILORE_FMT_INT8_BLK) {
                        const int b0 = (int)(int8_t)(cw[i] & 0xFF), b1 = (int)(int8_t)((cw[i] >> 8) & 0xFF);
                        const int b2 = (int)(int8_t)((cw[i] >> 16) & 0xFF), b3 = (int)(int8_t)(cw[i] >> 24);
                        const float qnan = __uint_as_float(0x7FC00000u);
                        f0 = (b0 == -128) ? qnan : (float)b0;
                        f1 = (b1 == -128) ? qnan : (float)b1;
                        f2 = (b2 == -128) ? qnan : (float)b2;
                        f3 = (b3 == -128) ? qnan : (float)b3;
                    } else {
                        const uint32_t h01 = cvt_e4m3x2_to_f16x2(cw[i] & 0xFFFFu);
                        const uint32_t h23 = cvt_e4m3x2_to_f16x2(cw[i] >> 16);
                        f0 = f16_lo_to_f32(h01);
                        f1 = f16_hi_to_f32(h01);
                        f2 = f16_lo_to_f32(h23);
                        f3 = f16_hi_to_f32(h23);
                    }
                    if (FMT != HILORE_FMT_E4M3FN_RAW) {
                        f0 = __fmul_rn(f0, s[j]);
                        f1 = __fmul_rn(f1, s[j]);
                        f2 = __fmul_rn(f2, s[j]);
                        f3 = __fmul_rn(f3, s[j]);
                    }
                    o[2 * i] = cvt_bf16x2(f1, f0);
                    o[2 * i + 1] = cvt_bf16x2(f3, f2);
                }
                st_global_256(out + chunk_offset(g, rb0, c, g.ld), o);
            }
        }
    }
}

} // namespace hilore
