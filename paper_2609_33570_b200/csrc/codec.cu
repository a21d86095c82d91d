// Entry points of the store / recover path: hilore_compress, hilore_recover, hilore_plan_apply.
// One kernel serves all three: every CTA walks the unit table, decides per unit (from the gating
// arrays in device memory) what to do, and processes its share of the unit's rows.  A whole
// microbatch of units therefore costs one launch per phase and no host synchronisation.
#include "codec.cuh"

namespace hilore {

struct CodecWork {
    const hilore_unit *units; // device table, or nullptr => `single`
    hilore_unit single;
    int U;
    int phase;                // HILORE_PHASE_* for table mode; CodecOp for single mode
    const uint8_t *avail;     // q_u
    const uint8_t *action;    // a_u
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

template <int UNR>
__global__ void __launch_bounds__(kCodecThreads) codec_kernel(const __grid_constant__ CodecWork wk)
{
    __shared__ float sm_blocksum[kBlockSumSlots];
    const int64_t nC = gridDim.x, cta = blockIdx.x;
    for (int ui = 0; ui < wk.U; ++ui) {
        const int op = unit_op(wk, ui);
        if (op == OP_NONE)
            continue;
        hilore_unit u = wk.units ? wk.units[ui] : wk.single;
        // balanced contiguous row ranges: CTA c owns rows [rows*c/nC, rows*(c+1)/nC)
        const int64_t r0 = (u.rows * cta) / nC, r1 = (u.rows * (cta + 1)) / nC;
        if (r0 >= r1)
            continue;
        const bool scaled = u.fmt != HILORE_FMT_E4M3FN_RAW;
        if ((op == OP_COMPRESS && (!u.x || !u.codes || (scaled && !u.scales))) || (op == OP_STATS && !u.x) ||
            (op == OP_RECOVER && (!u.out || !u.codes || (scaled && !u.scales))))
            continue; // the unit lacks a buffer this operation needs: leave it untouched
        if (op == OP_STATS) {
            if (u.row_rms != nullptr)
                compress_rows<HILORE_FMT_E4M3FN_RAW, false, UNR>(u, r0, r1, sm_blocksum);
            continue;
        }
        if (op == OP_COMPRESS && wk.units && wk.phase == HILORE_PHASE_ENCODE)
            u.row_rms = nullptr; // token magnitudes were collected at capture time
        switch (u.fmt) {
        case HILORE_FMT_E4M3FN_RAW:
            if (op == OP_COMPRESS) compress_rows<HILORE_FMT_E4M3FN_RAW, true, UNR>(u, r0, r1, sm_blocksum);
            else recover_rows<HILORE_FMT_E4M3FN_RAW, UNR>(u, r0, r1);
            break;
        case HILORE_FMT_E4M3FN_BLK:
            if (op == OP_COMPRESS) compress_rows<HILORE_FMT_E4M3FN_BLK, true, UNR>(u, r0, r1, sm_blocksum);
            else recover_rows<HILORE_FMT_E4M3FN_BLK, UNR>(u, r0, r1);
            break;
        case HILORE_FMT_INT8_BLK:
            if (op == OP_COMPRESS) compress_rows<HILORE_FMT_INT8_BLK, true, UNR>(u, r0, r1, sm_blocksum);
            else recover_rows<HILORE_FMT_INT8_BLK, UNR>(u, r0, r1);
            break;
        default:
            break;
        }
    }
}

// psi, threshold rule, availability demotion, recompute flags and retained bytes for U units.
__global__ void plan_decide_kernel(const hilore_unit *units, int U, const float *exposure, const float *kappa,
                                   const float *ebar, float tau_lo, float tau_hi, const uint8_t *avail,
                                   uint8_t *action_io, float *psi, uint8_t *recompute, uint64_t *retained_bytes)
{
    for (int u = blockIdx.x * blockDim.x + threadIdx.x; u < U; u += gridDim.x * blockDim.x) {
        uint32_t want = action_io[u];
        if (exposure != nullptr) {
            const float p = __fmul_rn(__fmul_rn(kappa[u], exposure[u]), ebar[u]);
            if (psi) psi[u] = p;
            want = (p < tau_lo) ? HILORE_ACT_L : ((p >= tau_hi) ? HILORE_ACT_H : HILORE_ACT_R);
        }
        const uint32_t q = avail[u];
        const bool ok = (q == HILORE_ACT_H) || (q == HILORE_ACT_L && want != HILORE_ACT_H) || (want == HILORE_ACT_R);
        uint32_t a = (ok && want <= HILORE_ACT_L) ? want : (uint32_t)HILORE_ACT_R;
        action_io[u] = (uint8_t)a;
        if (recompute) recompute[u] = (a == HILORE_ACT_R);
        if (retained_bytes) {
            const uint64_t n = (uint64_t)units[u].rows * (uint64_t)units[u].cols;
            uint64_t b = 0;
            if (a == HILORE_ACT_H) b = 2 * n;
            else if (a == HILORE_ACT_L) b = n + (units[u].fmt == HILORE_FMT_E4M3FN_RAW ? 0 : 4 * (n / HILORE_BLOCK));
            retained_bytes[u] = b;
        }
    }
}

// Host-side validation of one unit descriptor.  `strict` (single-unit entry points): the buffers the
// operation needs must be present.  Table mode: shapes and the alignment of whatever is present are
// checked here; a unit whose gate selects an operation for which it lacks a buffer is skipped on the
// device (the gates live in device memory, so the host cannot know which units will run).
static int check_unit(const hilore_unit &u, bool strict, bool need_x, bool need_codes, bool need_out)
{
    if (u.rows < 0 || u.cols <= 0)
        return HILORE_INVALID_ARG;
    if (u.fmt != HILORE_FMT_E4M3FN_RAW && u.fmt != HILORE_FMT_E4M3FN_BLK && u.fmt != HILORE_FMT_INT8_BLK)
        return HILORE_INVALID_ARG;
    if (u.fmt == HILORE_FMT_E4M3FN_RAW ? (u.block != 0) : (u.block != HILORE_BLOCK))
        return HILORE_INVALID_ARG;
    if (u.cols % HILORE_BLOCK != 0 || u.cols > (int64_t)kBlockSumSlots * HILORE_BLOCK)
        return HILORE_SHAPE;
    if (u.ld < u.cols)
        return HILORE_SHAPE;
    if (u.ld % 16 != 0)
        return HILORE_ALIGN;
    if (strict) {
        if (need_x && u.x == nullptr)
            return HILORE_INVALID_ARG;
        if (need_out && u.out == nullptr)
            return HILORE_INVALID_ARG;
        if (need_codes && (u.codes == nullptr || (u.fmt != HILORE_FMT_E4M3FN_RAW && u.scales == nullptr)))
            return HILORE_INVALID_ARG;
    }
    if (!aligned(u.x, 32) || !aligned(u.out, 32) || !aligned(u.codes, 16) || !aligned(u.scales, 4) ||
        !aligned(u.row_rms, 4))
        return HILORE_ALIGN;
    return HILORE_OK;
}

static int launch_codec(const CodecWork &wk, int64_t max_rows, cudaStream_t st)
{
    if (max_rows <= 0)
        return HILORE_OK;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, codec_kernel<2>, kCodecThreads, 0) != cudaSuccess ||
        per_sm <= 0)
        per_sm = 2;
    int64_t grid = (int64_t)sm_count() * per_sm;
    if (grid > max_rows)
        grid = max_rows;
    codec_kernel<2><<<(unsigned)grid, kCodecThreads, 0, st>>>(wk);
    return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
}

} // namespace hilore

using namespace hilore;

extern "C" int hilore_compress(const void *x, int64_t rows, int64_t cols, int64_t ld, int32_t fmt, int32_t block,
                               uint8_t *codes, float *scales, float *row_rms, void *stream)
{
    hilore_unit u{};
    u.x = x;
    u.codes = codes;
    u.scales = scales;
    u.row_rms = row_rms;
    u.rows = rows;
    u.cols = cols;
    u.ld = ld;
    u.fmt = fmt;
    u.block = block;
    if (codes == nullptr && row_rms == nullptr)
        return HILORE_INVALID_ARG;
    if (fmt == HILORE_FMT_E4M3FN_RAW && scales != nullptr)
        return HILORE_INVALID_ARG;
    const int st = check_unit(u, true, true, codes != nullptr, false);
    if (st != HILORE_OK)
        return st;
    CodecWork wk{};
    wk.units = nullptr;
    wk.single = u;
    wk.U = 1;
    wk.phase = codes ? OP_COMPRESS : OP_STATS;
    return launch_codec(wk, rows, static_cast<cudaStream_t>(stream));
}

extern "C" int hilore_recover(const uint8_t *codes, const float *scales, int64_t rows, int64_t cols, int32_t fmt,
                              int32_t block, void *out, int64_t ld_out, void *stream)
{
    hilore_unit u{};
    u.codes = const_cast<uint8_t *>(codes);
    u.scales = const_cast<float *>(scales);
    u.out = out;
    u.rows = rows;
    u.cols = cols;
    u.ld = ld_out;
    u.fmt = fmt;
    u.block = block;
    const int st = check_unit(u, true, false, true, true);
    if (st != HILORE_OK)
        return st;
    CodecWork wk{};
    wk.single = u;
    wk.U = 1;
    wk.phase = OP_RECOVER;
    return launch_codec(wk, rows, static_cast<cudaStream_t>(stream));
}

extern "C" int hilore_plan_apply(const hilore_unit *units_dev, const hilore_unit *units_host, int32_t U, int32_t phase,
                                 const float *exposure, const float *kappa, const float *ebar, float tau_lo,
                                 float tau_hi, const uint8_t *avail, uint8_t *action_io, float *psi,
                                 uint8_t *recompute, uint64_t *retained_bytes, void *stream)
{
    if (U < 0 || phase < HILORE_PHASE_DECIDE || phase > HILORE_PHASE_RECOVER)
        return HILORE_INVALID_ARG;
    if (U == 0)
        return HILORE_OK;
    if (units_dev == nullptr || units_host == nullptr || avail == nullptr || action_io == nullptr)
        return HILORE_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int64_t max_rows = 0;
    for (int u = 0; u < U; ++u) {
        const int s = check_unit(units_host[u], false, false, false, false);
        if (s != HILORE_OK)
            return s;
        if (units_host[u].rows > max_rows)
            max_rows = units_host[u].rows;
    }
    if (phase == HILORE_PHASE_DECIDE) {
        if (exposure != nullptr && (kappa == nullptr || ebar == nullptr))
            return HILORE_INVALID_ARG;
        plan_decide_kernel<<<1, 128, 0, st>>>(units_dev, U, exposure, kappa, ebar, tau_lo, tau_hi, avail, action_io,
                                              psi, recompute, retained_bytes);
        return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
    }
    CodecWork wk{};
    wk.units = units_dev;
    wk.U = U;
    wk.phase = phase;
    wk.avail = avail;
    wk.action = action_io;
    return launch_codec(wk, max_rows, st);
}
