// Entry points of the store / recover path: hilore_compress, hilore_recover, hilore_plan_apply.
// Two kernels (compress / token RMS, and recover), each compiled once per storage format and once for
// mixed tables.  Every CTA walks the unit table, decides per unit (from the gating arrays in device
// memory) what to do, and processes its share of the unit's rows: a whole microbatch of units costs one
// launch per phase and no host synchronisation.
#include "codec.cuh"

namespace hilore {

// Compress / token-RMS pass over rows [r0, r1) of one unit, specialised on what the unit asks for.
// Iterations of bulk L2 prefetch run-ahead of the compress pass (16 KB of bf16 per iteration and CTA), by what
// the pass writes.  Measured on B200 (TB/s at run-ahead 0 / 1 / 2 / 3): token RMS only, 7B-shaped table
// 6.6 / 6.8 / 7.1 / 7.1; codes + scales + RMS, 7B-shaped table 6.2 / 6.6 / 6.4 / 6.0, 4 GiB unit 6.3 / 6.7 / 6.0;
// the unscaled format on a 4 GiB unit 6.7 / 6.5 / 6.0; codes + scales only (post-forward encode) 6.7 / 6.4 / 6.1 /
// 5.9: the more a pass writes, the sooner lines pulled in ahead of time are in the way of the written ones.
constexpr int kPrefetchStats = 2, kPrefetchCodesRms = 1, kPrefetchCodesOnly = 0;

template <int FMT>
__device__ __forceinline__ void compress_unit(const hilore_unit &u, int op, int64_t r0, int64_t r1, int rpb, float *sm,
                                              const uint32_t *tab)
{
    const uint16_t *x = static_cast<const uint16_t *>(u.x);
    if (op == OP_STATS)
        compress_rows<HILORE_FMT_E4M3FN_RAW, false, true>(x, nullptr, nullptr, u.row_rms, u.cols, u.ld, r0, r1, rpb, sm, kPrefetchStats, tab);
    else if (u.row_rms != nullptr)
        compress_rows<FMT, true, true>(x, u.codes, u.scales, u.row_rms, u.cols, u.ld, r0, r1, rpb, sm, FMT == HILORE_FMT_E4M3FN_RAW ? kPrefetchCodesOnly : kPrefetchCodesRms, tab);
    else
        compress_rows<FMT, true, false>(x, u.codes, u.scales, nullptr, u.cols, u.ld, r0, r1, rpb, sm, kPrefetchCodesOnly, tab);
}

// FMT >= 0: every unit of the launch has this format (the common case; the hot loop is compiled for it).
// FMT < 0: formats differ between units; each unit is dispatched on its own format.
template <int FMT> __global__ void __launch_bounds__(kCodecThreads, 4) compress_kernel(const __grid_constant__ CodecWork wk)
{
    __shared__ float sm_blocksum[kBlockSumSlots];
    __shared__ uint32_t sm_tab[2][kScaleTableWords]; // scale tables: [0] Q = 448, [1] Q = 127
    if (FMT < 0 || FMT == HILORE_FMT_E4M3FN_BLK) fill_scale_table<HILORE_FMT_E4M3FN_BLK>(sm_tab[0]);
    if (FMT < 0 || FMT == HILORE_FMT_INT8_BLK) fill_scale_table<HILORE_FMT_INT8_BLK>(sm_tab[1]);
    grid_dependency_wait();    // everything above touched shared memory only
    grid_dependency_release(); // the next kernel's CTAs may take the place of ours as they finish
    // descriptors and gates of the launch once into shared memory: a CTA that meets a new unit every few iterations
    // would otherwise wait for a dependent global load before it can issue the unit's first data loads (+5 % on
    // the 1.5B-shaped table, +7 % on the token-RMS capture of the 7B-shaped one)
    __shared__ UnitStage stage;
    stage_units(wk, false, stage);
    __syncthreads();           // scale tables and descriptors are in place
    JobCursor cur;
    Job j;
    while (next_job(wk, stage, cur, j, kBlockSumSlots)) {
        const int fmt = FMT >= 0 ? FMT : j.u.fmt;
        if (fmt == HILORE_FMT_E4M3FN_RAW) compress_unit<HILORE_FMT_E4M3FN_RAW>(j.u, j.op, j.r0, j.r1, j.rows_per_batch, sm_blocksum, sm_tab[0]);
        else if (fmt == HILORE_FMT_E4M3FN_BLK) compress_unit<HILORE_FMT_E4M3FN_BLK>(j.u, j.op, j.r0, j.r1, j.rows_per_batch, sm_blocksum, sm_tab[0]);
        else compress_unit<HILORE_FMT_INT8_BLK>(j.u, j.op, j.r0, j.r1, j.rows_per_batch, sm_blocksum, sm_tab[1]);
    }
}

// Tiles of bulk L2 prefetch run-ahead of the recover pass (8 KB of codes per tile and CTA).  Measured on B200 (TB/s
// at run-ahead 0 / 1 / 2 / 3): block-scaled formats, whose decode waits for a scale as well, 4 GiB unit
// 6.12 / 6.40 / 6.30, 7B-shaped table 5.98 / 6.36 / 6.32; the unscaled format, 4 GiB unit 6.21 / 6.08 / 6.02 / 6.02.
constexpr int kPrefetchRecoverScaled = 1, kPrefetchRecoverUnscaled = 0;

template <int FMT> __device__ __forceinline__ void recover_unit(const hilore_unit &u, int64_t r0, int64_t r1, uint8_t *sm_out,
                                                                uint32_t &tile, int prefetch)
{
    uint16_t *out = static_cast<uint16_t *>(u.out);
    if (u.ld == u.cols || u.cols >= 1024) // wide enough rows: bulk stores also with a leading dimension
        recover_rows_bulk<FMT>(u.codes, u.scales, out, u.cols, u.ld, r0, r1, sm_out, tile, prefetch);
    else
        recover_rows<FMT>(u.codes, u.scales, out, u.cols, u.ld, r0, r1, prefetch);
}

template <int FMT> __global__ void __launch_bounds__(kCodecThreads, 4) recover_kernel(const __grid_constant__ CodecWork wk)
{
    __shared__ __align__(128) uint8_t sm_out[kRecoverStageBytes];
    __shared__ UnitStage stage;
    grid_dependency_wait();
    grid_dependency_release();
    stage_units(wk, true, stage);
    __syncthreads();
    uint32_t tile = 0;
    JobCursor cur;
    Job j;
    while (next_job(wk, stage, cur, j, 1)) {
        const int fmt = FMT >= 0 ? FMT : j.u.fmt;
        if (fmt == HILORE_FMT_E4M3FN_RAW) recover_unit<HILORE_FMT_E4M3FN_RAW>(j.u, j.r0, j.r1, sm_out, tile, kPrefetchRecoverUnscaled);
        else if (fmt == HILORE_FMT_E4M3FN_BLK) recover_unit<HILORE_FMT_E4M3FN_BLK>(j.u, j.r0, j.r1, sm_out, tile, kPrefetchRecoverScaled);
        else recover_unit<HILORE_FMT_INT8_BLK>(j.u, j.r0, j.r1, sm_out, tile, kPrefetchRecoverScaled);
    }
    if (threadIdx.x == 0)
        bulk_wait_all(); // every bulk store of this CTA is complete before it gives up its shared memory
}

// psi, threshold rule, availability demotion, recompute flags and retained bytes for U units.
__global__ void plan_decide_kernel(PlanTail p, int U, const float *exposure)
{
    grid_dependency_wait();
    grid_dependency_release();
    for (int u = blockIdx.x * blockDim.x + threadIdx.x; u < U; u += gridDim.x * blockDim.x)
        decide_unit(p, u, exposure ? exposure + u : nullptr);
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

// Scale of the windows of a unit that all CTAs sweep together (see plan_unit, next_job): units up to 1.5 x this size
// go in one piece, larger ones in windows of two thirds of it or more.  Measured on B200: a 4 GiB unit runs at
// 5.5 / 6.2 TB/s (compress / recover) uncut, 6.0 / 6.3 TB/s in windows of 64-96 MB; below about 48 MB the
// pieces per CTA become too short.
constexpr int64_t kSegmentBytes = 96ll << 20;

template <typename K> static int launch_one(K kernel, CodecWork wk, int64_t total_rows, cudaStream_t st)
{
    wk.seg_bytes = kSegmentBytes;
    int64_t grid = (int64_t)sm_count() * ctas_per_sm(kernel, kCodecThreads, 0, 2);
    if (grid > total_rows)
        grid = total_rows;
    wk.share_m = (1ull << 32) / (uint64_t)grid;
    wk.share_rem = (uint32_t)((1ull << 32) % (uint64_t)grid);
    // Rotation of the CTA index per window (see next_job): about 0.38 of the grid, coprime to it, so that the
    // rotated indices of consecutive windows fall evenly.
    wk.rot_step = 0;
    if (grid > 2) {
        uint32_t step = (uint32_t)(grid * 0.381966) | 1u;
        auto gcd = [](uint32_t a, uint32_t b) { while (b) { const uint32_t t = a % b; a = b; b = t; } return a; };
        while (gcd(step, (uint32_t)grid) != 1) step += 2;
        wk.rot_step = step % (uint32_t)grid;
    }
    // Programmatic dependent launch: the CTAs of this kernel may become resident while the previous kernel of the
    // stream drains; they wait (griddepcontrol.wait) before their first access to global memory.
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kCodecThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kernel, wk) != cudaSuccess)
        return HILORE_CUDA;
    return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
}

// fmt: the format shared by all units of the launch, or -1 if they differ.
static int launch_codec(const CodecWork &wk, int64_t total_rows, int fmt, bool recover, cudaStream_t st)
{
    if (total_rows <= 0)
        return HILORE_OK;
    if (recover) {
        switch (fmt) {
        case HILORE_FMT_E4M3FN_RAW: return launch_one(recover_kernel<HILORE_FMT_E4M3FN_RAW>, wk, total_rows, st);
        case HILORE_FMT_E4M3FN_BLK: return launch_one(recover_kernel<HILORE_FMT_E4M3FN_BLK>, wk, total_rows, st);
        case HILORE_FMT_INT8_BLK: return launch_one(recover_kernel<HILORE_FMT_INT8_BLK>, wk, total_rows, st);
        default: return launch_one(recover_kernel<-1>, wk, total_rows, st);
        }
    }
    switch (fmt) {
    case HILORE_FMT_E4M3FN_RAW: return launch_one(compress_kernel<HILORE_FMT_E4M3FN_RAW>, wk, total_rows, st);
    case HILORE_FMT_E4M3FN_BLK: return launch_one(compress_kernel<HILORE_FMT_E4M3FN_BLK>, wk, total_rows, st);
    case HILORE_FMT_INT8_BLK: return launch_one(compress_kernel<HILORE_FMT_INT8_BLK>, wk, total_rows, st);
    default: return launch_one(compress_kernel<-1>, wk, total_rows, st);
    }
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
    return launch_codec(wk, rows, fmt, false, static_cast<cudaStream_t>(stream));
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
    return launch_codec(wk, rows, fmt, true, static_cast<cudaStream_t>(stream));
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
    for (int u = 0; u < U; ++u) {
        const int s = check_unit(units_host[u], false, false, false, false);
        if (s != HILORE_OK)
            return s;
    }
    if (phase == HILORE_PHASE_DECIDE) {
        if (exposure != nullptr && (kappa == nullptr || ebar == nullptr))
            return HILORE_INVALID_ARG;
        PlanTail p{};
        p.units = units_dev;
        p.kappa = kappa;
        p.ebar = ebar;
        p.tau_lo = tau_lo;
        p.tau_hi = tau_hi;
        p.avail = avail;
        p.action_io = action_io;
        p.psi = psi;
        p.recompute = recompute;
        p.retained_bytes = retained_bytes;
        if (launch_dependent(plan_decide_kernel, dim3(1), dim3(128), 0, st, p, (int)U, exposure) != cudaSuccess)
            return HILORE_CUDA;
        return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
    }
    // one launch per slice of at most kStageUnits units (the kernels stage a slice's descriptors in shared memory)
    for (int u0 = 0; u0 < U; u0 += kStageUnits) {
        const int cnt = U - u0 < kStageUnits ? U - u0 : kStageUnits;
        int64_t slice_rows = 0;
        int slice_fmt = units_host[u0].fmt;
        for (int u = u0; u < u0 + cnt; ++u) {
            slice_rows += units_host[u].rows;
            if (units_host[u].fmt != slice_fmt)
                slice_fmt = -1;
        }
        CodecWork wk{};
        wk.units = units_dev + u0;
        wk.U = cnt;
        wk.phase = phase;
        wk.avail = avail + u0;
        wk.action = action_io + u0;
        const int s = launch_codec(wk, slice_rows, slice_fmt, phase == HILORE_PHASE_RECOVER, st);
        if (s != HILORE_OK)
            return s;
    }
    return HILORE_OK;
}
