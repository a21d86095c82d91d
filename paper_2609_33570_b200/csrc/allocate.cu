// Joint H/L/R allocation on the device: the paper's two-constraint multiple-choice knapsack, solved by
// dynamic programming on the conservative grid (Appendix "Joint Allocation and Schedule Validation",
// Eqs. "allocation-grid", "allocation-integer-costs", "allocation-dp").  The paper runs this DP on one CPU
// thread; for U = 84 units that is 2.6e8 state updates between forward and backward of every microbatch.
// Here layer i of the DP is one data-parallel pass over the (N+1)^2 states (it depends on layer i-1 only),
// and the chosen actions never leave the device.
#include "common.cuh"

#include <cooperative_groups.h>

namespace hilore {

struct AllocUnit {
    int b[3], r[3]; // integer memory / risk cost of actions R, H, L; -1 = the action cannot be taken
    double tau[3];  // utility
};

__device__ __forceinline__ AllocUnit alloc_prepare_unit(int u, const float *psi, const double *dtau, const double *dmem,
                                                        const uint8_t *avail, double M_res, double delta_b, int N)
{
    const double hB = M_res / (double)N, hD = delta_b / (double)N;
    const uint32_t q = avail[u];
    AllocUnit out;
    for (int a = 0; a < 3; ++a) {
        bool ok = (a == HILORE_ACT_R) || (q == HILORE_ACT_H) || (q == HILORE_ACT_L && a == HILORE_ACT_L);
        double dm = (a == HILORE_ACT_R) ? 0.0 : dmem[u * 3 + a];
        const double d = (a == HILORE_ACT_L) ? (double)psi[u] : 0.0;
        if (dm < 0.0) dm = 0.0;
        if (a == HILORE_ACT_L && (!(d >= 0.0) || delta_b == 0.0)) ok = false; // NaN / negative risk; zero budget
        if (!(dm == dm)) ok = false;
        if (q > HILORE_ACT_L) ok = (a == HILORE_ACT_R);
        long long b = 0, r = 0;
        if (ok) {
            if (M_res > 0.0) b = (long long)ceil(dm / hB);
            else if (dm > 0.0) ok = false;
            if (delta_b > 0.0) r = (long long)ceil(d / hD);
            if (b > N || r > N || b < 0 || r < 0) ok = false;
        }
        out.b[a] = ok ? (int)b : -1;
        out.r[a] = ok ? (int)r : -1;
        out.tau[a] = (a == HILORE_ACT_R) ? 0.0 : dtau[u * 3 + a];
    }
    return out;
}

struct Terminal {
    double F;
    int j, k;
};
constexpr int kNoState = 0x7FFFFFFF;

__device__ __forceinline__ bool better(const Terminal &a, const Terminal &b)
{ // larger utility; ties: lower risk state, then lower memory state
    if (a.F != b.F)
        return a.F > b.F;
    if (a.k != b.k)
        return a.k < b.k;
    return a.j < b.j;
}

struct AllocArgs {
    int U, N, KB, KD;
    const float *psi;
    const double *dtau, *dmem;
    const uint8_t *avail;
    double M_res, delta_b;
    AllocUnit *units;
    double *F0, *F1;
    uint8_t *pred;
    Terminal *partial; // one per CTA
    uint8_t *action, *recompute;
    double *totals;
};

constexpr int kAllocThreads = 1024;

// The whole allocation in one cooperative launch: integer costs, the U layers of the DP (each a grid-stride
// pass over the states, separated by grid-wide barriers), the terminal maximum and the backtracking.
//   F_i(j,k) = max over available a with b <= j, r <= k of F_{i-1}(j-b, k-r) + tau_i(a); candidates in the
//   order R, H, L, the first maximum wins.
__global__ void __launch_bounds__(kAllocThreads, 2) alloc_dp_kernel(const __grid_constant__ AllocArgs a)
{
    namespace cg = cooperative_groups;
    cg::grid_group grid = cg::this_grid();
    __shared__ Terminal sm[kAllocThreads];
    const int64_t S = (int64_t)a.KB * a.KD;
    const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, gsz = (int64_t)gridDim.x * blockDim.x;

    for (int64_t u = gid; u < a.U; u += gsz)
        a.units[u] = alloc_prepare_unit((int)u, a.psi, a.dtau, a.dmem, a.avail, a.M_res, a.delta_b, a.N);
    for (int64_t s = gid; s < S; s += gsz)
        a.F0[s] = (s == 0) ? 0.0 : -INFINITY;
    grid.sync();

    double *Fprev = a.F0, *Fcur = a.F1;
    const int KD = a.KD;
    // (j, k) of this thread's first state and the step between its states (no division in the loops)
    const int j0 = (int)(gid / KD), k0 = (int)(gid - (int64_t)j0 * KD);
    const int dj = (int)(gsz / KD), dk = (int)(gsz - (int64_t)dj * KD);
    const double ninf = -INFINITY;
    for (int u = 0; u < a.U; ++u) {
        // Candidates in the order R, H, L; R always costs (0, 0) and adds 0, so it is the state itself.
        // An unavailable action gets a cost no state can pay.
        const AllocUnit un = a.units[u]; // the same 48 bytes for every thread: one broadcast load per layer
        const int bH = un.b[HILORE_ACT_H] < 0 ? 0x3FFFFFFF : un.b[HILORE_ACT_H], rH = un.r[HILORE_ACT_H] < 0 ? 0 : un.r[HILORE_ACT_H];
        const int bL = un.b[HILORE_ACT_L] < 0 ? 0x3FFFFFFF : un.b[HILORE_ACT_L], rL = un.r[HILORE_ACT_L] < 0 ? 0 : un.r[HILORE_ACT_L];
        const int offH = bH < 0x3FFFFFFF ? bH * KD + rH : 0, offL = bL < 0x3FFFFFFF ? bL * KD + rL : 0;
        const double tH = un.tau[HILORE_ACT_H], tL = un.tau[HILORE_ACT_L];
        uint8_t *pred = a.pred + (size_t)u * S;
        int j = j0, k = k0;
        for (int s = (int)gid; s < (int)S; s += (int)gsz, j += dj, k += dk) {
            if (k >= KD) {
                k -= KD;
                ++j;
            }
            const bool canH = j >= bH && k >= rH, canL = j >= bL && k >= rL;
            // the three reads are issued together
            const double pR = Fprev[s];
            const double pH = canH ? Fprev[s - offH] : ninf;
            const double pL = canL ? Fprev[s - offL] : ninf;
            double best = pR; // pR + 0.0 is pR for every value the table can hold
            uint32_t arg = (pR == ninf) ? 255u : (uint32_t)HILORE_ACT_R;
            if (pH != ninf) {
                const double v = pH + tH;
                if (arg == 255u || v > best) {
                    best = v;
                    arg = HILORE_ACT_H;
                }
            }
            if (pL != ninf) {
                const double v = pL + tL;
                if (arg == 255u || v > best) {
                    best = v;
                    arg = HILORE_ACT_L;
                }
            }
            Fcur[s] = (arg == 255u) ? ninf : best;
            pred[s] = (uint8_t)arg;
        }
        grid.sync();
        double *t = Fprev;
        Fprev = Fcur;
        Fcur = t;
    }

    // terminal state: largest utility; ties: lower risk, then lower memory
    Terminal best{-INFINITY, kNoState, kNoState};
    for (int64_t s = gid; s < S; s += gsz) {
        const double v = Fprev[s];
        if (v == -INFINITY)
            continue;
        const int j = (int)(s / a.KD);
        const Terminal t{v, j, (int)(s - (int64_t)j * a.KD)};
        if (best.j == kNoState || better(t, best))
            best = t;
    }
    sm[threadIdx.x] = best;
    __syncthreads();
    for (int o = kAllocThreads / 2; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) {
            const Terminal other = sm[threadIdx.x + o];
            if (other.j != kNoState && (sm[threadIdx.x].j == kNoState || better(other, sm[threadIdx.x])))
                sm[threadIdx.x] = other;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0)
        a.partial[blockIdx.x] = sm[0];
    grid.sync();
    if (blockIdx.x != 0)
        return;
    best = Terminal{-INFINITY, kNoState, kNoState};
    for (int c = threadIdx.x; c < (int)gridDim.x; c += kAllocThreads) {
        const Terminal t = a.partial[c];
        if (t.j != kNoState && (best.j == kNoState || better(t, best)))
            best = t;
    }
    sm[threadIdx.x] = best;
    __syncthreads();
    for (int o = kAllocThreads / 2; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) {
            const Terminal other = sm[threadIdx.x + o];
            if (other.j != kNoState && (sm[threadIdx.x].j == kNoState || better(other, sm[threadIdx.x])))
                sm[threadIdx.x] = other;
        }
        __syncthreads();
    }
    if (threadIdx.x != 0)
        return;
    // backtracking (one thread; U dependent reads)
    int j = sm[0].j, k = sm[0].k;
    if (j == kNoState) { // cannot happen: the all-R assignment always reaches state (0, 0)
        j = 0;
        k = 0;
    }
    double tot_m = 0.0, tot_r = 0.0;
    for (int u = a.U - 1; u >= 0; --u) {
        uint32_t c = a.pred[(size_t)u * S + (int64_t)j * a.KD + k];
        if (c > HILORE_ACT_L)
            c = HILORE_ACT_R;
        a.action[u] = (uint8_t)c;
        if (a.recompute) a.recompute[u] = (c == HILORE_ACT_R);
        j -= a.units[u].b[c];
        k -= a.units[u].r[c];
        if (c != HILORE_ACT_R) tot_m += (a.dmem[u * 3 + c] < 0.0 ? 0.0 : a.dmem[u * 3 + c]);
        if (c == HILORE_ACT_L) tot_r += (double)a.psi[u];
    }
    if (a.totals) {
        a.totals[0] = sm[0].F;
        a.totals[1] = tot_m;
        a.totals[2] = tot_r;
    }
}

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct AllocLayout {
    size_t F0, F1, pred, units, term, total;
};

static AllocLayout alloc_layout(int U, int N, bool mem_axis, bool risk_axis)
{
    const size_t KB = mem_axis ? (size_t)N + 1 : 1, KD = risk_axis ? (size_t)N + 1 : 1, S = KB * KD;
    AllocLayout l;
    size_t off = 0;
    l.F0 = off; off = align_up(off + S * sizeof(double), 256);
    l.F1 = off; off = align_up(off + S * sizeof(double), 256);
    l.pred = off; off = align_up(off + S * (size_t)(U > 0 ? U : 1), 256);
    l.units = off; off = align_up(off + sizeof(AllocUnit) * (size_t)(U > 0 ? U : 1), 256);
    l.term = off; off = align_up(off + sizeof(Terminal) * 4096, 256); // one partial terminal state per CTA
    l.total = off;
    return l;
}

} // namespace hilore

using namespace hilore;

extern "C" size_t hilore_allocate_workspace_bytes(int32_t U, int32_t n_intervals)
{
    if (U < 0 || n_intervals <= 0)
        return 0;
    return alloc_layout(U, n_intervals, true, true).total;
}

extern "C" double hilore_risk_budget(double delta, int64_t N_b, int64_t N_total)
{
    return (N_total > 0) ? delta * (double)N_b / (double)N_total : 0.0;
}

extern "C" int hilore_allocate(int32_t U, const float *psi, const double *dtau, const double *dmem, const uint8_t *avail,
                               double M_res, double delta_b, int32_t n_intervals, uint8_t *action, uint8_t *recompute,
                               double *totals, void *workspace, size_t workspace_bytes, void *stream)
{
    if (U < 0 || n_intervals <= 0 || n_intervals > 8192)
        return HILORE_INVALID_ARG;
    if (!(M_res >= 0.0) || !(delta_b >= 0.0))
        return HILORE_INVALID_ARG; // a plan that exceeds the budget under all-R execution is excluded before capture
    if (U == 0)
        return HILORE_OK;
    if (!psi || !dtau || !dmem || !avail || !action || !workspace)
        return HILORE_INVALID_ARG;
    if (!aligned(workspace, 256) || !aligned(dtau, 8) || !aligned(dmem, 8) || !aligned(totals, 8) || !aligned(psi, 4))
        return HILORE_ALIGN;
    const bool mem_axis = M_res > 0.0, risk_axis = delta_b > 0.0;
    const AllocLayout l = alloc_layout(U, n_intervals, mem_axis, risk_axis);
    if (workspace_bytes < l.total)
        return HILORE_WORKSPACE;
    const int KB = mem_axis ? n_intervals + 1 : 1, KD = risk_axis ? n_intervals + 1 : 1;
    const int64_t S = (int64_t)KB * KD;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    double *F0 = reinterpret_cast<double *>(ws + l.F0), *F1 = reinterpret_cast<double *>(ws + l.F1);
    uint8_t *pred = ws + l.pred;
    AllocUnit *units = reinterpret_cast<AllocUnit *>(ws + l.units);
    Terminal *term = reinterpret_cast<Terminal *>(ws + l.term);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    AllocArgs args{};
    args.U = U;
    args.N = n_intervals;
    args.KB = KB;
    args.KD = KD;
    args.psi = psi;
    args.dtau = dtau;
    args.dmem = dmem;
    args.avail = avail;
    args.M_res = M_res;
    args.delta_b = delta_b;
    args.units = units;
    args.F0 = F0;
    args.F1 = F1;
    args.pred = pred;
    args.partial = term;
    args.action = action;
    args.recompute = recompute;
    args.totals = totals;
    // every CTA must be resident for the grid-wide barriers: size the grid from the occupancy
    int64_t grid = (int64_t)sm_count() * ctas_per_sm(alloc_dp_kernel, kAllocThreads, 0, 1);
    const int64_t need = (S + kAllocThreads - 1) / kAllocThreads;
    if (grid > need) grid = need;
    if (grid > 4096) grid = 4096;
    void *kargs[] = {&args};
    if (cudaLaunchCooperativeKernel(reinterpret_cast<const void *>(alloc_dp_kernel), dim3((unsigned)grid), dim3(kAllocThreads),
                                    kargs, 0, st) != cudaSuccess)
        return HILORE_CUDA;
    return cudaGetLastError() == cudaSuccess ? HILORE_OK : HILORE_CUDA;
}
