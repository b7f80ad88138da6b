// A generic space-time-transform executor for the 1-D convolution UREs (Sections 2 and 4): given only the
// allocation row P = (pc, pq) and the schedule row s = (sc, sq) over the iteration space (c, q), it derives the
// dependences, checks the validity conditions, and runs the resulting linear systolic array with one PE per
// lane in the paper's generic code pattern (Code 2): every recurrent variable keeps a register history as
// deep as its delay s.e, reads its neighbour P.e PEs away, and a PE computes only when its time comes
// (CheckTime).  Nothing is specialised per design: the six designs of Table 2 / Section 3.1 and every other
// valid transform run through the same kernel, which is therefore a reference rendering, not a fast one
// (the folded, unrolled kernels are the fast ones).
//
// UREs (source = point - e, sign chosen so that s.e >= 0):
//   X(c,q) = x(c+q)  outside the array, else X(point - ex),   ex = +-(-1, 1)   (same input along c+q = const)
//   W(c,q) = w(q)    outside the array, else W(point - ew),   ew = +-( 1, 0)   (same weight along c)
//   Z(c,q) = X*W + (0 outside the array, else Z(point - ez)), ez = +-( 0, 1)   (accumulation along q)
// A variable with s.e = 0 is a broadcast (read from its source in the same step), with P.e = 0 it stays in
// its PE, otherwise it is forwarded.  The paper's design letters follow from that.
#pragma once

#include "sysconv_common.cuh"

namespace sysconv {

constexpr int kStMaxDelay = 4;      // deepest register history (largest s.e) the executor keeps

struct StPlan {
    int pc, pq, sc, sq, det;
    int e[3][2];        // dependence vectors of X, W, Z
    int pd[3];          // P.e: PE distance of the source
    int dl[3];          // s.e: delay in time steps (0 = broadcast)
    int C;              // outputs per array (one warp = one array of up to 32 PEs)
    int pes;            // PEs the array uses
    int pmin, tmin, tmax;
    char name[4];       // input / weight / partial-sum letters, e.g. "FBS"
};

// Plans the array for filter length q.  Returns SYSCONV_OK, SYSCONV_EINVAL for a transform that violates a
// validity condition of Section 2.2 (processor availability: P and s linearly dependent; data availability:
// sums cannot accumulate within one time step), SYSCONV_EUNSUPPORTED for a valid one this executor does not
// cover (a delay above kStMaxDelay, an array of more than 32 PEs for a single output).
inline int spacetime_plan(int pc, int pq, int sc, int sq, int q, StPlan *pl)
{
    if (q < 1 || q > kMaxQ1) return SYSCONV_EINVAL;
    pl->pc = pc; pl->pq = pq; pl->sc = sc; pl->sq = sq;
    pl->det = pc * sq - pq * sc;
    if (pl->det == 0) return SYSCONV_EINVAL;                   // two points on one PE at one time
    const int base[3][2] = {{-1, 1}, {1, 0}, {0, 1}};
    for (int v = 0; v < 3; ++v) {
        int ec = base[v][0], eq = base[v][1];
        if (sc * ec + sq * eq < 0) { ec = -ec; eq = -eq; }     // data availability: s.e >= 0
        pl->e[v][0] = ec; pl->e[v][1] = eq;
        pl->pd[v] = pc * ec + pq * eq;
        pl->dl[v] = sc * ec + sq * eq;
    }
    if (pl->dl[2] == 0) return SYSCONV_EINVAL;                 // a sum needs a strict order along q
    for (int v = 0; v < 3; ++v)
        if (pl->dl[v] > kStMaxDelay) return SYSCONV_EUNSUPPORTED;
    const int apc = pc < 0 ? -pc : pc, apq = pq < 0 ? -pq : pq;
    const int room = kLanes - 1 - apq * (q - 1);
    if (room < 0) return SYSCONV_EUNSUPPORTED;
    pl->C = apc == 0 ? kLanes : room / apc + 1;
    if (pl->C > 1024) pl->C = 1024;
    pl->pes = apc * (pl->C - 1) + apq * (q - 1) + 1;
    auto lo = [](int a, int n) { return a < 0 ? a * n : 0; };
    auto hi = [](int a, int n) { return a > 0 ? a * n : 0; };
    pl->pmin = lo(pc, pl->C - 1) + lo(pq, q - 1);
    pl->tmin = lo(sc, pl->C - 1) + lo(sq, q - 1);
    pl->tmax = hi(sc, pl->C - 1) + hi(sq, q - 1);
    for (int v = 0; v < 2; ++v) pl->name[v] = pl->dl[v] == 0 ? 'B' : (pl->pd[v] == 0 ? 'S' : 'F');
    pl->name[2] = pl->pd[2] == 0 ? 'S' : 'M';
    pl->name[3] = 0;
    return SYSCONV_OK;
}

__device__ __forceinline__ float st_pick(const float (&h)[kStMaxDelay], int k)
{
    return k == 0 ? h[0] : k == 1 ? h[1] : k == 2 ? h[2] : h[3];
}

constexpr int kStWarps = 4;

__global__ void __launch_bounds__(kStWarps *kLanes)
spacetime_conv1d_kernel(const float *__restrict__ x, float *__restrict__ y, long long n_out,
                        const __grid_constant__ Taps1D taps, int Q, const __grid_constant__ StPlan pl)
{
    dependent_launch_enter();
    const int lane = threadIdx.x & (kLanes - 1);
    const long long gw = static_cast<long long>(blockIdx.x) * kStWarps + threadIdx.x / kLanes;
    const long long warps = static_cast<long long>(gridDim.x) * kStWarps;
    const int p = lane + pl.pmin;                   // this lane's PE
    for (long long blk = gw; blk * pl.C < n_out; blk += warps) {
        const long long c0 = blk * pl.C;
        const int Cb = static_cast<int>(n_out - c0 < pl.C ? n_out - c0 : pl.C);
        float H[3][kStMaxDelay];                    // register histories of X, W, Z (newest first)
#pragma unroll
        for (int v = 0; v < 3; ++v)
#pragma unroll
            for (int k = 0; k < kStMaxDelay; ++k) H[v][k] = 0.f;
        for (int t = pl.tmin; t <= pl.tmax; ++t) {
            // the point (c, q) that runs on PE p at time t, if any (CheckTime)
            const int nc = pl.sq * p - pl.pq * t, nq = pl.pc * t - pl.sc * p;
            const int c = nc / pl.det, q = nq / pl.det;
            const bool active = nc % pl.det == 0 && nq % pl.det == 0 && c >= 0 && c < Cb && q >= 0 && q < Q;
            float val[3];
#pragma unroll
            for (int v = 0; v < 3; ++v) {
                // what the PE P.e away produced s.e steps ago (every lane takes part in the exchange)
                const float mine = st_pick(H[v], pl.dl[v] > 0 ? pl.dl[v] - 1 : 0);
                const float from = __shfl_sync(kFullMask, mine, (lane - pl.pd[v]) & (kLanes - 1));
                const int sc_ = c - pl.e[v][0], sq_ = q - pl.e[v][1];
                const bool inside = pl.dl[v] > 0 && sc_ >= 0 && sc_ < Cb && sq_ >= 0 && sq_ < Q;
                float src = 0.f;                     // outside the array: x(c+q), w(q), 0
                if (active && !inside) src = v == 0 ? x[c0 + c + q] : v == 1 ? taps.w[q] : 0.f;
                val[v] = inside ? from : src;
            }
            const float z = fmaf(val[0], val[1], val[2]);
#pragma unroll
            for (int v = 0; v < 3; ++v) {
#pragma unroll
                for (int k = kStMaxDelay - 1; k > 0; --k) H[v][k] = H[v][k - 1];
                H[v][0] = v == 2 ? z : val[v];
            }
            // the sum leaves the array where its chain ends
            const int qn = q + pl.e[2][1];
            if (active && (qn < 0 || qn >= Q)) y[c0 + c] = z;
        }
    }
}

}  // namespace sysconv
