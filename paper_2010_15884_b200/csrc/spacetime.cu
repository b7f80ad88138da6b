// Generic space-time-transform executor: host planning and launch.
#include "spacetime.cuh"

namespace sysconv {

int spacetime_describe(int pc, int pq, int sc, int sq, int q, int *out10, char *name4)
{
    StPlan pl;
    const int st = spacetime_plan(pc, pq, sc, sq, q, &pl);
    if (st != SYSCONV_OK) return st;
    if (out10) {
        for (int v = 0; v < 3; ++v) { out10[2 * v] = pl.pd[v]; out10[2 * v + 1] = pl.dl[v]; }
        out10[6] = pl.C; out10[7] = pl.pes; out10[8] = pl.tmax - pl.tmin + 1; out10[9] = pl.det;
    }
    if (name4) for (int i = 0; i < 4; ++i) name4[i] = pl.name[i];
    return SYSCONV_OK;
}

cudaError_t launch_spacetime_conv1d(const float *x, long long n, const float *w, int q, float *y, int pc, int pq, int sc,
                                    int sq, int sm_count, cudaStream_t s, int *status, int *launches)
{
    StPlan pl;
    *status = spacetime_plan(pc, pq, sc, sq, q, &pl);
    if (*status != SYSCONV_OK) return cudaSuccess;
    Taps1D taps;
    for (int k = 0; k < kMaxQ1; ++k) taps.w[k] = k < q ? w[k] : 0.f;
    const long long n_out = n - q + 1;
    const long long blocks = (n_out + pl.C - 1) / pl.C;
    long long ctas = (blocks + kStWarps - 1) / kStWarps;
    const long long cap = static_cast<long long>(sm_count) * 16;
    if (ctas > cap) ctas = cap;
    launch_kernel(spacetime_conv1d_kernel, static_cast<unsigned>(ctas), kStWarps * kLanes, s, x, y, n_out, taps, q, pl);
    const cudaError_t err = cudaGetLastError();
    if (err == cudaSuccess && launches) *launches += 1;
    return err;
}

}  // namespace sysconv
