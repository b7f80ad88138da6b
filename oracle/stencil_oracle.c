/*
 * CPU oracle for the iterated 2-D stencil (TEST INFRASTRUCTURE ONLY; shares no code with the CUDA path).
 *
 * The paper motivates systolic arrays on GPUs with stencils beside convolution (Section 1); this library's
 * second workload is a Jacobi-type sweep of a 3x3 stencil with fixed (Dirichlet) boundary values:
 *
 *   one sweep:  v(r, c) = sum_{dr,dc in {-1,0,1}} k(dr, dc) * u(r+dr, c+dc)   for 0 < r < H-1, 0 < c < W-1
 *               v(r, c) = u(r, c)                                              on the outermost ring
 *   T sweeps:   the sweep applied T times, each on the result of the one before.
 *
 * k is stored row-major as k[dr+1][dc+1] (a five-point stencil has zero corner coefficients).  Written
 * out as the definition: a loop over sweeps around plain nested loops over the grid, two buffers swapped
 * between sweeps, no blocking and no fusion of sweeps.  The grid and the coefficients are fp32 values;
 * every product, sum and every intermediate grid is kept in fp64.
 *
 * Beside the result the oracle returns S: the same T sweeps applied to |u| with the coefficients |k|,
 * which bounds sum |w||x| of the composite (2T+1)x(2T+1) operator at every point and is the scale of the
 * parity tolerance |y_gpu - y| <= 1e-5 * S.
 *
 * Pins (tests/test_stencil_oracle_pins.py): a constant field under coefficients that sum to one, a linear
 * field under a symmetric averaging stencil, the response to an impulse (orientation of k), a Dirichlet
 * eigenfunction of the five-point stencil with its closed-form decay, scipy's 2-D correlation for one
 * sweep and for the composite of two, and a pure-Python brute force.
 */
#include <stdlib.h>
#include <string.h>
#include <math.h>

/* one sweep from `src` to `dst` (both h*w doubles); use_abs: coefficients and nothing else made non-negative
 * by the caller */
static void sweep_once(const double *src, double *dst, int w, int h, const double k[9])
{
#pragma omp parallel for schedule(static)
    for (int r = 0; r < h; ++r) {
        for (int c = 0; c < w; ++c) {
            if (r == 0 || r == h - 1 || c == 0 || c == w - 1) {
                dst[(long long)r * w + c] = src[(long long)r * w + c];
                continue;
            }
            double acc = 0.0;
            for (int dr = -1; dr <= 1; ++dr)
                for (int dc = -1; dc <= 1; ++dc)
                    acc += k[(dr + 1) * 3 + (dc + 1)] * src[(long long)(r + dr) * w + (c + dc)];
            dst[(long long)r * w + c] = acc;
        }
    }
}

/* u: h rows of w floats, `pitch` floats apart.  k: 9 floats.  y, s: h*w doubles, dense (s may be NULL).
 * Returns 0, or -1 if memory for the two work grids could not be had. */
int oracle_stencil2d_f32(const float *u, int w, int h, long long pitch, const float *k, int sweeps,
                         double *y, double *s)
{
    const long long n = (long long)w * h;
    double *a = (double *)malloc(sizeof(double) * (size_t)n);
    double *b = (double *)malloc(sizeof(double) * (size_t)n);
    if (!a || !b) { free(a); free(b); return -1; }
    for (int pass = 0; pass < (s ? 2 : 1); ++pass) {
        double kk[9];
        for (int i = 0; i < 9; ++i) kk[i] = pass ? fabs((double)k[i]) : (double)k[i];
        for (int r = 0; r < h; ++r)
            for (int c = 0; c < w; ++c) {
                const double v = (double)u[(long long)r * pitch + c];
                a[(long long)r * w + c] = pass ? fabs(v) : v;
            }
        double *src = a, *dst = b;
        for (int t = 0; t < sweeps; ++t) {
            sweep_once(src, dst, w, h, kk);
            double *tmp = src; src = dst; dst = tmp;
        }
        memcpy(pass ? s : y, src, sizeof(double) * (size_t)n);
    }
    free(a);
    free(b);
    return 0;
}
