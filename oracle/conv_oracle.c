/*
 * CPU oracle for valid-mode 1-D and 2-D convolution (correlation form).
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing on the product path (the CUDA library and
 * its Python binding) may include, link or call this file; it shares no code
 * with the CUDA kernels.  Only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg use it.
 *
 * What it computes is the plain definition, written out with the outputs in
 * the outer loops and the taps in the inner loops, no blocking or reordering:
 *
 *   1-D (Eq. 2 of the paper):  Z(c)    = sum_q        x(c+q)      * w(q)
 *   2-D (Eq. 3 of the paper):  Z(c, r) = sum_q sum_p  x(c+q, r+p) * w(q, p)
 *
 * "c" is the column (contiguous in memory), "r" the row; the filter is stored
 * row-major as w[p][q] (p = filter row).  No filter flip; valid mode only:
 * C = N-Q+1 outputs in 1-D, (H-P+1) x (W-Q+1) in 2-D.
 *
 * Floating point: inputs and taps are fp32 values, every product and the sum
 * are formed in fp64 (a product of two fp32 values is exact in fp64).  Beside
 * each output the oracle returns S = sum |w|*|x| over the same taps, which is
 * the scale of the parity tolerance |y_gpu - y| <= 1e-5 * S.
 * Integer: x is uint8 (zero-extended), w is int8 (sign-extended), the sum is
 * exact in int32 (the *_i64 variant keeps it in int64 as a cross-check).
 *
 * A second statement of the same sums with the loops in the other order (taps
 * outer, outputs inner: y += w[k] * shift(x, k)) is provided as a brute-force
 * cross-check of the first.
 *
 * Pins (tests/test_oracle_pins.py): impulse filters, constant inputs, ramp
 * inputs with closed forms, linearity, shift invariance, separable filters,
 * Q=1 and N=Q special cases, numpy.correlate, pure-Python brute force.
 */
#include <stdint.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Eq. 2: y[c] = sum_q w[q] * x[c+q], c in [0, n-q]. s may be NULL. */
void oracle_conv1d_f32(const float *x, long long n, const float *w, int q,
                       double *y, double *s)
{
    long long C = n - q + 1;
#pragma omp parallel for schedule(static)
    for (long long c = 0; c < C; ++c) {
        double acc = 0.0, mag = 0.0;
        for (int k = 0; k < q; ++k) {
            double prod = (double)w[k] * (double)x[c + k];
            acc += prod;
            mag += fabs(prod);
        }
        y[c] = acc;
        if (s) s[c] = mag;
    }
}

/* Same sums, taps in the outer loop (y must hold n-q+1 doubles). */
void oracle_conv1d_f32_taps_outer(const float *x, long long n, const float *w,
                                  int q, double *y)
{
    long long C = n - q + 1;
    for (long long c = 0; c < C; ++c) y[c] = 0.0;
    for (int k = 0; k < q; ++k)
        for (long long c = 0; c < C; ++c)
            y[c] += (double)w[k] * (double)x[c + k];
}

/* Eq. 2 at a list of output positions only (for full-size sampled parity). */
void oracle_conv1d_f32_at(const float *x, long long n, const float *w, int q,
                          const long long *pos, long long count,
                          double *y, double *s)
{
    (void)n;
#pragma omp parallel for schedule(static)
    for (long long i = 0; i < count; ++i) {
        long long c = pos[i];
        double acc = 0.0, mag = 0.0;
        for (int k = 0; k < q; ++k) {
            double prod = (double)w[k] * (double)x[c + k];
            acc += prod;
            mag += fabs(prod);
        }
        y[i] = acc;
        if (s) s[i] = mag;
    }
}

/* Strided form of Eq. 2 (the stride-2 FBS cell of Table 2 reads x(2c+q)):
 * y[c] = sum_q w[q] * x[stride*c + q], c in [0, (n-q)/stride]. s may be NULL. */
void oracle_conv1d_f32_strided(const float *x, long long n, const float *w, int q,
                               int stride, double *y, double *s)
{
    long long C = (n - q) / stride + 1;
#pragma omp parallel for schedule(static)
    for (long long c = 0; c < C; ++c) {
        double acc = 0.0, mag = 0.0;
        for (int k = 0; k < q; ++k) {
            double prod = (double)w[k] * (double)x[(long long)stride * c + k];
            acc += prod;
            mag += fabs(prod);
        }
        y[c] = acc;
        if (s) s[c] = mag;
    }
}

/* Strided form of Eq. 3: y[r][c] = sum_p sum_q w[p][q] * x[sr*r + p][sc*c + q],
 * r in [0, (height-p)/sr], c in [0, (width-q)/sc]. s may be NULL. */
void oracle_conv2d_f32_strided(const float *x, int width, int height, long long x_pitch,
                               const float *w, int p, int q, int sr, int sc,
                               double *y, double *s, long long y_pitch)
{
    int out_h = (height - p) / sr + 1, out_w = (width - q) / sc + 1;
#pragma omp parallel for schedule(static)
    for (int r = 0; r < out_h; ++r)
        for (int c = 0; c < out_w; ++c) {
            double acc = 0.0, mag = 0.0;
            for (int i = 0; i < p; ++i)
                for (int k = 0; k < q; ++k) {
                    double prod = (double)w[i * q + k] *
                                  (double)x[(long long)(sr * r + i) * x_pitch + sc * c + k];
                    acc += prod;
                    mag += fabs(prod);
                }
            y[(long long)r * y_pitch + c] = acc;
            if (s) s[(long long)r * y_pitch + c] = mag;
        }
}

/* Eq. 3: y[r][c] = sum_p sum_q w[p][q] * x[r+p][c+q].
 * x_pitch / y_pitch are row pitches in elements.  s may be NULL. */
void oracle_conv2d_f32(const float *x, int width, int height, long long x_pitch,
                       const float *w, int q, int p,
                       double *y, double *s, long long y_pitch)
{
    int R = height - p + 1, C = width - q + 1;
#pragma omp parallel for schedule(static)
    for (int r = 0; r < R; ++r) {
        for (int c = 0; c < C; ++c) {
            double acc = 0.0, mag = 0.0;
            for (int pp = 0; pp < p; ++pp)
                for (int qq = 0; qq < q; ++qq) {
                    double prod = (double)w[pp * q + qq] *
                                  (double)x[(long long)(r + pp) * x_pitch + (c + qq)];
                    acc += prod;
                    mag += fabs(prod);
                }
            y[(long long)r * y_pitch + c] = acc;
            if (s) s[(long long)r * y_pitch + c] = mag;
        }
    }
}

/* Same sums, taps in the outer loops. */
void oracle_conv2d_f32_taps_outer(const float *x, int width, int height,
                                  long long x_pitch, const float *w, int q, int p,
                                  double *y, long long y_pitch)
{
    int R = height - p + 1, C = width - q + 1;
    for (int r = 0; r < R; ++r)
        for (int c = 0; c < C; ++c) y[(long long)r * y_pitch + c] = 0.0;
    for (int pp = 0; pp < p; ++pp)
        for (int qq = 0; qq < q; ++qq)
            for (int r = 0; r < R; ++r)
                for (int c = 0; c < C; ++c)
                    y[(long long)r * y_pitch + c] +=
                        (double)w[pp * q + qq] *
                        (double)x[(long long)(r + pp) * x_pitch + (c + qq)];
}

/* Eq. 3 at a list of (row, col) output positions only. */
void oracle_conv2d_f32_at(const float *x, int width, int height, long long x_pitch,
                          const float *w, int q, int p,
                          const long long *rows, const long long *cols,
                          long long count, double *y, double *s)
{
    (void)width; (void)height;
#pragma omp parallel for schedule(static)
    for (long long i = 0; i < count; ++i) {
        long long r = rows[i], c = cols[i];
        double acc = 0.0, mag = 0.0;
        for (int pp = 0; pp < p; ++pp)
            for (int qq = 0; qq < q; ++qq) {
                double prod = (double)w[pp * q + qq] *
                              (double)x[(r + pp) * x_pitch + (c + qq)];
                acc += prod;
                mag += fabs(prod);
            }
        y[i] = acc;
        if (s) s[i] = mag;
    }
}

/* Integer form of Eq. 2: uint8 inputs, int8 taps, exact int32 sums. */
void oracle_conv1d_u8s8_s32(const uint8_t *x, long long n, const int8_t *w, int q,
                            int32_t *y)
{
    long long C = n - q + 1;
#pragma omp parallel for schedule(static)
    for (long long c = 0; c < C; ++c) {
        int32_t acc = 0;
        for (int k = 0; k < q; ++k)
            acc += (int32_t)w[k] * (int32_t)x[c + k];
        y[c] = acc;
    }
}

/* Integer form of Eq. 3: uint8 pixels, int8 taps, exact int32 sums. */
void oracle_conv2d_u8s8_s32(const uint8_t *x, int width, int height, long long x_pitch,
                            const int8_t *w, int q, int p,
                            int32_t *y, long long y_pitch)
{
    int R = height - p + 1, C = width - q + 1;
#pragma omp parallel for schedule(static)
    for (int r = 0; r < R; ++r) {
        for (int c = 0; c < C; ++c) {
            int32_t acc = 0;
            for (int pp = 0; pp < p; ++pp)
                for (int qq = 0; qq < q; ++qq)
                    acc += (int32_t)w[pp * q + qq] *
                           (int32_t)x[(long long)(r + pp) * x_pitch + (c + qq)];
            y[(long long)r * y_pitch + c] = acc;
        }
    }
}

/* The same integer sums kept in int64 (overflow cross-check of the int32 form). */
void oracle_conv2d_u8s8_i64(const uint8_t *x, int width, int height, long long x_pitch,
                            const int8_t *w, int q, int p,
                            int64_t *y, long long y_pitch)
{
    int R = height - p + 1, C = width - q + 1;
    for (int r = 0; r < R; ++r)
        for (int c = 0; c < C; ++c) {
            int64_t acc = 0;
            for (int pp = 0; pp < p; ++pp)
                for (int qq = 0; qq < q; ++qq)
                    acc += (int64_t)w[pp * q + qq] *
                           (int64_t)x[(long long)(r + pp) * x_pitch + (c + qq)];
            y[(long long)r * y_pitch + c] = acc;
        }
}
