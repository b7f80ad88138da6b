// 2-D fp32 input-stationary (SBM, two projections) convolution, paired form for the larger filters.
//
// Same array as conv2d_is_kernel: PE s keeps the P-deep input column x(r .. r+P-1, s), the sums move one PE
// up per step, four PEs per lane.  Here the sums of two neighbouring outputs o (even) and o+1 of a row travel
// TOGETHER in one 64-bit register pair: in PE s = o+t the first takes the filter column t and the second the
// filter column t-1 of the SAME inputs, so each of the P taps is ONE packed fp32x2 FMA with the multiplicand
// (x, x) and the aligned tap pair (w(p,t), w(p,t-1)) from the kernel parameters.  The pair (o, o+1) sits in PE
// o+t at step t: the PEs with the parity of t hold the live pairs, a step is P packed FMAs on every second PE,
// and the scalar kernel's P*Q FMAs per output become P*(Q-1)/2 packed ones plus P scalar ones (the first and
// the last step touch only one sum of each pair and stay scalar, so no zero tap ever multiplies an input).
// Up to ten filter rows, two output rows are processed together, so that every tap pair read from the
// parameters serves four packed FMAs (with one row it serves two, and the uniform loads take a quarter of the
// issue slots).
// The scalar kernel is issue-bound (81-87 % of the issue slots at 60-63 % of the FMA pipe).
#pragma once

#include "conv2d_kernels.cuh"

namespace sysconv {

struct TapsColPairs {
    float2 w[kMaxP2 * (kMaxQ2 + 1)];    // w[p * (Q+1) + t] = (w(p,t), w(p,t-1)); taps outside 0..Q-1 are zero
};

template <int Q>
struct IsPairGeom {
    // moves without arithmetic after the last step, until a lane's four outputs start at a multiple of four
    static constexpr int drain()
    {
        for (int d = 0; d < 4; ++d)
            if (((Q + d) - (Q + d) % 2) % 4 == 0) return d;
        return 0;
    }
    static constexpr int kMoves = Q + drain();              // the pair (o, o+1) is stored from PE o + kMoves
    static constexpr int kPar = kMoves % 2;                 // parity of the PEs that hold the pairs then
    static constexpr int kShift = kMoves - kPar;            // lane l holds outputs 4l - kShift .. +3
    static constexpr int kValid = kStrip2 - kShift;         // outputs per strip
};

template <int P, int Q, int ROWS, int MIN_CTAS>
__global__ void __launch_bounds__(kThreads2, MIN_CTAS)
conv2d_is_pair_kernel(const Conv2DArgs a, const __grid_constant__ Taps2D taps, const __grid_constant__ TapsColPairs tp,
                      const int band_h)
{
    dependent_launch_enter();
    using Tr = F32Traits;
    using G = IsPairGeom<Q>;
    constexpr int R = R2;
    static_assert(R == 4 && Q >= 2, "four PEs per lane; a pair needs two filter columns");
    const int lane = threadIdx.x & (kLanes - 1);
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;    // (a block of fewer warps is the only one of its row)
    const int c0 = strip * G::kValid;           // first output column = first input column (PE 0)
    if (c0 >= a.out_w) return;
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const float *xb = static_cast<const float *>(a.x) + blockIdx.z * a.x_bstride;
    float *yb = static_cast<float *>(a.y) + blockIdx.z * a.y_bstride;
    const bool x_vec = row_alignment(static_cast<const float *>(a.x), a.x_pitch, a.x_bstride, a.batch) == 4;
    const int y_align = row_alignment(static_cast<const float *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const int col = c0 + R * lane;              // columns held by this lane's PEs
    const int ocol = col - G::kShift;           // output columns its PEs end up holding
    const int oend = min(a.out_w, c0 + G::kValid);

    // PE registers: the input column of each PE for ROWS output rows, rows r .. r+P+ROWS-2 (row r+p feeds
    // output row r+h through filter row p-h, so one tap pair read serves all ROWS rows)
    auto load_row = [&](int row, float *v) {
        load_group<Tr>(xb + static_cast<long long>(min(row, a.height - 1)) * a.x_pitch, col, a.width, x_vec, v);
    };
    constexpr int XR = P + ROWS - 1;
    float X[XR][R];
#pragma unroll
    for (int p = 0; p + ROWS < XR; ++p) load_row(r0 + p, X[p + ROWS]);
    float nX[ROWS][R];
#pragma unroll
    for (int h = 0; h < ROWS; ++h) load_row(r0 + P - 1 + h, nX[h]);

#pragma unroll 1
    for (int r = r0; r < r1; r += ROWS) {
        // the window of input rows slides down by ROWS
#pragma unroll
        for (int p = 0; p + ROWS < XR; ++p)
#pragma unroll
            for (int j = 0; j < R; ++j) X[p][j] = X[p + ROWS][j];
#pragma unroll
        for (int h = 0; h < ROWS; ++h)
#pragma unroll
            for (int j = 0; j < R; ++j) X[P - 1 + h][j] = nX[h][j];
        if (r + ROWS < r1) {
#pragma unroll
            for (int h = 0; h < ROWS; ++h) load_row(r + ROWS + P - 1 + h, nX[h]);
        }

        float2 Z[ROWS][R];                      // Z[h][j]: output row r+h; live while j has the parity of the step
        // step 0: the even PEs open the pairs; only the first sum of a pair has a tap (filter column 0)
#pragma unroll
        for (int j = 0; j < R; j += 2) {
#pragma unroll
            for (int h = 0; h < ROWS; ++h) {
                float z = X[h][j] * taps.w[0];
#pragma unroll
                for (int p = 1; p < P; ++p) z = fmaf(X[p + h][j], taps.w[p * Q], z);
                Z[h][j] = make_float2(z, 0.f);
            }
        }
#pragma unroll
        for (int t = 1; t <= G::kMoves; ++t) {
            float2 up[ROWS];
#pragma unroll
            for (int h = 0; h < ROWS; ++h) {
                up[h] = make_float2(0.f, 0.f);
                if (t % 2 == 0)                 // the pairs move one PE up (lane 0 has no left neighbour: invalid PEs)
                    up[h] = make_float2(__shfl_up_sync(kFullMask, Z[h][R - 1].x, 1), __shfl_up_sync(kFullMask, Z[h][R - 1].y, 1));
            }
#pragma unroll
            for (int j = R - 1; j >= 0; --j) {
                if (j % 2 != t % 2) continue;
                float2 z[ROWS];
#pragma unroll
                for (int h = 0; h < ROWS; ++h) z[h] = j == 0 ? up[h] : Z[h][j - 1];
                if (t < Q) {
#pragma unroll
                    for (int p = 0; p < P; ++p) {   // time p + P*t of the two-projection schedule
                        const float2 wp = tp.w[p * (Q + 1) + t];
#pragma unroll
                        for (int h = 0; h < ROWS; ++h) z[h] = __ffma2_rn(make_float2(X[p + h][j], X[p + h][j]), wp, z[h]);
                    }
                } else if (t == Q) {
                    // only the second sum still lacks a tap: filter column Q-1
#pragma unroll
                    for (int p = 0; p < P; ++p) {
                        const float wl = taps.w[p * Q + Q - 1];
#pragma unroll
                        for (int h = 0; h < ROWS; ++h) z[h].y = fmaf(X[p + h][j], wl, z[h].y);
                    }
                }
#pragma unroll
                for (int h = 0; h < ROWS; ++h) Z[h][j] = z[h];
            }
        }
        if (ocol >= c0) {
#pragma unroll
            for (int h = 0; h < ROWS; ++h) {
                if (r + h >= r1) break;
                const float out[4] = {Z[h][G::kPar].x, Z[h][G::kPar].y, Z[h][G::kPar + 2].x, Z[h][G::kPar + 2].y};
                store_group<Tr>(yb + static_cast<long long>(r + h) * a.y_pitch, ocol, oend, y_align, out);
            }
        }
    }
}

template <int P, int Q>
cudaError_t launch_conv2d_is_pair(const Conv2DArgs &a, const Taps2D &taps, cudaStream_t s)
{
    static_assert(P * (Q + 1) <= kMaxP2 * (kMaxQ2 + 1), "tap-pair table too small");
    TapsColPairs tp{};
    for (int p = 0; p < P; ++p)
        for (int t = 0; t <= Q; ++t) {
            const float cur = t < Q ? taps.w[p * Q + t] : 0.f;
            const float prev = t >= 1 ? taps.w[p * Q + t - 1] : 0.f;
            tp.w[p * (Q + 1) + t] = make_float2(cur, prev);
        }
    const int per_strip = IsPairGeom<Q>::kValid;
    const int strips = (a.out_w + per_strip - 1) / per_strip;
    const int band_h = pick_band_height(a.out_h, static_cast<long long>(strips) * a.batch, P, Q);
    const int wpb = block_warps(strips, kWarps2);
    dim3 grid((strips + wpb - 1) / wpb, (a.out_h + band_h - 1) / band_h, a.batch);
    if (grid.y > 65535) return cudaErrorInvalidConfiguration;
    // two output rows per pass up to ten filter rows (measured: 9x9 0.96 -> 0.85 ms); beyond that the
    // second row's registers cost more than the shared tap reads save (15x15: 2.33 ms with one row, 2.63 with two)
    constexpr int ROWS = P <= 10 ? 2 : 1;
    launch_kernel(conv2d_is_pair_kernel<P, Q, ROWS, ROWS == 2 ? 4 : 1>, grid, wpb * kLanes, s, a, taps, tp, band_h);
    return cudaGetLastError();
}

// the larger filters (more than 25 taps, or seven and more rows; at least three columns) run the paired packed-FMA
// kernel (2 x 2048 x 4096: 7x3 48 -> 38 us, 8x3 53 -> 40 us against the scalar kernel)
template <int P, int Q>
struct FastPath2D<F32Traits, SYSCONV_IS, P, Q> {
    static bool launch(const Conv2DArgs &a, const Taps2D &taps, cudaStream_t s, cudaError_t *err)
    {
        if constexpr ((P * Q > 25 || P >= 7) && Q >= 3) {
            *err = launch_conv2d_is_pair<P, Q>(a, taps, s);
            return true;
        } else {
            return false;
        }
    }
};

}  // namespace sysconv
