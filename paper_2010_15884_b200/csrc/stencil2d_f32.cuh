// Second workload on the folded warp array: T Jacobi sweeps of a 3x3 stencil over an fp32 grid whose
// outermost ring keeps its values (the paper's Section 1 names stencils beside convolution as the
// workloads systolic arrays on GPUs are for).
//
//   one sweep:  v(r, c) = sum_{dr,dc} k(dr, dc) * u(r+dr, c+dc)  inside,   v = u on the ring.
//
// Mapping.  As in the 2-D output-stationary convolution, the PE dimension is the column: lane l of a warp
// holds four consecutive PEs of a 128-PE array and the warp marches down the rows of a band.  Inputs are
// FORWARDED between neighbouring PEs (the FBS way): a PE needs its left and right neighbours' values of
// each row, which cross the lane boundary by one shuffle per side and row; inside a lane the forwarding is
// register renaming.  What is new is the time dimension: the T sweeps are fused in ONE pass over the grid
// (temporal blocking in registers).  Each time level t < T keeps a three-row window of its values in PE
// registers; when row i of the input arrives, level 1 finishes row i-2, level 2 row i-4, ... and level T row
// i-2T, which is stored (a lag of two rows per level makes the levels of one step independent of each other).
// The grid is read once and written once for T sweeps: 8/T bytes per point and sweep instead of 8.
//
// A PE at the edge of a strip (or a row at the edge of a band) lacks a neighbour, so what it computes is
// wrong from level 1 on and the error moves one PE inwards per level: a strip of 128 PEs yields 128 - 2*HL
// correct columns after T levels (HL = T rounded up to a multiple of 4, so that the correct part is made
// of whole lanes and leaves as aligned 128-bit words), strips and bands overlap accordingly, and the
// values computed in the overlap are never stored.  The grid's own ring is different: its values are fixed,
// so it needs no neighbours and is exact at every level.
#pragma once

#include "conv2d_kernels.cuh"

namespace sysconv {

constexpr int kStencilMaxFused = 4;     // sweeps fused in one launch

struct StencilCoef {
    float k[9];     // k[(dr+1)*3 + (dc+1)]
};

template <int T>
struct StencilGeom {
    static constexpr int kHalo = (T + 3) / 4 * 4;               // columns given up on each side of a strip
    static constexpr int kValid = kLanes * 4 - 2 * kHalo;       // correct columns per strip
};

// FIVE: the four corner coefficients are zero (five-point stencil): their multiply-adds are left out.
template <int T, bool FIVE>
__global__ void __launch_bounds__(kThreads2, 4)
stencil2d_kernel(const Conv2DArgs a, const __grid_constant__ StencilCoef coef, const int band_h)
{
    dependent_launch_enter();
    using Tr = F32Traits;
    constexpr int R = 4;
    constexpr int HL = StencilGeom<T>::kHalo;
    constexpr int V = StencilGeom<T>::kValid;
    const int lane = threadIdx.x & (kLanes - 1);
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;
    const int c_out0 = strip * V;                   // first column this strip is responsible for
    if (c_out0 >= a.width) return;
    const int col = c_out0 - HL + R * lane;         // first column of this lane's PEs (may lie outside the grid)
    const int r_out0 = blockIdx.y * band_h;
    const int r_out1 = min(r_out0 + band_h, a.height);          // one past the band's last row
    const float *xb = static_cast<const float *>(a.x) + blockIdx.z * a.x_bstride;
    float *yb = static_cast<float *>(a.y) + blockIdx.z * a.y_bstride;
    const bool x_vec = row_alignment(static_cast<const float *>(a.x), a.x_pitch, a.x_bstride, a.batch) == 4;
    const int y_align = row_alignment(static_cast<const float *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const int last_row = a.height - 1, last_col = a.width - 1;

    // PEs on the grid's ring columns (and the ones outside the grid, whose values nobody uses) keep their values
    bool keeps[R];
#pragma unroll
    for (int j = 0; j < R; ++j) keeps[j] = col + j <= 0 || col + j >= last_col;
    const bool stores = lane >= HL / R && lane < kLanes - HL / R && col < a.width;

    // PE registers: for each time level 0 .. T-1 the window of its last three rows; a row is the lane's four
    // values with the left neighbour's last and the right neighbour's first value beside them
    float win[T][3][R + 2];
#pragma unroll
    for (int t = 0; t < T; ++t)
#pragma unroll
        for (int d = 0; d < 3; ++d)
#pragma unroll
            for (int j = 0; j < R + 2; ++j) win[t][d][j] = 0.f;

    // A new row of a level enters its window: the neighbours' edge values are forwarded by one shuffle per side.
    // The windows are rings: the row loop is unrolled three times and at position u of the unrolled group every
    // level writes slot u (its oldest row), so no row is ever moved between registers.
    auto push = [&](int t, int slot, const float (&v)[R]) {
        win[t][slot][0] = __shfl_up_sync(kFullMask, v[R - 1], 1);   // lane 0 keeps its own: the strip's edge
#pragma unroll
        for (int j = 0; j < R; ++j) win[t][slot][j + 1] = v[j];
        win[t][slot][R + 1] = __shfl_down_sync(kFullMask, v[0], 1); // lane 31 likewise
    };
    // Schedule: input row i enters level 0 at step i, and at the same step level t completes its row i-2t from the
    // rows i-2t-1 .. i-2t+1 that level t-1 had completed BEFORE this step.  Every level thus lags its predecessor
    // by two rows, and the T levels of one step do not depend on each other: they are issued highest level first
    // (each reads its predecessor's window before that one is overwritten) and overlap in the pipelines.
    //
    // One step exists in two forms.  The checked form chooses, per PE and level, between the stencil and the fixed
    // value (ring columns, ring rows); the plain form carries no test at all and is taken whenever the strip holds
    // no ring column and none of the T rows completed in this step is a ring row -- almost always.  The choice is
    // warp-uniform and made once per step, so that inside a step nothing separates the T independent levels.
    const int r_in0 = max(r_out0 - T, 0);           // first input row the band needs
    const int i_end = r_out1 + 2 * T;               // level T completes the band's last row at step r_out1-1+2T
    const float *xrow = xb + static_cast<long long>(r_in0) * a.x_pitch;     // the row that is loaded next
    int next_row = r_in0;
    auto load_next = [&](float (&v)[R]) {
        if (next_row <= last_row && col >= 0) {
            load_group<Tr>(xrow, col, a.width, x_vec, v);
        } else {
            // rows beyond the grid (and PEs left of it) enter as zeros and only keep the windows in step
#pragma unroll
            for (int j = 0; j < R; ++j) v[j] = 0.f;
        }
        xrow += a.x_pitch;
        ++next_row;
    };
    const int c_end = min(a.width, c_out0 + V);
    // does any PE of this strip sit on (or outside) the grid's first or last column?
    const bool edge_strip = c_out0 - HL <= 0 || c_out0 - HL + kLanes * R > last_col;
    float nxt[R];
    load_next(nxt);
    auto step = [&](auto checked_tag, auto phase_tag, int i) {
        constexpr bool CHECKED = decltype(checked_tag)::value;
        constexpr int u = decltype(phase_tag)::value;
        // before this step's push, level t-1 holds its three newest rows in the slots u (oldest), u+1, u+2
        constexpr int top = u % 3, mid = (u + 1) % 3, bot = (u + 2) % 3;
        float cur[R];
#pragma unroll
        for (int j = 0; j < R; ++j) cur[j] = nxt[j];
        load_next(nxt);
#pragma unroll
        for (int t = T; t >= 1; --t) {
            const int ri = i - 2 * t;
            const bool ring_row = CHECKED && (ri <= 0 || ri >= last_row);
            float v[R];
#pragma unroll
            for (int j = 0; j < R; ++j) {
                const float centre = win[t - 1][mid][j + 1];
                float acc = centre * coef.k[4];
                acc = fmaf(coef.k[1], win[t - 1][top][j + 1], acc);
                acc = fmaf(coef.k[3], win[t - 1][mid][j], acc);
                acc = fmaf(coef.k[5], win[t - 1][mid][j + 2], acc);
                acc = fmaf(coef.k[7], win[t - 1][bot][j + 1], acc);
                if (!FIVE) {
                    acc = fmaf(coef.k[0], win[t - 1][top][j], acc);
                    acc = fmaf(coef.k[2], win[t - 1][top][j + 2], acc);
                    acc = fmaf(coef.k[6], win[t - 1][bot][j], acc);
                    acc = fmaf(coef.k[8], win[t - 1][bot][j + 2], acc);
                }
                v[j] = (CHECKED && (ring_row || keeps[j])) ? centre : acc;   // a value on the ring stays
            }
            if (t < T) {
                push(t, u, v);
            } else if (ri >= r_out0 && ri < r_out1 && stores) {
                store_group<Tr>(yb + static_cast<long long>(ri) * a.y_pitch, col, c_end, y_align, v);
            }
        }
        push(0, u, cur);
    };
#pragma unroll 1
    for (int ib = r_in0; ib < i_end; ib += 3) {
        // rows completed in the three steps ib .. ib+2: level 1's ib-2 .. ib (the highest), level T's ib-2T .. (the lowest)
        const bool checked = edge_strip || ib - 2 * T <= 0 || ib >= last_row;
        if (checked) {
            step(std::true_type{}, std::integral_constant<int, 0>{}, ib);
            if (ib + 1 < i_end) step(std::true_type{}, std::integral_constant<int, 1>{}, ib + 1);
            if (ib + 2 < i_end) step(std::true_type{}, std::integral_constant<int, 2>{}, ib + 2);
        } else {
            step(std::false_type{}, std::integral_constant<int, 0>{}, ib);
            if (ib + 1 < i_end) step(std::false_type{}, std::integral_constant<int, 1>{}, ib + 1);
            if (ib + 2 < i_end) step(std::false_type{}, std::integral_constant<int, 2>{}, ib + 2);
        }
    }
}

template <int T>
cudaError_t launch_stencil2d_t(const Conv2DArgs &a, const StencilCoef &coef, bool five, cudaStream_t s)
{
    constexpr int V = StencilGeom<T>::kValid;
    const int strips = (a.width + V - 1) / V;
    const int wpb = block_warps(strips, kWarps2);       // narrow grids: blocks of as many warps as there are strips
    const long long per_band = static_cast<long long>((strips + wpb - 1) / wpb) * a.batch;
    // bands re-read and re-compute 2T rows each: long bands for large grids, bands by the number of block waves
    // for small ones
    int band_h = 128;
    static const long long slots4 = 148LL * resident_blocks_per_sm(stencil2d_kernel<T, false>, kThreads2);
    const long long slots = slots4 * kWarps2 / wpb;
    if (small_problem(a.height, per_band, 8, slots)) band_h = pick_band_height_small(a.height, per_band, 2 * T + 1, 8, 128, slots);
    dim3 grid((strips + wpb - 1) / wpb, (a.height + band_h - 1) / band_h, a.batch);
    if (grid.y > 65535 || a.batch > 65535) return cudaErrorInvalidConfiguration;
    if (five) launch_kernel(stencil2d_kernel<T, true>, grid, wpb * kLanes, s, a, coef, band_h);
    else launch_kernel(stencil2d_kernel<T, false>, grid, wpb * kLanes, s, a, coef, band_h);
    return cudaGetLastError();
}

}  // namespace sysconv
