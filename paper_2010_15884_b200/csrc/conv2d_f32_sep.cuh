// Separable 2-D convolution, y(r, c) = sum_p sum_q u(p) v(q) x(r+p, c+q), fp32: a second workload on the same
// folded array.  It is Section 6's "multiple FBS 1-D convolutions" taken literally: every input row goes
// through ONE 1-D output-stationary (FBS) pass with the horizontal taps v (inputs forwarded one PE down per
// step, weights broadcast), and the resulting row feeds the P partial output rows that sediment in the PEs
// through the vertical taps u.  P + Q multiply-adds per output instead of P * Q, so every filter size up to
// 15 x 15 stays HBM-bound.  Strip / band decomposition, halo registers and row prefetch as in conv2d_os_kernel.
#pragma once

#include "conv2d_kernels.cuh"

namespace sysconv {

struct TapsSep {
    float u[kMaxP2];        // vertical taps (filter rows)
    float v[kMaxQ2];        // horizontal taps (filter columns)
};

template <int P, int Q, int R, int PF>
__global__ void __launch_bounds__(kThreads2)
conv2d_sep_os_kernel(const Conv2DArgs a, const __grid_constant__ TapsSep taps, const int band_h)
{
    dependent_launch_enter();
    using Tr = F32Traits;
    static_assert(R == 4 || R == 8, "R = PEs per lane");
    constexpr int kStrip = kLanes * R;
    constexpr bool kHalo = Q > 1;
    constexpr bool kHaloChain = Q - 1 > 4;      // the halo spans more than one lane
    const int lane = threadIdx.x & (kLanes - 1);
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;
    const int c0 = strip * kStrip;
    if (c0 >= a.out_w) return;
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const float *xb = static_cast<const float *>(a.x) + blockIdx.z * a.x_bstride;
    float *yb = static_cast<float *>(a.y) + blockIdx.z * a.y_bstride;
    const bool x_vec = row_alignment(static_cast<const float *>(a.x), a.x_pitch, a.x_bstride, a.batch) == 4;
    const int y_align = row_alignment(static_cast<const float *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const int col = c0 + R * lane;              // first column of this lane's PEs
    const int hcol = c0 + kStrip + 4 * lane;    // halo columns (lanes 0 .. ceil((Q-1)/4)-1)
    const bool has_halo = kHalo && 4 * lane < Q - 1;
    const int i_end = r1 + P - 1;               // input rows r0 .. i_end-1

    float Z[P][R];
#pragma unroll
    for (int p = 0; p < P; ++p)
#pragma unroll
        for (int j = 0; j < R; ++j) Z[p][j] = 0.f;

    float nX[PF][R], nH[PF][4];
#pragma unroll
    for (int f = 0; f < PF; ++f)
#pragma unroll
        for (int j = 0; j < 4; ++j) nH[f][j] = 0.f;
    auto fetch = [&](int row, float *dx, float *dh) {
        if (row < i_end) {
            const float *rowp = xb + static_cast<long long>(row) * a.x_pitch;
#pragma unroll
            for (int g = 0; g < R / 4; ++g) load_group<Tr>(rowp, col + 4 * g, a.width, x_vec, dx + 4 * g);
            if (has_halo) load_group<Tr>(rowp, hcol, a.width, x_vec, dh);
        }
    };
    auto process = [&](int i, int f) {
        float X[R], H[4], S[R];
#pragma unroll
        for (int j = 0; j < R; ++j) X[j] = nX[f][j];
#pragma unroll
        for (int j = 0; j < 4; ++j) H[j] = nH[f][j];
        fetch(i + PF, nX[f], nH[f]);
        // one 1-D FBS pass over the row: S(c) = sum_q v(q) x(i, c+q)
#pragma unroll
        for (int q = 0; q < Q; ++q) {
#pragma unroll
            for (int j = 0; j < R; ++j) S[j] = q == 0 ? X[j] * taps.v[0] : fmaf(X[j], taps.v[q], S[j]);
            if (q < Q - 1) {
                // forward the inputs one PE down; the strip's last PE takes the halo from lane 0
                const float send = (lane == 0) ? H[0] : X[0];
                const float in0 = __shfl_sync(kFullMask, send, (lane + 1) & (kLanes - 1));
#pragma unroll
                for (int j = 0; j < R - 1; ++j) X[j] = X[j + 1];
                X[R - 1] = in0;
                float in1 = 0.f;
                if (kHaloChain) in1 = __shfl_down_sync(kFullMask, H[0], 1);
                H[0] = H[1]; H[1] = H[2]; H[2] = H[3]; H[3] = in1;
            }
        }
        // the row's result feeds output rows i-p through the vertical tap u(p); the partial rows rotate:
        // the sums of output row i-p were in Z[p-1]
#pragma unroll
        for (int p = P - 1; p > 0; --p)
#pragma unroll
            for (int j = 0; j < R; ++j) Z[p][j] = fmaf(S[j], taps.u[p], Z[p - 1][j]);
#pragma unroll
        for (int j = 0; j < R; ++j) Z[0][j] = S[j] * taps.u[0];
        const int r = i - (P - 1);              // output row completed by this input row
        if (r >= r0) {
            float *orow = yb + static_cast<long long>(r) * a.y_pitch;
#pragma unroll
            for (int g = 0; g < R / 4; ++g) store_group<Tr>(orow, col + 4 * g, a.out_w, y_align, &Z[P - 1][4 * g]);
        }
    };

#pragma unroll
    for (int f = 0; f < PF; ++f) fetch(r0 + f, nX[f], nH[f]);
#pragma unroll 1
    for (int i = r0; i < i_end; i += PF) {
        process(i, 0);
#pragma unroll
        for (int f = 1; f < PF; ++f)
            if (i + f < i_end) process(i + f, f);
    }
}

template <int P, int Q>
cudaError_t launch_conv2d_sep_pq(const Conv2DArgs &a, const TapsSep &taps, cudaStream_t s)
{
    if (a.batch > 65535) return cudaErrorInvalidConfiguration;
    // eight PEs per lane and two rows in flight (the memory-bound shape) while the P partial rows fit 128 registers
    // (measured 9+9: 0.487 -> 0.456 ms against four PEs; 11 rows need 159 registers and ran 47-58 us on 2 x 2048 x 4096
    // where 9 rows take 35-39, 10 rows with more than 9 columns 70-77 against 58); four PEs per lane for taller
    // filters and on small images
    constexpr int RW = (P <= 9 || (P == 10 && Q <= 9)) ? 8 : 4;
    const long long strips8 = (a.out_w + 255) / 256;
    const bool narrow = RW == 8 && strips8 * a.batch * ((a.out_h + 7) / 8) < 148LL * 8 * 4;
    const int per_strip = narrow ? kLanes * 4 : kLanes * RW;
    const int strips = (a.out_w + per_strip - 1) / per_strip;
    const int band_h = pick_band_height(a.out_h, static_cast<long long>(strips) * a.batch, P, 1);
    const int wpb = block_warps(strips, kWarps2);       // narrow images: blocks of as many warps as there are strips
    dim3 grid((strips + wpb - 1) / wpb, (a.out_h + band_h - 1) / band_h, a.batch);
    if (narrow) launch_kernel(conv2d_sep_os_kernel<P, Q, 4, 2>, grid, wpb * kLanes, s, a, taps, band_h);
    else launch_kernel(conv2d_sep_os_kernel<P, Q, RW, 2>, grid, wpb * kLanes, s, a, taps, band_h);
    return cudaGetLastError();
}

template <int P>
cudaError_t launch_conv2d_sep_p(const Conv2DArgs &a, const TapsSep &taps, int q, cudaStream_t s)
{
    switch (q) {
#define SYSCONV_CASE(QQ) case QQ: return launch_conv2d_sep_pq<P, QQ>(a, taps, s);
        SYSCONV_CASE(1) SYSCONV_CASE(2) SYSCONV_CASE(3) SYSCONV_CASE(4) SYSCONV_CASE(5)
        SYSCONV_CASE(6) SYSCONV_CASE(7) SYSCONV_CASE(8) SYSCONV_CASE(9) SYSCONV_CASE(10)
        SYSCONV_CASE(11) SYSCONV_CASE(12) SYSCONV_CASE(13) SYSCONV_CASE(14) SYSCONV_CASE(15)
#undef SYSCONV_CASE
        default: return kNoInstantiation;
    }
}

}  // namespace sysconv
