// 2-D fp32 weight-stationary convolution for the smaller filters (at most 8 filter columns and a window of at most
// 96 registers: up to 9 x 8 and 15 x 4; wider filters of one or two rows): the arrays
// side by side ALONG THE ROWS, everything in registers, no shared memory.
//
// As in the other weight-stationary kernels an array (Q PEs, PE q keeps the P taps of filter column q) is folded
// into one lane, the taps are uniform operands and the sums of two neighbouring outputs travel as a register
// pair updated by one packed fp32x2 FMA per tap.  Here array a (lane a) takes the SEG = 4, 8 or 16 image columns
// [c0 + SEG*a, c0 + SEG*(a+1)) of a row group: exactly the columns its lane fetches with its own 128-bit loads,
// which are contiguous across the warp -- the broadcast input of macro-step T is simply register T of that load,
// so no transpose and no staging is needed.  Every array runs exactly SEG macro-steps, neither filling nor
// draining: the sums still in flight when array a stops are continued by array a+1 from empty PEs (linearity),
// and what array a+1 emits for them is handed back to lane a by one shuffle per value and added to the in-flight
// registers there.  Lane 31 has no successor in its warp: it only serves as lane 30's successor, its own outputs
// belong to the next slice, so a warp yields 31 * SEG output columns.
//
// The K = P+3 input rows that feed four output rows stay in registers as a window that slides down four rows per
// pass (four new loads per lane and pass, issued one pass ahead), so every input is read from memory once per
// band.  The earlier form of this kernel (arrays stacked over the rows, two transposes through shared memory)
// was bound by the load/store unit at these filter sizes (49 % of the HBM roofline at 3x3).
#pragma once

#include "conv2d_f32_is_pair.cuh"

namespace sysconv {

constexpr int kWsrM = 4;                        // output rows per pass
constexpr int kWsrWarps = 4;

template <int P, int Q>
struct WsrShape {
    static constexpr int kSeg = Q <= 4 ? 4 : Q <= 8 ? 8 : 16;   // image columns per array and pass
    // window registers: (P+3) x segment.  Measured on 2 x 2048 x 4096 against the form with transposed staging: 6x5
    // 65 -> 37 us, 7x7 72 -> 50, 8x6 73 -> 52, 9x7 79 -> 70, 9x8 level; 11 rows: 11x5 76 -> 66 but 11x8 86 -> 104
    // 16-column segments (filters of 9 to 15 columns) pay for one and two filter rows (1x15 52 -> 38 us, 2x13 66 -> 45);
    // with three rows the two forms are level
    static constexpr bool kFits = kSeg == 16 ? P <= 2 : (P + kWsrM - 1) * kSeg <= 96;
    static constexpr int kOut = (kLanes - 1) * kSeg;            // output columns per warp
};

template <int P, int Q>
__global__ void __launch_bounds__(kWsrWarps *kLanes)
conv2d_ws_reg_kernel(const Conv2DArgs a, const __grid_constant__ Taps2D taps, const __grid_constant__ TapsColPairs tp,
                     const int band_h)
{
    dependent_launch_enter();
    using Tr = F32Traits;
    constexpr int M = kWsrM, K = M + P - 1, SEG = WsrShape<P, Q>::kSeg, W4 = SEG / 4;
    constexpr int kTail = Q - Q % 2;            // outputs at the end of a segment whose sums are still in flight
    static_assert(Q <= SEG, "a filter row longer than a segment breaks the hand-over");
    const int lane = threadIdx.x & (kLanes - 1);
    const int slice = blockIdx.x * kWsrWarps + threadIdx.x / kLanes;    // (a block of fewer warps is the only one of its row)
    const int c0 = slice * WsrShape<P, Q>::kOut;        // first output column of the slice
    if (c0 >= a.out_w) return;
    const int col0 = c0 + lane * SEG;                   // first image column of this lane's segment
    const int c_end = min(a.out_w, c0 + WsrShape<P, Q>::kOut);
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const float *xb = static_cast<const float *>(a.x) + blockIdx.z * a.x_bstride;
    float *yb = static_cast<float *>(a.y) + blockIdx.z * a.y_bstride;
    const bool x_vec = row_alignment(static_cast<const float *>(a.x), a.x_pitch, a.x_bstride, a.batch) == 4;
    const int y_align = row_alignment(static_cast<const float *>(a.y), a.y_pitch, a.y_bstride, a.batch);

    auto load_row = [&](int row, float (&v)[SEG]) {
        const float *rowp = xb + static_cast<long long>(min(row, a.height - 1)) * a.x_pitch;
#pragma unroll
        for (int g = 0; g < W4; ++g) load_group<Tr>(rowp, col0 + 4 * g, a.width, x_vec, &v[4 * g]);
    };

    // PE-side registers: the window of K input rows of this lane's segment
    float X[K][SEG];
#pragma unroll
    for (int kk = 0; kk < K - M; ++kk) load_row(r0 + kk, X[kk + M]);      // rows the first slide moves to the top
    float nX[M][SEG];
#pragma unroll
    for (int m = 0; m < M; ++m) load_row(r0 + K - M + m, nX[m]);

#pragma unroll 1
    for (int rg = r0; rg < r1; rg += M) {
        // the window slides down four rows: the rows it keeps move up, the four prefetched rows enter
#pragma unroll
        for (int kk = 0; kk < K - M; ++kk)
#pragma unroll
            for (int t = 0; t < SEG; ++t) X[kk][t] = X[kk + M][t];
#pragma unroll
        for (int m = 0; m < M; ++m)
#pragma unroll
            for (int t = 0; t < SEG; ++t) X[K - M + m][t] = nX[m][t];
        if (rg + M < r1) {
#pragma unroll
            for (int m = 0; m < M; ++m) load_row(rg + M + K - M + m, nX[m]);
        }

#pragma unroll
        for (int m = 0; m < M; ++m) {
            float2 Z[Q];                        // Z[s]: the pair in PE s (live at the parity of the macro-step)
#pragma unroll
            for (int s = 0; s < Q; ++s) Z[s] = make_float2(0.f, 0.f);
            float own[SEG];                     // outputs of this segment (the last kTail of them: in-flight parts)
            float part[kTail > 0 ? kTail : 1];  // this array's share of the previous segment's last kTail outputs
#pragma unroll
            for (int t = 0; t < SEG; ++t) {
                if (t % 2 == Q % 2) {
                    // the pair that left PE Q-1 one step ago: outputs t-Q and t-Q+1 of the segment
                    float z = Z[Q - 1].y;
#pragma unroll
                    for (int p = 0; p < P; ++p) z = fmaf(X[m + p][t], taps.w[p * Q + Q - 1], z);
                    const int o = t - Q;
                    if (o >= 0) {
                        own[o] = Z[Q - 1].x;
                        own[o + 1] = z;
                    } else {
                        part[o + kTail] = Z[Q - 1].x;
                        part[o + kTail + 1] = z;
                    }
                }
#pragma unroll
                for (int s = Q - 1; s >= 1; --s) {
                    if (s % 2 != t % 2) continue;
                    float2 z = Z[s - 1];
#pragma unroll
                    for (int p = 0; p < P; ++p)         // sub-steps p of macro-step t
                        z = __ffma2_rn(make_float2(X[m + p][t], X[m + p][t]), tp.w[p * (Q + 1) + s], z);
                    Z[s] = z;
                }
                if (t % 2 == 0) {
                    float z = X[m][t] * taps.w[0];      // PE 0 opens a pair: filter column 0, first sum only
#pragma unroll
                    for (int p = 1; p < P; ++p) z = fmaf(X[m + p][t], taps.w[p * Q], z);
                    Z[0] = make_float2(z, 0.f);
                }
            }
            // the odd PEs stopped while holding the pairs of outputs SEG-1-s and SEG-s: this array's part of them;
            // the successor (lane + 1) holds the other part and hands it back by shuffle
#pragma unroll
            for (int s = 1; s < Q; s += 2) {
                own[SEG - 1 - s] = Z[s].x;
                own[SEG - s] = Z[s].y;
            }
#pragma unroll
            for (int j = 0; j < kTail; ++j) own[SEG - kTail + j] += __shfl_down_sync(kFullMask, part[j], 1);
            if (rg + m < r1 && lane < kLanes - 1) {
                float *orow = yb + static_cast<long long>(rg + m) * a.y_pitch;
#pragma unroll
                for (int g = 0; g < W4; ++g) store_group<Tr>(orow, col0 + 4 * g, c_end, y_align, &own[4 * g]);
            }
        }
    }
}

template <int P, int Q>
cudaError_t launch_conv2d_ws_reg(const Conv2DArgs &a, const Taps2D &taps, cudaStream_t s)
{
    TapsColPairs tp{};
    for (int p = 0; p < P; ++p)
        for (int t = 0; t <= Q; ++t)
            tp.w[p * (Q + 1) + t] = make_float2(t < Q ? taps.w[p * Q + t] : 0.f, t >= 1 ? taps.w[p * Q + t - 1] : 0.f);
    constexpr int kOut = WsrShape<P, Q>::kOut;
    const int slices = (a.out_w + kOut - 1) / kOut;
    const int wpb = block_warps(slices, kWsrWarps);
    const long long per_band = static_cast<long long>((slices + wpb - 1) / wpb) * a.batch;
    // bands of four-row passes; every band re-reads the P-1 rows above it
    static const long long slots4 = 148LL * resident_blocks_per_sm(conv2d_ws_reg_kernel<P, Q>, kWsrWarps * kLanes);
    const long long slots = slots4 * kWsrWarps / wpb;       // smaller blocks: as many more of them are resident
    long long band_h;
    if (small_problem(a.out_h, per_band, kWsrM, slots)) {
        band_h = pick_band_height_small(a.out_h, per_band, P, kWsrM, 64, slots);
    } else {
        const long long bands = (148LL * 16 + per_band - 1) / per_band;
        band_h = (a.out_h + bands - 1) / bands;
        if (band_h > 64) band_h = 64;
    }
    band_h = (band_h + kWsrM - 1) / kWsrM * kWsrM;
    if ((a.out_h + band_h - 1) / band_h > 65535) band_h = ((a.out_h + 65534) / 65535 + kWsrM - 1) / kWsrM * kWsrM;
    dim3 grid((slices + wpb - 1) / wpb, static_cast<unsigned>((a.out_h + band_h - 1) / band_h), a.batch);
    launch_kernel(conv2d_ws_reg_kernel<P, Q>, grid, wpb * kLanes, s, a, taps, tp, static_cast<int>(band_h));
    return cudaGetLastError();
}

}  // namespace sysconv
