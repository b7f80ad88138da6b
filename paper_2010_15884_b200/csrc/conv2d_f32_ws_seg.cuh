// 2-D fp32 weight-stationary convolution (derived from BSM: PE = q keeps the P taps of filter column q,
// t = P*(c+q)+p) with the arrays laid side by side ALONG THE ROWS, as in the 1-D weight-stationary kernel.
//
// An array (Q <= 15 PEs) is folded entirely into one lane: PE-to-PE transfer is register renaming and the
// stationary taps are uniform operands.  The 32 arrays of a warp take 32 consecutive 20-column segments of the
// same four output rows; array a streams the image columns of segment a and nothing else.  Macro-step T
// broadcasts the P+3 inputs of image column T that feed the four rows to the array; the sums of two neighbouring
// outputs travel together in a register pair (one packed fp32x2 FMA per tap, multiplicand (x, x), multiplier the
// aligned tap pair); PE 0 opens a pair, the pair leaves PE Q-1 one filter column short and the emission adds it.
//
// Arrays neither fill nor drain: each runs exactly the 20 macro-steps of its segment.  The sums still in flight
// when array a stops are continued by array a+1, which starts from empty PEs: what it emits during its first
// steps are the missing parts of segment a's last outputs, so they are written into segment a's tail and array a
// adds its in-flight registers to them afterwards.  The last array of a warp (lane 31) is only such a successor:
// its own outputs belong to the next slice and are not stored, so a warp yields 31 x 20 = 620 output columns.
//
// Data movement: a lane reads the inputs of its own segment straight from memory (128-bit loads; the 32 lanes of
// a warp together cover one contiguous 2560-byte piece of every row, so each sector is fetched from L2 once and
// served from L1 after that); the outputs of the four rows are collected in shared memory, where the hand-over
// above takes place, and leave as contiguous 128-bit stores.  The previous form of this kernel had the arrays
// stacked over the rows and moved every input and output through a transpose in shared memory, which bound it
// to the load/store unit (49 % of the HBM roofline at 3x3).
#pragma once

#include "conv2d_f32_is_pair.cuh"

namespace sysconv {

constexpr int kWsgM = 4;                        // output rows per pass
constexpr int kWsgSeg = 20;                     // image columns per array and pass (even, >= the longest filter row)
constexpr int kWsgIn = kLanes * kWsgSeg;        // 640 columns read per warp
constexpr int kWsgOut = (kLanes - 1) * kWsgSeg; // 620 columns written per warp
constexpr int kWsgPitch = kWsgIn + 4;           // floats per row of the output tile

template <int P, int Q>
__global__ void __launch_bounds__(kLanes)
conv2d_ws_seg_kernel(const Conv2DArgs a, const __grid_constant__ Taps2D taps, const __grid_constant__ TapsColPairs tp,
                     const int band_h)
{
    dependent_launch_enter();
    using Tr = F32Traits;
    constexpr int M = kWsgM, K = M + P - 1, SEG = kWsgSeg;
    // image columns fetched per load: four (128-bit loads) while the K rows of a chunk fit the registers beside
    // the 4 x Q pairs, two (64-bit loads) for the taller filters
    constexpr int CW = K <= 9 ? 4 : 2;
    static_assert(Q <= SEG && SEG % 4 == 0, "a filter row longer than a segment breaks the hand-over");
    __shared__ __align__(16) float s_o[M * kWsgPitch];

    const int lane = threadIdx.x;
    const int c0 = blockIdx.x * kWsgOut;                // first output column of the slice
    const int col0 = c0 + lane * SEG;                   // first image column of this lane's segment
    const int c_end = min(a.out_w, c0 + kWsgOut);       // one past the last output column this warp stores
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const float *xb = static_cast<const float *>(a.x) + blockIdx.z * a.x_bstride;
    float *yb = static_cast<float *>(a.y) + blockIdx.z * a.y_bstride;
    const int x_align = row_alignment(static_cast<const float *>(a.x), a.x_pitch, a.x_bstride, a.batch);
    const int y_align = row_alignment(static_cast<const float *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    float *yo = s_o + lane * SEG;                       // this array's segment in row 0 of the output tile

#pragma unroll 1
    for (int rg = r0; rg < r1; rg += M) {
        float2 Z[M][Q];                                 // Z[m][s]: the pair in PE s of output row rg+m
#pragma unroll
        for (int m = 0; m < M; ++m)
#pragma unroll
            for (int s = 0; s < Q; ++s) Z[m][s] = make_float2(0.f, 0.f);

#pragma unroll 1
        for (int kc = 0; kc < SEG / CW; ++kc) {
            // the inputs of CW image columns for the K rows that feed the four output rows
            float xk[K][CW];
#pragma unroll
            for (int kk = 0; kk < K; ++kk) {
                const float *rowp = xb + static_cast<long long>(min(rg + kk, a.height - 1)) * a.x_pitch;
                const int c = col0 + CW * kc;
                if (CW == 4) {
                    load_group<Tr>(rowp, c, a.width, x_align == 4, xk[kk]);
                } else if (x_align >= 2 && c + 1 < a.width) {
                    const float2 t2 = __ldg(reinterpret_cast<const float2 *>(rowp + c));
                    xk[kk][0] = t2.x; xk[kk][1] = t2.y;
                } else {
#pragma unroll
                    for (int e = 0; e < CW; ++e) xk[kk][e] = c + e < a.width ? __ldg(rowp + c + e) : 0.f;
                }
            }
#pragma unroll
            for (int v = 0; v < CW; ++v) {
                const int t = CW * kc + v;              // macro-step = column inside the segment; t and v have the same parity
                if (v % 2 == Q % 2) {
                    // the pairs that left PE Q-1 one step ago: outputs t-Q and t-Q+1 of the segment.  Negative
                    // positions are the tail of the previous segment and receive this array's share of those sums
                    // (the slice's first array has no predecessor here: the previous slice's last lane does that)
                    const int o = t - Q;
                    if (o >= 0 || lane > 0) {
#pragma unroll
                        for (int m = 0; m < M; ++m) {
                            float z = Z[m][Q - 1].y;
#pragma unroll
                            for (int p = 0; p < P; ++p) z = fmaf(xk[m + p][v], taps.w[p * Q + Q - 1], z);
                            *reinterpret_cast<float2 *>(yo + m * kWsgPitch + o) = make_float2(Z[m][Q - 1].x, z);
                        }
                    }
                }
#pragma unroll
                for (int m = 0; m < M; ++m) {
#pragma unroll
                    for (int s = Q - 1; s >= 1; --s) {
                        if (s % 2 != v % 2) continue;
                        float2 z = Z[m][s - 1];
#pragma unroll
                        for (int p = 0; p < P; ++p)     // sub-steps p of macro-step t
                            z = __ffma2_rn(make_float2(xk[m + p][v], xk[m + p][v]), tp.w[p * (Q + 1) + s], z);
                        Z[m][s] = z;
                    }
                    if (v % 2 == 0) {
                        float z = xk[m][v] * taps.w[0]; // PE 0 opens a pair: filter column 0, first sum only
#pragma unroll
                        for (int p = 1; p < P; ++p) z = fmaf(xk[m + p][v], taps.w[p * Q], z);
                        Z[m][0] = make_float2(z, 0.f);
                    }
                }
            }
        }
        __syncwarp();
        // the odd PEs stopped while holding the pairs of outputs SEG-1-s and SEG-s of the segment: add them to what
        // the successor has written there (lane 31 has no successor in this warp; its outputs are not stored)
#pragma unroll
        for (int m = 0; m < M; ++m)
#pragma unroll
            for (int s = 1; s < Q; s += 2) {
                yo[m * kWsgPitch + SEG - 1 - s] += Z[m][s].x;
                yo[m * kWsgPitch + SEG - s] += Z[m][s].y;
            }
        __syncwarp();
        // the tile's four rows leave as contiguous 128-bit words
#pragma unroll
        for (int m = 0; m < M; ++m) {
            if (rg + m < r1) {
                float *orow = yb + static_cast<long long>(rg + m) * a.y_pitch;
                for (int i = lane; i < kWsgOut / 4; i += kLanes) {
                    const float4 t4 = *reinterpret_cast<const float4 *>(s_o + m * kWsgPitch + 4 * i);
                    const float v4[4] = {t4.x, t4.y, t4.z, t4.w};
                    store_group<Tr>(orow, c0 + 4 * i, c_end, y_align, v4);
                }
            }
        }
        __syncwarp();                                   // the tile is free for the next four rows
    }
}

template <int P, int Q>
cudaError_t launch_conv2d_ws_seg(const Conv2DArgs &a, const Taps2D &taps, cudaStream_t s)
{
    TapsColPairs tp{};
    for (int p = 0; p < P; ++p)
        for (int t = 0; t <= Q; ++t)
            tp.w[p * (Q + 1) + t] = make_float2(t < Q ? taps.w[p * Q + t] : 0.f, t >= 1 ? taps.w[p * Q + t - 1] : 0.f);
    const long long slices = (a.out_w + kWsgOut - 1) / kWsgOut;
    // one-warp blocks: bands of four-row passes, short enough to give every SM a few dozen blocks
    const long long want = 148LL * 48;
    long long bands = (want + slices * a.batch - 1) / (slices * a.batch);
    long long band_h = (a.out_h + bands - 1) / bands;
    band_h = (band_h + kWsgM - 1) / kWsgM * kWsgM;
    if (band_h < kWsgM) band_h = kWsgM;
    if ((a.out_h + band_h - 1) / band_h > 65535) band_h = ((a.out_h + 65534) / 65535 + kWsgM - 1) / kWsgM * kWsgM;
    dim3 grid(static_cast<unsigned>(slices), static_cast<unsigned>((a.out_h + band_h - 1) / band_h), a.batch);
    launch_kernel(conv2d_ws_seg_kernel<P, Q>, grid, kLanes, s, a, taps, tp, static_cast<int>(band_h));
    return cudaGetLastError();
}

}  // namespace sysconv
