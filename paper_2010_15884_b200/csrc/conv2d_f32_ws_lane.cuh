// 2-D fp32 weight-stationary convolution (derived from BSM: PE = q keeps the P taps of filter column q,
// t = P*(c+q)+p), arrays folded into single lanes, paired packed-FMA form.
//
// An array has only Q <= 15 PEs, so it lives entirely in one lane (PE-to-PE transfer = register renaming, no
// shuffle); all arrays hold the same filter, so the stationary taps are uniform operands from the kernel
// parameters.  A CTA is one warp = 32 arrays stacked over 128 output rows (array a: rows 4a .. 4a+3, which
// share the broadcast inputs); it streams a segment of the image width, 8 (small filters: 16) image columns at a time.
//
// Macro-step T broadcasts the P+3 inputs x(4a .. 4a+P+2, T) of image column T to the array.  The sums of two
// neighbouring outputs o (even) and o+1 of a row travel together in one 64-bit register pair, which sits in
// PE s = T-o: that PE adds, for each of its P taps, x * (w(p,s), w(p,s-1)) with ONE packed fp32x2 FMA
// (multiplicand (x, x), multiplier the aligned tap pair from the kernel parameters).  PEs with the parity of
// T hold the live pairs.  PE 0 opens a pair with P scalar FMAs (only the first sum has a tap there) and the
// pair leaves PE Q-1 with its second sum one filter column short, which the emission adds with P scalar
// FMAs: no zero tap ever multiplies an input.
//
// Data movement: the chunk of 8 (16) image columns x 142 rows is loaded with 128-bit loads (one or two 32-byte
// sectors per row), held in registers while the previous chunk is processed, and written TRANSPOSED ([column][row]) to
// shared memory, so that an array reads its inputs of one image column with 128-bit loads that are contiguous
// across the lanes.  Outputs go the other way: the four rows' results of one column leave as one 128-bit
// store into a transposed ring of 16 or 32 columns, and complete groups of 8 (16) columns are written to memory
// as full 32-byte sectors per row.
#pragma once

#include "conv2d_f32_is_pair.cuh"
#include "conv2d_f32_ws_reg.cuh"
#include "conv2d_f32_ws_seg.cuh"

namespace sysconv {

constexpr int kWlM = 4;                         // output rows per array
constexpr int kWlRows = kLanes * kWlM;          // 128 output rows per CTA (one warp)
// Image columns per staged chunk.  Small filters are bound by the load/store unit: a warp's 128-bit global
// access covers 16 rows (16 cache lines) with 8-column chunks, 8 rows with 16-column chunks, so the wider chunk
// halves the work of the memory pipe per byte; larger filters keep the narrow chunk (registers, shared memory).
template <int P, int Q>
struct WlShape {
    static constexpr int kChunk = P * Q <= 25 ? 16 : 8;
    // how the multiply-adds of a macro-step are written out (see the kernel): 1 = sub-step outermost, 0 = chain by chain
    static constexpr int kOrder = P >= 12 ? 1 : 0;
};
constexpr int kWlPitch = 164;                   // rows per staged column: >= 128 + 14, = 4 mod 32 (conflict-free transposes)
constexpr int kWlPitchO = 132;                  // rows per column of the output ring: >= 128, = 4 mod 32

template <int P, int Q>
__global__ void __launch_bounds__(kLanes)
conv2d_ws_lane_kernel(const Conv2DArgs a, const __grid_constant__ Taps2D taps, const __grid_constant__ TapsColPairs tp,
                      const int seg_w)
{
    dependent_launch_enter();
    using Tr = F32Traits;
    constexpr int M = kWlM;
    constexpr int K = M + P - 1;                // input rows feeding M output rows
    constexpr int KG = (K + 3) / 4;
    constexpr int kRowsUsed = kWlRows + P - 1;  // staged rows that are ever read (the last group may read up to 3 more)
    constexpr int kWlChunk = WlShape<P, Q>::kChunk;
    constexpr int WPR = kWlChunk / 4;           // 128-bit words per row of a chunk
    constexpr int kGroupDelay = (Q - 1 + kWlChunk - 1) / kWlChunk;  // chunks between an output group's first input and its completion
    // columns of the output ring: groups j-delay .. j are alive (a power of two)
    constexpr int kWlRing = (kGroupDelay + 1) * kWlChunk <= 16 ? 16 : ((kGroupDelay + 1) * kWlChunk <= 32 ? 32 : 64);
    static_assert(kWlRows + 4 * KG - M <= kWlPitch, "staged column too short");
    __shared__ __align__(16) float s_x[kWlChunk * kWlPitch];
    __shared__ __align__(16) float s_o[kWlRing * kWlPitchO];

    const int lane = threadIdx.x;
    const int band0 = blockIdx.y * kWlRows;             // first output row of the CTA
    const int c0 = blockIdx.x * seg_w;                  // first output column of the segment (multiple of 8)
    const int c1 = min(c0 + seg_w, a.out_w);            // one past its last output column
    const float *xb = static_cast<const float *>(a.x) + blockIdx.z * a.x_bstride;
    float *yb = static_cast<float *>(a.y) + blockIdx.z * a.y_bstride;
    const bool x_vec = row_alignment(static_cast<const float *>(a.x), a.x_pitch, a.x_bstride, a.batch) == 4;
    const int y_align = row_alignment(static_cast<const float *>(a.y), a.y_pitch, a.y_bstride, a.batch);

    // staging of image columns [cc, cc+chunk) x rows [band0, band0 + kRowsUsed): WPR 128-bit words per row
    // (a permutation that makes the transposed stores of the four-word case conflict-free was measured: no gain)
    constexpr int kStageVec = (kRowsUsed * WPR + kLanes - 1) / kLanes;
    float pf[kStageVec][4];
    auto stage_load = [&](int cc) {
#pragma unroll
        for (int n = 0; n < kStageVec; ++n) {
            const int idx = lane + n * kLanes;
            const int row = idx / WPR, i = idx % WPR;
            if (idx < kRowsUsed * WPR) {
                const float *rowp = xb + static_cast<long long>(min(band0 + row, a.height - 1)) * a.x_pitch;
                load_group<Tr>(rowp, cc + 4 * i, a.width, x_vec, pf[n]);
            }
        }
    };
    auto stage_store = [&]() {
#pragma unroll
        for (int n = 0; n < kStageVec; ++n) {
            const int idx = lane + n * kLanes;
            const int row = idx / WPR, i = idx % WPR;
            if (idx < kRowsUsed * WPR) {
#pragma unroll
                for (int e = 0; e < 4; ++e) s_x[(4 * i + e) * kWlPitch + row] = pf[n][e];
            }
        }
    };
    // write output columns [c0 + chunk*g, c0 + chunk*(g+1)) of the CTA's 128 rows from the ring to memory
    auto flush = [&](int g) {
        const int ocol = c0 + kWlChunk * g;
#pragma unroll
        for (int n = 0; n < kWlRows * WPR / kLanes; ++n) {
            const int idx = lane + n * kLanes;
            const int row = idx / WPR, i = idx % WPR;
            float v[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) v[e] = s_o[((kWlChunk * g + 4 * i + e) & (kWlRing - 1)) * kWlPitchO + row];
            if (band0 + row < a.out_h)
                store_group<Tr>(yb + static_cast<long long>(band0 + row) * a.y_pitch, ocol + 4 * i, c1, y_align, v);
        }
    };

    float2 Z[M][Q];                             // Z[m][s]: the pair in PE s of output row 4a+m (live at the parity of T)
#pragma unroll
    for (int m = 0; m < M; ++m)
#pragma unroll
        for (int s = 0; s < Q; ++s) Z[m][s] = make_float2(0.f, 0.f);

    const int n_out = c1 - c0;
    stage_load(c0);
    stage_store();
    __syncwarp();
#pragma unroll 1
    for (int j = 0; (j - kGroupDelay) * kWlChunk < n_out; ++j) {
        stage_load(c0 + (j + 1) * kWlChunk);
        // small filters: all macro-steps of the chunk unrolled (immediate shared-memory offsets, the reads
        // of later columns can be issued early); larger ones: two macro-steps per iteration (code size)
        constexpr int kUnrollU = P * Q <= 25 ? kWlChunk / 2 : 1;
#pragma unroll kUnrollU
        for (int u = 0; u < kWlChunk / 2; ++u) {
#pragma unroll
            for (int v = 0; v < 2; ++v) {
                const int c = 2 * u + v;                // column inside the chunk; the macro-step has the parity of v
                float xk[4 * KG];                       // broadcast: the K inputs of this image column
#pragma unroll
                for (int g = 0; g < KG; ++g) {
                    const float4 t = *reinterpret_cast<const float4 *>(s_x + c * kWlPitch + 4 * (lane + g));
                    xk[4 * g] = t.x; xk[4 * g + 1] = t.y; xk[4 * g + 2] = t.z; xk[4 * g + 3] = t.w;
                }
                if (v == Q % 2) {
                    // the pairs that left PE Q-1 one step ago: output columns T-Q and T-Q+1 of the four rows
                    float e0[M], e1[M];
#pragma unroll
                    for (int m = 0; m < M; ++m) {
                        float z = Z[m][Q - 1].y;
#pragma unroll
                        for (int p = 0; p < P; ++p) z = fmaf(xk[m + p], taps.w[p * Q + Q - 1], z);
                        e0[m] = Z[m][Q - 1].x;
                        e1[m] = z;
                    }
                    const int o = j * kWlChunk + c - Q;     // may be negative during the fill: those slots are rewritten
                    *reinterpret_cast<float4 *>(s_o + (o & (kWlRing - 1)) * kWlPitchO + 4 * lane) =
                        make_float4(e0[0], e0[1], e0[2], e0[3]);
                    *reinterpret_cast<float4 *>(s_o + ((o + 1) & (kWlRing - 1)) * kWlPitchO + 4 * lane) =
                        make_float4(e1[0], e1[1], e1[2], e1[3]);
                }
                // The pairs move one PE up (register renaming), then the P sub-steps of macro-step T in every PE.  The
                // order in which the independent chains (rows x PEs) are written matters to the compiler's schedule.
                // Tall filters: sub-step outermost, the tap pair of (p, s) serves the four rows and all chains
                // advance side by side (15x15: 74 against 61 % of the FP32 peak); smaller ones: chain by chain (9x9: 64 against
                // 52 % the other way round).
#pragma unroll
                for (int m = 0; m < M; ++m)
#pragma unroll
                    for (int s = Q - 1; s >= 1; --s)
                        if (s % 2 == v) Z[m][s] = Z[m][s - 1];
                if constexpr (WlShape<P, Q>::kOrder == 1) {
#pragma unroll
                    for (int p = 0; p < P; ++p) {
#pragma unroll
                        for (int s = Q - 1; s >= 1; --s) {
                            if (s % 2 != v) continue;
                            const float2 w2 = tp.w[p * (Q + 1) + s];
#pragma unroll
                            for (int m = 0; m < M; ++m)
                                Z[m][s] = __ffma2_rn(make_float2(xk[m + p], xk[m + p]), w2, Z[m][s]);
                        }
                    }
                } else {
#pragma unroll
                    for (int m = 0; m < M; ++m)
#pragma unroll
                        for (int s = Q - 1; s >= 1; --s) {
                            if (s % 2 != v) continue;
                            float2 z = Z[m][s];
#pragma unroll
                            for (int p = 0; p < P; ++p)
                                z = __ffma2_rn(make_float2(xk[m + p], xk[m + p]), tp.w[p * (Q + 1) + s], z);
                            Z[m][s] = z;
                        }
                }
#pragma unroll
                for (int m = 0; m < M; ++m) {
                    if (v == 0) {
                        float z = xk[m] * taps.w[0];    // PE 0 opens a pair: filter column 0, first sum only
#pragma unroll
                        for (int p = 1; p < P; ++p) z = fmaf(xk[m + p], taps.w[p * Q], z);
                        Z[m][0] = make_float2(z, 0.f);
                    }
                }
            }
        }
        __syncwarp();                                   // chunk j consumed, its emissions are in the ring
        stage_store();
        if (j >= kGroupDelay) flush(j - kGroupDelay);
        __syncwarp();                                   // chunk j+1 staged
    }
}

template <int P, int Q>
cudaError_t launch_conv2d_ws_lane(const Conv2DArgs &a, const Taps2D &taps, cudaStream_t s)
{
    TapsColPairs tp{};
    for (int p = 0; p < P; ++p)
        for (int t = 0; t <= Q; ++t)
            tp.w[p * (Q + 1) + t] = make_float2(t < Q ? taps.w[p * Q + t] : 0.f, t >= 1 ? taps.w[p * Q + t - 1] : 0.f);
    // CTAs = width segments x bands of 128 rows x images; a segment costs Q-1 extra macro-steps, so segments are
    // as long as the grid allows (about 32 one-warp CTAs per SM in total), at least 128 columns, multiples of 8
    const long long bands = (a.out_h + kWlRows - 1) / kWlRows;
    const long long want = 148LL * 32;
    long long segs = (want + bands * a.batch - 1) / (bands * a.batch);
    const long long max_segs = (a.out_w + 127) / 128;
    if (segs > max_segs) segs = max_segs;
    if (segs < 1) segs = 1;
    int seg_w = static_cast<int>((a.out_w + segs - 1) / segs);
    constexpr int kChunk = WlShape<P, Q>::kChunk;
    seg_w = (seg_w + kChunk - 1) / kChunk * kChunk;
    dim3 grid((a.out_w + seg_w - 1) / seg_w, static_cast<unsigned>(bands), a.batch);
    if (grid.y > 65535) return cudaErrorInvalidConfiguration;
    launch_kernel(conv2d_ws_lane_kernel<P, Q>, grid, kLanes, s, a, taps, tp, seg_w);
    return cudaGetLastError();
}

// fp32 dispatch.  Small filters (at most 8 columns, P*Q up to about 32): the all-register form with the arrays side by
// side along the rows (conv2d_f32_ws_reg.cuh).  Larger filters: the arrays stacked over the rows with transposed
// staging (this file) when the problem gives its one-warp blocks a few warps per SM, else the segment form with
// the hand-over in shared memory (conv2d_f32_ws_seg.cuh), which reads its inputs straight from memory and so suits
// problems that live in L2 (1920 x 1080, 5 x 5: 13 us against 20 us for four-lane arrays with register taps).
// None of the three pads with zero taps: an input outside an output's window never enters its sum.
template <int P, int Q>
struct FastPath2D<F32Traits, SYSCONV_WS, P, Q> {
    static bool launch(const Conv2DArgs &a, const Taps2D &taps, cudaStream_t s, cudaError_t *err)
    {
        if constexpr (WsrShape<P, Q>::kFits) {
            *err = launch_conv2d_ws_reg<P, Q>(a, taps, s);
            return true;
        } else {
            const long long bands = (a.out_h + kWlRows - 1) / kWlRows;
            const long long max_segs = (a.out_w + 127) / 128;
            if (bands * max_segs * a.batch < 148LL * 4) *err = launch_conv2d_ws_seg<P, Q>(a, taps, s);
            else *err = launch_conv2d_ws_lane<P, Q>(a, taps, s);
            return true;
        }
    }
};

}  // namespace sysconv
