// Stride-2 2-D convolution, y(r, c) = sum_p sum_q x(2r+p, 2c+q) w(p, q), fp32, filters up to 7 x 7:
// rows of the stride-2 FBS array of Table 2 (output-stationary) and the matching input-stationary array,
// folded onto a warp like their stride-1 forms.  A strip is 256 input columns (eight per lane); its first
// PE has no left neighbour and its last no right neighbour, so a strip yields 120 outputs and consecutive
// strips overlap by 16 input columns.
#pragma once

#include "conv2d_kernels.cuh"

namespace sysconv {

constexpr int kMaxPQS2 = 7;                    // largest filter side of the stride-2 kernels
constexpr int kStripInS2 = kLanes * 8;         // 256 input columns per strip
constexpr int kStripOutS2 = 120;               // outputs per strip (2*119 + 14 < 256)

// eight consecutive inputs of one row (zeros beyond the image)
__device__ __forceinline__ void load8_f32(const float *rowp, int col, int width, bool vec_ok, float *v)
{
    load_group<F32Traits>(rowp, col, width, vec_ok, v);
    load_group<F32Traits>(rowp, col + 4, width, vec_ok, v + 4);
}

// ---------------------------------------------------------------------------
// OS / FBS, stride 2.  PE c keeps the partial sums of output column c for the ceil(P/2) output rows the
// current PAIR of input rows (2m, 2m+1) contributes to: row 2m feeds output row m-k through filter row 2k,
// row 2m+1 through filter row 2k+1.  Along a row the inputs are forwarded as in the 1-D stride-2 array:
// X(c, q) = X(c+1, q-2), i.e. the even and the odd input columns form two chains that move one PE down
// every second step.  A lane holds four PEs.
// ---------------------------------------------------------------------------
template <int P, int Q>
__global__ void __launch_bounds__(kThreads2)
conv2d_os_s2_kernel(const Conv2DArgs a, const __grid_constant__ Taps2D taps, const int band_h)
{
    dependent_launch_enter();
    constexpr int KP = (P + 1) / 2;             // partial output rows alive
    const int lane = threadIdx.x & (kLanes - 1);
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;
    const int c0 = strip * kStripOutS2;         // first output column of the strip
    if (c0 >= a.out_w) return;
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const float *xb = static_cast<const float *>(a.x) + blockIdx.z * a.x_bstride;
    float *yb = static_cast<float *>(a.y) + blockIdx.z * a.y_bstride;
    const bool x_vec = row_alignment(static_cast<const float *>(a.x), a.x_pitch, a.x_bstride, a.batch) == 4;
    const int y_align = row_alignment(static_cast<const float *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const int icol = 2 * c0 + 8 * lane;         // first input column of this lane's PEs
    const int ocol = c0 + 4 * lane;             // its four output columns
    const int oend = min(a.out_w, c0 + kStripOutS2);
    const int m_end = r1 + KP - 1;              // row pairs r0 .. m_end-1

    auto fetch = [&](int m, float (&v)[2][8]) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int row = 2 * m + h;
            if (m < m_end && row < a.height) {
                load8_f32(xb + static_cast<long long>(row) * a.x_pitch, icol, a.width, x_vec, v[h]);
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) v[h][j] = 0.f;
            }
        }
    };

    float Z[KP][4];
#pragma unroll
    for (int k = 0; k < KP; ++k)
#pragma unroll
        for (int j = 0; j < 4; ++j) Z[k][j] = 0.f;

    float nV[2][8];
    fetch(r0, nV);
#pragma unroll 1
    for (int m = r0; m < m_end; ++m) {
        float V[2][8];
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int j = 0; j < 8; ++j) V[h][j] = nV[h][j];
        fetch(m + 1, nV);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float E[4], O[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                E[j] = V[h][2 * j];
                O[j] = V[h][2 * j + 1];
            }
#pragma unroll
            for (int q = 0; q < Q; ++q) {
                float(&S)[4] = (q % 2 == 0) ? E : O;
#pragma unroll
                for (int k = KP - 1; k >= 0; --k) {
                    const int p = 2 * k + h;
                    if (p >= P) continue;
                    const float wt = taps.w[p * Q + q];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        // the pair's first step rotates the partial rows: the sums of output row m-k were in Z[k-1]
                        if (h == 0 && q == 0) Z[k][j] = k > 0 ? fmaf(S[j], wt, Z[k - 1][j]) : S[j] * wt;
                        else Z[k][j] = fmaf(S[j], wt, Z[k][j]);
                    }
                }
                if (q + 2 < Q) {
                    const float in = __shfl_down_sync(kFullMask, S[0], 1);   // lane 31 keeps its own: invalid PEs
                    S[0] = S[1]; S[1] = S[2]; S[2] = S[3]; S[3] = in;
                }
            }
        }
        const int r = m - (KP - 1);             // output row completed by this pair
        if (r >= r0) store_group<F32Traits>(yb + static_cast<long long>(r) * a.y_pitch, ocol, oend, y_align, Z[KP - 1]);
    }
}

// ---------------------------------------------------------------------------
// IS / SBM, stride 2.  PE s keeps the P-deep input column x(2r .. 2r+P-1, s); the window slides down two
// rows per output row.  The sum of output column c sits in PE 2c+q at step q and moves one PE up per step,
// so only the PEs with the parity of q hold live sums: a step is P multiply-adds on every second PE.
// After the Q steps the sums move on without arithmetic until their offset is a multiple of eight PEs, so
// that a lane's four outputs leave as one aligned 128-bit word.  A lane holds eight PEs.
// ---------------------------------------------------------------------------
template <int Q>
struct IsGeomS2 {
    static constexpr int kShift = ((Q - 1 + 7) / 8) * 8;          // PEs a sum has moved when it is stored
    static constexpr int kValid = (kStripInS2 - kShift) / 2;      // outputs per strip (124 or 128)
};

template <int P, int Q>
__global__ void __launch_bounds__(kThreads2)
conv2d_is_s2_kernel(const Conv2DArgs a, const __grid_constant__ Taps2D taps, const int band_h)
{
    dependent_launch_enter();
    constexpr int kShift = IsGeomS2<Q>::kShift;
    constexpr int kValid = IsGeomS2<Q>::kValid;
    const int lane = threadIdx.x & (kLanes - 1);
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;
    const int c0 = strip * kValid;              // first output column of the strip; PE 0 holds input column 2*c0
    if (c0 >= a.out_w) return;
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const float *xb = static_cast<const float *>(a.x) + blockIdx.z * a.x_bstride;
    float *yb = static_cast<float *>(a.y) + blockIdx.z * a.y_bstride;
    const bool x_vec = row_alignment(static_cast<const float *>(a.x), a.x_pitch, a.x_bstride, a.batch) == 4;
    const int y_align = row_alignment(static_cast<const float *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const int icol = 2 * c0 + 8 * lane;         // input columns held by this lane's PEs
    const int ocol = c0 + (8 * lane - kShift) / 2;      // output columns its PEs end up holding
    const int oend = min(a.out_w, c0 + kValid);

    auto load_row = [&](int row, float *v) {
        if (row < a.height) {
            load8_f32(xb + static_cast<long long>(row) * a.x_pitch, icol, a.width, x_vec, v);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = 0.f;
        }
    };

    // PE registers: input rows 2r .. 2r+P-1; NEW of them are new for every output row
    constexpr int NEW = P < 2 ? P : 2;
    float X[P][8];
#pragma unroll
    for (int p = 0; p + NEW < P; ++p) load_row(2 * r0 + p, X[p + 2]);
    float nX[NEW][8];
#pragma unroll
    for (int h = 0; h < NEW; ++h) load_row(2 * r0 + P - NEW + h, nX[h]);

#pragma unroll 1
    for (int r = r0; r < r1; ++r) {
        // the window of input rows slides down by two
#pragma unroll
        for (int p = 0; p + NEW < P; ++p)
#pragma unroll
            for (int j = 0; j < 8; ++j) X[p][j] = X[p + 2][j];
#pragma unroll
        for (int h = 0; h < NEW; ++h)
#pragma unroll
            for (int j = 0; j < 8; ++j) X[P - NEW + h][j] = nX[h][j];
        if (r + 1 < r1) {
#pragma unroll
            for (int h = 0; h < NEW; ++h) load_row(2 * (r + 1) + P - NEW + h, nX[h]);
        }

        float Z[8];
#pragma unroll
        for (int t = 0; t < kShift + 1; ++t) {
            // live sums: PEs with the parity of t
            float up = 0.f;
            if (t > 0 && t % 2 == 0) up = __shfl_up_sync(kFullMask, Z[7], 1);   // lane 0: its own, invalid PEs
#pragma unroll
            for (int j = 7; j >= 0; --j) {
                if (j % 2 != t % 2) continue;
                float z = (t == 0) ? 0.f : (j == 0 ? up : Z[j - 1]);
                if (t < Q) {
#pragma unroll
                    for (int p = 0; p < P; ++p) z = (t == 0 && p == 0) ? X[0][j] * taps.w[0] : fmaf(X[p][j], taps.w[p * Q + t], z);
                }
                Z[j] = z;
            }
        }
        // kShift is even: the live sums are in the even PEs
        if (ocol >= c0) {
            const float out[4] = {Z[0], Z[2], Z[4], Z[6]};
            store_group<F32Traits>(yb + static_cast<long long>(r) * a.y_pitch, ocol, oend, y_align, out);
        }
    }
}

template <int DESIGN, int P, int Q>
cudaError_t launch_conv2d_s2_pq(const Conv2DArgs &a, const Taps2D &taps, cudaStream_t s)
{
    if (a.batch > 65535) return cudaErrorInvalidConfiguration;
    const int per_strip = DESIGN == SYSCONV_OS ? kStripOutS2 : IsGeomS2<Q>::kValid;
    const int strips = (a.out_w + per_strip - 1) / per_strip;
    const int band_h = pick_band_height(a.out_h, static_cast<long long>(strips) * a.batch, P, Q);
    const int wpb = block_warps(strips, kWarps2);       // narrow images: blocks of as many warps as there are strips
    dim3 grid((strips + wpb - 1) / wpb, (a.out_h + band_h - 1) / band_h, a.batch);
    if (DESIGN == SYSCONV_OS) launch_kernel(conv2d_os_s2_kernel<P, Q>, grid, wpb * kLanes, s, a, taps, band_h);
    else launch_kernel(conv2d_is_s2_kernel<P, Q>, grid, wpb * kLanes, s, a, taps, band_h);
    return cudaGetLastError();
}

template <int DESIGN, int P>
cudaError_t launch_conv2d_s2_p(const Conv2DArgs &a, const Taps2D &taps, int q, cudaStream_t s)
{
    switch (q) {
        case 1: return launch_conv2d_s2_pq<DESIGN, P, 1>(a, taps, s);
        case 2: return launch_conv2d_s2_pq<DESIGN, P, 2>(a, taps, s);
        case 3: return launch_conv2d_s2_pq<DESIGN, P, 3>(a, taps, s);
        case 4: return launch_conv2d_s2_pq<DESIGN, P, 4>(a, taps, s);
        case 5: return launch_conv2d_s2_pq<DESIGN, P, 5>(a, taps, s);
        case 6: return launch_conv2d_s2_pq<DESIGN, P, 6>(a, taps, s);
        case 7: return launch_conv2d_s2_pq<DESIGN, P, 7>(a, taps, s);
        default: return kNoInstantiation;
    }
}

template <int DESIGN>
cudaError_t launch_conv2d_s2(const Conv2DArgs &a, const float *w, int q, int p, cudaStream_t s, int *launches)
{
    Taps2D taps;
    for (int i = 0; i < kMaxP2 * kMaxQ2; ++i) taps.w[i] = i < p * q ? w[i] : 0.f;
    cudaError_t err = kNoInstantiation;
    switch (p) {
        case 1: err = launch_conv2d_s2_p<DESIGN, 1>(a, taps, q, s); break;
        case 2: err = launch_conv2d_s2_p<DESIGN, 2>(a, taps, q, s); break;
        case 3: err = launch_conv2d_s2_p<DESIGN, 3>(a, taps, q, s); break;
        case 4: err = launch_conv2d_s2_p<DESIGN, 4>(a, taps, q, s); break;
        case 5: err = launch_conv2d_s2_p<DESIGN, 5>(a, taps, q, s); break;
        case 6: err = launch_conv2d_s2_p<DESIGN, 6>(a, taps, q, s); break;
        case 7: err = launch_conv2d_s2_p<DESIGN, 7>(a, taps, q, s); break;
        default: break;
    }
    if (err == cudaSuccess && launches) *launches += 1;
    return err;
}

}  // namespace sysconv
