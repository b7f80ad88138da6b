// 2-D convolution (Eq. 3) as folded linear systolic arrays on a warp, for fp32
// and for uint8 x int8 -> int32 data (same kernels, different arithmetic traits).
//
// The PE dimension is the image column c (contiguous in memory); the image row r
// is the outer loop that the paper leaves untouched (Section 5).  Lane l of a
// warp holds the R2 = 4 consecutive PEs 4l .. 4l+3 of a 128-PE array; a warp
// marches down a band of rows, loading each input row exactly once into
// registers with one 128-bit (fp32) or 32-bit (uint8) load per lane.
//
//  * OS / FBS ("multiple FBS 1-D convolutions"): PE c keeps the partial sums of
//    column c for the P output rows the current input row contributes to.  The
//    Q time steps of one FBS pass forward the input row one PE down per step;
//    every forwarded value feeds all P filter rows.  The last PE takes its
//    inputs from memory (the halo registers), as in the paper's URE
//    X(c,q) = select(q==0 || c==C-1, x(c+q), X(c+1,q-1)), so all 128 PEs of a
//    strip produce valid outputs.  Rotating the P partial rows costs nothing:
//    the first step of every pass writes Z[p] = Z[p-1] + X*w.
//  * IS / SBM (two projections, PE = c+q, t = p + P*q): PE s keeps the P-deep
//    column x(s, r..r+P-1); per output row, for each q the P taps of filter
//    column q are applied in place, then the partial sums move one PE up.  The
//    first Q-1 PEs of a strip hold incomplete sums (lane 0 has no left
//    neighbour), so a strip yields 128-(Q-1)-drain outputs.
//  * WS (derived from BSM, PE = q, t = P*(c+q)+p): PE q keeps the P taps of
//    filter column q; the inputs of image column T are broadcast to the array at
//    macro-step T; partial sums move one PE up per macro-step; the last PE emits
//    one output per macro-step.  A warp holds eight 4-lane arrays working on
//    eight groups of M output rows.
#pragma once

#include <type_traits>

#include "sysconv_common.cuh"

namespace sysconv {

constexpr int R2 = 4;                       // PEs (columns) per lane
constexpr int kStrip2 = kLanes * R2;        // 128 PEs per warp
constexpr int kWarps2 = 4;
constexpr int kThreads2 = kWarps2 * kLanes;

struct F32Traits {
    using in_t = float;
    using acc_t = float;
    using out_t = float;
    using taps_t = Taps2D;
    static __device__ __forceinline__ acc_t mad(acc_t x, acc_t w, acc_t z) { return fmaf(x, w, z); }
    static __device__ __forceinline__ acc_t mul(acc_t x, acc_t w) { return x * w; }
    // four consecutive elements starting at p (16-byte aligned)
    static __device__ __forceinline__ void load4v(const in_t *p, acc_t (&v)[4])
    {
        const float4 t = __ldg(reinterpret_cast<const float4 *>(p));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    static __device__ __forceinline__ acc_t load1(const in_t *p) { return __ldg(p); }
};

struct U8Traits {
    using in_t = uint8_t;
    using acc_t = int;
    using out_t = int;
    using taps_t = Taps2DInt;
    static __device__ __forceinline__ acc_t mad(acc_t x, acc_t w, acc_t z) { return x * w + z; }
    static __device__ __forceinline__ acc_t mul(acc_t x, acc_t w) { return x * w; }
    static __device__ __forceinline__ void load4v(const in_t *p, acc_t (&v)[4])
    {
        const unsigned t = __ldg(reinterpret_cast<const unsigned *>(p));
        v[0] = t & 0xff; v[1] = (t >> 8) & 0xff; v[2] = (t >> 16) & 0xff; v[3] = t >> 24;
    }
    static __device__ __forceinline__ acc_t load1(const in_t *p) { return __ldg(p); }
};

// Four consecutive inputs of one row starting at column col; zeros beyond the row's end.
template <typename Tr>
__device__ __forceinline__ void load_group(const typename Tr::in_t *__restrict__ rowp, int col, int width,
                                           bool vec_ok, typename Tr::acc_t (&v)[4])
{
    if (vec_ok && col + 3 < width) {
        Tr::load4v(rowp + col, v);
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = (col + j < width) ? Tr::load1(rowp + col + j) : typename Tr::acc_t(0);
    }
}

// Four consecutive outputs of one row starting at column col; align = 4, 2 or 1 elements.
template <typename Tr>
__device__ __forceinline__ void store_group(typename Tr::out_t *__restrict__ rowp, int col, int col_end,
                                            int align, const typename Tr::acc_t (&v)[4])
{
    using out_t = typename Tr::out_t;
    if (col + 3 < col_end && align == 4) {
        using vec4 = typename std::conditional<std::is_same<out_t, float>::value, float4, int4>::type;
        vec4 t;
        t.x = v[0]; t.y = v[1]; t.z = v[2]; t.w = v[3];
        *reinterpret_cast<vec4 *>(rowp + col) = t;
    } else if (col + 3 < col_end && align == 2) {
        using vec2 = typename std::conditional<std::is_same<out_t, float>::value, float2, int2>::type;
        vec2 t0, t1;
        t0.x = v[0]; t0.y = v[1]; t1.x = v[2]; t1.y = v[3];
        *reinterpret_cast<vec2 *>(rowp + col) = t0;
        *reinterpret_cast<vec2 *>(rowp + col + 2) = t1;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (col + j < col_end) rowp[col + j] = v[j];
    }
}

// alignment class (in elements) shared by every row start of an array
template <typename T>
__device__ __forceinline__ int row_alignment(const T *base, long long pitch, long long bstride, int batch)
{
    const unsigned long long addr = reinterpret_cast<unsigned long long>(base);
    const long long bs = batch > 1 ? bstride : 0;
    if ((addr % (4 * sizeof(T))) == 0 && pitch % 4 == 0 && bs % 4 == 0) return 4;
    if ((addr % (2 * sizeof(T))) == 0 && pitch % 2 == 0 && bs % 2 == 0) return 2;
    return 1;
}

// ---------------------------------------------------------------------------
// OS / FBS
// ---------------------------------------------------------------------------
template <typename Tr, int P, int Q>
__global__ void __launch_bounds__(kThreads2)
conv2d_os_kernel(const Conv2DArgs a, const __grid_constant__ typename Tr::taps_t taps, const int band_h)
{
    using in_t = typename Tr::in_t;
    using acc_t = typename Tr::acc_t;
    using out_t = typename Tr::out_t;
    constexpr bool kHalo = Q > 1;
    constexpr bool kHaloChain = Q - 1 > R2;     // the halo spans more than one lane
    const int lane = threadIdx.x & (kLanes - 1);
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;
    const int c0 = strip * kStrip2;
    if (c0 >= a.out_w) return;
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const in_t *xb = static_cast<const in_t *>(a.x) + blockIdx.z * a.x_bstride;
    out_t *yb = static_cast<out_t *>(a.y) + blockIdx.z * a.y_bstride;
    const bool x_vec = row_alignment(static_cast<const in_t *>(a.x), a.x_pitch, a.x_bstride, a.batch) == 4;
    const int y_align = row_alignment(static_cast<const out_t *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const int col = c0 + R2 * lane;             // first column of this lane's PEs
    const int hcol = c0 + kStrip2 + R2 * lane;  // halo columns (lanes 0 .. ceil((Q-1)/4)-1)
    const bool has_halo = kHalo && R2 * lane < Q - 1;

    acc_t Z[P][R2];
#pragma unroll
    for (int p = 0; p < P; ++p)
#pragma unroll
        for (int j = 0; j < R2; ++j) Z[p][j] = 0;

    acc_t nX[R2], nH[R2];
#pragma unroll
    for (int j = 0; j < R2; ++j) nH[j] = 0;
    {
        const in_t *rowp = xb + static_cast<long long>(r0) * a.x_pitch;
        load_group<Tr>(rowp, col, a.width, x_vec, nX);
        if (has_halo) load_group<Tr>(rowp, hcol, a.width, x_vec, nH);
    }
    const int i_end = r1 + P - 1;               // input rows r0 .. i_end-1
#pragma unroll 1
    for (int i = r0; i < i_end; ++i) {
        acc_t X[R2], H[R2];
#pragma unroll
        for (int j = 0; j < R2; ++j) { X[j] = nX[j]; H[j] = nH[j]; }
        if (i + 1 < i_end) {                    // prefetch the next input row
            const in_t *rowp = xb + static_cast<long long>(i + 1) * a.x_pitch;
            load_group<Tr>(rowp, col, a.width, x_vec, nX);
            if (has_halo) load_group<Tr>(rowp, hcol, a.width, x_vec, nH);
        }
        // input row i contributes to output rows i-p through filter row p: one
        // FBS pass of Q steps, every forwarded input feeding all P rows
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            if (q == 0) {
                // partial rows rotate: the sums of output row i-p were in Z[p-1]
#pragma unroll
                for (int p = P - 1; p > 0; --p)
#pragma unroll
                    for (int j = 0; j < R2; ++j) Z[p][j] = Tr::mad(X[j], taps.w[p * Q], Z[p - 1][j]);
#pragma unroll
                for (int j = 0; j < R2; ++j) Z[0][j] = Tr::mul(X[j], taps.w[0]);
            } else {
#pragma unroll
                for (int p = 0; p < P; ++p)
#pragma unroll
                    for (int j = 0; j < R2; ++j) Z[p][j] = Tr::mad(X[j], taps.w[p * Q + q], Z[p][j]);
            }
            if (q < Q - 1) {
                // forward the inputs one PE down; the strip's last PE takes the halo from lane 0
                const acc_t send = (lane == 0) ? H[0] : X[0];
                const acc_t in0 = __shfl_sync(kFullMask, send, (lane + 1) & (kLanes - 1));
                X[0] = X[1]; X[1] = X[2]; X[2] = X[3]; X[3] = in0;
                acc_t in1 = 0;
                if (kHaloChain) in1 = __shfl_down_sync(kFullMask, H[0], 1);
                H[0] = H[1]; H[1] = H[2]; H[2] = H[3]; H[3] = in1;
            }
        }
        const int r = i - (P - 1);              // output row completed by this input row
        if (r >= r0) store_group<Tr>(yb + static_cast<long long>(r) * a.y_pitch, col, a.out_w, y_align, Z[P - 1]);
    }
}

// ---------------------------------------------------------------------------
// IS / SBM
// ---------------------------------------------------------------------------
template <int Q>
struct IsGeom {
    static constexpr int kDrain = (4 - ((Q - 1) & 3)) & 3;
    static constexpr int kShift = Q - 1 + kDrain;         // multiple of 4
    static constexpr int kValid = kStrip2 - kShift;       // outputs per strip
};

template <typename Tr, int P, int Q>
__global__ void __launch_bounds__(kThreads2)
conv2d_is_kernel(const Conv2DArgs a, const __grid_constant__ typename Tr::taps_t taps, const int band_h)
{
    using in_t = typename Tr::in_t;
    using acc_t = typename Tr::acc_t;
    using out_t = typename Tr::out_t;
    constexpr int kShift = IsGeom<Q>::kShift;
    constexpr int kValid = IsGeom<Q>::kValid;
    const int lane = threadIdx.x & (kLanes - 1);
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;
    const int c0 = strip * kValid;              // first output column = first input column (PE 0)
    if (c0 >= a.out_w) return;
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const in_t *xb = static_cast<const in_t *>(a.x) + blockIdx.z * a.x_bstride;
    out_t *yb = static_cast<out_t *>(a.y) + blockIdx.z * a.y_bstride;
    const bool x_vec = row_alignment(static_cast<const in_t *>(a.x), a.x_pitch, a.x_bstride, a.batch) == 4;
    const int y_align = row_alignment(static_cast<const out_t *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const int col = c0 + R2 * lane;             // columns held by this lane's PEs
    const int ocol = col - kShift;              // output columns its PEs end up holding
    const int oend = min(a.out_w, c0 + kValid);

    // PE registers: the P-deep input column of each PE, rows r .. r+P-1
    acc_t X[P][R2];
#pragma unroll
    for (int p = 0; p < P - 1; ++p)
        load_group<Tr>(xb + static_cast<long long>(min(r0 + p, a.height - 1)) * a.x_pitch, col, a.width, x_vec, X[p + 1]);
    acc_t nX[R2];
    load_group<Tr>(xb + static_cast<long long>(r0 + P - 1) * a.x_pitch, col, a.width, x_vec, nX);

#pragma unroll 1
    for (int r = r0; r < r1; ++r) {
        // the window of input rows slides down by one
#pragma unroll
        for (int p = 0; p < P - 1; ++p)
#pragma unroll
            for (int j = 0; j < R2; ++j) X[p][j] = X[p + 1][j];
#pragma unroll
        for (int j = 0; j < R2; ++j) X[P - 1][j] = nX[j];
        if (r + 1 < r1)
            load_group<Tr>(xb + static_cast<long long>(r + P) * a.x_pitch, col, a.width, x_vec, nX);

        acc_t Z[R2];
#pragma unroll
        for (int q = 0; q < Q + IsGeom<Q>::kDrain; ++q) {
            if (q > 0) {
                // partial sums move one PE up (lane 0 has no left neighbour: invalid PEs)
                const acc_t up = __shfl_up_sync(kFullMask, Z[R2 - 1], 1);
                Z[3] = Z[2]; Z[2] = Z[1]; Z[1] = Z[0]; Z[0] = up;
            }
            if (q < Q) {
#pragma unroll
                for (int p = 0; p < P; ++p)     // t = p + P*q
#pragma unroll
                    for (int j = 0; j < R2; ++j)
                        Z[j] = (q == 0 && p == 0) ? Tr::mul(X[0][j], taps.w[0])
                                                  : Tr::mad(X[p][j], taps.w[p * Q + q], Z[j]);
            }
        }
        if (ocol >= c0) store_group<Tr>(yb + static_cast<long long>(r) * a.y_pitch, ocol, oend, y_align, Z);
    }
}

// ---------------------------------------------------------------------------
// WS (derived from BSM)
// ---------------------------------------------------------------------------
constexpr int kWsM2 = 4;                        // output rows per array pass
constexpr int kWsRows2 = kWsArrays * kWsM2;     // 32 output rows per warp pass
constexpr int kWsCols2 = 128;                   // output columns streamed per warp pass

template <typename Tr, int P, int Q>
__global__ void __launch_bounds__(kThreads2)
conv2d_ws_kernel(const Conv2DArgs a, const __grid_constant__ typename Tr::taps_t taps)
{
    using in_t = typename Tr::in_t;
    using acc_t = typename Tr::acc_t;
    using out_t = typename Tr::out_t;
    constexpr int RW = (Q + kWsLanes - 1) / kWsLanes;    // PEs per lane
    constexpr int QP = RW * kWsLanes;                    // PEs per array (taps beyond Q are zero)
    constexpr int K = kWsM2 + P - 1;                     // input rows feeding M output rows
    const int lane = threadIdx.x & (kLanes - 1);
    const int m_lane = lane & (kWsLanes - 1);
    const int arr = lane / kWsLanes;
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;
    const int c0 = strip * kWsCols2;
    if (c0 >= a.out_w) return;
    const int r0 = blockIdx.y * kWsRows2 + arr * kWsM2;  // first output row of this array
    const in_t *xb = static_cast<const in_t *>(a.x) + blockIdx.z * a.x_bstride;
    out_t *yb = static_cast<out_t *>(a.y) + blockIdx.z * a.y_bstride;

    // PE registers: the P taps of each PE's filter column
    acc_t W[RW][P];
#pragma unroll
    for (int i = 0; i < RW; ++i) {
        const int s = m_lane * RW + i;
#pragma unroll
        for (int p = 0; p < P; ++p) W[i][p] = s < Q ? taps.w[p * Q + s] : acc_t(0);
    }
    acc_t Z[kWsM2][RW];
#pragma unroll
    for (int m = 0; m < kWsM2; ++m)
#pragma unroll
        for (int i = 0; i < RW; ++i) Z[m][i] = 0;

    const in_t *rowp[K];
#pragma unroll
    for (int k = 0; k < K; ++k) rowp[k] = xb + static_cast<long long>(min(r0 + k, a.height - 1)) * a.x_pitch;

    const int c_end = min(c0 + kWsCols2, a.out_w);       // output columns [c0, c_end)
    const int steps = (c_end - c0) + QP - 1;             // macro-steps T = 0 .. steps-1
#pragma unroll 1
    for (int T = 0; T < steps; ++T) {
        const int xc = min(c0 + T, a.width - 1);         // image column broadcast at this macro-step
        acc_t xk[K];
#pragma unroll
        for (int k = 0; k < K; ++k) xk[k] = Tr::load1(rowp[k] + xc);
#pragma unroll
        for (int m = 0; m < kWsM2; ++m) {
            acc_t up = __shfl_up_sync(kFullMask, Z[m][RW - 1], 1, kWsLanes);
            if (m_lane == 0) up = 0;                     // PE 0 starts a new sum
            // sub-step p = 0 also moves the sums one PE up
#pragma unroll
            for (int i = RW - 1; i > 0; --i) Z[m][i] = Tr::mad(xk[m], W[i][0], Z[m][i - 1]);
            Z[m][0] = Tr::mad(xk[m], W[0][0], up);
#pragma unroll
            for (int p = 1; p < P; ++p)
#pragma unroll
                for (int i = 0; i < RW; ++i) Z[m][i] = Tr::mad(xk[m + p], W[i][p], Z[m][i]);
        }
        const int oc = c0 + T - (QP - 1);                // column completed by the array's last PE
        if (m_lane == kWsLanes - 1 && oc >= c0) {
#pragma unroll
            for (int m = 0; m < kWsM2; ++m)
                if (r0 + m < a.out_h) yb[static_cast<long long>(r0 + m) * a.y_pitch + oc] = Z[m][RW - 1];
        }
    }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
inline int pick_band_height(int out_h, long long strips_times_batch, int p)
{
    const long long target = 148LL * 16;                 // warps wanted in flight
    long long bands = (target + strips_times_batch - 1) / strips_times_batch;
    if (bands < 1) bands = 1;
    long long h = (out_h + bands - 1) / bands;
    const long long lo = p > 8 ? p : 8;
    if (h < lo) h = lo;
    if (h > 256) h = 256;
    return static_cast<int>(h);
}

template <typename Tr, int DESIGN, int P, int Q>
cudaError_t launch_conv2d_pq(const Conv2DArgs &a, const typename Tr::taps_t &taps, cudaStream_t s)
{
    if (a.batch > 65535) return cudaErrorInvalidConfiguration;
    if (DESIGN == SYSCONV_WS) {
        const int strips = (a.out_w + kWsCols2 - 1) / kWsCols2;
        dim3 grid((strips + kWarps2 - 1) / kWarps2, (a.out_h + kWsRows2 - 1) / kWsRows2, a.batch);
        if (grid.y > 65535) return cudaErrorInvalidConfiguration;
        conv2d_ws_kernel<Tr, P, Q><<<grid, kThreads2, 0, s>>>(a, taps);
    } else {
        const int per_strip = DESIGN == SYSCONV_OS ? kStrip2 : IsGeom<Q>::kValid;
        const int strips = (a.out_w + per_strip - 1) / per_strip;
        const int band_h = pick_band_height(a.out_h, static_cast<long long>(strips) * a.batch, P);
        dim3 grid((strips + kWarps2 - 1) / kWarps2, (a.out_h + band_h - 1) / band_h, a.batch);
        if (grid.y > 65535) return cudaErrorInvalidConfiguration;
        if (DESIGN == SYSCONV_OS) conv2d_os_kernel<Tr, P, Q><<<grid, kThreads2, 0, s>>>(a, taps, band_h);
        else conv2d_is_kernel<Tr, P, Q><<<grid, kThreads2, 0, s>>>(a, taps, band_h);
    }
    return cudaGetLastError();
}

template <typename Tr, int DESIGN, int P>
cudaError_t launch_conv2d_p(const Conv2DArgs &a, const typename Tr::taps_t &taps, int q, cudaStream_t s)
{
    switch (q) {
#define SYSCONV_CASE(QQ) case QQ: return launch_conv2d_pq<Tr, DESIGN, P, QQ>(a, taps, s);
        SYSCONV_CASE(1) SYSCONV_CASE(2) SYSCONV_CASE(3) SYSCONV_CASE(4) SYSCONV_CASE(5)
        SYSCONV_CASE(6) SYSCONV_CASE(7) SYSCONV_CASE(8) SYSCONV_CASE(9) SYSCONV_CASE(10)
        SYSCONV_CASE(11) SYSCONV_CASE(12) SYSCONV_CASE(13) SYSCONV_CASE(14) SYSCONV_CASE(15)
#undef SYSCONV_CASE
        default: return kNoInstantiation;
    }
}

// Dispatch over the filter heights P_LO .. P_HI compiled into the calling translation unit.
template <typename Tr, int DESIGN, int P_LO, int P_HI, typename W>
cudaError_t launch_conv2d_range(const Conv2DArgs &a, const W *w, int q, int p, cudaStream_t s, int *launches)
{
    typename Tr::taps_t taps;
    for (int k = 0; k < kMaxP2 * kMaxQ2; ++k) taps.w[k] = k < p * q ? w[k] : 0;
    cudaError_t err = kNoInstantiation;
    switch (p) {
#define SYSCONV_CASE(PP) \
    case PP: if (PP >= P_LO && PP <= P_HI) err = launch_conv2d_p<Tr, DESIGN, (PP >= P_LO && PP <= P_HI) ? PP : P_LO>(a, taps, q, s); break;
        SYSCONV_CASE(1) SYSCONV_CASE(2) SYSCONV_CASE(3) SYSCONV_CASE(4) SYSCONV_CASE(5)
        SYSCONV_CASE(6) SYSCONV_CASE(7) SYSCONV_CASE(8) SYSCONV_CASE(9) SYSCONV_CASE(10)
        SYSCONV_CASE(11) SYSCONV_CASE(12) SYSCONV_CASE(13) SYSCONV_CASE(14) SYSCONV_CASE(15)
#undef SYSCONV_CASE
        default: break;
    }
    if (err == cudaSuccess && launches) *launches += 1;
    return err;
}

}  // namespace sysconv
