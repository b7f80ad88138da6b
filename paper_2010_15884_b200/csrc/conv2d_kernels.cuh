// 2-D convolution (Eq. 3) as folded linear systolic arrays on a warp, for fp32
// and for uint8 x int8 -> int32 data (same kernels, different arithmetic traits).
//
// The PE dimension is the image column c (contiguous in memory); the image row r
// is the outer loop that the paper leaves untouched (Section 5).  Lane l of a
// warp holds R consecutive PEs (R = 4 or 8) of a 32R-PE array; a warp
// marches down a band of rows, loading each input row exactly once into
// registers with 128-bit (fp32) or 32-bit (uint8) loads (R = 4 or 8 PEs per lane).
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
    static __device__ __forceinline__ void load4v(const in_t *p, acc_t *v)
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
    static __device__ __forceinline__ void load4v(const in_t *p, acc_t *v)
    {
        const unsigned t = __ldg(reinterpret_cast<const unsigned *>(p));
        v[0] = t & 0xff; v[1] = (t >> 8) & 0xff; v[2] = (t >> 16) & 0xff; v[3] = t >> 24;
    }
    static __device__ __forceinline__ acc_t load1(const in_t *p) { return __ldg(p); }
};

// Four consecutive inputs of one row starting at column col; zeros beyond the row's end.
template <typename Tr>
__device__ __forceinline__ void load_group(const typename Tr::in_t *__restrict__ rowp, int col, int width,
                                           bool vec_ok, typename Tr::acc_t *v)
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
                                            int align, const typename Tr::acc_t *v)
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
template <typename Tr, int P, int Q, int R, int MIN_CTAS, int PF>
__global__ void __launch_bounds__(kThreads2, MIN_CTAS)
conv2d_os_kernel(const Conv2DArgs a, const __grid_constant__ typename Tr::taps_t taps, const int band_h)
{
    dependent_launch_enter();
    using in_t = typename Tr::in_t;
    using acc_t = typename Tr::acc_t;
    using out_t = typename Tr::out_t;
    static_assert(R == 4 || R == 8, "R = PEs per lane");
    static_assert(PF == 1 || PF == 2 || PF == 4, "PF = input rows in flight ahead of the one being processed");
    constexpr int kStrip = kLanes * R;          // PEs (= output columns) per strip
    constexpr bool kHalo = Q > 1;
    constexpr bool kHaloChain = Q - 1 > 4;      // the halo spans more than one lane
    const int lane = threadIdx.x & (kLanes - 1);
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;    // (a block of fewer warps is the only one of its row)
    const int c0 = strip * kStrip;
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const in_t *xb = static_cast<const in_t *>(a.x) + blockIdx.z * a.x_bstride;
    out_t *yb = static_cast<out_t *>(a.y) + blockIdx.z * a.y_bstride;
    if (c0 >= a.out_w) return;
    const bool x_vec = row_alignment(static_cast<const in_t *>(a.x), a.x_pitch, a.x_bstride, a.batch) == 4;
    const int y_align = row_alignment(static_cast<const out_t *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const int col = c0 + R * lane;              // first column of this lane's PEs
    const int hcol = c0 + kStrip + 4 * lane;    // halo columns (lanes 0 .. ceil((Q-1)/4)-1)
    const bool has_halo = kHalo && 4 * lane < Q - 1;
    const int i_end = r1 + P - 1;               // input rows r0 .. i_end-1

    acc_t Z[P][R];
#pragma unroll
    for (int p = 0; p < P; ++p)
#pragma unroll
        for (int j = 0; j < R; ++j) Z[p][j] = 0;

    // rows in flight: buffer f holds input row (i + 1 + f) while row i is processed
    acc_t nX[PF][R], nH[PF][4];
#pragma unroll
    for (int f = 0; f < PF; ++f)
#pragma unroll
        for (int j = 0; j < 4; ++j) nH[f][j] = 0;
    auto fetch = [&](int row, acc_t *dx, acc_t *dh) {
        if (row < i_end) {
            const in_t *rowp = xb + static_cast<long long>(row) * a.x_pitch;
#pragma unroll
            for (int g = 0; g < R / 4; ++g) load_group<Tr>(rowp, col + 4 * g, a.width, x_vec, dx + 4 * g);
            if (has_halo) load_group<Tr>(rowp, hcol, a.width, x_vec, dh);
        }
    };
    // process input row i, whose data sit in buffer f; refill that buffer with row i + PF
    auto process = [&](int i, int f) {
        acc_t X[R], H[4];
#pragma unroll
        for (int j = 0; j < R; ++j) X[j] = nX[f][j];
#pragma unroll
        for (int j = 0; j < 4; ++j) H[j] = nH[f][j];
        fetch(i + PF, nX[f], nH[f]);
        // input row i contributes to output rows i-p through filter row p: one
        // FBS pass of Q steps, every forwarded input feeding all P rows
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            if (q == 0) {
                // partial rows rotate: the sums of output row i-p were in Z[p-1]
#pragma unroll
                for (int p = P - 1; p > 0; --p)
#pragma unroll
                    for (int j = 0; j < R; ++j) Z[p][j] = Tr::mad(X[j], taps.w[p * Q], Z[p - 1][j]);
#pragma unroll
                for (int j = 0; j < R; ++j) Z[0][j] = Tr::mul(X[j], taps.w[0]);
            } else {
#pragma unroll
                for (int p = 0; p < P; ++p)
#pragma unroll
                    for (int j = 0; j < R; ++j) Z[p][j] = Tr::mad(X[j], taps.w[p * Q + q], Z[p][j]);
            }
            if (q < Q - 1) {
                // forward the inputs one PE down; the strip's last PE takes the halo from lane 0
                const acc_t send = (lane == 0) ? H[0] : X[0];
                const acc_t in0 = __shfl_sync(kFullMask, send, (lane + 1) & (kLanes - 1));
#pragma unroll
                for (int j = 0; j < R - 1; ++j) X[j] = X[j + 1];
                X[R - 1] = in0;
                acc_t in1 = 0;
                if (kHaloChain) in1 = __shfl_down_sync(kFullMask, H[0], 1);
                H[0] = H[1]; H[1] = H[2]; H[2] = H[3]; H[3] = in1;
            }
        }
        const int r = i - (P - 1);              // output row completed by this input row
        if (r >= r0) {
            out_t *orow = yb + static_cast<long long>(r) * a.y_pitch;
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

// ---------------------------------------------------------------------------
// OS / FBS, fp32, row-paired form for filters with six or more rows.
//
// Same dataflow as conv2d_os_kernel, two input rows per iteration.  The partial sums of two consecutive
// output rows share a 64-bit register pair and are updated by ONE packed fp32x2 FMA (fma.rn.f32x2, new on
// sm_100): the multiplicand is (x, x), the multiplier a pair of taps of two consecutive filter rows, which
// comes straight from the kernel parameters as a uniform-register pair.  Each of the two input rows feeds
// pair m with its own tap pair, so a step costs (P+1) packed FMAs per PE instead of 2P scalar ones; the
// scalar kernel is issue-bound (81 % of its instructions are FMAs at 89 % issue-slot use), this form is
// FMA-pipe-bound.  Both rows' inputs are forwarded exactly as before (one shuffle per row and step).
// With P odd the P+1 slots fill the pairs exactly; with P even one slot of the last pair stays zero.
// Slots without a tap for one of the two rows: scalar FMAs on the other half for P <= 11 (exact), a zero tap
// for P >= 12 (measured faster there), where a NON-FINITE input can therefore also turn the outputs one row
// above and one row below its window rows into NaN; finite inputs are unaffected.
// ---------------------------------------------------------------------------
// Slots and slot pairs of the row-paired kernel: P + 1 partial rows are alive while two input rows are
// processed; pair m holds the slots 2m and 2m+1.
template <int P>
struct F2R {
    static constexpr int S = P + 1, SP = (S + 1) / 2;
};
// Tap pairs [m][q], m < 8: a = (w[2m][q], w[2m+1][q]) for the later input row, b = (w[2m-1][q], w[2m][q]) for the
// earlier one; taps outside 0..P-1 are zero.
struct TapsRowPairs {
    float2 a[8 * kMaxQ2];
    float2 b[8 * kMaxQ2];
};
template <int P, int Q, int R, int MIN_CTAS, bool EXACT_HALVES>
__global__ void __launch_bounds__(kThreads2, MIN_CTAS)
conv2d_os_rowpair_kernel(const Conv2DArgs a, const __grid_constant__ TapsRowPairs taps, const int band_h)
{
    dependent_launch_enter();
    using Tr = F32Traits;
    constexpr int SP = F2R<P>::SP;
    constexpr bool kHalo = Q > 1;
    constexpr bool kHaloChain = Q - 1 > 4;
    constexpr int kStrip = kLanes * R;
    const int lane = threadIdx.x & (kLanes - 1);
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;    // (a block of fewer warps is the only one of its row)
    const int c0 = strip * kStrip;
    if (c0 >= a.out_w) return;
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const float *xb = static_cast<const float *>(a.x) + blockIdx.z * a.x_bstride;
    float *yb = static_cast<float *>(a.y) + blockIdx.z * a.y_bstride;
    const bool x_vec = row_alignment(static_cast<const float *>(a.x), a.x_pitch, a.x_bstride, a.batch) == 4;
    const int y_align = row_alignment(static_cast<const float *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const int col = c0 + R * lane;
    const int hcol = c0 + kStrip + 4 * lane;
    const bool has_halo = kHalo && 4 * lane < Q - 1;
    const int i_end = r1 + P - 1;

    float2 Z[SP][R];
#pragma unroll
    for (int m = 0; m < SP; ++m)
#pragma unroll
        for (int j = 0; j < R; ++j) Z[m][j] = make_float2(0.f, 0.f);
    float nX[2][R], nH[2][4];
#pragma unroll
    for (int t = 0; t < 2; ++t)
#pragma unroll
        for (int j = 0; j < 4; ++j) nH[t][j] = 0;
    auto fetch = [&](int i) {
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const float *rowp = xb + static_cast<long long>(min(i + t, a.height - 1)) * a.x_pitch;
#pragma unroll
            for (int g = 0; g < R / 4; ++g) load_group<Tr>(rowp, col + 4 * g, a.width, x_vec, &nX[t][4 * g]);
            if (has_halo) load_group<Tr>(rowp, hcol, a.width, x_vec, nH[t]);
        }
    };
    fetch(r0);
#pragma unroll 1
    for (int i = r0; i < i_end; i += 2) {
        float X[2][R], H[2][4];
#pragma unroll
        for (int t = 0; t < 2; ++t) {
#pragma unroll
            for (int j = 0; j < R; ++j) X[t][j] = nX[t][j];
#pragma unroll
            for (int j = 0; j < 4; ++j) H[t][j] = nH[t][j];
        }
        if (i + 2 < i_end) fetch(i + 2);
        // slot k holds output row (i+1)-k; pair m = slots (2m, 2m+1); all slots move up by two per iteration
#pragma unroll
        for (int q = 0; q < Q; ++q) {
            float2 D0[R], D1[R];
#pragma unroll
            for (int j = 0; j < R; ++j) { D0[j] = make_float2(X[0][j], X[0][j]); D1[j] = make_float2(X[1][j], X[1][j]); }
#pragma unroll
            for (int m = SP - 1; m >= 0; --m) {
                const float2 wa = taps.a[m * Q + q];      // row i+1 reaches slots 2m, 2m+1 through filter rows 2m, 2m+1
                const float2 wb = taps.b[m * Q + q];      // row i   reaches them through filter rows 2m-1, 2m
                // slots of a pair that have no tap for one of the two rows: either a scalar FMA on the other half
                // (EXACT_HALVES: nothing outside an output's window enters its sum) or a packed FMA with a zero tap
                const bool a_both = !EXACT_HALVES || 2 * m + 1 < P, a_first = 2 * m < P;
                const bool b_both = !EXACT_HALVES || (m > 0 && 2 * m < P), b_second = m == 0, b_first = 2 * m - 1 < P;
#pragma unroll
                for (int j = 0; j < R; ++j) {
                    float2 z = (q == 0) ? (m > 0 ? Z[m - 1][j] : make_float2(0.f, 0.f)) : Z[m][j];
                    if (a_both) z = __ffma2_rn(D1[j], wa, z);
                    else if (a_first) z.x = fmaf(D1[j].x, wa.x, z.x);
                    if (b_both) z = __ffma2_rn(D0[j], wb, z);
                    else if (b_second) z.y = fmaf(D0[j].x, wb.y, z.y);
                    else if (b_first) z.x = fmaf(D0[j].x, wb.x, z.x);
                    Z[m][j] = z;
                }
            }
            if (q < Q - 1) {
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const float send = (lane == 0) ? H[t][0] : X[t][0];
                    const float in0 = __shfl_sync(kFullMask, send, (lane + 1) & (kLanes - 1));
#pragma unroll
                    for (int j = 0; j < R - 1; ++j) X[t][j] = X[t][j + 1];
                    X[t][R - 1] = in0;
                    float in1 = 0;
                    if (kHaloChain) in1 = __shfl_down_sync(kFullMask, H[t][0], 1);
                    H[t][0] = H[t][1]; H[t][1] = H[t][2]; H[t][2] = H[t][3]; H[t][3] = in1;
                }
            }
        }
        // slots P-1 (output row i-P+2) and P (output row i-P+1) are complete
        float lo[R], hi[R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            hi[j] = (P & 1) ? Z[(P - 1) / 2][j].x : Z[(P - 1) / 2][j].y;     // slot P-1
            lo[j] = (P & 1) ? Z[P / 2][j].y : Z[P / 2][j].x;                 // slot P
        }
        const int rl = i - (P - 1), rh = rl + 1;
#pragma unroll
        for (int g = 0; g < R / 4; ++g) {
            if (rl >= r0 && rl < r1) store_group<Tr>(yb + static_cast<long long>(rl) * a.y_pitch, col + 4 * g, a.out_w, y_align, &lo[4 * g]);
            if (rh >= r0 && rh < r1) store_group<Tr>(yb + static_cast<long long>(rh) * a.y_pitch, col + 4 * g, a.out_w, y_align, &hi[4 * g]);
        }
    }
}

// ---------------------------------------------------------------------------
// IS / SBM
// ---------------------------------------------------------------------------
template <int Q, int R>
struct IsGeom {
    static constexpr int kDrain = (4 - ((Q - 1) & 3)) & 3;
    static constexpr int kShift = Q - 1 + kDrain;             // multiple of 4
    static constexpr int kValid = kLanes * R - kShift;        // outputs per strip
};

// The P-deep input column of a PE is a window that slides down one row per output row.  Where the code stays
// small the row loop is unrolled P times and the window is a ring (input row r+p sits in slot (u+p) mod P, u =
// position in the unrolled group), so sliding costs nothing; otherwise the window is shifted by (P-1)*R moves.
// (Measured: the ring pays for the four-PE-per-lane kernels of the small problems -- 1920 x 1080, 5 x 5: 7.9 -> 6.4 us;
// with eight PEs per lane its registers cost residency -- 16 x 4096^2, 3 x 3: 0.39 -> 0.45 ms -- so those shift.)
template <int P, int Q, int R>
constexpr bool kIsRing = P > 1 && R == 4 && P * P * Q * R <= 2048;

template <typename Tr, int P, int Q, int R, int MIN_CTAS>
__global__ void __launch_bounds__(kThreads2, MIN_CTAS)
conv2d_is_kernel(const Conv2DArgs a, const __grid_constant__ typename Tr::taps_t taps, const int band_h)
{
    dependent_launch_enter();
    using in_t = typename Tr::in_t;
    using acc_t = typename Tr::acc_t;
    using out_t = typename Tr::out_t;
    static_assert(R == 4 || R == 8, "R = PEs per lane");
    constexpr int kShift = IsGeom<Q, R>::kShift;
    constexpr int kValid = IsGeom<Q, R>::kValid;
    constexpr bool kRing = kIsRing<P, Q, R>;
    constexpr int U = kRing ? P : 1;            // output rows per trip of the row loop
    const int lane = threadIdx.x & (kLanes - 1);
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;    // (a block of fewer warps is the only one of its row)
    const int c0 = strip * kValid;              // first output column = first input column (PE 0)
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const in_t *xb = static_cast<const in_t *>(a.x) + blockIdx.z * a.x_bstride;
    out_t *yb = static_cast<out_t *>(a.y) + blockIdx.z * a.y_bstride;
    if (c0 >= a.out_w) return;
    const bool x_vec = row_alignment(static_cast<const in_t *>(a.x), a.x_pitch, a.x_bstride, a.batch) == 4;
    const int y_align = row_alignment(static_cast<const out_t *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const int col = c0 + R * lane;              // columns held by this lane's PEs
    const int ocol = col - kShift;              // output columns its PEs end up holding
    const int oend = min(a.out_w, c0 + kValid);

    auto fetch = [&](int row, acc_t *dx) {
        const in_t *rowp = xb + static_cast<long long>(min(row, a.height - 1)) * a.x_pitch;
#pragma unroll
        for (int g = 0; g < R / 4; ++g) load_group<Tr>(rowp, col + 4 * g, a.width, x_vec, dx + 4 * g);
    };

    // PE registers: the P-deep input column of each PE.  Before output row r0 the rows r0 .. r0+P-2 sit in the
    // slots they will have at the first trip (ring: slot p; shifting window: slot p+1, shifted down first).
    acc_t X[P][R];
#pragma unroll
    for (int p = 0; p < P - 1; ++p) fetch(r0 + p, X[kRing ? p : p + 1]);
    acc_t nX[R];
    fetch(r0 + P - 1, nX);

#pragma unroll 1
    for (int rb = r0; rb < r1; rb += U) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int r = rb + u;
            if (r >= r1) break;
            if (!kRing) {
                // the window of input rows slides down by one
#pragma unroll
                for (int p = 0; p < P - 1; ++p)
#pragma unroll
                    for (int j = 0; j < R; ++j) X[p][j] = X[p + 1][j];
            }
#pragma unroll
            for (int j = 0; j < R; ++j) X[(u + P - 1) % P][j] = nX[j];
            if (r + 1 < r1) fetch(r + P, nX);

            acc_t Z[R];
#pragma unroll
            for (int q = 0; q < Q + IsGeom<Q, R>::kDrain; ++q) {
                if (q > 0) {
                    // partial sums move one PE up (lane 0 has no left neighbour: invalid PEs)
                    const acc_t up = __shfl_up_sync(kFullMask, Z[R - 1], 1);
#pragma unroll
                    for (int j = R - 1; j > 0; --j) Z[j] = Z[j - 1];
                    Z[0] = up;
                }
                if (q < Q) {
#pragma unroll
                    for (int p = 0; p < P; ++p)     // t = p + P*q
#pragma unroll
                        for (int j = 0; j < R; ++j)
                            Z[j] = (q == 0 && p == 0) ? Tr::mul(X[u % P][j], taps.w[0])
                                                      : Tr::mad(X[(u + p) % P][j], taps.w[p * Q + q], Z[j]);
                }
            }
            out_t *orow = yb + static_cast<long long>(r) * a.y_pitch;
#pragma unroll
            for (int g = 0; g < R / 4; ++g)
                if (ocol + 4 * g >= c0) store_group<Tr>(orow, ocol + 4 * g, oend, y_align, &Z[4 * g]);
        }
    }
}

// ---------------------------------------------------------------------------
// WS (derived from BSM): PE q keeps the P taps of filter column q; at macro-step T the P+M-1 inputs of
// image column T that feed the array's M output rows are broadcast to its PEs; every PE adds its P
// products (sub-steps p = 0..P-1) and the partial sums move one PE up; the last PE emits one output per
// row and macro-step.
//
// An array is four lanes (RW = ceil(Q/4) PEs per lane, unused PEs keep zero taps), a warp holds eight
// arrays and a CTA 32, stacked over 32*M = 128 output rows.  The CTA streams a segment of the image
// width through shared memory in chunks of 32 columns, stored TRANSPOSED ([column][row], rows in
// XOR-swizzled groups of four) so that an array reads the inputs of one image column with 128-bit
// same-address (broadcast) loads; arrays never refill inside a segment.  The up to three PEs beyond the filter
// width keep zero taps (guarding them was measured 15-60 % slower), so with fp32 data a NON-FINITE input can
// also turn the up to three outputs to the left of its window columns into NaN; finite inputs are unaffected.
// ---------------------------------------------------------------------------
constexpr int kWsM2 = 4;                        // output rows per array
constexpr int kWsRows2 = kWarps2 * kWsArrays * kWsM2;   // 128 output rows per CTA
constexpr int kWsChunk = 32;                    // image columns per staged chunk
constexpr int kWsPitch = 160;                   // rows per staged column (>= 128 + 14 + 2, multiple of 32)

// word index of (column c of the chunk, row) in a staged chunk
__device__ __forceinline__ int ws_word(int c, int row)
{
    return c * kWsPitch + 4 * ((row >> 2) ^ ((c >> 2) & 7)) + (row & 3);
}

template <typename Tr, int P, int Q>
__global__ void __launch_bounds__(kThreads2)
conv2d_ws_kernel(const Conv2DArgs a, const __grid_constant__ typename Tr::taps_t taps, const int seg_w)
{
    dependent_launch_enter();
    using in_t = typename Tr::in_t;
    using acc_t = typename Tr::acc_t;
    using out_t = typename Tr::out_t;
    constexpr int RW = (Q + kWsLanes - 1) / kWsLanes;    // PEs per lane
    constexpr int QP = RW * kWsLanes;                    // PEs per array (taps beyond Q are zero)
    constexpr int M = kWsM2;
    constexpr int K = M + P - 1;                         // input rows feeding M output rows
    constexpr int KG = (K + 3) / 4;                      // ... in groups of four
    constexpr int kRowsUsed = kWsRows2 + P - 1;          // staged rows that are ever read
    __shared__ __align__(16) acc_t s_x[2][kWsChunk * kWsPitch];

    const int lane = threadIdx.x & (kLanes - 1);
    const int warp = threadIdx.x / kLanes;
    const int m_lane = lane & (kWsLanes - 1);
    const int arr = warp * kWsArrays + lane / kWsLanes;  // array index inside the CTA, 0..31
    const int band0 = blockIdx.y * kWsRows2;             // first output row of the CTA
    const int r0 = band0 + arr * M;                      // first output row of this array
    const int c0 = blockIdx.x * seg_w;                   // first output column of the segment (multiple of 32)
    const int c1 = min(c0 + seg_w, a.out_w);             // one past its last output column
    const in_t *xb = static_cast<const in_t *>(a.x) + blockIdx.z * a.x_bstride;
    out_t *yb = static_cast<out_t *>(a.y) + blockIdx.z * a.y_bstride;
    const bool x_vec = row_alignment(static_cast<const in_t *>(a.x), a.x_pitch, a.x_bstride, a.batch) == 4;
    const int y_align = row_alignment(static_cast<const out_t *>(a.y), a.y_pitch, a.y_bstride, a.batch);

    // PE registers: the P taps of each PE's filter column
    acc_t W[RW][P];
#pragma unroll
    for (int i = 0; i < RW; ++i) {
        const int sidx = m_lane * RW + i;
#pragma unroll
        for (int p = 0; p < P; ++p) W[i][p] = sidx < Q ? taps.w[p * Q + sidx] : acc_t(0);
    }
    acc_t Z[M][RW];
#pragma unroll
    for (int m = 0; m < M; ++m)
#pragma unroll
        for (int i = 0; i < RW; ++i) Z[m][i] = 0;
    acc_t obuf[M][4];                                    // outputs of four macro-steps, one 128-bit word per row
#pragma unroll
    for (int m = 0; m < M; ++m)
#pragma unroll
        for (int v = 0; v < 4; ++v) obuf[m][v] = 0;

    // Staging of image columns [cc, cc+32) x rows [band0, band0 + kRowsUsed): the loads of the next chunk
    // are issued into registers before the current chunk is processed and written (transposed) after it.
    constexpr int kStageVec = (kRowsUsed * (kWsChunk / 4) + kThreads2 - 1) / kThreads2;
    acc_t pf[kStageVec][4];
    auto stage_load = [&](int cc) {
#pragma unroll
        for (int n = 0; n < kStageVec; ++n) {
            const int idx = threadIdx.x + n * kThreads2;
            const int row = idx >> 3, i = idx & 7;
            if (idx < kRowsUsed * (kWsChunk / 4)) {
                const in_t *rowp = xb + static_cast<long long>(min(band0 + row, a.height - 1)) * a.x_pitch;
                load_group<Tr>(rowp, cc + 4 * i, a.width, x_vec, pf[n]);
            }
        }
    };
    auto stage_store = [&](int buf) {
        acc_t *dst = s_x[buf];
#pragma unroll
        for (int n = 0; n < kStageVec; ++n) {
            const int idx = threadIdx.x + n * kThreads2;
            const int row = idx >> 3, i = idx & 7;
            if (idx < kRowsUsed * (kWsChunk / 4)) {
#pragma unroll
                for (int e = 0; e < 4; ++e) dst[ws_word(4 * i + e, row)] = pf[n][e];
            }
        }
    };

    // macro-steps T = 0 .. (c1-c0)+QP-2 produce the segment; up to three more complete the last 128-bit word
    const int steps = (c1 - c0) + QP - 1 + 3;
    const int chunks = (steps + kWsChunk - 1) / kWsChunk;
    stage_load(c0);
    stage_store(0);
    __syncthreads();
    const int row_in_cta = arr * M;                      // first staged row this array reads (multiple of 4)
#pragma unroll 1
    for (int j = 0; j < chunks; ++j) {
        if (j + 1 < chunks) stage_load(c0 + (j + 1) * kWsChunk);
        const acc_t *src = s_x[j & 1];
#pragma unroll 1
        for (int u = 0; u < kWsChunk / 4; ++u) {
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const int c = 4 * u + v;                 // column inside the chunk
                // broadcast: the K inputs of this image column, 128 bits at a time
                acc_t xk[4 * KG];
#pragma unroll
                for (int g = 0; g < KG; ++g) {
                    const int word = c * kWsPitch + 4 * (((row_in_cta >> 2) + g) ^ (u & 7));
                    if (sizeof(acc_t) == 4) {
                        const int4 t = *reinterpret_cast<const int4 *>(src + word);
                        xk[4 * g] = *reinterpret_cast<const acc_t *>(&t.x);
                        xk[4 * g + 1] = *reinterpret_cast<const acc_t *>(&t.y);
                        xk[4 * g + 2] = *reinterpret_cast<const acc_t *>(&t.z);
                        xk[4 * g + 3] = *reinterpret_cast<const acc_t *>(&t.w);
                    }
                }
#pragma unroll
                for (int m = 0; m < M; ++m) {
                    acc_t up = __shfl_up_sync(kFullMask, Z[m][RW - 1], 1, kWsLanes);
                    if (m_lane == 0) up = 0;             // PE 0 starts a new sum
                    // sub-step p = 0 also moves the sums one PE up
#pragma unroll
                    for (int i = RW - 1; i > 0; --i) Z[m][i] = Tr::mad(xk[m], W[i][0], Z[m][i - 1]);
                    Z[m][0] = Tr::mad(xk[m], W[0][0], up);
#pragma unroll
                    for (int p = 1; p < P; ++p)
#pragma unroll
                        for (int i = 0; i < RW; ++i) Z[m][i] = Tr::mad(xk[m + p], W[i][p], Z[m][i]);
                    // the array's last PE now holds output column T-(QP-1); QP is a multiple of 4 and so
                    // is c0, hence that column is congruent to v+1 modulo 4
                    obuf[m][(v + 1) & 3] = Z[m][RW - 1];
                }
                if (v == 2) {
                    // columns oc-3 .. oc are complete (oc = T-(QP-1), oc & 3 == 3)
                    const int oc = c0 + j * kWsChunk + c - (QP - 1);
                    if (m_lane == kWsLanes - 1 && oc >= c0 + 3 && oc - 3 < c1) {
#pragma unroll
                        for (int m = 0; m < M; ++m)
                            if (r0 + m < a.out_h)
                                store_group<Tr>(yb + static_cast<long long>(r0 + m) * a.y_pitch, oc - 3, c1, y_align,
                                                obuf[m]);
                    }
                }
            }
        }
        if (j + 1 < chunks) stage_store((j + 1) & 1);    // buffer (j+1)&1 was last read in iteration j-1
        __syncthreads();                                 // chunk j consumed, chunk j+1 staged
    }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------
// Shape of the OS/IS kernels per filter size (measured on B200, 16 x 4096 x 4096 fp32):
//   small filters are memory-bound: eight PEs per lane, short bands (many CTAs in flight) and two input
//     rows in flight per warp (four measured slower); on small images four PEs per lane instead (twice as many warps);
//   fp32 OS filters with six or more rows use the row-paired kernel (launch_conv2d_os_rowpair) instead;
//   the scalar OS kernel with 6 <= P <= 11 (integer data) takes eight PEs per lane under a 128-register cap;
//   IS beyond the small filters keeps four PEs per lane: P*8 stationary inputs no longer fit.
template <typename Tr, int DESIGN, int P, int Q>
struct Shape2D {
    static constexpr bool kF32 = std::is_same<Tr, F32Traits>::value;
    static constexpr bool kSmall = P * Q <= 25;
    static constexpr int kR = !kF32 ? 4 : kSmall ? 8 : (DESIGN == SYSCONV_OS && P <= 11) ? 8 : 4;
    static constexpr int kMinCtas = (kF32 && DESIGN == SYSCONV_OS && !kSmall && P <= 11) ? 4 : 1;
    static constexpr int kPrefetch = kSmall ? 2 : 1;
    static constexpr bool kAlsoNarrow = kF32 && kSmall;     // a four-PE variant exists for small images
};

inline int pick_band_height(int out_h, long long strips_times_batch, int p, int q)
{
    // enough CTAs to fill the machine a few times over; bands never shorter than 2*P rows (halo rows are
    // recomputed per band) nor longer than 256 (64 for the memory-bound small filters)
    const long long target = 148LL * 16;
    long long bands = (target + strips_times_batch - 1) / strips_times_batch;
    if (bands < 1) bands = 1;
    long long h = (out_h + bands - 1) / bands;
    const long long lo = 2 * p > 8 ? 2 * p : 8;
    const long long hi = p * q <= 25 ? 64 : 256;
    if (h > hi) h = hi;
    if (h < lo) h = lo;
    const long long fit = (out_h + 65534LL) / 65535;       // grid.y limit
    if (h < fit) h = fit;
    return static_cast<int>(h);
}

template <typename Tr, int DESIGN, int P, int Q, int R>
cudaError_t launch_conv2d_osis(const Conv2DArgs &a, const typename Tr::taps_t &taps, cudaStream_t s)
{
    using Sh = Shape2D<Tr, DESIGN, P, Q>;
    const int per_strip = DESIGN == SYSCONV_OS ? kLanes * R : IsGeom<Q, R>::kValid;
    const int strips = (a.out_w + per_strip - 1) / per_strip;
    int band_h = pick_band_height(a.out_h, static_cast<long long>(strips) * a.batch, P, Q);
    const int wpb = block_warps(strips, kWarps2);
    {
        // a problem of a few waves of blocks: short bands, chosen by the number of waves they give
        static const long long slots4 = 148LL * [] {
            if constexpr (DESIGN == SYSCONV_OS)
                return resident_blocks_per_sm(conv2d_os_kernel<Tr, P, Q, R, Sh::kMinCtas, Sh::kPrefetch>, kThreads2);
            else
                return resident_blocks_per_sm(conv2d_is_kernel<Tr, P, Q, R, Sh::kMinCtas>, kThreads2);
        }();
        const long long slots = slots4 * kWarps2 / wpb;      // smaller blocks: as many more of them are resident
        const long long per_band = static_cast<long long>((strips + wpb - 1) / wpb) * a.batch;
        if (small_problem(a.out_h, per_band, 4, slots)) band_h = pick_band_height_small(a.out_h, per_band, P, 4, 64, slots);
    }
    dim3 grid((strips + wpb - 1) / wpb, (a.out_h + band_h - 1) / band_h, a.batch);
    if (grid.y > 65535) return cudaErrorInvalidConfiguration;
    if constexpr (DESIGN == SYSCONV_OS)
        launch_kernel(conv2d_os_kernel<Tr, P, Q, R, Sh::kMinCtas, Sh::kPrefetch>, grid, wpb * kLanes, s, a, taps, band_h);
    else
        launch_kernel(conv2d_is_kernel<Tr, P, Q, R, Sh::kMinCtas>, grid, wpb * kLanes, s, a, taps, band_h);
    return cudaGetLastError();
}

// scalar half-steps where a slot pair has a tap for only one slot: exact for non-finite inputs and measured
// faster up to 11 filter rows (9x9: 72 % vs 68 % of FP32 peak), slower from 12 on (15x15: 69 % vs 79 %)
template <int P>
constexpr bool kRowPairExact = P <= 11;

template <int P, int Q>
cudaError_t launch_conv2d_os_rowpair(const Conv2DArgs &a, const float *w, cudaStream_t s)
{
    constexpr int R = 4, MINB = 4;
    TapsRowPairs t;
    auto tap = [&](int p, int q) { return (p >= 0 && p < P) ? w[p * Q + q] : 0.f; };
    for (int m = 0; m < 8; ++m)
        for (int q = 0; q < Q; ++q) {
            t.a[m * Q + q] = make_float2(tap(2 * m, q), tap(2 * m + 1, q));
            t.b[m * Q + q] = make_float2(tap(2 * m - 1, q), tap(2 * m, q));
        }
    const int strips = (a.out_w + kLanes * R - 1) / (kLanes * R);
    const int band_h = pick_band_height(a.out_h, static_cast<long long>(strips) * a.batch, P, Q);
    const int wpb = block_warps(strips, kWarps2);
    dim3 grid((strips + wpb - 1) / wpb, (a.out_h + band_h - 1) / band_h, a.batch);
    if (grid.y > 65535) return cudaErrorInvalidConfiguration;
    launch_kernel(conv2d_os_rowpair_kernel<P, Q, R, MINB, kRowPairExact<P>>, grid, wpb * kLanes, s, a, t, band_h);
    return cudaGetLastError();
}

// Hook for a faster kernel of a (traits, design) pair defined in another header: returns true and sets
// *err if it launched.  The default does nothing.
template <typename Tr, int DESIGN, int P, int Q>
struct FastPath2D {
    static bool launch(const Conv2DArgs &, const typename Tr::taps_t &, cudaStream_t, cudaError_t *) { return false; }
};

template <typename Tr, int DESIGN, int P, int Q>
cudaError_t launch_conv2d_pq(const Conv2DArgs &a, const typename Tr::taps_t &taps, cudaStream_t s)
{
    if (a.batch > 65535) return cudaErrorInvalidConfiguration;
    {
        cudaError_t err = cudaSuccess;
        if (FastPath2D<Tr, DESIGN, P, Q>::launch(a, taps, s, &err)) return err;
    }
    if constexpr (DESIGN == SYSCONV_WS && !std::is_same<Tr, F32Traits>::value) {
        // (integer data; fp32 has its own weight-stationary kernels behind the hook above)
        // CTAs = width segments x bands of 128 rows x images; segments are multiples of 32 columns and as
        // long as possible (each costs QP-1 fill steps) while still giving a few CTAs per SM
        const long long bands = (a.out_h + kWsRows2 - 1) / kWsRows2;
        const long long want = 148LL * 6;
        long long segs = (want + bands * a.batch - 1) / (bands * a.batch);
        const long long max_segs = (a.out_w + 127) / 128;          // segments of at least 128 columns
        if (segs > max_segs) segs = max_segs;
        if (segs < 1) segs = 1;
        int seg_w = static_cast<int>((a.out_w + segs - 1) / segs);
        seg_w = (seg_w + kWsChunk - 1) / kWsChunk * kWsChunk;
        dim3 grid((a.out_w + seg_w - 1) / seg_w, static_cast<unsigned>(bands), a.batch);
        if (grid.y > 65535) return cudaErrorInvalidConfiguration;
        launch_kernel(conv2d_ws_kernel<Tr, P, Q>, grid, kThreads2, s, a, taps, seg_w);
        return cudaGetLastError();
    }
    if constexpr (DESIGN == SYSCONV_WS) return kNoInstantiation;
    using Sh = Shape2D<Tr, DESIGN, P, Q>;
    if constexpr (std::is_same<Tr, F32Traits>::value && DESIGN == SYSCONV_OS && P >= 6)
        return launch_conv2d_os_rowpair<P, Q>(a, taps.w, s);
    if (Sh::kAlsoNarrow) {
        // small image: with eight PEs per lane there would be fewer than ~8 warps per SM even with the
        // shortest bands, so take four PEs per lane
        const long long strips8 = (a.out_w + 255) / 256;
        const long long warps8 = strips8 * a.batch * ((a.out_h + 7) / 8);
        if (warps8 < 148LL * 8 * 4) return launch_conv2d_osis<Tr, DESIGN, P, Q, 4>(a, taps, s);
        // narrow image: 256-PE strips would stand idle for a quarter or more of what 128-PE strips cover
        // (batches of short signals arrive here as images of a few dozen to a few hundred columns)
        const long long cover8 = strips8 * 256, cover4 = (a.out_w + 127) / 128 * 128LL;
        if (cover4 * 5 <= cover8 * 4) return launch_conv2d_osis<Tr, DESIGN, P, Q, 4>(a, taps, s);
    }
    return launch_conv2d_osis<Tr, DESIGN, P, Q, Sh::kR>(a, taps, s);
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
