// 2-D uint8 x int8 -> int32 convolution, weight-stationary design on the packed integer datapath.
//
// The stationary operand of a PE is a WORD of four taps: word-PE g keeps, for every filter row p, the taps
// w(p, 4g .. 4g+3) (uniform operands, as in the fp32 weight-stationary kernels).  At macro-step T the four pixels
// x(r+p, T .. T+3) are broadcast to the array; word-PE g adds their dot product with its taps (one dp4a.u32.s32 per
// filter row, exact int32) to the sum of output c = T - 4g, which it took over from word-PE g-1 four steps earlier
// and hands to word-PE g+1 four steps later.  An array has ceil(Q/4) <= 4 word-PEs and is folded into one lane
// (PE-to-PE transfer = register renaming); the 32 arrays of a warp lie side by side along the rows: array a (lane
// a) streams the 16 pixels its own 128-bit load fetches, so the loads of a warp are contiguous and nothing is
// staged.  The broadcast words that straddle two aligned words are built with byte permutes (PRMT), the three that
// reach into the next segment with one shuffle per row.
//
// Arrays neither fill nor drain: each runs exactly the 16 macro-steps of its segment.  The sums of the last
// 4*(G-1) outputs of a segment are completed by the next array, which starts from empty PEs and hands its share
// back by shuffle (integer addition is exact in any order).  Lane 31 is only such a successor: a warp yields
// 31 * 16 output columns.  Four output rows (two for filters of up to four rows) are computed per pass; every input
// row of the pass is fetched once, its 16 shifted words are built once and used by up to four output rows.
#pragma once

#include "conv2d_u8_dp4a.cuh"

namespace sysconv {

constexpr int kU8WsM = 4;                       // output rows per pass (two for filters of up to four rows)
constexpr int kU8WsWarps = 4;
constexpr int kU8WsSeg = 16;                    // pixels per array and pass (one 128-bit load)
constexpr int kU8WsOut = (kLanes - 1) * kU8WsSeg;
constexpr int kU8WsPitch = kU8WsSeg + 4;        // ints per lane block of the output staging row

template <int P, int Q, int MROWS = kU8WsM>
__global__ void __launch_bounds__(kU8WsWarps *kLanes)
conv2d_u8_ws_dp4a_kernel(const Conv2DArgs a, const __grid_constant__ TapsPacked taps, const int band_h)
{
    dependent_launch_enter();
    constexpr int M = MROWS, K = M + P - 1, G = (Q + 3) / 4, SEG = kU8WsSeg, TAIL = 4 * (G - 1);
    const int lane = threadIdx.x & (kLanes - 1);
    const int slice = blockIdx.x * kU8WsWarps + threadIdx.x / kLanes;    // (a block of fewer warps is the only one of its row)
    const int c0 = slice * kU8WsOut;                    // first output column of the slice
    if (c0 >= a.out_w) return;
    const int col0 = c0 + lane * SEG;                   // first pixel of this lane's segment
    const int c_end = min(a.out_w, c0 + kU8WsOut);
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const uint8_t *xb = static_cast<const uint8_t *>(a.x) + blockIdx.z * a.x_bstride;
    int *yb = static_cast<int *>(a.y) + blockIdx.z * a.y_bstride;
    const int y_align = row_alignment(static_cast<const int *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const bool whole = col0 + SEG <= a.width;           // the segment lies inside the image: one 128-bit load per row
    __shared__ __align__(16) int s_out[kU8WsWarps][kLanes * kU8WsPitch];
    int *so = s_out[threadIdx.x / kLanes];

#pragma unroll 1
    for (int rg = r0; rg < r1; rg += M) {
        // acc[m][TAIL + c]: sum of output column c of the segment, row rg+m; c < 0 = the previous segment's last outputs
        int acc[M][SEG + TAIL];
#pragma unroll
        for (int m = 0; m < M; ++m)
#pragma unroll
            for (int c = 0; c < SEG + TAIL; ++c) acc[m][c] = 0;
        // One input row: fetched once, its 16 shifted words built once, used by every output row it reaches.  FULL:
        // the row reaches all four output rows (kk in [M-1, P-1]), through the filter rows kk-m.
        auto load_row = [&](int kk, unsigned (&W)[5]) {
            const uint8_t *rowp = xb + static_cast<long long>(min(rg + kk, a.height - 1)) * a.x_pitch + col0;
            if (whole) {
                const uint4 t = __ldg(reinterpret_cast<const uint4 *>(rowp));
                W[0] = t.x; W[1] = t.y; W[2] = t.z; W[3] = t.w;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    unsigned v = 0;
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (col0 + 4 * j + e < a.width) v |= static_cast<unsigned>(rowp[4 * j + e]) << (8 * e);
                    W[j] = v;
                }
            }
        };
        auto use_row = [&](auto full_tag, int kk, unsigned (&W)[5]) {
            constexpr bool FULL = decltype(full_tag)::value;
            W[4] = __shfl_down_sync(kFullMask, W[0], 1);        // the first pixels of the next segment
            int wt[M][G];                                       // the taps through which this row reaches the four output rows
#pragma unroll
            for (int m = 0; m < M; ++m)
#pragma unroll
                for (int g = 0; g < G; ++g) wt[m][g] = (FULL || (kk - m >= 0 && kk - m < P)) ? taps.w[(kk - m) * 4 + g] : 0;
#pragma unroll
            for (int t = 0; t < SEG; ++t) {
                // the broadcast input of macro-step t: the four pixels starting at pixel t of the segment
                const int j = t / 4, sh = t % 4;
                const unsigned xw = sh == 0 ? W[j] : __byte_perm(W[j], W[j + 1], sh == 1 ? 0x4321 : sh == 2 ? 0x5432 : 0x6543);
#pragma unroll
                for (int m = 0; m < M; ++m) {
                    if (!FULL && (kk - m < 0 || kk - m >= P)) continue;     // (kk is a constant where FULL is false)
#pragma unroll
                    for (int g = 0; g < G; ++g)                 // word-PE g works on output column t - 4g
                        acc[m][TAIL + t - 4 * g] = dp4a_u8s8(xw, wt[m][g], acc[m][TAIL + t - 4 * g]);
                }
            }
        };
        // Short filters: every input row of a pass unrolled.  From five rows on the rows that reach all four output
        // rows run in a loop (measured on 2 x 2048 x 4096: 7x13 90 -> 67 us, 5x13 71 -> 54, 7x7 44 -> 40; narrow
        // filters of 5 to 7 rows are the exception: 7x3 36 -> 43 us, so they stay unrolled; from eight rows on the
        // unrolled code also takes minutes to compile)
        constexpr bool kRolled = P >= 8 || (P >= 5 && Q > 4);
        if constexpr (!kRolled) {
#pragma unroll
            for (int kk = 0; kk < K; ++kk) {
                unsigned W[5];
                load_row(kk, W);
                use_row(std::false_type{}, kk, W);
            }
        } else {
            // the rows that reach all four output rows run in a loop, the others unrolled; the next row is fetched
            // before the current one is used
#pragma unroll
            for (int kk = 0; kk < M - 1; ++kk) {
                unsigned W[5];
                load_row(kk, W);
                use_row(std::false_type{}, kk, W);
            }
            unsigned Wn[5];
            load_row(M - 1, Wn);
#pragma unroll 1
            for (int kk = M - 1; kk < P; ++kk) {
                unsigned W[5] = {Wn[0], Wn[1], Wn[2], Wn[3], 0u};
                load_row(kk + 1, Wn);
                use_row(std::true_type{}, kk, W);
            }
#pragma unroll
            for (int kk = P; kk < K; ++kk) {
                unsigned W[5] = {Wn[0], Wn[1], Wn[2], Wn[3], 0u};
                if (kk + 1 < K) load_row(kk + 1, Wn);
                use_row(std::false_type{}, kk, W);
            }
        }
        // the successor's share of this segment's last TAIL outputs comes back by shuffle
#pragma unroll
        for (int m = 0; m < M; ++m)
#pragma unroll
            for (int j = 0; j < TAIL; ++j) acc[m][TAIL + SEG - TAIL + j] += __shfl_down_sync(kFullMask, acc[m][j], 1);
        // A lane's 16 outputs of a row are 64 contiguous bytes; stored from the lanes directly, every 128-bit store
        // of a warp would touch 32 sectors half filled.  They pass through a small shared-memory row instead (lane
        // blocks 80 bytes apart: conflict-free both ways) and leave as contiguous 128-bit words.
#pragma unroll
        for (int m = 0; m < M; ++m) {
            if (rg + m >= r1) break;
#pragma unroll
            for (int i = 0; i < SEG / 4; ++i)
                *reinterpret_cast<int4 *>(so + lane * kU8WsPitch + 4 * i) =
                    make_int4(acc[m][TAIL + 4 * i], acc[m][TAIL + 4 * i + 1], acc[m][TAIL + 4 * i + 2], acc[m][TAIL + 4 * i + 3]);
            __syncwarp();
            int *orow = yb + static_cast<long long>(rg + m) * a.y_pitch;
#pragma unroll
            for (int i = 0; i < SEG / 4; ++i) {
                const int u = lane + kLanes * i;                // 128-bit word of the slice's row
                if (u < (kLanes - 1) * (SEG / 4)) {             // lane 31's words belong to the next slice
                    const int4 t = *reinterpret_cast<const int4 *>(so + (u / (SEG / 4)) * kU8WsPitch + 4 * (u % (SEG / 4)));
                    const int v4[4] = {t.x, t.y, t.z, t.w};
                    store_group<U8Traits>(orow, c0 + 4 * u, c_end, y_align, v4);
                }
            }
            __syncwarp();
        }
    }
}

// true if every row of every image starts 16-byte aligned (128-bit loads of 16 pixels)
inline bool u8_ws_dp4a_eligible(const Conv2DArgs &a)
{
    const unsigned long long xa = reinterpret_cast<unsigned long long>(a.x);
    return (xa & 15ull) == 0 && (a.x_pitch & 15) == 0 && (a.batch == 1 || (a.x_bstride & 15) == 0);
}

template <int P, int Q, int MROWS>
cudaError_t launch_conv2d_u8_ws_dp4a_m(const Conv2DArgs &a, const Taps2DInt &t, cudaStream_t s)
{
    TapsPacked pk;
    for (int p = 0; p < kMaxP2; ++p)
        for (int g = 0; g < 4; ++g) {
            unsigned v = 0;
            for (int e = 0; e < 4; ++e) {
                const int q = 4 * g + e;
                const int w = (p < P && q < Q) ? t.w[p * Q + q] : 0;
                v |= (static_cast<unsigned>(w) & 0xffu) << (8 * e);
            }
            pk.w[p * 4 + g] = static_cast<int>(v);
        }
    const int slices = (a.out_w + kU8WsOut - 1) / kU8WsOut;
    const int wpb = block_warps(slices, kU8WsWarps);
    const long long per_band = static_cast<long long>((slices + wpb - 1) / wpb) * a.batch;
    static const long long slots4 = 148LL * resident_blocks_per_sm(conv2d_u8_ws_dp4a_kernel<P, Q, MROWS>, kU8WsWarps * kLanes);
    const long long slots = slots4 * kU8WsWarps / wpb;      // smaller blocks: as many more of them are resident
    long long band_h;
    if (small_problem(a.out_h, per_band, MROWS, slots)) {
        band_h = pick_band_height_small(a.out_h, per_band, P, MROWS, 64, slots);
    } else {
        const long long bands = (148LL * 16 + per_band - 1) / per_band;
        band_h = (a.out_h + bands - 1) / bands;
        if (band_h > 64) band_h = 64;
    }
    band_h = (band_h + MROWS - 1) / MROWS * MROWS;
    if ((a.out_h + band_h - 1) / band_h > 65535) band_h = ((a.out_h + 65534) / 65535 + MROWS - 1) / MROWS * MROWS;
    dim3 grid((slices + wpb - 1) / wpb, static_cast<unsigned>((a.out_h + band_h - 1) / band_h), a.batch);
    launch_kernel(conv2d_u8_ws_dp4a_kernel<P, Q, MROWS>, grid, wpb * kLanes, s, a, pk, static_cast<int>(band_h));
    return cudaGetLastError();
}

template <int P, int Q>
cudaError_t launch_conv2d_u8_ws_dp4a(const Conv2DArgs &a, const Taps2DInt &t, cudaStream_t s)
{
    // up to four filter rows: two output rows per pass (half the accumulators, more blocks per SM; 3840 x 2160, 3x3:
    // 15.9 -> 14.1 us); taller filters: four, so that an input row serves up to four output rows
    if constexpr (P <= 4) return launch_conv2d_u8_ws_dp4a_m<P, Q, 2>(a, t, s);
    else return launch_conv2d_u8_ws_dp4a_m<P, Q, kU8WsM>(a, t, s);
}

// uint8 rows that start 16-byte aligned run on the packed weight-stationary kernel
template <int P, int Q>
struct FastPath2D<U8Traits, SYSCONV_WS, P, Q> {
    static bool launch(const Conv2DArgs &a, const Taps2DInt &taps, cudaStream_t s, cudaError_t *err)
    {
        if (!u8_ws_dp4a_eligible(a)) return false;
        *err = launch_conv2d_u8_ws_dp4a<P, Q>(a, taps, s);
        return true;
    }
};

}  // namespace sysconv
