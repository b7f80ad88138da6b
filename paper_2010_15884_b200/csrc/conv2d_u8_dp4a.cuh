// 2-D uint8 x int8 -> int32 convolution, output-stationary (FBS) design on the packed integer datapath.
//
// Same dataflow as conv2d_os_kernel: PE c keeps the partial sums of column c for the P output rows the
// current input row contributes to, inputs are forwarded between PEs, taps are broadcast.  Pixels stay
// packed four to a 32-bit word: a lane holds PX/4 pixel words (groups of four consecutive PEs), the
// forwarding between lanes moves whole words (one shuffle per word and tap group), the forwarding inside a
// lane is a byte selection (PRMT builds the words that start 1, 2 and 3 pixels later), and one time step
// applies FOUR taps at once: dp4a.u32.s32 multiplies four unsigned pixels by four signed taps and adds the
// products to the 32-bit sum, exactly (|sum| <= 225*255*128 < 2^31).
// On B200 dp4a and the 32-bit integer multiply-add both issue at 64 lanes per clock per SM (measured), so
// this form has four times the multiply-add rate of the one-tap-per-step integer kernel.
#pragma once

#include "conv2d_kernels.cuh"

namespace sysconv {

struct TapsPacked {
    int w[kMaxP2 * 4];          // w[p * 4 + g]: taps 4g .. 4g+3 of filter row p as four signed bytes (zeros beyond Q)
};

__device__ __forceinline__ int dp4a_u8s8(unsigned pixels, int taps, int acc)
{
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(pixels), "r"(taps), "r"(acc));
    return d;
}

template <int P, int Q, int PX, int PF>
__global__ void __launch_bounds__(kThreads2)
conv2d_u8_os_dp4a_kernel(const Conv2DArgs a, const __grid_constant__ TapsPacked taps, const int band_h)
{
    dependent_launch_enter();
    static_assert(PX % 4 == 0 && PX <= 16, "PX = PEs (pixels) per lane");
    static_assert(PF >= 1 && PF <= 4, "PF = input rows in flight ahead of the one being processed");
    constexpr int NW = PX / 4;                  // pixel words (groups of four PEs) per lane
    constexpr int G = (Q + 3) / 4;              // tap groups (time steps) per filter row
    constexpr int kStrip = kLanes * PX;
    // A strip is NW runs of 32 words; lane l holds word l of every run, so that each load and each 128-bit
    // store of a warp covers one contiguous piece of the row.
    const int lane = threadIdx.x & (kLanes - 1);
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;    // (a block of fewer warps is the only one of its row)
    const int c0 = strip * kStrip;
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const uint8_t *xb = static_cast<const uint8_t *>(a.x) + blockIdx.z * a.x_bstride;
    int *yb = static_cast<int *>(a.y) + blockIdx.z * a.y_bstride;
    if (c0 >= a.out_w) return;
    const int y_align = row_alignment(static_cast<const int *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const int col = c0 + 4 * lane;              // first column of this lane's word in run 0
    const int i_end = r1 + P - 1;

    // Everything that is the same for every row of the band is decided here, so that the row loop carries no
    // comparisons: which of the lane's words are loaded whole, which ragged (the image's last, partial word),
    // which groups of four outputs leave as one 128-bit word and which element by element.
    bool ld_whole[NW + 1], ld_ragged[NW + 1], st_vec[NW], st_part[NW];
#pragma unroll
    for (int k = 0; k <= NW; ++k) {
        const int c = col + 4 * kLanes * k;
        const bool mine = k < NW || lane < G;   // the words that follow the strip are fetched by lanes 0 .. G-1
        ld_whole[k] = mine && c + 4 <= a.width;
        ld_ragged[k] = mine && !ld_whole[k] && c < a.width;
    }
#pragma unroll
    for (int k = 0; k < NW; ++k) {
        const int c = col + 4 * kLanes * k;
        st_vec[k] = y_align == 4 && c + 4 <= a.out_w;
        st_part[k] = !st_vec[k] && c < a.out_w;
    }
    // row pointers advance by one pitch per row: the row to fetch next, the output row to store next
    const uint8_t *xnext = xb + static_cast<long long>(r0) * a.x_pitch + col;
    int *onext = yb + static_cast<long long>(r0) * a.y_pitch + col;
    int next_row = r0;                          // image row xnext points at

    // the lane's NW words of the next input row plus, in lanes 0 .. G-1, the words that follow the strip;
    // rows are 4-byte aligned (checked by the launcher), pixels beyond the image read as zero
    auto fetch = [&](unsigned (&w)[NW + 1]) {
        if (next_row >= i_end) return;
#pragma unroll
        for (int k = 0; k <= NW; ++k) {
            unsigned v = 0;
            if (ld_whole[k]) {
                v = __ldg(reinterpret_cast<const unsigned *>(xnext + 4 * kLanes * k));
            } else if (ld_ragged[k]) {
                const int c = col + 4 * kLanes * k;
#pragma unroll
                for (int e = 0; e < 3; ++e)
                    if (c + e < a.width) v |= static_cast<unsigned>(xnext[4 * kLanes * k + e]) << (8 * e);
            }
            w[k] = v;
        }
        xnext += a.x_pitch;
        ++next_row;
    };

    int Z[P][PX];
#pragma unroll
    for (int p = 0; p < P; ++p)
#pragma unroll
        for (int j = 0; j < PX; ++j) Z[p][j] = 0;

    // rows in flight: buffer f holds input row i + f while row i is processed
    unsigned nW[PF][NW + 1];
#pragma unroll
    for (int f = 0; f < PF; ++f) {
#pragma unroll
        for (int k = 0; k <= NW; ++k) nW[f][k] = 0;
        fetch(nW[f]);
    }
    // process input row i, whose data sit in buffer f; refill that buffer with row i + PF
    auto process = [&](int i, int f) {
        unsigned W[NW + 1];
#pragma unroll
        for (int k = 0; k <= NW; ++k) W[k] = nW[f][k];
        fetch(nW[f]);
#pragma unroll
        for (int k = 0; k < NW; ++k) {
            // inputs forwarded from the next PEs: word e further on sits in lane (l+e) mod 32, in the same run
            // or, past lane 31, in the next one (the sender knows which of its words the reader wants)
            unsigned V[G + 1];
            V[0] = W[k];
#pragma unroll
            for (int e = 1; e <= G; ++e) {
                const unsigned send = lane < e ? W[k + 1] : W[k];
                V[e] = __shfl_sync(kFullMask, send, (lane + e) & (kLanes - 1));
            }
            // S[s][m] = the four pixels starting s pixels after word m
            unsigned S[4][G];
#pragma unroll
            for (int m = 0; m < G; ++m) {
                S[0][m] = V[m];
                S[1][m] = __byte_perm(V[m], V[m + 1], 0x4321);
                S[2][m] = __byte_perm(V[m], V[m + 1], 0x5432);
                S[3][m] = __byte_perm(V[m], V[m + 1], 0x6543);
            }
            // one FBS pass over this group's four PEs: G steps of four taps; the sums of output row i-p
            // were in Z[p-1]
#pragma unroll
            for (int g = 0; g < G; ++g) {
#pragma unroll
                for (int p = P - 1; p >= 0; --p) {
                    const int wt = taps.w[p * 4 + g];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int base = (g == 0) ? (p > 0 ? Z[p - 1][4 * k + j] : 0) : Z[p][4 * k + j];
                        Z[p][4 * k + j] = dp4a_u8s8(S[j][g], wt, base);
                    }
                }
            }
        }
        if (i - (P - 1) >= r0) {
            // output row i-(P-1) is complete
#pragma unroll
            for (int k = 0; k < NW; ++k) {
                if (st_vec[k])
                    *reinterpret_cast<int4 *>(onext + 4 * kLanes * k) =
                        make_int4(Z[P - 1][4 * k], Z[P - 1][4 * k + 1], Z[P - 1][4 * k + 2], Z[P - 1][4 * k + 3]);
                else if (st_part[k])
                    store_group<U8Traits>(onext - col, col + 4 * kLanes * k, a.out_w, y_align, &Z[P - 1][4 * k]);
            }
            onext += a.y_pitch;
        }
    };
#pragma unroll 1
    for (int i = r0; i < i_end; i += PF) {
#pragma unroll
        for (int f = 0; f < PF; ++f)
            if (i + f < i_end) process(i + f, f);
    }
}

// true if the packed kernel can run: every input row must start 4-byte aligned
inline bool u8_dp4a_eligible(const Conv2DArgs &a)
{
    const unsigned long long xa = reinterpret_cast<unsigned long long>(a.x);
    return (xa & 3ull) == 0 && (a.x_pitch & 3) == 0 && (a.batch == 1 || (a.x_bstride & 3) == 0);
}

// Eight PEs per lane and two rows in flight measured best (3x3 and 7x7 on 3840x2160, launches back to back over
// rotating buffers: 3x3 10.8 -> 9.3 us, 7x7 20.0 -> 16.5 us against one row in flight; 4 or 16 PEs slower or equal).
template <int P, int Q>
cudaError_t launch_conv2d_u8_os_dp4a(const Conv2DArgs &a, const Taps2DInt &t, cudaStream_t s)
{
    constexpr int PX = 8, PF = 2;
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
    const int strips = (a.out_w + kLanes * PX - 1) / (kLanes * PX);
    // bands: about 32 warps per SM in total, between 2P (at least 6) and 32 rows each
    const long long warps = static_cast<long long>(strips) * a.batch;
    const long long bands = (148LL * 32 + warps - 1) / warps;
    long long h = (a.out_h + bands - 1) / bands;
    const long long lo = 2 * P > 6 ? 2 * P : 6;
    if (h > 32) h = 32;
    if (h < lo) h = lo;
    const long long fit = (a.out_h + 65534LL) / 65535;     // grid.y limit
    if (h < fit) h = fit;
    int band_h = static_cast<int>(h);
    const int wpb = block_warps(strips, kWarps2);
    {
        // a problem of a few waves of blocks: bands chosen by the number of waves they give
        static const long long slots4 = 148LL * resident_blocks_per_sm(conv2d_u8_os_dp4a_kernel<P, Q, PX, PF>, kThreads2);
        const long long slots = slots4 * kWarps2 / wpb;     // smaller blocks: as many more of them are resident
        const long long per_band = static_cast<long long>((strips + wpb - 1) / wpb) * a.batch;
        if (small_problem(a.out_h, per_band, 4, slots)) band_h = pick_band_height_small(a.out_h, per_band, P, 4, 64, slots);
    }
    dim3 grid((strips + wpb - 1) / wpb, (a.out_h + band_h - 1) / band_h, a.batch);
    if (grid.y > 65535) return cudaErrorInvalidConfiguration;
    launch_kernel(conv2d_u8_os_dp4a_kernel<P, Q, PX, PF>, grid, wpb * kLanes, s, a, pk, band_h);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// IS / SBM on the packed integer datapath, filters up to 7 rows.  A word-PE keeps four consecutive pixels of
// each of the P input rows of the window, together with the three words that start 1, 2 and 3 pixels later
// (built once per input row with PRMT from the next PE's word): the stationary inputs.  The sums of the four
// outputs 4k .. 4k+3 start in word-PE k and move one word-PE up per step; a step applies FOUR taps of each of
// the P filter rows with dp4a, so a pass is ceil(Q/4) steps and the four sums end up 128-bit aligned in
// word-PE k + ceil(Q/4) - 1 without any drain.  A strip is two runs of 32 words (lane l holds word l of each
// run: contiguous loads and stores), its last word-PE has no right neighbour and its first ones no left
// neighbour, so a strip yields 4*(64 - ceil(Q/4)) outputs and consecutive strips overlap by ceil(Q/4) words.
// ---------------------------------------------------------------------------
template <int Q>
struct IsDp4aGeom {
    static constexpr int G = (Q + 3) / 4;
    static constexpr int kValid = 4 * (64 - G);         // outputs per strip
};

template <int P, int Q>
__global__ void __launch_bounds__(kThreads2)
conv2d_u8_is_dp4a_kernel(const Conv2DArgs a, const __grid_constant__ TapsPacked taps, const int band_h)
{
    dependent_launch_enter();
    constexpr int G = IsDp4aGeom<Q>::G;
    constexpr int kValid = IsDp4aGeom<Q>::kValid;
    const int lane = threadIdx.x & (kLanes - 1);
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;    // (a block of fewer warps is the only one of its row)
    const int c0 = strip * kValid;              // first output column = first input column of the strip
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const uint8_t *xb = static_cast<const uint8_t *>(a.x) + blockIdx.z * a.x_bstride;
    int *yb = static_cast<int *>(a.y) + blockIdx.z * a.y_bstride;
    if (c0 >= a.out_w) return;
    const int y_align = row_alignment(static_cast<const int *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const int oend = min(a.out_w, c0 + kValid);

    // decided once per band, so that the row loop carries no comparisons: which of the lane's two words are loaded
    // whole or ragged (the image's last, partial word), which of its two output groups leave as one 128-bit word
    bool ld_whole[2], ld_ragged[2], st_vec[2], st_part[2];
#pragma unroll
    for (int n = 0; n < 2; ++n) {
        const int c = c0 + 4 * (kLanes * n + lane);
        ld_whole[n] = c + 4 <= a.width;
        ld_ragged[n] = !ld_whole[n] && c < a.width;
        const int k = kLanes * n + lane - (G - 1);              // word-PE whose outputs end up here
        st_vec[n] = k >= 0 && y_align == 4 && c0 + 4 * k + 4 <= oend;
        st_part[n] = k >= 0 && !st_vec[n] && c0 + 4 * k < oend;
    }
    const uint8_t *xnext = xb + static_cast<long long>(r0) * a.x_pitch + c0 + 4 * lane;
    int *onext = yb + static_cast<long long>(r0) * a.y_pitch + c0 + 4 * (lane - (G - 1));

    // the lane's two words of the next input row (pixels beyond the image read as zero)
    auto fetch = [&](unsigned (&w)[2]) {
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            unsigned v = 0;
            if (ld_whole[n]) {
                v = __ldg(reinterpret_cast<const unsigned *>(xnext + 4 * kLanes * n));
            } else if (ld_ragged[n]) {
                const int c = c0 + 4 * (kLanes * n + lane);
#pragma unroll
                for (int e = 0; e < 3; ++e)
                    if (c + e < a.width) v |= static_cast<unsigned>(xnext[4 * kLanes * n + e]) << (8 * e);
            }
            w[n] = v;
        }
        xnext += a.x_pitch;
    };
    // the four stationary words of both word-PEs for one input row
    auto expand = [&](const unsigned (&w)[2], unsigned (&s)[2][4]) {
        // the next PE's word: the next lane's, and for lane 31 of run 0 the first word of run 1
        const unsigned send = lane == 0 ? w[1] : w[0];
        const unsigned n0 = __shfl_sync(kFullMask, send, (lane + 1) & (kLanes - 1));
        const unsigned n1 = __shfl_down_sync(kFullMask, w[1], 1);    // the strip's last PE keeps its own: invalid sums
        const unsigned nx[2] = {n0, n1};
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            s[n][0] = w[n];
            s[n][1] = __byte_perm(w[n], nx[n], 0x4321);
            s[n][2] = __byte_perm(w[n], nx[n], 0x5432);
            s[n][3] = __byte_perm(w[n], nx[n], 0x6543);
        }
    };

    // PE registers: the window of P input rows is a ring -- the row loop is unrolled P times and input row r+p sits
    // in slot (u+p) mod P, u = position in the unrolled group, so sliding the window costs no moves
    unsigned S[P][2][4];
#pragma unroll
    for (int p = 0; p < P; ++p)
#pragma unroll
        for (int n = 0; n < 2; ++n)
#pragma unroll
            for (int i = 0; i < 4; ++i) S[p][n][i] = 0;
#pragma unroll
    for (int p = 0; p < P - 1; ++p) {
        unsigned w[2] = {0u, 0u};
        fetch(w);
        expand(w, S[p]);
    }
    unsigned nW[2] = {0u, 0u};
    fetch(nW);

#pragma unroll 1
    for (int rb = r0; rb < r1; rb += P) {
#pragma unroll
        for (int u = 0; u < P; ++u) {
            const int r = rb + u;
            if (r >= r1) break;
            expand(nW, S[(u + P - 1) % P]);
            if (r + 1 < r1) fetch(nW);

            int Z[2][4];
#pragma unroll
            for (int g = 0; g < G; ++g) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    int z0 = 0, z1 = 0;
                    if (g > 0) {
                        // the sums move one word-PE up: run 0 from the previous lane, run 1 likewise, its first PE
                        // from the last PE of run 0 (the strip's first PE has no left neighbour: invalid sums)
                        const int send = lane == kLanes - 1 ? Z[0][i] : Z[1][i];
                        z0 = __shfl_up_sync(kFullMask, Z[0][i], 1);
                        z1 = __shfl_sync(kFullMask, send, (lane - 1) & (kLanes - 1));
                    }
#pragma unroll
                    for (int p = 0; p < P; ++p) {
                        z0 = dp4a_u8s8(S[(u + p) % P][0][i], taps.w[p * 4 + g], z0);
                        z1 = dp4a_u8s8(S[(u + p) % P][1][i], taps.w[p * 4 + g], z1);
                    }
                    Z[0][i] = z0;
                    Z[1][i] = z1;
                }
            }
            // word-PE k holds the outputs that started in word-PE k - (G-1)
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                if (st_vec[n])
                    *reinterpret_cast<int4 *>(onext + 4 * kLanes * n) = make_int4(Z[n][0], Z[n][1], Z[n][2], Z[n][3]);
                else if (st_part[n])
                    store_group<U8Traits>(onext - (c0 + 4 * (lane - (G - 1))), c0 + 4 * (kLanes * n + lane - (G - 1)), oend,
                                          y_align, Z[n]);
            }
            onext += a.y_pitch;
        }
    }
}

// Input-stationary form that rebuilds the shifted words (filters of 8 to 15 rows, and of up to 4).  The kernel above
// keeps the four shifted words of every stationary row in registers (8 P of them) and unrolls the row loop P
// times; beyond seven rows neither fits, and for very short filters those registers cost more than they save.  Here a
// word-PE keeps only each row's word and its right neighbour's word (4 P registers for the lane's two word-PEs), the
// window slides by register moves, and the shifted words are rebuilt (PRMT) when they are used -- once per shift and
// row, shared by the ceil(Q/4) tap groups: for one shift the products of all tap groups are summed first
// (A_g = sum_p dp4a(x_p, w(p, g))), then the sums take their way up the word-PEs, z = shuffle(z) + A_g (integer
// addition is exact in any order).  Geometry, loads and stores are those of the kernel above.
template <int P, int Q>
__global__ void __launch_bounds__(kThreads2)
conv2d_u8_is_dp4a_rebuild_kernel(const Conv2DArgs a, const __grid_constant__ TapsPacked taps, const int band_h)
{
    dependent_launch_enter();
    constexpr int G = IsDp4aGeom<Q>::G;
    constexpr int kValid = IsDp4aGeom<Q>::kValid;
    const int lane = threadIdx.x & (kLanes - 1);
    const int strip = blockIdx.x * kWarps2 + threadIdx.x / kLanes;    // (a block of fewer warps is the only one of its row)
    const int c0 = strip * kValid;
    const int r0 = blockIdx.y * band_h;
    const int r1 = min(r0 + band_h, a.out_h);
    const uint8_t *xb = static_cast<const uint8_t *>(a.x) + blockIdx.z * a.x_bstride;
    int *yb = static_cast<int *>(a.y) + blockIdx.z * a.y_bstride;
    if (c0 >= a.out_w) return;
    const int y_align = row_alignment(static_cast<const int *>(a.y), a.y_pitch, a.y_bstride, a.batch);
    const int oend = min(a.out_w, c0 + kValid);

    bool ld_whole[2], ld_ragged[2], st_vec[2], st_part[2];
#pragma unroll
    for (int n = 0; n < 2; ++n) {
        const int c = c0 + 4 * (kLanes * n + lane);
        ld_whole[n] = c + 4 <= a.width;
        ld_ragged[n] = !ld_whole[n] && c < a.width;
        const int k = kLanes * n + lane - (G - 1);              // word-PE whose outputs end up here
        st_vec[n] = k >= 0 && y_align == 4 && c0 + 4 * k + 4 <= oend;
        st_part[n] = k >= 0 && !st_vec[n] && c0 + 4 * k < oend;
    }
    const uint8_t *xnext = xb + static_cast<long long>(r0) * a.x_pitch + c0 + 4 * lane;
    int *onext = yb + static_cast<long long>(r0) * a.y_pitch + c0 + 4 * (lane - (G - 1));

    auto fetch = [&](unsigned (&w)[2]) {
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            unsigned v = 0;
            if (ld_whole[n]) {
                v = __ldg(reinterpret_cast<const unsigned *>(xnext + 4 * kLanes * n));
            } else if (ld_ragged[n]) {
                const int c = c0 + 4 * (kLanes * n + lane);
#pragma unroll
                for (int e = 0; e < 3; ++e)
                    if (c + e < a.width) v |= static_cast<unsigned>(xnext[4 * kLanes * n + e]) << (8 * e);
            }
            w[n] = v;
        }
        xnext += a.x_pitch;
    };
    // the next PE's words: the next lane's, and for lane 31 of run 0 the first word of run 1
    auto neighbours = [&](const unsigned (&w)[2], unsigned (&nx)[2]) {
        const unsigned send = lane == 0 ? w[1] : w[0];
        nx[0] = __shfl_sync(kFullMask, send, (lane + 1) & (kLanes - 1));
        nx[1] = __shfl_down_sync(kFullMask, w[1], 1);           // the strip's last PE keeps its own: invalid sums
    };

    // PE registers: the window of P input rows, each as the PE's word and its right neighbour's word
    unsigned W[P][2], N[P][2];
#pragma unroll
    for (int p = 0; p < P; ++p)
#pragma unroll
        for (int n = 0; n < 2; ++n) W[p][n] = N[p][n] = 0;
#pragma unroll
    for (int p = 1; p < P; ++p) fetch(W[p]);    // rows r0 .. r0+P-2 sit one slot low: the first slide moves them up
#pragma unroll
    for (int p = 1; p < P; ++p) neighbours(W[p], N[p]);         // (after all the loads: they are in flight together)
    unsigned nW[2] = {0u, 0u};
    fetch(nW);

#pragma unroll 1
    for (int r = r0; r < r1; ++r) {
        // the window slides down one row
#pragma unroll
        for (int p = 0; p < P - 1; ++p)
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                W[p][n] = W[p + 1][n];
                N[p][n] = N[p + 1][n];
            }
        W[P - 1][0] = nW[0];
        W[P - 1][1] = nW[1];
        neighbours(nW, N[P - 1]);
        if (r + 1 < r1) fetch(nW);

        int Z[2][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            // products of every tap group with the inputs shifted by i pixels
            int A[G][2];
#pragma unroll
            for (int g = 0; g < G; ++g) A[g][0] = A[g][1] = 0;
#pragma unroll
            for (int p = 0; p < P; ++p) {
#pragma unroll
                for (int n = 0; n < 2; ++n) {
                    const unsigned sw = i == 0 ? W[p][n]
                                               : __byte_perm(W[p][n], N[p][n], i == 1 ? 0x4321 : i == 2 ? 0x5432 : 0x6543);
#pragma unroll
                    for (int g = 0; g < G; ++g) A[g][n] = dp4a_u8s8(sw, taps.w[p * 4 + g], A[g][n]);
                }
            }
            // the sums move one word-PE up per tap group: run 0 from the previous lane, run 1 likewise, its first PE
            // from the last PE of run 0 (the strip's first PE has no left neighbour: invalid sums)
            int z0 = A[0][0], z1 = A[0][1];
#pragma unroll
            for (int g = 1; g < G; ++g) {
                const int send = lane == kLanes - 1 ? z0 : z1;
                const int u0 = __shfl_up_sync(kFullMask, z0, 1);
                const int u1 = __shfl_sync(kFullMask, send, (lane - 1) & (kLanes - 1));
                z0 = u0 + A[g][0];
                z1 = u1 + A[g][1];
            }
            Z[0][i] = z0;
            Z[1][i] = z1;
        }
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            if (st_vec[n])
                *reinterpret_cast<int4 *>(onext + 4 * kLanes * n) = make_int4(Z[n][0], Z[n][1], Z[n][2], Z[n][3]);
            else if (st_part[n])
                store_group<U8Traits>(onext - (c0 + 4 * (lane - (G - 1))), c0 + 4 * (kLanes * n + lane - (G - 1)), oend,
                                      y_align, Z[n]);
        }
        onext += a.y_pitch;
    }
}

template <int P, int Q>
cudaError_t launch_conv2d_u8_is_dp4a(const Conv2DArgs &a, const Taps2DInt &t, cudaStream_t s)
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
    const int strips = (a.out_w + IsDp4aGeom<Q>::kValid - 1) / IsDp4aGeom<Q>::kValid;
    const long long warps = static_cast<long long>(strips) * a.batch;
    const long long bands = (148LL * 32 + warps - 1) / warps;
    long long h = (a.out_h + bands - 1) / bands;
    const long long lo = 2 * P > 8 ? 2 * P : 8;         // the first P-1 rows of a band are loaded twice
    if (h > 64) h = 64;
    if (h < lo) h = lo;
    const long long fit = (a.out_h + 65534LL) / 65535;  // grid.y limit
    if (h < fit) h = fit;
    int band_h = static_cast<int>(h);
    // which form: the ring of expanded rows pays for 5 to 7 filter rows (3840 x 2160, 7x7: 16.3 against 16.9 us);
    // with fewer rows rebuilding the shifted words costs less than the ring's registers (3x3: 9.4 against 11.8 us),
    // with more rows the ring does not fit
    constexpr bool kRebuild = P <= 4 || P > 7;
    const int wpb = block_warps(strips, kWarps2);
    {
        static const long long slots4 = 148LL * [] {
            if constexpr (kRebuild) return resident_blocks_per_sm(conv2d_u8_is_dp4a_rebuild_kernel<P, Q>, kThreads2);
            else return resident_blocks_per_sm(conv2d_u8_is_dp4a_kernel<P, Q>, kThreads2);
        }();
        const long long slots = slots4 * kWarps2 / wpb;
        const long long per_band = static_cast<long long>((strips + wpb - 1) / wpb) * a.batch;
        if (small_problem(a.out_h, per_band, 4, slots)) band_h = pick_band_height_small(a.out_h, per_band, P, 4, 64, slots);
    }
    dim3 grid((strips + wpb - 1) / wpb, (a.out_h + band_h - 1) / band_h, a.batch);
    if constexpr (kRebuild) launch_kernel(conv2d_u8_is_dp4a_rebuild_kernel<P, Q>, grid, wpb * kLanes, s, a, pk, band_h);
    else launch_kernel(conv2d_u8_is_dp4a_kernel<P, Q>, grid, wpb * kLanes, s, a, pk, band_h);
    return cudaGetLastError();
}

template <int P, int Q>
struct FastPath2D<U8Traits, SYSCONV_IS, P, Q> {
    static bool launch(const Conv2DArgs &a, const Taps2DInt &taps, cudaStream_t s, cudaError_t *err)
    {
        if (!u8_dp4a_eligible(a)) return false;
        *err = launch_conv2d_u8_is_dp4a<P, Q>(a, taps, s);
        return true;
    }
};

// uint8 rows that start 4-byte aligned run on the packed (dp4a) kernel
template <int P, int Q>
struct FastPath2D<U8Traits, SYSCONV_OS, P, Q> {
    static bool launch(const Conv2DArgs &a, const Taps2DInt &taps, cudaStream_t s, cudaError_t *err)
    {
        if (!u8_dp4a_eligible(a)) return false;
        *err = launch_conv2d_u8_os_dp4a<P, Q>(a, taps, s);
        return true;
    }
};

}  // namespace sysconv
